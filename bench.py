"""Benchmark of the BMU search hot path on B200.

A step is one pass of the whole hot path -- codebook norms, the neuron-chunked
gather-accumulate sweep with the fused argmin, outputs in document order --
over one synthetic corpus batch.  Default workload: the 512x512 map
(M=262144, D=16384, 17 GB fp32 codebook) against 2,000,000 documents.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--config cfg4] [--impl reference]

With N > 1 every rank holds a replica of the codebook and its own batch of
documents (documents are independent: no collective on the data path, weak
scaling); the time is the maximum over ranks.  Under torchrun the ranks are the
launcher's; a plain `python bench.py --gpus N` starts N ranks itself.
Prints one JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from inputs import synth  # noqa: E402

METRIC = "bmu_search_docs_per_s"
UNIT = "docs/s"


# ----------------------------------------------------------------------------- helpers
def dist_env():
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            return json.load(f), "measured"
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "sm_max_mhz": 1965.0}, "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, device):
        self.uuid = None
        try:
            u = str(torch.cuda.get_device_properties(device).uuid)
            self.uuid = u if u.startswith("GPU-") else "GPU-" + u
        except Exception:
            pass
        self.tmp = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.proc = None

    def start(self):
        cmd = ["nvidia-smi", "--query-gpu=" + self.FIELDS, "--format=csv,noheader,nounits",
               "-lms", "200"]
        if self.uuid:
            cmd += ["-i", self.uuid]
        try:
            self.proc = subprocess.Popen(cmd, stdout=self.tmp, stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None

    def stop(self):
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.proc.kill()
        self.tmp.flush()
        self.tmp.seek(0)
        if not self.tmp.read().strip():
            # the timed region was shorter than one sampling period: one reading right after it
            cmd = ["nvidia-smi", "--query-gpu=" + self.FIELDS, "--format=csv,noheader,nounits"]
            if self.uuid:
                cmd += ["-i", self.uuid]
            try:
                self.tmp.write(subprocess.run(cmd, capture_output=True, text=True, timeout=20).stdout)
            except (OSError, subprocess.SubprocessError):
                pass
            self.tmp.flush()
        self.tmp.seek(0)
        sm, mx, pw, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.tmp.read().splitlines():
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            try:
                pw.append(float(parts[2]))
            except ValueError:
                pass
            for n, v in zip(names, parts[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        self.tmp.close()
        os.unlink(self.tmp.name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx),
                "power_w": statistics.median(pw) if pw else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def union_rows_per_block(rowptr, colidx, D, docs_per_block, order=None):
    """Sum over blocks of `docs_per_block` documents, consecutive in the planned order
    (`order[p]` = the document at position p; None = the corpus order), of the number of
    distinct features the block touches: the rows an SM has to fetch at least once per slab
    when those documents share it (the design's own grouping)."""
    N = rowptr.numel() - 1
    lens = (rowptr[1:] - rowptr[:-1]).to(torch.int64)
    doc = torch.repeat_interleave(torch.arange(N, device=rowptr.device), lens)
    if order is not None:
        pos = torch.empty(N, dtype=torch.int64, device=rowptr.device)
        pos[order.to(torch.int64)] = torch.arange(N, device=rowptr.device)
        doc = pos[doc]
    key = (doc // docs_per_block) * D + colidx.to(torch.int64)
    del doc
    key = torch.sort(key).values
    return int((key[1:] != key[:-1]).sum().item()) + (1 if key.numel() else 0)


# ----------------------------------------------------------------------------- reference arm
def run_reference(args, cfg):
    """The CPU oracle, as it stands, on the host cores: the reference arm and the
    cpu_baseline leg.  A step = full norms + BMU search of a bounded sample of documents;
    the value extrapolates that to the whole batch (documents are independent)."""
    import numpy as np
    import oracle

    n_docs = args.docs or synth.batch_size(cfg)
    gen_dev = "cuda" if torch.cuda.is_available() else "cpu"
    W = synth.make_codebook(cfg.D, cfg.M, synth.codebook_seed(cfg), device=gen_dev).cpu().numpy()
    sample = min(n_docs, args.ref_sample)
    rowptr, colidx = synth.make_corpus(cfg, device=gen_dev, n_docs=sample)
    rowptr, colidx = rowptr.cpu().numpy(), colidx.cpu().numpy()
    cores = oracle.max_threads()
    times = []
    for it in range(args.warmup + args.steps):
        t0 = time.perf_counter()
        nrm = oracle.norms(W)
        t1 = time.perf_counter()
        oracle.bmu(W, rowptr, colidx, nrm)
        t2 = time.perf_counter()
        if it >= args.warmup:
            times.append(((t1 - t0), (t2 - t1)))
    t_norm = statistics.mean(t[0] for t in times)
    t_bmu = statistics.mean(t[1] for t in times)
    step_s = t_norm + t_bmu * (n_docs / sample)
    value = n_docs / step_s
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": step_s * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic",
        "config": workload_config(cfg, n_docs, 1),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                         "sample": "norms of the full codebook (%.2f s, one thread) + BMU of the "
                                   "first %d documents (%.2f s, %d threads), extrapolated to %d "
                                   "documents" % (t_norm, sample, t_bmu, cores, n_docs)},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    return line


def cpu_baseline(cfg, W_dev, rowptr, colidx, n_docs, budget_s=15.0):
    """Oracle timed on a bounded sample of this run's own arrays (rank 0, N=1)."""
    import oracle
    W = W_dev.cpu().numpy()
    cores = oracle.max_threads()
    t0 = time.perf_counter()
    nrm = oracle.norms(W)
    t_norm = time.perf_counter() - t0
    rp = rowptr.cpu().numpy()

    def run(k):
        ci = colidx[: int(rp[k])].cpu().numpy()
        t = time.perf_counter()
        oracle.bmu(W, rp[: k + 1], ci, nrm)
        return time.perf_counter() - t

    probe = min(n_docs, 4 * cores)
    t_probe = run(probe)
    sample = int(max(probe, min(n_docs, probe * budget_s / max(t_probe, 1e-6))))
    t_bmu = run(sample)
    step_s = t_norm + t_bmu * (n_docs / sample)
    return {"value": n_docs / step_s, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": "norms of the full codebook (%.2f s, one thread) + BMU of the first %d "
                      "documents (%.2f s, %d threads), extrapolated to %d documents"
                      % (t_norm, sample, t_bmu, cores, n_docs)}


def workload_config(cfg, n_docs, world, corpus="zipf"):
    return {
        "workload": "%s: %dx%d map (M=%d), D=%d, fp32 feature-major codebook U[0,1), "
                    "N=%d docs per GPU, nnz/doc %s, Zipf(s=%.1f) ids without replacement"
                    % (cfg.name, cfg.edge, cfg.edge, cfg.M, cfg.D, n_docs,
                       "Poisson(%g)>=1" % cfg.nnz_param if cfg.nnz_kind == "poisson"
                       else "lognormal(median %g, sigma 0.5) in [1,400]" % cfg.nnz_param,
                       cfg.zipf_s),
        "docs_per_gpu": n_docs, "global_docs": n_docs * world, "corpus": corpus,
        "parallelism": "docs sharded over %d GPU(s), codebook replicated, no collective" % world,
        "l2_policy": "inputs larger than L2 (codebook %.1f GB); no flush between steps"
                     % (cfg.D * cfg.M * 4 / 1e9),
    }


# ----------------------------------------------------------------------------- our arm
def dram_traffic_record():
    """DRAM bytes per sweep launch from the committed ncu capture of a small case, with the
    rule that scales it to another launch (see the file itself)."""
    p = os.path.join(ROOT, "profiles", "dram_traffic_sweep_mma2.json")
    if not os.path.exists(p):
        return None
    with open(p) as f:
        return json.load(f)


def scaled_traffic(rec, cfg, desc, opts, n_docs_per_launch):
    """The capture's DRAM bytes scaled to this launch: the codebook chunk is read once per
    launch whatever the number of documents, the rest (tile id matrices, masks, per-document
    state) grows with the documents."""
    if rec is None or desc.kernel != 6 or opts.tile_order or opts.repack or opts.relabel:
        return None
    b = rec["build"]
    if desc.head_rows != b["head_rows"] or int(desc.chunk_neurons) != b["chunk_neurons"] or cfg.D != b["D"]:
        return None
    fixed = 4.0 * b["D"] * b["chunk_neurons"]
    per_doc = max(0.0, rec["dram_bytes_per_launch"] - fixed) / rec["docs_per_launch"]
    return fixed + per_doc * n_docs_per_launch


def measure_roofs(bmu, dev):
    """On-chip ceilings of this GPU, measured now.  The L2 -> SM ceiling is the largest rate
    any committed microbenchmark reaches: loads alone, bulk copies alone, both together."""
    r = {"l2_ldg": bmu.bmu_measure_roof("l2_ldg", device=dev),
         "l2_bulk_16k": bmu.bmu_measure_roof("l2_bulk", piece=16384, device=dev),
         "smem": bmu.bmu_measure_roof("smem", device=dev),
         "fadd2": bmu.bmu_measure_roof("fadd2", device=dev)}
    for piece in (4096, 8192, 16384):
        r["l2_mixed_%dk" % (piece // 1024)] = bmu.bmu_measure_roof("l2_mixed", piece=piece, device=dev)
    r["l2"] = max(v for k, v in r.items() if k.startswith("l2_"))
    return r


def measure_config(bmu, cfg, args, dev, rank, world, roofs, peaks, steps, warmup, opts,
                   detail=True):
    """Times `steps` steps of the whole hot path on one configuration (after `warmup`), and
    derives the roofline figures of its sweep kernel.  Returns (line fragment, arrays)."""
    n_batches = min(synth.num_batches(cfg), args.batches) if args.batches else synth.num_batches(cfg)
    W = synth.make_codebook(cfg.D, cfg.M, synth.codebook_seed(cfg), device=dev)
    batches = []
    for b in range(n_batches):
        bsz = min(synth.batch_size(cfg), cfg.N - b * synth.batch_size(cfg))
        if args.corpus == "topical":               # an extra input with co-occurrence structure
            rp_b, ci_b = synth.make_topical_corpus(cfg, device=dev,
                                                   n_docs=min(bsz, args.docs) if args.docs else bsz,
                                                   seed=synth.corpus_seed(cfg, 50 + b) + 1000 * rank)
        else:
            rp_b, ci_b = synth.make_corpus(cfg, batch=b, device=dev,
                                           n_docs=min(bsz, args.docs) if args.docs else bsz,
                                           seed=synth.corpus_seed(cfg, b) + 1000 * rank)
        batches.append((rp_b, ci_b))
    n_docs = sum(rp_b.numel() - 1 for rp_b, _ in batches)
    rowptr, colidx = batches[0]
    total_nnz = sum(ci_b.numel() for _, ci_b in batches)
    max_n = max(rp_b.numel() - 1 for rp_b, _ in batches)
    max_nnz = max(ci_b.numel() for _, ci_b in batches)
    ws = torch.empty(bmu.bmu_search_workspace_bytes(cfg.D, cfg.M, max_n, max_nnz, opts) + 256,
                     dtype=torch.uint8, device=dev)
    norms = torch.empty(cfg.M, dtype=torch.float32, device=dev)
    out_bmu = torch.empty(max_n, dtype=torch.int32, device=dev)
    out_dist = torch.empty(max_n, dtype=torch.float32, device=dev)
    # what the library does for this size and these options (it answers, nothing is mirrored here)
    desc = bmu.bmu_describe_search(cfg.D, cfg.M, max_n, max_nnz, opts, device=dev)
    kernel_name = {1: "sweep_direct_kernel", 3: "sweep_rows_kernel", 4: "sweep_tiles_kernel",
                   6: "sweep_mma2_kernel"}[desc.kernel]
    n_chunks = int(desc.sweep_launches)
    # neurons per launch, averaged over the launches of one search (the last one may be shorter)
    chunk = (cfg.M - desc.ragged_neurons) / float(n_chunks)

    def step(e0=None, e1=None, e2=None):
        if e0 is not None:
            e0.record()
        bmu.bmu_codebook_norms(W, norms)
        if e1 is not None:
            e1.record()
        for rp_b, ci_b in batches:
            nb = rp_b.numel() - 1
            bmu.bmu_search_ws(W, rp_b, ci_b, norms=norms, opts=opts, workspace=ws,
                              out_bmu=out_bmu[:nb], out_dist=out_dist[:nb])
        if e2 is not None:
            e2.record()

    def barrier():
        torch.cuda.synchronize(dev)
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize(dev)

    for _ in range(warmup):
        step()
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(steps)]
    barrier()
    sampler = ClockSampler(dev)
    sampler.start()
    launches0 = bmu.bmu_kernel_launches()
    for k in range(steps):
        step(*ev[k])
    launches = bmu.bmu_kernel_launches() - launches0
    barrier()
    clocks = sampler.stop()
    total_ms = ev[0][0].elapsed_time(ev[-1][2])
    sweep_ms = sum(e[1].elapsed_time(e[2]) for e in ev) / steps
    norms_ms = sum(e[0].elapsed_time(e[1]) for e in ev) / steps
    t = torch.tensor([total_ms, sweep_ms, norms_ms], dtype=torch.float64, device=dev)
    if world > 1:
        import torch.distributed as dist
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    total_ms, sweep_ms, norms_ms = t.tolist()
    ms_per_step = total_ms / steps
    value = n_docs * world / (ms_per_step * 1e-3)     # all ranks' documents / slowest rank

    # ---- roofline of the dominant kernel (the sweep): algorithmic units per launch / time.
    # The sweep launches are timed together with the tiling pass that precedes them (one
    # search call); on the large configurations the pass is under 1 % of it.
    launch_s = sweep_ms * 1e-3 / (n_chunks * len(batches))
    nnz = total_nnz / len(batches)                              # mean batch
    N = n_docs / len(batches)
    adds = float(nnz) * chunk                                   # one update per (nnz, neuron)
    order = None
    if desc.kernel != 1:                        # the order the tiling pass gives the documents
        plan = bmu.Plan(rowptr, colidx, cfg.D, cfg.M, opts)
        order = plan.order()
        plan.close()
        del plan
    union_rows = union_rows_per_block(rowptr, colidx, cfg.D, desc.docs_per_block, order) * (
        nnz / max(1, colidx.numel()))
    # listings per distinct row among the documents that share a block / an 8-document tile
    reuse = {"per_block_of_%d" % desc.docs_per_block: nnz / max(1.0, union_rows),
             "per_tile_of_8": colidx.numel() / max(1, union_rows_per_block(rowptr, colidx, cfg.D, 8, order))}
    del order
    alg = {
        "alu": (adds / launch_s, roofs["fadd2"], "add/s"),
        "l1": (4.0 * adds / launch_s, roofs["smem"], "B/s"),           # one 4-byte operand per add
        "l2": (4.0 * union_rows * chunk / launch_s, roofs["l2"], "B/s"),
        "hbm": ((4.0 * cfg.D * chunk + 4.0 * nnz + 24.0 * N) / launch_s,
                peaks["hbm_gbs"] * 1e9, "B/s"),
    }
    extra = {}
    if desc.kernel == 6:
        # the frequent features' updates are MMAs, not loads and adds: only the tail's updates
        # pass through L1 and the fp32 pipe.  The L2 figure is the algorithmic one (each block
        # of 128 documents fetches every distinct row it touches once per slab); what the
        # design really moves is the tail's rows per document plus the head image per block.
        head = desc.head_rows
        tail_share = float((colidx >= head).sum().item()) / max(1, colidx.numel())
        alg["alu"] = (tail_share * adds / launch_s, roofs["fadd2"], "add/s")
        alg["l1"] = (4.0 * tail_share * adds / launch_s, roofs["smem"], "B/s")
        moved = 4.0 * chunk * (tail_share * nnz + head * (N / float(desc.docs_per_block)))
        mma_flops = 2.0 * 2.0 * head * N * chunk        # hi and lo parts, 2 flops per MAC
        extra = {"tail_share_of_updates": tail_share,
                 "l2_bytes_moved_by_design_GBs": moved / launch_s / 1e9,
                 "l2_moved_frac_of_roof": moved / launch_s / roofs["l2"],
                 "head_mma_TFLOPs": mma_flops / launch_s / 1e12,
                 "head_mma_frac_of_bf16_peak": mma_flops / launch_s / 1e12 /
                 peaks.get("bf16_tflops_sustained", peaks.get("bf16_tflops", 1590.0))}
    bound = max(alg, key=lambda k: alg[k][0] / alg[k][1])
    ach, peak, unit = alg[bound]
    traffic = scaled_traffic(dram_traffic_record(), cfg, desc, opts, N)
    roofline = {
        "kernel": kernel_name, "bound": bound,
        "achieved": ach / 1e9, "peak": peak / 1e9,
        "unit": "GB/s" if unit == "B/s" else "Gadd/s", "frac": ach / peak,
        "traffic": traffic,
        "traffic_source": (None if traffic is None else
                           "profiles/dram_traffic_sweep_mma2.json (ncu on a small case, scaled "
                           "to this launch: codebook chunk once + the rest per document)"),
        "launch_ms": launch_s * 1e3, "launches_per_step": n_chunks * len(batches),
        "units_per_launch": {"adds": adds, "union_rows_x_chunk": float(union_rows) * chunk},
        "tile_reuse": reuse,
        "fractions": {k: v[0] / v[1] for k, v in alg.items()},
        **extra,
    }
    frag = {
        "value": value, "ms_per_step": ms_per_step,
        "updates_per_s": float(total_nnz) * cfg.M * world / (ms_per_step * 1e-3),
        "phases_ms": {"norms": norms_ms, "sweep_and_output": sweep_ms},
        "clocks": clocks, "gpu_launches": int(launches), "roofline": roofline,
        "search": {"kernel": desc.kernel, "head_rows": desc.head_rows, "slab": desc.slab,
                   "docs_per_block": desc.docs_per_block, "chunk_neurons": int(desc.chunk_neurons),
                   "sweep_launches": n_chunks, "repack": desc.repack},
    }
    arrays = dict(W=W, batches=batches, ws=ws, norms=norms, out_bmu=out_bmu, out_dist=out_dist,
                  n_docs=n_docs, total_nnz=total_nnz, barrier=barrier)
    return frag, arrays


def planned_steps(bmu, cfg, a, opts, steps, dev):
    """The same step with the tiling pass done beforehand (a frozen corpus, reused per epoch)."""
    rowptr, colidx = a["batches"][0]
    n0 = rowptr.numel() - 1
    plan = bmu.Plan(rowptr, colidx, cfg.D, cfg.M, opts)
    plan.search(a["W"], norms=a["norms"], out_bmu=a["out_bmu"][:n0], out_dist=a["out_dist"][:n0])
    torch.cuda.synchronize(dev)
    p0, p1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    p0.record()
    for _ in range(steps):
        bmu.bmu_codebook_norms(a["W"], a["norms"])
        plan.search(a["W"], norms=a["norms"], out_bmu=a["out_bmu"][:n0], out_dist=a["out_dist"][:n0])
    p1.record()
    torch.cuda.synchronize(dev)
    planned_ms = p0.elapsed_time(p1) / steps
    plan.close()
    return {"ms_per_step": planned_ms, "value": n0 / (planned_ms * 1e-3), "unit": UNIT,
            "api": "bmu_plan_create once, then bmu_codebook_norms + bmu_search_planned per step "
                   "(rank 0's figure)"}


def run_ours(args, cfg, rank, local_rank, world):
    import paper_2609_05138_b200 as bmu
    bmu.load()                                    # fails loudly if the CUDA library is missing
    dev = torch.device("cuda", local_rank)
    torch.cuda.set_device(dev)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    opts = bmu.Opts()
    for kv in args.opt:
        k, v = kv.split("=")
        setattr(opts, k, int(v))
    peaks, peaks_kind = measured_peaks()
    roofs = measure_roofs(bmu, dev)

    frag, a = measure_config(bmu, cfg, args, dev, rank, world, roofs, peaks, args.steps,
                             args.warmup, opts)
    W, batches, ws, norms = a["W"], a["batches"], a["ws"], a["norms"]
    out_bmu, out_dist, n_docs, total_nnz = a["out_bmu"], a["out_dist"], a["n_docs"], a["total_nnz"]
    rowptr, colidx = batches[0]
    N = rowptr.numel() - 1

    # ---- end to end through the host entry point (pinned CSR in, results out)
    host = [(rp_b.cpu().pin_memory(), ci_b.cpu().pin_memory()) for rp_b, ci_b in batches]
    outs = [(torch.empty(rp_b.numel() - 1, dtype=torch.int32).pin_memory(),
             torch.empty(rp_b.numel() - 1, dtype=torch.float32).pin_memory()) for rp_b, _ in host]
    rp_h, ci_h = host[0]
    ob_h, od_h = outs[0]

    def e2e_step():
        if len(host) == 1:
            bmu.bmu_search_host(W, rp_h, ci_h, ob_h, od_h)
        else:
            bmu.bmu_search_batches_host(W, host, outs)

    e2e_step()                                              # warm-up (grows the scratch)
    e2e_steps = max(1, min(args.steps, 2))
    a["barrier"]()
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        e2e_step()
    torch.cuda.synchronize(dev)
    e2e_s = (time.perf_counter() - t0) / e2e_steps
    te = torch.tensor([e2e_s], dtype=torch.float64, device=dev)
    if world > 1:
        import torch.distributed as dist
        dist.all_reduce(te, op=dist.ReduceOp.MAX)
    e2e_s = te.item()
    bmu.bmu_search_ws(W, rowptr, colidx, norms=norms, opts=opts, workspace=ws,
                      out_bmu=out_bmu[:N], out_dist=out_dist[:N])
    same = bool(torch.equal(ob_h, out_bmu[:N].cpu()))
    del host, outs
    bmu.bmu_release_scratch()

    if rank != 0:
        return None

    frag["roofline"]["peaks"] = {
        "hbm_GBs": peaks["hbm_gbs"], "hbm_source": "MEASURED_PEAKS.json (%s)" % peaks_kind,
        "l2_GBs": roofs["l2"] / 1e9,
        "l2_variants_GBs": {k: v / 1e9 for k, v in roofs.items() if k.startswith("l2_")},
        "l2_rule": "largest of: 128-bit loads, 16 KB bulk copies, loads and bulk copies together",
        "l1_smem_GBs": roofs["smem"] / 1e9, "fp32_Gadds": roofs["fadd2"] / 1e9,
        "on_chip_source": "bmu_measure_roof, this run"}
    line = {
        "metric": METRIC, "value": frag["value"], "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": frag["ms_per_step"],
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
        "data": "synthetic", "config": workload_config(cfg, n_docs, world, args.corpus),
        "updates_per_s": frag["updates_per_s"], "phases_ms": frag["phases_ms"],
        "clocks": frag["clocks"],
        "e2e": {"value": n_docs * world / e2e_s, "unit": UNIT,
                "h2d_bytes_per_step": int((n_docs + len(batches) + total_nnz) * 4),
                "d2h_bytes_per_step": int(n_docs * 8),
                "api": ("bmu_search_host" if len(batches) == 1 else
                        "bmu_search_batches_host (%d batches, upload of the next batch overlapped "
                        "with the search of the current one)" % len(batches)) +
                       " (codebook resident in HBM; CSR from pinned host memory; results back "
                       "to host)", "matches_device_path": same},
        "gpu_launches": frag["gpu_launches"],
        "gpu_launches_source": "bmu_kernel_launches(): the library's own count of its kernel "
                               "launches across the timed region (library sort/scan kernels and "
                               "memsets not counted)",
        "search": frag["search"],
        "roofline": frag["roofline"],
    }
    if len(batches) == 1:
        line["planned"] = planned_steps(bmu, cfg, a, opts, min(args.steps, 5), dev)
    if args.comparator:
        line["comparator"] = comparator_spmm(cfg, W, norms, rowptr, colidx, peaks)
    if args.f16 and len(batches) == 1:
        line["f16_codebook"] = f16_codebook(bmu, cfg, W, rowptr, colidx, args)
    if args.epoch:
        line["epoch"] = epoch_phases(bmu, cfg, W, batches, opts, ws, norms, out_bmu, out_dist,
                                     peaks, args.sigma)
    if world == 1 and not args.no_cpu_baseline:
        line["cpu_baseline"] = cpu_baseline(cfg, W, rowptr, colidx, rowptr.numel() - 1)
    # ---- the other benchmark configurations, briefly (same protocol, fewer steps)
    if (world == 1 and args.all_configs and not args.docs and not args.batches and not args.opt
            and args.corpus == "zipf"):
        del W, batches, ws, norms, out_bmu, out_dist, rowptr, colidx
        a.clear()
        torch.cuda.empty_cache()
        line["all_configs"] = {cfg.name: {k: frag[k] for k in ("value", "ms_per_step", "updates_per_s")}
                               | {"unit": UNIT, "bound": frag["roofline"]["bound"],
                                  "frac": frag["roofline"]["frac"],
                                  "sm_mhz": frag["clocks"].get("sm_mhz")}}
        for name in sorted(synth.CONFIGS):
            if name == cfg.name:
                continue
            line["all_configs"][name] = brief_config(bmu, synth.CONFIGS[name], args, dev, roofs, peaks)
    return line


def brief_config(bmu, cfg, args, dev, roofs, peaks):
    """One of the other benchmark configurations: 3 warm-up + 3 timed steps (the 0.2 ms
    configuration: 100 back-to-back steps), docs/s, updates/s and the roofline fraction."""
    small = cfg.N * cfg.M < 10 ** 9
    steps, warmup = (100, 10) if small else (3, 3)
    opts = bmu.Opts()
    frag, a = measure_config(bmu, cfg, args, dev, 0, 1, roofs, peaks, steps, warmup, opts)
    out = {"value": frag["value"], "unit": UNIT, "ms_per_step": frag["ms_per_step"],
           "updates_per_s": frag["updates_per_s"], "steps": steps, "warmup": warmup,
           "kernel": frag["roofline"]["kernel"], "bound": frag["roofline"]["bound"],
           "frac": frag["roofline"]["frac"], "fractions": frag["roofline"]["fractions"],
           "l2_moved_frac_of_roof": frag["roofline"].get("l2_moved_frac_of_roof"),
           "sm_mhz": frag["clocks"].get("sm_mhz"), "clock_reasons": frag["clocks"].get("reasons"),
           "gpu_launches": frag["gpu_launches"], "docs": a["n_docs"]}
    if len(a["batches"]) == 1:
        out["planned_ms_per_step"] = planned_steps(bmu, cfg, a, opts, steps, dev)["ms_per_step"]
    a.clear()
    torch.cuda.empty_cache()
    return out


def f16_codebook(bmu, cfg, W, rowptr, colidx, args):
    """The same sweep with the paper's own storage (Section 4.2: two bytes per half-precision
    weight): the codebook rounded to fp16 once, sums and distances still fp32.  Context beside
    the fp32 headline, not a substitute for it: the rounding changes the weights."""
    W16 = W.half()
    n16 = bmu.bmu_codebook_norms_f16(W16)
    n0, nnz = rowptr.numel() - 1, colidx.numel()
    D, M = W16.shape
    o16 = bmu.Opts()
    o16.head_rows = args.f16_head
    import ctypes
    need = int(bmu.load().bmu_search_f16_workspace_bytes(D, M, n0, nnz, ctypes.byref(o16)))
    ws = torch.empty(need + 256, dtype=torch.uint8, device=W.device)
    for _ in range(max(1, args.warmup)):
        bmu.bmu_search_f16_ws(W16, rowptr, colidx, norms=n16, opts=o16, workspace=ws)
    torch.cuda.synchronize(W.device)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        bmu.bmu_codebook_norms_f16(W16)
        bmu.bmu_search_f16_ws(W16, rowptr, colidx, norms=n16, opts=o16, workspace=ws)
    e1.record()
    torch.cuda.synchronize(W.device)
    ms = e0.elapsed_time(e1) / args.steps
    return {"ms_per_step": ms, "value": n0 / (ms * 1e-3), "unit": UNIT,
            "updates_per_s": nnz * float(M) / (ms * 1e-3), "dtype": "f16 storage, f32 sums",
            "api": "bmu_codebook_norms_f16 + bmu_search_f16_ws per step (rank 0's figure)"}


def comparator_spmm(cfg, W, norms, rowptr, colidx, peaks, budget_docs=0):
    """The other side of the paper's comparison (Section 3: a library sparse-dense product that
    materialises the score block, then a separate arg-min read-back), tuned the way the paper
    tunes it (Section 4.4): score block in fp32 and in fp16, batch size swept, and the read-back
    done by a warp-per-row kernel with 128-bit loads that forms n_j - 2 s_ij on the fly
    (bmu_score_block_argmin) -- next to the untuned torch.argmin read-back for contrast.  The
    product is torch.sparse CSR x dense (cuSPARSE SpMM): the library stays the library.  Timed on
    a bounded prefix of the workload (documents are independent, so docs/s extrapolates)."""
    import warnings
    import paper_2609_05138_b200 as bmu
    dev = W.device
    if not budget_docs:
        budget_docs = 100_000 if cfg.M > 100_000 else 400_000
    n_docs = min(rowptr.numel() - 1, budget_docs)
    rp32 = rowptr[: n_docs + 1].contiguous()
    rp64 = rp32.to(torch.int64)
    ci64 = colidx[: int(rp64[-1])].to(torch.int64)
    W16 = None
    cells = []

    def one_pass(dtype, batch, tuned):
        Wd = W if dtype == torch.float32 else W16
        ones = torch.ones(ci64.numel(), device=dev, dtype=dtype)
        ob = torch.empty(n_docs, dtype=torch.int32, device=dev)
        od = torch.empty(n_docs, dtype=torch.float32, device=dev)
        t_rb = 0.0
        for lo in range(0, n_docs, batch):
            hi = min(n_docs, lo + batch)
            a, b = int(rp64[lo]), int(rp64[hi])
            X = torch.sparse_csr_tensor(rp64[lo:hi + 1] - a, ci64[a:b], ones[a:b],
                                        size=(hi - lo, cfg.D))
            S = X @ Wd                                      # the materialised score block
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            if tuned:
                bmu.bmu_score_block_argmin(S, norms, rp32[lo:hi + 1], ob[lo:hi], od[lo:hi])
            else:
                d = torch.addcmul(norms[None, :], S.float(), S.new_full((), -2.0, dtype=torch.float32))
                ob[lo:hi] = torch.argmin(d, dim=1).to(torch.int32)
            e1.record()
            torch.cuda.synchronize(dev)
            t_rb += e0.elapsed_time(e1)
            del X, S
        return ob, t_rb

    with warnings.catch_warnings():
        warnings.simplefilter("ignore")
        for dtype in (torch.float32, torch.float16):
            esize = 4 if dtype == torch.float32 else 2
            if dtype == torch.float16:
                W16 = W.half()
            for batch in (1024, 4096, 16384, 65536):
                if batch * cfg.M * esize > (4 << 30) or batch > 4 * n_docs:
                    continue
                for tuned in (True, False):
                    if not tuned and (dtype == torch.float16 or batch != 4096):
                        continue                      # the untuned read-back once, for contrast
                    try:
                        one_pass(dtype, batch, tuned)             # warm-up
                        torch.cuda.synchronize(dev)
                        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                        e0.record()
                        _, t_rb = one_pass(dtype, batch, tuned)
                        e1.record()
                        torch.cuda.synchronize(dev)
                    except RuntimeError as ex:        # e.g. no half-precision SpMM in this library build
                        cells.append({"score_dtype": str(dtype).replace("torch.", ""), "batch": batch,
                                      "tuned_readback": tuned, "unavailable": str(ex)[:120]})
                        continue
                    ms = e0.elapsed_time(e1)
                    cells.append({"score_dtype": str(dtype).replace("torch.", ""), "batch": batch,
                                  "tuned_readback": tuned, "ms": ms, "value": n_docs / (ms * 1e-3),
                                  "readback_ms": t_rb,
                                  "readback_frac_of_hbm": (n_docs * cfg.M * esize / (t_rb * 1e-3) /
                                                           (peaks["hbm_gbs"] * 1e9)) if tuned else None})
        del W16
    ok = [c for c in cells if "value" in c and c["tuned_readback"]]
    best = max(ok, key=lambda c: c["value"]) if ok else None
    return {"kind": "materialised score block: torch.sparse CSR x dense (cuSPARSE SpMM) into an fp32 "
                    "or fp16 block, then a warp-per-row 128-bit arg-min read-back "
                    "(bmu_score_block_argmin); batch size and score dtype swept",
            "sample_docs": n_docs, "unit": UNIT, "best": best, "cells": cells}


def epoch_phases(bmu, cfg, W, batches, opts, ws, norms, out_bmu, out_dist, peaks, sigma):
    """One whole batch epoch (Table 4 of the paper: norms, search, stopping metric on held-out
    documents, scatter, blur, write-back),
    timed phase by phase with CUDA events; HBM-bound phases against the measured copy roof.
    The codebook is overwritten by the update (random data either way)."""
    dev = W.device
    D, M = cfg.D, cfg.M
    num = torch.zeros((D, M), dtype=torch.int32, device=dev)
    cnt = torch.zeros(M, dtype=torch.int32, device=dev)
    nnz = sum(ci.numel() for _, ci in batches)
    n_docs = sum(rp.numel() - 1 for rp, _ in batches)
    names = ["norms", "search", "stopping_metric", "scatter", "blur", "writeback"]
    acc = {k: 0.0 for k in names}
    # held-out documents for the stopping metrics: a tenth of the corpus (the paper trains on
    # 90 % and holds 10 % out, Section 5), drawn as a batch of its own
    n_held = max(1, n_docs // 9)
    held_rp, held_ci = synth.make_corpus(cfg, n_docs=min(n_held, synth.batch_size(cfg)),
                                         seed=synth.corpus_seed(cfg, 40), device=dev)
    quality = None

    def timed(name, fn):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        r = fn()
        e1.record()
        torch.cuda.synchronize(dev)
        acc[name] += e0.elapsed_time(e1)
        return r

    for rep in range(2):                              # the second pass is the one reported
        for k in names:
            acc[k] = 0.0
        num.zero_()
        cnt.zero_()
        timed("norms", lambda: bmu.bmu_codebook_norms(W, norms))

        def stopping_metric():
            b1, d1, b2, _ = bmu.bmu_search_top2_ws(W, held_rp, held_ci, norms=norms, opts=opts)
            return bmu.bmu_map_errors(b1, b2, d1, cfg.edge, cfg.edge, 4)
        quality = timed("stopping_metric", stopping_metric)
        for rp_b, ci_b in batches:
            nb = rp_b.numel() - 1
            timed("search", lambda: bmu.bmu_search_ws(W, rp_b, ci_b, norms=norms, opts=opts,
                                                      workspace=ws, out_bmu=out_bmu[:nb],
                                                      out_dist=out_dist[:nb]))
            timed("scatter", lambda: bmu.bmu_update_scatter(rp_b, ci_b, out_bmu[:nb], num, cnt))
        nbl, cbl = timed("blur", lambda: bmu.bmu_update_blur(num, cnt, cfg.edge, cfg.edge, sigma))
        timed("writeback", lambda: bmu.bmu_update_writeback(nbl, cbl, W))
        del nbl, cbl
    total = sum(acc.values())
    hbm = peaks["hbm_gbs"] * 1e9
    plane = 4.0 * D * M
    alg = {"scatter": 12.0 * nnz + 12.0 * n_docs,      # id + counter read-modify-write per listing
           "blur": 2.0 * plane, "writeback": 3.0 * plane, "norms": plane}
    q = quality.cpu().tolist()
    return {"sigma": sigma, "phases_ms": dict(acc), "total_ms": total,
            "search_share": acc["search"] / total,
            "held_out_docs": held_rp.numel() - 1,
            "held_out_quality": {"mean_sq_quantisation_error": q[0], "quantisation_error": q[1],
                                 "topographic_error_4": q[2]},
            "hbm_frac": {k: alg[k] / (acc[k] * 1e-3) / hbm for k in alg if acc[k] > 0},
            "note": "paper (RTX 4090, Table 4): search 73.7-94.0 % of the epoch"}


def launch_ranks(n_ranks, argv):
    """Re-runs this script as `n_ranks` ranks on this node (one process per GPU) through
    torch.distributed.run and returns its exit code; rank 0 of the children prints the line."""
    import socket
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1",
           "--nproc-per-node", str(n_ranks), "--master-addr", "127.0.0.1",
           "--master-port", str(port), os.path.abspath(__file__), *argv]
    return subprocess.call(cmd)


def selfcheck_ranks(rank, world):
    """No GPU work: the ranks meet over gloo on the host and rank 0 reports how many came."""
    import torch.distributed as dist
    if "MASTER_ADDR" not in os.environ:              # a single rank started by hand
        os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT="29533", RANK="0", WORLD_SIZE="1")
    dist.init_process_group("gloo")
    t = torch.ones(1, dtype=torch.int64)
    dist.all_reduce(t)
    dist.barrier()
    if rank == 0:
        print(json.dumps({"selfcheck": "ranks", "n_gpus": int(t.item()), "world_size": world}))
    dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=3)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="cfg4", choices=sorted(synth.CONFIGS))
    ap.add_argument("--docs", type=int, default=0, help="documents per batch (0 = the config's)")
    ap.add_argument("--batches", type=int, default=0, help="batches per step (0 = the config's)")
    ap.add_argument("--opt", action="append", default=[], help="bmu_opts field=value")
    ap.add_argument("--ref-sample", type=int, default=4000)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--comparator", action="store_true",
                    help="also time the materialised-score route (library SpMM + argmin)")
    ap.add_argument("--f16", action="store_true",
                    help="also time the same sweep on the codebook rounded to fp16 (the paper's storage)")
    ap.add_argument("--f16-head", type=int, default=0, help="head_rows of the --f16 sweep (0 = default)")
    ap.add_argument("--epoch", action="store_true",
                    help="also time one whole epoch (search + scatter + blur + write-back)")
    ap.add_argument("--sigma", type=float, default=2.0, help="neighbourhood width of --epoch")
    ap.add_argument("--corpus", default="zipf", choices=["zipf", "topical"],
                    help="zipf: the configuration's own recipe (ids drawn independently); topical: "
                         "the same sizes with topics, i.e. documents that share rare features")
    ap.add_argument("--no-all-configs", dest="all_configs", action="store_false",
                    help="skip the brief runs of the other benchmark configurations")
    ap.add_argument("--selfcheck-ranks", action="store_true",
                    help="start the ranks, let them meet on the host and report their number")
    args = ap.parse_args()
    cfg = synth.CONFIGS[args.config]
    if "WORLD_SIZE" not in os.environ and args.gpus > 1 and (args.impl == "ours" or args.selfcheck_ranks):
        sys.exit(launch_ranks(args.gpus, sys.argv[1:]))
    rank, local_rank, world = dist_env()
    if args.selfcheck_ranks:
        selfcheck_ranks(rank, world)
        return
    if args.warmup < 3 and args.impl == "ours" and rank == 0:
        print("note: fewer than 3 warm-up steps", file=sys.stderr)

    if args.impl == "reference":
        if rank == 0:
            print(json.dumps(run_reference(args, cfg)))
        return
    line = run_ours(args, cfg, rank, local_rank, world)
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()
    if line is not None:
        print(json.dumps(line))


if __name__ == "__main__":
    main()
