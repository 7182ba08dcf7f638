"""Parity at the benchmark's full sizes, in the launch configuration bench.py times.

The oracle cannot sweep 2,000,000 documents against 262,144 neurons in test
time, so the full-size run is checked (a) on a seeded sample of documents the
oracle computes one by one, (b) by properties that hold for every document,
and (c) against an independent computation by a library sparse-dense product (test-only
code): every document of the 64x64 and 128x128 configurations, and 96 windows of 2,048
documents spread evenly over the whole corpus of the 512x512 one.
"""
import numpy as np
import pytest
import torch

from inputs import synth
from tests import parity

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def bmu():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    import paper_2609_05138_b200 as lib
    lib.load()
    return lib


def check_sample(W_dev, rowptr, colidx, ob, od, n_sample, seed):
    g = torch.Generator().manual_seed(seed)
    N = rowptr.numel() - 1
    docs = torch.sort(torch.randperm(N, generator=g)[:n_sample]).values.numpy()
    res = parity.compare(ob.cpu().numpy(), od.cpu().numpy(), W_dev.cpu().numpy(),
                         rowptr.cpu().numpy(), colidx.cpu().numpy(), docs=docs)
    assert res["docs"] == n_sample and res["failed"] == 0
    return res


def check_properties(W_dev, norms, rowptr, colidx, ob, od, M):
    N = rowptr.numel() - 1
    assert int(ob.min()) >= 0 and int(ob.max()) < M
    assert bool(torch.isfinite(od).all())
    # the returned distance is the distance of the returned neuron (recomputed for every
    # document with plain torch gathers, fp64)
    lens = (rowptr[1:] - rowptr[:-1]).to(torch.int64)
    doc = torch.repeat_interleave(torch.arange(N, device=rowptr.device), lens)
    w = W_dev[colidx.to(torch.int64), ob.to(torch.int64)[doc]].double()
    s = torch.zeros(N, dtype=torch.float64, device=rowptr.device).index_add_(0, doc, w)
    d = lens.double() + norms.double()[ob.to(torch.int64)] - 2.0 * s
    assert bool(((od.double() - d).abs() <= 1e-5 * d.abs()).all())


def test_cfg4_full_size_sampled(bmu):
    cfg = synth.CONFIGS["cfg4"]
    dev = torch.device("cuda")
    W = synth.make_codebook(cfg.D, cfg.M, synth.codebook_seed(cfg), device=dev)
    rowptr, colidx = synth.make_corpus(cfg, device=dev)
    assert rowptr.numel() - 1 == cfg.N
    norms = bmu.bmu_codebook_norms(W)
    ob, od = bmu.bmu_search_ws(W, rowptr, colidx, norms=norms)     # bench.py's call and options
    torch.cuda.synchronize()
    check_properties(W, norms, rowptr, colidx, ob, od, cfg.M)
    check_sample(W, rowptr, colidx, ob, od, 2000, seed=4)


def test_cfg3_full_size_sampled(bmu):
    cfg = synth.CONFIGS["cfg3"]
    dev = torch.device("cuda")
    W = synth.make_codebook(cfg.D, cfg.M, synth.codebook_seed(cfg), device=dev)
    rowptr, colidx = synth.make_corpus(cfg, device=dev)
    assert rowptr.numel() - 1 == cfg.N
    norms = bmu.bmu_codebook_norms(W)
    ob, od = bmu.bmu_search_ws(W, rowptr, colidx, norms=norms)
    torch.cuda.synchronize()
    check_properties(W, norms, rowptr, colidx, ob, od, cfg.M)
    check_sample(W, rowptr, colidx, ob, od, 2000, seed=3)


def test_cfg3_full_size_half_precision_codebook_sampled(bmu):
    """The paper's storage at full size: the codebook rounded to fp16 once; the oracle reads the
    same rounded weights widened to fp32, so the rule and its tolerance are unchanged."""
    cfg = synth.CONFIGS["cfg3"]
    dev = torch.device("cuda")
    W16 = synth.make_codebook(cfg.D, cfg.M, synth.codebook_seed(cfg), device=dev).half()
    Ww = W16.float()
    rowptr, colidx = synth.make_corpus(cfg, device=dev)
    n16 = bmu.bmu_codebook_norms_f16(W16)
    ob, od = bmu.bmu_search_f16_ws(W16, rowptr, colidx, norms=n16)   # the wide tensor-core sweep
    torch.cuda.synchronize()
    check_properties(Ww, n16, rowptr, colidx, ob, od, cfg.M)
    check_sample(Ww, rowptr, colidx, ob, od, 2000, seed=33)


def test_cfg5_one_streamed_batch_sampled(bmu):
    cfg = synth.CONFIGS["cfg5"]
    dev = torch.device("cuda")
    W = synth.make_codebook(cfg.D, cfg.M, synth.codebook_seed(cfg), device=dev)
    norms = bmu.bmu_codebook_norms(W)
    for batch in (0, 26):                                            # a full and the short batch
        rowptr, colidx = synth.make_corpus(cfg, batch=batch, device=dev)
        assert rowptr.numel() - 1 == (1_000_000 if batch == 0 else 900_000)
        ob, od = bmu.bmu_search_ws(W, rowptr, colidx, norms=norms)
        torch.cuda.synchronize()
        check_properties(W, norms, rowptr, colidx, ob, od, cfg.M)
        check_sample(W, rowptr, colidx, ob, od, 1500, seed=5 + batch)


@pytest.mark.parametrize("name,n_windows,step", [("cfg2", 0, 50_000), ("cfg3", 0, 20_000),
                                                 ("cfg4", 96, 2_048)])
def test_full_size_against_library_product(bmu, name, n_windows, step):
    """Every document of configs 2 and 3, and 96 windows of 2,048 documents spread evenly over
    all of config 4's full search (the planned order is by length, so evenly spaced windows of
    the caller's order reach every part of every launch), against an independent computation:
    a library sparse-dense product per document batch, the distance formula and an arg-min in
    fp64 (test-only code)."""
    cfg = synth.CONFIGS[name]
    dev = torch.device("cuda")
    W = synth.make_codebook(cfg.D, cfg.M, synth.codebook_seed(cfg), device=dev)
    rowptr, colidx = synth.make_corpus(cfg, device=dev)
    N = cfg.N
    ob, od = bmu.bmu_search(W, rowptr, colidx)
    torch.cuda.synchronize()
    check_sample(W, rowptr, colidx, ob, od, 3000 if cfg.M <= 16384 else 200, seed=2)
    norms = (W.double() ** 2).sum(0)
    bad_d = bad_j = 0
    starts = (range(0, N, step) if not n_windows else
              [min(N - step, k * (N // n_windows) + (k * 977) % (N // n_windows - step))
               for k in range(n_windows)])
    for lo in starts:
        hi = min(N, lo + step)
        rp = (rowptr[lo:hi + 1] - rowptr[lo]).to(torch.int64)
        ci = colidx[int(rowptr[lo]):int(rowptr[hi])].to(torch.int64)
        X = torch.sparse_csr_tensor(rp, ci, torch.ones(ci.numel(), device=dev),
                                    size=(hi - lo, cfg.D))
        S = (X @ W).double()                                         # library sparse-dense product
        d = S.mul_(-2.0).add_(norms[None, :]).add_((rp[1:] - rp[:-1]).double()[:, None])
        dmin, jmin = d.min(dim=1)
        got_d = od[lo:hi].double()
        got_j = ob[lo:hi].to(torch.int64)
        tol = 1e-5 * dmin.abs()
        bad_d += int(((got_d - dmin).abs() > tol).sum())
        d_at = d.gather(1, got_j[:, None])[:, 0]
        bad_j += int(((got_j != jmin) & (d_at > dmin + tol)).sum())
        del X, S, d
    assert bad_d == 0 and bad_j == 0


def test_cfg2_full_size_update_step_properties(bmu):
    """Scatter, blur and write-back at full size: what must hold at any size (integer totals,
    a weighted mean of binary vectors stays in [0, 1], untouched units keep their weights),
    plus sampled planes against the oracle."""
    import oracle
    cfg = synth.CONFIGS["cfg2"]
    dev = torch.device("cuda")
    W = synth.make_codebook(cfg.D, cfg.M, synth.codebook_seed(cfg), device=dev)
    rowptr, colidx = synth.make_corpus(cfg, device=dev)
    units, _ = bmu.bmu_search(W, rowptr, colidx)
    num = torch.zeros((cfg.D, cfg.M), dtype=torch.int32, device=dev)
    cnt = torch.zeros(cfg.M, dtype=torch.int32, device=dev)
    bmu.bmu_update_scatter(rowptr, colidx, units, num, cnt)
    torch.cuda.synchronize()
    assert int(cnt.sum()) == cfg.N
    assert int(num.sum(dtype=torch.int64)) == colidx.numel()
    assert torch.equal(num.sum(1, dtype=torch.int64), torch.bincount(colidx.long(), minlength=cfg.D))
    assert torch.equal(cnt.long(), torch.bincount(units.long(), minlength=cfg.M))
    sigma = 1.5
    nb, cb = bmu.bmu_update_blur(num, cnt, cfg.edge, cfg.edge, sigma)
    for f in (0, 17, 4095, cfg.D - 1):                               # sampled planes
        ref = oracle.blur(num[f].cpu().numpy(), cfg.edge, cfg.edge, sigma)
        got = nb[f].cpu().numpy()
        assert np.all(np.abs(got - ref) <= 2e-6 * max(1.0, np.abs(ref).max()))
    W1 = W.clone()
    bmu.bmu_update_writeback(nb, cb, W1)
    torch.cuda.synchronize()
    live = cb > 0
    assert float(W1[:, live].min()) >= 0.0 and float(W1[:, live].max()) <= 1.0 + 1e-6
    assert torch.equal(W1[:, ~live], W[:, ~live])


@pytest.mark.parametrize("M", [256, 512])           # planned kernel; wide tensor-core sweep
def test_listing_count_next_to_the_32_bit_limit(bmu, M):
    """nnz = 2.1e9 of the 2^31 - 1 a CSR batch with int32 offsets can hold (16.5 M documents of
    120-134 listings, repeats allowed: rows are multisets): offsets, the tiling pass and the
    kernels must not wrap.  Checked on sampled documents against a plain fp64 recomputation and
    by agreement of the planned and the generic kernel."""
    dev = torch.device("cuda")
    D, N = 4096, 16_500_000
    g = torch.Generator(device=dev).manual_seed(1)
    lens = torch.randint(120, 135, (N,), generator=g, device=dev, dtype=torch.int64)
    rowptr64 = torch.zeros(N + 1, dtype=torch.int64, device=dev)
    rowptr64[1:] = torch.cumsum(lens, 0)
    nnz = int(rowptr64[-1])
    assert 2_000_000_000 < nnz < 2 ** 31
    rowptr = rowptr64.to(torch.int32)
    del rowptr64, lens
    colidx = torch.randint(0, D, (nnz,), generator=g, device=dev, dtype=torch.int32)
    W = torch.rand((D, M), generator=g, device=dev) * 0.05
    norms64 = (W.double() ** 2).sum(0)
    outs = []
    for kernel in (0, 1):
        o = bmu.Opts()
        o.kernel = kernel
        ob, od = bmu.bmu_search_ws(W, rowptr, colidx, opts=o)
        torch.cuda.synchronize()
        assert int(ob.min()) >= 0 and int(ob.max()) < M
        sample = list(range(0, 50)) + list(range(N - 50, N)) + \
            torch.randint(0, N, (100,), generator=torch.Generator().manual_seed(2)).tolist()
        for i in sample:
            ids = colidx[int(rowptr[i]):int(rowptr[i + 1])].long()
            d = float(ids.numel()) + norms64 - 2.0 * W[ids].double().sum(0)
            j = int(torch.argmin(d))
            assert abs(float(od[i]) - float(d[j])) <= 1e-5 * abs(float(d[j]))
            assert int(ob[i]) == j or abs(float(d[int(ob[i])]) - float(d[j])) <= 1e-5 * abs(float(d[j]))
        outs.append((ob, od))
    assert float((outs[0][0] == outs[1][0]).float().mean()) > 0.9999      # near-ties aside
    assert float(((outs[0][1] - outs[1][1]).abs() / outs[1][1].abs()).max()) < 1e-6


def test_cfg5_whole_corpus_streamed_in_batches_against_library_product(bmu):
    """Config 5 as it is meant to run: all 27 batches (26.9 M documents) from host memory through
    bmu_search_batches_host, every document checked against the library sparse-dense product."""
    cfg = synth.CONFIGS["cfg5"]
    dev = torch.device("cuda")
    W = synth.make_codebook(cfg.D, cfg.M, synth.codebook_seed(cfg), device=dev)
    n_batches = (cfg.N + synth.batch_size(cfg) - 1) // synth.batch_size(cfg)
    assert n_batches == 27
    host = []
    for k in range(n_batches):
        rp, ci = synth.make_corpus(cfg, batch=k, device=dev)
        host.append((rp.cpu(), ci.cpu()))
    assert sum(rp.numel() - 1 for rp, _ in host) == cfg.N
    outs = bmu.bmu_search_batches_host(W, host)
    norms = (W.double() ** 2).sum(0)
    bad_d = bad_j = 0
    step = 25_000
    for (rp_h, ci_h), (ob_h, od_h) in zip(host, outs):
        rowptr, colidx, ob, od = rp_h.to(dev), ci_h.to(dev), ob_h.to(dev), od_h.to(dev)
        n = rowptr.numel() - 1
        for lo in range(0, n, step):
            hi = min(n, lo + step)
            rp = (rowptr[lo:hi + 1] - rowptr[lo]).to(torch.int64)
            ci = colidx[int(rowptr[lo]):int(rowptr[hi])].to(torch.int64)
            X = torch.sparse_csr_tensor(rp, ci, torch.ones(ci.numel(), device=dev),
                                        size=(hi - lo, cfg.D))
            S = (X @ W).double()
            d = S.mul_(-2.0).add_(norms[None, :]).add_((rp[1:] - rp[:-1]).double()[:, None])
            dmin, jmin = d.min(dim=1)
            got_j = ob[lo:hi].to(torch.int64)
            tol = 1e-5 * dmin.abs()
            bad_d += int(((od[lo:hi].double() - dmin).abs() > tol).sum())
            bad_j += int(((got_j != jmin) & (d.gather(1, got_j[:, None])[:, 0] > dmin + tol)).sum())
            del X, S, d
    assert bad_d == 0 and bad_j == 0
