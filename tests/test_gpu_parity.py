"""Parity of the CUDA path against the fp64 oracle, through the C ABI.

Same seeded arrays on both sides; the rule is tests/parity.py (indices equal
except inside a 1e-5 near-tie, distances within 1e-5 relative).
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


def dev(*arrays):
    return [a.cuda() if isinstance(a, torch.Tensor) else torch.from_numpy(np.ascontiguousarray(a)).cuda()
            for a in arrays]


def run_and_check(bmu, W, rowptr, colidx, opts=None, cancel_floor=False, one_shot=False):
    Wd, rp, ci = dev(W, rowptr, colidx)
    if one_shot:
        ob, od = bmu.bmu_search(Wd, rp, ci)
    else:
        ob, od = bmu.bmu_search_ws(Wd, rp, ci, opts=opts)
    torch.cuda.synchronize()
    return parity.compare(ob.cpu().numpy(), od.cpu().numpy(), W.numpy(), rowptr.numpy(),
                          colidx.numpy(), cancel_floor=cancel_floor)


def make_opts(bmu, **kw):
    o = bmu.Opts()
    for k, v in kw.items():
        setattr(o, k, v)
    return o


# ------------------------------------------------------------------ norms
@pytest.mark.parametrize("D,M,kind", [(4096, 1024, "uniform"), (16384, 4096, "uniform"),
                                      (513, 1000, "signed"), (77, 37, "uniform"),
                                      (1, 5, "uniform"), (300, 130, "scaled"),
                                      # every column layout of the kernel: 2, 8 and 32 lanes
                                      # across, rows of 16-byte pieces and ragged rows
                                      (64, 8192, "uniform"), (8, 65536, "signed"),
                                      (33, 1301, "uniform"), (5, 9999, "scaled")])
def test_norms_match_oracle(bmu, D, M, kind):
    import oracle
    W = synth.make_codebook(D, M, 5, kind=kind)
    got = bmu.bmu_codebook_norms(W.cuda()).cpu().numpy().astype(np.float64)
    ref = oracle.norms(W.numpy())
    # fp64 accumulation rounded once to fp32: half an ulp
    np.testing.assert_allclose(got, ref, rtol=6e-8, atol=0)


# ------------------------------------------------------------------ benchmark shapes
def test_cfg1_full(bmu):
    cfg = synth.CONFIGS["cfg1"]
    rowptr, colidx = synth.make_corpus(cfg)
    W = synth.make_codebook(cfg.D, cfg.M, synth.codebook_seed(cfg))
    res = run_and_check(bmu, W, rowptr, colidx, one_shot=True)
    assert res["docs"] == cfg.N and res["exact"] > 0.98 * cfg.N


@pytest.mark.parametrize("name,n_docs,M", [("cfg2", 3000, 4096), ("cfg3", 600, 16384),
                                           ("cfg5", 600, 16384)])
def test_reduced_benchmark_shapes(bmu, name, n_docs, M):
    cfg = synth.CONFIGS[name]
    rowptr, colidx = synth.make_corpus(cfg, n_docs=n_docs)
    W = synth.make_codebook(cfg.D, M, synth.codebook_seed(cfg))
    run_and_check(bmu, W, rowptr, colidx)


# ------------------------------------------------------------------ codebooks where the sum decides
@pytest.mark.parametrize("kind,floor", [("scaled", False), ("sparse", False), ("signed", False),
                                        ("dupes", False), ("const", False),
                                        ("prototype", True)])
def test_codebook_kinds(bmu, kind, floor):
    cfg = synth.CONFIGS["cfg1"]
    rowptr, colidx = synth.make_corpus(cfg, n_docs=1500)
    W = synth.make_codebook(cfg.D, 640, 77, kind=kind, docs=(rowptr, colidx))
    res = run_and_check(bmu, W, rowptr, colidx, cancel_floor=floor)
    if kind == "dupes":
        Wd, rp, ci = dev(W, rowptr, colidx)
        ob, _ = bmu.bmu_search_ws(Wd, rp, ci)
        assert int((ob % 2).sum()) == 0            # equal columns: the lower index wins
    if kind == "const":
        Wd, rp, ci = dev(W, rowptr, colidx)
        ob, _ = bmu.bmu_search_ws(Wd, rp, ci)
        assert int(ob.abs().sum()) == 0            # every neuron ties: index 0
    assert res["failed"] == 0


# ------------------------------------------------------------------ ragged sizes and chunking
@pytest.mark.parametrize("N,D,M,chunk", [
    (1, 1, 1, 0), (3, 9, 4, 0), (257, 300, 1000, 0), (130, 64, 1028, 256), (515, 128, 37, 0),
    (99, 2048, 2500, 512), (1000, 512, 4100, 1024), (64, 100, 131, 0), (200, 50, 6, 0),
])
def test_ragged_shapes(bmu, N, D, M, chunk):
    r = np.random.default_rng(N * 7 + M)
    rows = [np.sort(r.choice(D, size=int(r.integers(0, min(D, 40) + 1)), replace=False))
            for _ in range(N)]
    rowptr = np.zeros(N + 1, dtype=np.int32)
    rowptr[1:] = np.cumsum([len(x) for x in rows])
    colidx = np.concatenate(rows).astype(np.int32) if rowptr[-1] else np.zeros(0, np.int32)
    W = synth.make_codebook(D, M, 3 + M, kind="scaled")
    opts = make_opts(bmu, chunk_neurons=chunk) if chunk else None
    run_and_check(bmu, W, torch.from_numpy(rowptr), torch.from_numpy(colidx), opts=opts)


def test_long_and_empty_rows(bmu):
    D, M = 16384, 1536
    nnz = torch.tensor([400, 0, 1, 33, 0, 400, 97, 64, 32, 31, 0])
    rowptr, colidx = synth.draw_corpus(nnz.numel(), D, 1.1, nnz, seed=4)
    assert rowptr[-1] == nnz.sum()
    W = synth.make_codebook(D, M, 8)
    run_and_check(bmu, W, rowptr, colidx)


def test_unsorted_rows(bmu):
    cfg = synth.CONFIGS["cfg1"]
    rowptr, colidx = synth.make_corpus(cfg, n_docs=300)
    ci = colidx.numpy().copy()
    r = np.random.default_rng(0)
    rp = rowptr.numpy()
    for i in range(300):
        r.shuffle(ci[rp[i]:rp[i + 1]])
    W = synth.make_codebook(cfg.D, 512, 9, kind="scaled")
    run_and_check(bmu, W, rowptr, torch.from_numpy(ci))


# ------------------------------------------------------------------ every lever gives the same answer
@pytest.mark.parametrize("vec", [4, 8])
@pytest.mark.parametrize("docs_per_warp", [1, 2, 4])
@pytest.mark.parametrize("warps", [8, 32])
def test_direct_kernel_options(bmu, vec, docs_per_warp, warps):
    cfg = synth.CONFIGS["cfg2"]
    rowptr, colidx = synth.make_corpus(cfg, n_docs=777)
    W = synth.make_codebook(cfg.D, 2048 + 128, 13, kind="scaled")
    opts = make_opts(bmu, kernel=1, vec=vec, docs_per_warp=docs_per_warp, warps=warps,
                     chunk_neurons=768)
    run_and_check(bmu, W, rowptr, colidx, opts=opts)


def test_chunk_count_does_not_change_result(bmu):
    """Merging the per-chunk minima gives the single-pass BMU (Section 4.2)."""
    cfg = synth.CONFIGS["cfg1"]
    rowptr, colidx = synth.make_corpus(cfg, n_docs=2000)
    W = synth.make_codebook(cfg.D, 4096, 21, kind="scaled")
    Wd, rp, ci = dev(W, rowptr, colidx)
    base = None
    for chunk in (4096, 2048, 512, 128):
        ob, od = bmu.bmu_search_ws(Wd, rp, ci, opts=make_opts(bmu, chunk_neurons=chunk))
        if base is None:
            base = (ob.clone(), od.clone())
        assert torch.equal(ob, base[0]) and torch.equal(od, base[1])


def test_deterministic_and_norms_reuse(bmu):
    cfg = synth.CONFIGS["cfg1"]
    rowptr, colidx = synth.make_corpus(cfg, n_docs=3000)
    W = synth.make_codebook(cfg.D, cfg.M, 2)
    Wd, rp, ci = dev(W, rowptr, colidx)
    a = bmu.bmu_search_ws(Wd, rp, ci)
    b = bmu.bmu_search(Wd, rp, ci)
    n = bmu.bmu_codebook_norms(Wd)
    c = bmu.bmu_search_ws(Wd, rp, ci, norms=n)
    for x in (b, c):
        assert torch.equal(a[0], x[0]) and torch.equal(a[1], x[1])


def test_host_entry_point_matches_device_one(bmu):
    cfg = synth.CONFIGS["cfg1"]
    rowptr, colidx = synth.make_corpus(cfg, n_docs=2500)
    W = synth.make_codebook(cfg.D, cfg.M, 2)
    Wd, rp, ci = dev(W, rowptr, colidx)
    a = bmu.bmu_search(Wd, rp, ci)
    hb, hd = bmu.bmu_search_host(Wd, rowptr.pin_memory(), colidx.pin_memory())
    assert torch.equal(a[0].cpu(), hb) and torch.equal(a[1].cpu(), hd)


def test_validate_csr(bmu):
    rp = torch.tensor([0, 2, 3], dtype=torch.int32).cuda()
    ci = torch.tensor([0, 5, 2], dtype=torch.int32).cuda()
    bmu.bmu_validate_csr(rp, ci, 6)
    with pytest.raises(bmu.BmuError, match="outside"):
        bmu.bmu_validate_csr(rp, ci, 5)
    with pytest.raises(bmu.BmuError, match="decreases"):
        bmu.bmu_validate_csr(torch.tensor([0, 3, 2, 3], dtype=torch.int32).cuda(), ci, 6)
    long_rp = torch.tensor([0, 65535, 65535 + 65536], dtype=torch.int32).cuda()
    long_ci = torch.zeros(65535 + 65536, dtype=torch.int32).cuda()
    with pytest.raises(bmu.BmuError, match="more than 65535"):
        bmu.bmu_validate_csr(long_rp, long_ci, 6)
    bmu.bmu_validate_csr(long_rp[:2], long_ci[:65535], 6)          # exactly 65535 is allowed


def test_workspace_errors(bmu):
    W = torch.zeros(8, 8, device="cuda")
    rp = torch.tensor([0, 1], dtype=torch.int32).cuda()
    ci = torch.tensor([0], dtype=torch.int32).cuda()
    with pytest.raises(bmu.BmuError) as e:
        bmu.bmu_search_ws(W, rp, ci, workspace=torch.empty(300, dtype=torch.uint8, device="cuda"))
    assert e.value.status == 3


# ------------------------------------------------------------------ planned warp-per-document kernel
@pytest.mark.parametrize("vec", [4, 8])
@pytest.mark.parametrize("warps", [4, 8, 32])
def test_planned_kernel_matches_generic_bitwise(bmu, vec, warps):
    cfg = synth.CONFIGS["cfg2"]
    rowptr, colidx = synth.make_corpus(cfg, n_docs=1500)
    W = synth.make_codebook(cfg.D, 2048 + 36, 15, kind="scaled")   # ragged last slab
    Wd, rp, ci = dev(W, rowptr, colidx)
    a = bmu.bmu_search_ws(Wd, rp, ci, opts=make_opts(bmu, kernel=3, vec=vec, warps=warps,
                                                     chunk_neurons=512))
    g = bmu.bmu_search_ws(Wd, rp, ci, opts=make_opts(bmu, kernel=1))
    assert torch.equal(a[0], g[0]) and torch.equal(a[1], g[1])
    parity.compare(a[0].cpu().numpy(), a[1].cpu().numpy(), W.numpy(), rowptr.numpy(),
                   colidx.numpy())


def test_planned_kernel_long_empty_unsorted_rows(bmu):
    D, M = 16384, 384
    nnz = torch.tensor([400, 0, 1, 33, 0, 400, 97, 64, 32, 31, 0, 8, 16, 7, 9, 1500] * 9)
    rowptr, colidx = synth.draw_corpus(nnz.numel(), D, 1.1, nnz, seed=6)
    ci = colidx.numpy().copy()
    rp = rowptr.numpy()
    r = np.random.default_rng(2)
    for i in range(0, nnz.numel(), 2):
        r.shuffle(ci[rp[i]:rp[i + 1]])
    W = synth.make_codebook(D, M, 10, kind="scaled")
    run_and_check(bmu, W, rowptr, torch.from_numpy(ci), opts=make_opts(bmu, kernel=3))


def test_streamed_batches_match_single_calls(bmu):
    cfg = synth.CONFIGS["cfg5"]
    W = synth.make_codebook(cfg.D, 1024, 3).cuda()
    batches = []
    for k, n in enumerate((3000, 0, 4100, 1, 2500)):
        rp, ci = synth.make_corpus(cfg, batch=k, n_docs=n) if n else (
            torch.zeros(1, dtype=torch.int32), torch.zeros(0, dtype=torch.int32))
        batches.append((rp.pin_memory(), ci.pin_memory()))
    outs = bmu.bmu_search_batches_host(W, batches)
    for (rp, ci), (ob, od) in zip(batches, outs):
        if rp.numel() == 1:
            continue
        rb, rd = bmu.bmu_search(W, rp.cuda(), ci.cuda())
        assert torch.equal(rb.cpu(), ob) and torch.equal(rd.cpu(), od)


def test_status_word_of_the_one_shot_search_is_readable(bmu):
    """bmu_search keeps its status word in library-owned scratch; bmu_last_status hands it back
    (clean run: 0), also after the streamed-batches form, which collects every batch's word."""
    cfg = synth.CONFIGS["cfg2"]
    rowptr, colidx = synth.make_corpus(cfg, n_docs=700)
    W = synth.make_codebook(cfg.D, 1024, 5).cuda()
    bmu.bmu_search(W, rowptr.cuda(), colidx.cuda())
    assert bmu.bmu_last_status() == (0, 0)
    batches = [(rowptr.pin_memory(), colidx.pin_memory())] * 3
    bmu.bmu_search_batches_host(W, batches)
    assert bmu.bmu_last_status() == (0, 0)
    bmu.bmu_selftest_wait_timeout()                       # leaves the searches' word alone
    assert bmu.bmu_last_status() == (0, 0)


def test_bounded_wait_reports_timeout_and_context_survives(bmu):
    """A device-side wait that cannot succeed ends through the status word, not a hang."""
    assert bmu.bmu_selftest_wait_timeout() == 5            # BMU_ERR_TIMEOUT
    assert b"wait ran out" in bmu.load().bmu_last_error()
    cfg = synth.CONFIGS["cfg1"]                            # the context still works
    rowptr, colidx = synth.make_corpus(cfg, n_docs=200)
    W = synth.make_codebook(cfg.D, 256, 5)
    run_and_check(bmu, W, rowptr, colidx)


# ------------------------------------------------------------------ tiled kernel (8 documents per warp)
@pytest.mark.parametrize("tile_order,tile_head", [(0, 0), (1, 0), (0, 1), (1, 1)])
@pytest.mark.parametrize("name,n_docs,M", [("cfg1", 4001, 1024 + 36), ("cfg5", 1203, 2048)])
def test_tiled_kernel_matches_oracle(bmu, name, n_docs, M, tile_order, tile_head):
    cfg = synth.CONFIGS[name]
    rowptr, colidx = synth.make_corpus(cfg, n_docs=n_docs)
    W = synth.make_codebook(cfg.D, M, 16, kind="scaled")
    opts = make_opts(bmu, kernel=4, tile_order=tile_order, tile_head=tile_head, chunk_neurons=512)
    run_and_check(bmu, W, rowptr, colidx, opts=opts)
    Wd, rp, ci = dev(W, rowptr, colidx)
    a = bmu.bmu_search_ws(Wd, rp, ci, opts=opts)
    b = bmu.bmu_search_ws(Wd, rp, ci, opts=opts)      # tiles are cut differently run to run
    assert torch.equal(a[0], b[0]) and torch.equal(a[1], b[1])
    if tile_order == 1:                                # ascending sums: the planned kernel's bits
        p = bmu.bmu_search_ws(Wd, rp, ci, opts=make_opts(bmu, kernel=3))
        assert torch.equal(a[0], p[0]) and torch.equal(a[1], p[1])


@pytest.mark.parametrize("kind,floor", [("dupes", False), ("const", False), ("sparse", False),
                                        ("signed", False), ("prototype", True)])
def test_tiled_kernel_codebook_kinds(bmu, kind, floor):
    cfg = synth.CONFIGS["cfg1"]
    rowptr, colidx = synth.make_corpus(cfg, n_docs=1500)
    W = synth.make_codebook(cfg.D, 640, 79, kind=kind, docs=(rowptr, colidx))
    run_and_check(bmu, W, rowptr, colidx, opts=make_opts(bmu, kernel=4), cancel_floor=floor)


def test_tiled_kernel_long_empty_unsorted_and_repeated_rows(bmu):
    D, M = 16384, 384
    nnz = torch.tensor([400, 0, 1, 33, 0, 400, 97, 64, 32, 31, 0, 8, 16, 7, 9, 1500, 40] * 9)
    rowptr, colidx = synth.draw_corpus(nnz.numel(), D, 1.1, nnz, seed=8)
    ci = colidx.numpy().copy()
    rp = rowptr.numpy()
    r = np.random.default_rng(3)
    for i in range(0, nnz.numel(), 2):
        r.shuffle(ci[rp[i]:rp[i + 1]])
    # a row that lists a frequent id twice keeps multiset semantics (added twice, counted twice)
    ci[rp[3]:rp[3] + 2] = 5
    W = synth.make_codebook(D, M, 11, kind="scaled")
    run_and_check(bmu, W, rowptr, torch.from_numpy(ci), opts=make_opts(bmu, kernel=4))
    run_and_check(bmu, W, rowptr, torch.from_numpy(ci), opts=make_opts(bmu, kernel=3))


def test_tiled_kernel_refuses_unordered_tiles(bmu):
    W = torch.zeros(300, 256, device="cuda")
    rp = torch.tensor([0, 1], dtype=torch.int32).cuda()
    ci = torch.tensor([0], dtype=torch.int32).cuda()
    with pytest.raises(bmu.BmuError) as e:
        bmu.bmu_search_ws(W, rp, ci, opts=make_opts(bmu, kernel=4, cluster=2))
    assert e.value.status == 2
