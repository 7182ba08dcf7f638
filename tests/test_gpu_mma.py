"""Parity of the tensor-core head + gathered tail sweep (bmu_opts.kernel = 6: 256-neuron
slabs, double-buffered tensor memory, head of 64 .. 2048 features) against the fp64
oracle, through the C ABI.  Same rule as every other kernel
(tests/parity.py): indices equal except inside a 1e-5 near-tie, distances within
1e-5 relative.  The head sums come from fp16 (hi, lo) parts of the weights and a
tensor-core fp32 accumulator, so results are not bit-equal to the gathered
kernels; they are held to the oracle alone.
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


def opts_of(bmu, kernel=6, **kw):
    o = bmu.Opts()
    o.kernel = kernel
    for k, v in kw.items():
        setattr(o, k, v)
    return o


def run_and_check(bmu, W, rowptr, colidx, opts, cancel_floor=False):
    Wd, rp, ci = W.cuda(), rowptr.cuda(), colidx.cuda()
    need = bmu.bmu_search_workspace_bytes(W.shape[0], W.shape[1], rowptr.numel() - 1,
                                          colidx.numel(), opts)
    ws = torch.empty(need + 256, dtype=torch.uint8, device="cuda")
    ob, od = bmu.bmu_search_ws(Wd, rp, ci, opts=opts, workspace=ws)
    torch.cuda.synchronize()
    off = (-ws.data_ptr()) % 256
    assert int(ws[off:off + 4].view(torch.int32)[0]) == 0, "a bounded device-side wait ran out"
    return parity.compare(ob.cpu().numpy(), od.cpu().numpy(), W.numpy(), rowptr.numpy(),
                          colidx.numpy(), cancel_floor=cancel_floor)


@pytest.mark.parametrize("kernel,tile_order,head_rows", [(6, 0, 0), (6, 2, 64), (6, 1, 512),
                                                         (6, 0, 1024), (6, 2, 320), (6, 0, 2048),
                                                         (6, 1, 768), (6, 2, 256)])
@pytest.mark.parametrize("name,n_docs,M,chunk", [("cfg3", 2500, 2048, 1024), ("cfg5", 1203, 1536, 512),
                                                 ("cfg1", 4001, 1024 + 36, 0), ("cfg2", 777, 512, 0)])
def test_mma_kernel_matches_oracle(bmu, name, n_docs, M, chunk, kernel, tile_order, head_rows):
    cfg = synth.CONFIGS[name]
    rowptr, colidx = synth.make_corpus(cfg, n_docs=n_docs)
    for kind in ("uniform", "scaled"):
        W = synth.make_codebook(cfg.D, M, 21, kind=kind)
        res = run_and_check(bmu, W, rowptr, colidx,
                            opts_of(bmu, kernel, tile_order=tile_order, chunk_neurons=chunk,
                                    head_rows=head_rows))
        assert res["failed"] == 0 and res["docs"] == n_docs


@pytest.mark.parametrize("kernel", [6])
@pytest.mark.parametrize("kind,floor", [("dupes", False), ("const", False), ("sparse", False),
                                        ("signed", False), ("prototype", True)])
def test_mma_kernel_codebook_kinds(bmu, kind, floor, kernel):
    cfg = synth.CONFIGS["cfg1"]
    rowptr, colidx = synth.make_corpus(cfg, n_docs=1500)
    W = synth.make_codebook(cfg.D, 1024, 83, kind=kind, docs=(rowptr, colidx))
    run_and_check(bmu, W, rowptr, colidx, opts_of(bmu, kernel), cancel_floor=floor)
    if kind in ("dupes", "const"):
        ob, _ = bmu.bmu_search_ws(W.cuda(), rowptr.cuda(), colidx.cuda(), opts=opts_of(bmu, kernel))
        if kind == "dupes":
            assert int((ob % 2).sum()) == 0        # equal columns: the lower index wins
        else:
            assert int(ob.abs().sum()) == 0        # every neuron ties: index 0


@pytest.mark.parametrize("kernel", [6])
@pytest.mark.parametrize("scale", [1e-6, 1.0, 3e4, 1e9])
def test_mma_kernel_weight_magnitudes(bmu, scale, kernel):
    """The power-of-two scaling of the fp16 parts follows the largest head weight."""
    cfg = synth.CONFIGS["cfg3"]
    rowptr, colidx = synth.make_corpus(cfg, n_docs=700)
    W = synth.make_codebook(cfg.D, 512, 5, kind="signed") * scale
    run_and_check(bmu, W, rowptr, colidx, opts_of(bmu, kernel))


def test_mma_kernel_long_empty_unsorted_and_repeated_rows(bmu):
    D, M = 16384, 1024
    nnz = torch.tensor([400, 0, 1, 33, 0, 400, 97, 64, 32, 31, 0, 8, 16, 7, 9, 1500, 40] * 19)
    rowptr, colidx = synth.draw_corpus(nnz.numel(), D, 1.1, nnz, seed=8)
    ci = colidx.numpy().copy()
    rp = rowptr.numpy()
    r = np.random.default_rng(3)
    for i in range(0, nnz.numel(), 2):
        r.shuffle(ci[rp[i]:rp[i + 1]])
    # a row that lists a frequent id twice keeps multiset semantics (added twice, counted twice)
    ci[rp[3]:rp[3] + 2] = 5
    # a row made of frequent ids only (no tail at all), one with a single frequent id
    ci[rp[8]:rp[8 + 1]] = np.arange(32, dtype=np.int32) * 7
    ci[rp[2]] = 255
    W = synth.make_codebook(D, M, 11, kind="scaled")
    run_and_check(bmu, W, rowptr, torch.from_numpy(ci), opts_of(bmu))
    run_and_check(bmu, W, rowptr, torch.from_numpy(ci), opts_of(bmu, head_rows=512))
    run_and_check(bmu, W, rowptr, torch.from_numpy(ci), opts_of(bmu, 6, head_rows=256, tile_order=2))


@pytest.mark.parametrize("kernel", [6])
@pytest.mark.parametrize("relabel", [0, 2])
def test_mma_kernel_unlabelled_vocabulary(bmu, kernel, relabel):
    """Feature ids that are not frequency-ordered: the tiling pass ranks the features itself
    (relabel = 0); with relabel = 2 the head is the ids below head_rows -- exact either way."""
    cfg = synth.CONFIGS["cfg1"]
    rowptr, colidx = synth.make_corpus(cfg, n_docs=900)
    perm = torch.from_numpy(np.random.default_rng(1).permutation(cfg.D).astype(np.int32))
    ci = perm[colidx.long()]                              # rows are no longer ascending either
    W = synth.make_codebook(cfg.D, 512, 9, kind="scaled")
    run_and_check(bmu, W, rowptr, ci, opts_of(bmu, kernel, relabel=relabel))


def test_mma_kernel_relabel_off_matches_on_for_ordered_ids(bmu):
    """On a vocabulary already labelled by frequency both choices of head pass the oracle rule
    (they differ only in which of the near-equally frequent features fall inside the head)."""
    cfg = synth.CONFIGS["cfg3"]
    rowptr, colidx = synth.make_corpus(cfg, n_docs=1500)
    W = synth.make_codebook(cfg.D, 1024, 4, kind="scaled")
    for relabel in (0, 2):
        run_and_check(bmu, W, rowptr, colidx, opts_of(bmu, 6, relabel=relabel))


def test_mma_kernel_refuses_what_it_cannot_do(bmu):
    rp = torch.tensor([0, 1], dtype=torch.int32).cuda()
    ci = torch.tensor([0], dtype=torch.int32).cuda()
    for kernel, D, M in ((6, 32, 1024), (6, 2048, 128)):
        with pytest.raises(bmu.BmuError) as e:
            bmu.bmu_search_ws(torch.zeros(D, M, device="cuda"), rp, ci, opts=opts_of(bmu, kernel))
        assert e.value.status == 2


@pytest.mark.parametrize("kernel", [6])
@pytest.mark.parametrize("N", [1, 7, 9, 129, 257])
def test_mma_kernel_few_documents_and_empty_corpus_rows(bmu, kernel, N):
    """Blocks and tiles that are mostly padding; a corpus whose rows are all empty."""
    cfg = synth.CONFIGS["cfg1"]
    rowptr, colidx = synth.make_corpus(cfg, n_docs=N)
    W = synth.make_codebook(cfg.D, 512, 5 + N, kind="scaled")
    run_and_check(bmu, W, rowptr, colidx, opts_of(bmu, kernel))
    empty_rp = torch.zeros(N + 1, dtype=torch.int32)
    res = run_and_check(bmu, W, empty_rp, torch.zeros(0, dtype=torch.int32), opts_of(bmu, kernel))
    assert res["docs"] == N


@pytest.mark.parametrize("kernel", [0, 3, 4, 6])
def test_largest_vocabulary_with_16_bit_ids(bmu, kernel):
    """D = 65024, the most the 16-bit id lists hold: ids up to 65023 sit next to the 0xffff
    sentinel of a ragged row."""
    D, M, N = 65024, 512, 300
    r = np.random.default_rng(kernel)
    rows = []
    for i in range(N):
        n = int(r.integers(0, 60))
        low = r.choice(2000, size=n // 2, replace=False)
        high = D - 1 - r.choice(3000, size=n - n // 2, replace=False)      # 62024 .. 65023
        rows.append(np.sort(np.concatenate([low, high])))
    rows[5] = np.array([D - 1])
    rows[6] = np.arange(D - 40, D)
    rowptr = np.zeros(N + 1, dtype=np.int32)
    rowptr[1:] = np.cumsum([len(x) for x in rows])
    colidx = np.concatenate(rows).astype(np.int32)
    W = synth.make_codebook(D, M, 60, kind="scaled")
    run_and_check(bmu, W, torch.from_numpy(rowptr), torch.from_numpy(colidx), opts_of(bmu, kernel))


def test_vocabulary_beyond_16_bit_ids_takes_the_generic_kernel(bmu):
    D, M, N = 70000, 260, 150
    r = np.random.default_rng(3)
    rows = [np.sort(r.choice(D, size=int(r.integers(0, 50)), replace=False)) for _ in range(N)]
    rows[0] = np.array([D - 1, 65535, 65536, 65024])
    rowptr = np.zeros(N + 1, dtype=np.int32)
    rowptr[1:] = np.cumsum([len(x) for x in rows])
    colidx = np.concatenate(rows).astype(np.int32)
    W = synth.make_codebook(D, M, 61, kind="scaled")
    run_and_check(bmu, W, torch.from_numpy(rowptr), torch.from_numpy(colidx), opts_of(bmu, 0))
    with pytest.raises(bmu.BmuError) as e:
        run_and_check(bmu, W, torch.from_numpy(rowptr), torch.from_numpy(colidx), opts_of(bmu, 6))
    assert e.value.status == 2


@pytest.mark.parametrize("kernel", [2, 5, 7, 8, -1])
def test_unknown_kernel_numbers_are_refused(bmu, kernel):
    rp = torch.tensor([0, 1], dtype=torch.int32).cuda()
    ci = torch.tensor([0], dtype=torch.int32).cuda()
    with pytest.raises(bmu.BmuError) as e:
        bmu.bmu_search_ws(torch.zeros(2048, 1024, device="cuda"), rp, ci, opts=opts_of(bmu, kernel))
    assert e.value.status == 1


@pytest.mark.parametrize("cluster", [3, 4])
@pytest.mark.parametrize("kernel", [3, 4, 6])
@pytest.mark.parametrize("corpus", ["iid", "topical"])
def test_content_clustering_changes_no_result(bmu, cluster, kernel, corpus):
    """Tile membership by content (bmu_opts.cluster = 3, 4) only reorders documents: every
    document is reduced on its own, so any order is valid and the outputs still match the oracle
    -- also on a corpus with topics, where the ordering actually groups documents."""
    cfg = synth.CONFIGS["cfg3"]
    if corpus == "iid":
        rowptr, colidx = synth.make_corpus(cfg, n_docs=2300)
    else:
        rowptr, colidx = synth.make_topical_corpus(cfg, n_docs=2300, n_topics=40)
    W = synth.make_codebook(cfg.D, 768, 17, kind="scaled")
    res = run_and_check(bmu, W, rowptr, colidx, opts_of(bmu, kernel, cluster=cluster, chunk_neurons=512))
    assert res["docs"] == 2300 and res["failed"] == 0
    if kernel == 6:                                        # and with the features ranked by the pass
        run_and_check(bmu, W, rowptr, colidx, opts_of(bmu, 6, cluster=cluster, relabel=1, head_rows=256))


def test_single_slab_codebook(bmu):
    """M = 256: one 256-neuron slab, the smallest codebook the tensor-core sweep takes."""
    cfg = synth.CONFIGS["cfg1"]
    rowptr, colidx = synth.make_corpus(cfg, n_docs=700)
    W = synth.make_codebook(cfg.D, 256, 5, kind="scaled")
    run_and_check(bmu, W, rowptr, colidx, opts_of(bmu, 6))
    W = synth.make_codebook(cfg.D, 256 * 3 + 20, 6, kind="scaled")      # three slabs and a ragged rest
    run_and_check(bmu, W, rowptr, colidx, opts_of(bmu, 6, chunk_neurons=256))
