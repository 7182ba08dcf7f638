"""Half-precision codebook (the paper's storage, Section 4.2 / 4.3): the fp16
weights are exact in fp32, so the oracle simply runs on their fp32 copies."""
import numpy as np
import pytest
import torch

import oracle
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


@pytest.mark.parametrize("name,n_docs,M,kind", [("cfg1", 4000, 1024, "uniform"),
                                                ("cfg2", 1500, 4096, "uniform"),
                                                ("cfg5", 700, 2048, "scaled"),
                                                ("cfg1", 900, 512, "signed"),
                                                ("cfg1", 900, 256, "dupes")])
def test_f16_search_matches_oracle(bmu, name, n_docs, M, kind):
    cfg = synth.CONFIGS[name]
    rowptr, colidx = synth.make_corpus(cfg, n_docs=n_docs)
    W16 = synth.make_codebook(cfg.D, M, 50, kind=kind).half()
    W32 = W16.float()                                   # exact widening: what the kernel sees
    norms = bmu.bmu_codebook_norms_f16(W16.cuda())
    ref = oracle.norms(W32.numpy())
    np.testing.assert_allclose(norms.cpu().numpy().astype(np.float64), ref, rtol=6e-8)
    o = bmu.Opts()
    o.chunk_neurons = 512
    ob, od = bmu.bmu_search_f16_ws(W16.cuda(), rowptr.cuda(), colidx.cuda(), opts=o)
    torch.cuda.synchronize()
    parity.compare(ob.cpu().numpy(), od.cpu().numpy(), W32.numpy(), rowptr.numpy(),
                   colidx.numpy())
    # the fp32 kernels on the widened codebook add the same fp32 values in the same order
    o3 = bmu.Opts()
    o3.kernel = 3
    fb, fd = bmu.bmu_search_ws(W32.cuda(), rowptr.cuda(), colidx.cuda(), opts=o3)
    assert torch.equal(ob, fb) and torch.equal(od, fd)
    if kind == "dupes":
        assert int((ob % 2).sum()) == 0


def test_f16_top2_and_limits(bmu):
    cfg = synth.CONFIGS["cfg1"]
    rowptr, colidx = synth.make_corpus(cfg, n_docs=800)
    W16 = synth.make_codebook(cfg.D, 768, 51, kind="scaled").half()
    b1, d1, b2, d2 = bmu.bmu_search_f16_ws(W16.cuda(), rowptr.cuda(), colidx.cuda(), top2=True)
    e1, f1, e2, f2 = oracle.bmu2(W16.float().numpy(), rowptr.numpy(), colidx.numpy())
    clear = (f2 - f1) > 1e-4 * np.abs(f1)
    assert np.array_equal(b1.cpu().numpy()[clear], e1[clear])
    np.testing.assert_allclose(d2.cpu().numpy(), f2, rtol=1e-5)
    with pytest.raises(bmu.BmuError) as e:
        bmu.bmu_search_f16_ws(W16[:, :100].contiguous().cuda(), rowptr.cuda(), colidx.cuda())
    assert e.value.status == 2


@pytest.mark.parametrize("name,n_docs,M,kind,head", [("cfg1", 4000, 1024, "uniform", 0),
                                                     ("cfg3", 1500, 2048, "scaled", 0),
                                                     ("cfg5", 700, 512, "signed", 256),
                                                     ("cfg1", 900, 512, "dupes", 1024),
                                                     ("cfg3", 600, 1024, "scaled", 2048),
                                                     ("cfg2", 500, 512, "uniform", 64)])
def test_f16_tensor_core_sweep_matches_oracle(bmu, name, n_docs, M, kind, head):
    """The wide tensor-core sweep on a half-precision codebook: the weights are fp16 already, so
    the head image has one part and the tail gathers 16-byte pieces."""
    cfg = synth.CONFIGS[name]
    rowptr, colidx = synth.make_corpus(cfg, n_docs=n_docs)
    W16 = synth.make_codebook(cfg.D, M, 52, kind=kind).half()
    W32 = W16.float()
    o = bmu.Opts()
    o.kernel = 6
    o.head_rows = head
    ob, od = bmu.bmu_search_f16_ws(W16.cuda(), rowptr.cuda(), colidx.cuda(), opts=o)
    torch.cuda.synchronize()
    parity.compare(ob.cpu().numpy(), od.cpu().numpy(), W32.numpy(), rowptr.numpy(), colidx.numpy())
    if kind == "dupes":
        assert int((ob % 2).sum()) == 0
    b1, d1, b2, d2 = bmu.bmu_search_f16_ws(W16.cuda(), rowptr.cuda(), colidx.cuda(), opts=o, top2=True)
    assert torch.equal(b1, ob) and torch.equal(d1, od) and bool((b2 != b1).all())


def _csr(rows):
    rowptr = np.zeros(len(rows) + 1, dtype=np.int32)
    rowptr[1:] = np.cumsum([len(r) for r in rows])
    colidx = np.concatenate([np.asarray(r, dtype=np.int32) for r in rows]) if rowptr[-1] else \
        np.zeros(0, dtype=np.int32)
    return torch.from_numpy(rowptr), torch.from_numpy(colidx)


@pytest.mark.parametrize("n_docs", [1, 7, 129, 300])
def test_f16_tensor_core_sweep_ragged_documents(bmu, n_docs):
    """Few documents (less than a block, a block and a bit), rows that are empty, only head ids,
    only gathered ids, one long row, unsorted rows; several chunks of neurons."""
    D, M = 2048, 1536
    r = np.random.default_rng(n_docs)
    rows = []
    for i in range(n_docs):
        kind = i % 5
        if kind == 0:
            rows.append([])
        elif kind == 1:
            rows.append(r.choice(512, size=int(r.integers(1, 40)), replace=False))        # head only
        elif kind == 2:
            rows.append(512 + r.choice(D - 512, size=int(r.integers(1, 40)), replace=False))
        elif kind == 3:
            rows.append(r.permutation(D)[:400])                                            # long, unsorted
        else:
            rows.append(r.choice(D, size=int(r.integers(1, 90)), replace=False))
    rowptr, colidx = _csr(rows)
    W16 = (synth.make_codebook(D, M, 53, kind="scaled")).half()
    o = bmu.Opts()
    o.kernel = 6
    o.chunk_neurons = 512
    ob, od = bmu.bmu_search_f16_ws(W16.cuda(), rowptr.cuda(), colidx.cuda(), opts=o)
    torch.cuda.synchronize()
    parity.compare(ob.cpu().numpy(), od.cpu().numpy(), W16.float().numpy(), rowptr.numpy(),
                   colidx.numpy())
    # one chunk or three: the same bits
    o.chunk_neurons = 1536
    ob1, od1 = bmu.bmu_search_f16_ws(W16.cuda(), rowptr.cuda(), colidx.cuda(), opts=o)
    assert torch.equal(ob, ob1) and torch.equal(od, od1)


def test_f16_tensor_core_sweep_second_best_and_unlabelled_vocabulary(bmu):
    cfg = synth.CONFIGS["cfg3"]
    rowptr, colidx = synth.make_corpus(cfg, n_docs=1200)
    g = torch.Generator().manual_seed(9)
    relabel = torch.randperm(cfg.D, generator=g).to(torch.int32)       # frequent ids anywhere
    colidx = relabel[colidx.long()]
    W16 = synth.make_codebook(cfg.D, 1024, 54, kind="scaled").half()
    o = bmu.Opts()
    o.kernel = 6
    b1, d1, b2, d2 = bmu.bmu_search_f16_ws(W16.cuda(), rowptr.cuda(), colidx.cuda(), opts=o, top2=True)
    torch.cuda.synchronize()
    W32 = W16.float().numpy()
    parity.compare(b1.cpu().numpy(), d1.cpu().numpy(), W32, rowptr.numpy(), colidx.numpy())
    e1, f1, e2, f2 = oracle.bmu2(W32, rowptr.numpy(), colidx.numpy())
    np.testing.assert_allclose(d2.cpu().numpy(), f2, rtol=1e-5)
    clear = (f2 - f1) > 1e-4 * np.abs(f1)
    assert np.array_equal(b1.cpu().numpy()[clear], e1[clear])
    # the second-best index wherever the third-best distance is clearly apart: recompute its
    # distance with the oracle's pair evaluation
    sample = np.arange(0, 1200, 37)
    nrm = oracle.norms(W32)
    for i in sample:
        got = oracle.eval_pair(W32, rowptr.numpy(), colidx.numpy(), nrm, int(i), int(b2[i]))
        assert abs(got - f2[i]) <= 1e-5 * abs(f2[i])
