"""The materialised-score route (Section 3: library sparse-dense product into a score block,
then an arg-min read-back; Section 4.4: the read-back tuned to a warp per row with vector
loads): bmu_score_block_argmin against the oracle, through the C ABI, under the rule of every
other parity test."""
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


def score_block(W, rowptr, colidx, dtype=torch.float32):
    """Library SpMM (test-side stand-in for the comparison system's first half)."""
    rp = rowptr.to(torch.int64).cuda()
    ci = colidx.to(torch.int64).cuda()
    X = torch.sparse_csr_tensor(rp, ci, torch.ones(ci.numel(), device="cuda"),
                                size=(rowptr.numel() - 1, W.shape[0]))
    return (X @ W.cuda()).to(dtype).contiguous()


@pytest.mark.parametrize("name,n_docs,M", [("cfg1", 3000, 1024), ("cfg2", 900, 4096),
                                           ("cfg3", 257, 16384), ("cfg1", 31, 8)])
@pytest.mark.parametrize("kind", ["uniform", "scaled", "dupes"])
def test_fp32_score_block_readback_matches_oracle(bmu, name, n_docs, M, kind):
    cfg = synth.CONFIGS[name]
    rowptr, colidx = synth.make_corpus(cfg, n_docs=n_docs)
    W = synth.make_codebook(cfg.D, M, 3, kind=kind)
    S = score_block(W, rowptr, colidx)
    norms = bmu.bmu_codebook_norms(W.cuda())
    ob, od = bmu.bmu_score_block_argmin(S, norms, rowptr.cuda())
    torch.cuda.synchronize()
    res = parity.compare(ob.cpu().numpy(), od.cpu().numpy(), W.numpy(), rowptr.numpy(), colidx.numpy())
    assert res["docs"] == n_docs and res["failed"] == 0
    if kind == "dupes":
        assert int((ob % 2).sum()) == 0                 # equal columns: the lower index wins


@pytest.mark.parametrize("M", [8, 1000, 4096 + 8])
def test_fp16_score_block_readback_matches_oracle(bmu, M):
    """Weights on a 1/64 grid and rows of at most 16 ids: every score is exact in fp16, so the
    fp16 block holds the very sums the oracle forms and the usual rule applies."""
    D, N = 500, 700
    r = np.random.default_rng(M)
    W = torch.from_numpy((r.integers(0, 64, size=(D, M)) / 64.0).astype(np.float32))
    rows = [np.sort(r.choice(D, size=int(r.integers(0, 17)), replace=False)) for _ in range(N)]
    rowptr = np.zeros(N + 1, dtype=np.int32)
    rowptr[1:] = np.cumsum([len(x) for x in rows])
    colidx = np.concatenate(rows).astype(np.int32)
    S32 = score_block(W, torch.from_numpy(rowptr), torch.from_numpy(colidx))
    S16 = S32.half()
    assert torch.equal(S16.float(), S32)                # nothing was rounded
    norms = bmu.bmu_codebook_norms(W.cuda())
    ob, od = bmu.bmu_score_block_argmin(S16, norms, torch.from_numpy(rowptr).cuda())
    torch.cuda.synchronize()
    res = parity.compare(ob.cpu().numpy(), od.cpu().numpy(), W.numpy(), rowptr, colidx)
    assert res["failed"] == 0
    ob32, od32 = bmu.bmu_score_block_argmin(S32, norms, torch.from_numpy(rowptr).cuda())
    assert torch.equal(ob, ob32) and torch.equal(od, od32)


def test_readback_refuses_what_it_cannot_do(bmu):
    S = torch.zeros(4, 6, device="cuda")
    n = torch.zeros(8, device="cuda")
    rp = torch.zeros(5, dtype=torch.int32, device="cuda")
    with pytest.raises(bmu.BmuError) as e:
        bmu.bmu_score_block_argmin(S, n, rp)
    assert e.value.status == 2
