"""The synthetic corpus generator: structure and the distribution facts the
design relies on (row sizes, distinct ascending ids, Zipf head mass)."""
import numpy as np
import torch

from inputs import synth


def test_rows_are_distinct_ascending_and_sized():
    cfg = synth.CONFIGS["cfg1"]
    rowptr, colidx = synth.make_corpus(cfg, n_docs=3000)
    rp, ci = rowptr.numpy(), colidx.numpy()
    assert rp.dtype == np.int32 and ci.dtype == np.int32 and rp[0] == 0
    lens = np.diff(rp)
    assert lens.min() >= 1 and abs(lens.mean() - 64) < 1.0
    assert ci.min() >= 0 and ci.max() < cfg.D
    inner = np.ones(ci.size, dtype=bool)
    inner[rp[1:-1]] = False                       # first entry of every row but row 0
    assert np.all(np.diff(ci)[inner[1:]] > 0)


def test_seeded_and_batches_differ():
    cfg = synth.CONFIGS["cfg5"]
    a = synth.make_corpus(cfg, batch=2, n_docs=500)
    b = synth.make_corpus(cfg, batch=2, n_docs=500)
    c = synth.make_corpus(cfg, batch=3, n_docs=500)
    assert torch.equal(a[0], b[0]) and torch.equal(a[1], b[1])
    assert not torch.equal(a[0], c[0])
    lens = (a[0][1:] - a[0][:-1])
    assert lens.min() >= 1 and lens.max() <= 400
    assert synth.num_batches(cfg) == 27 and synth.batch_size(cfg) == 1_000_000


def test_zipf_head_mass_cfg4():
    cfg = synth.CONFIGS["cfg4"]
    n = 20000
    rowptr, colidx = synth.make_corpus(cfg, n_docs=n)
    inc = torch.bincount(colidx.long(), minlength=cfg.D).double() / n
    assert inc[0] > 0.99 and abs(inc[15] - 0.59) < 0.03 and abs(inc[127] - 0.086) < 0.01
    share = inc.cumsum(0) / inc.sum()
    assert abs(share[127] - 0.445) < 0.02 and abs(share[1023] - 0.71) < 0.02


def test_dense_rows_and_codebook_kinds():
    nnz = torch.tensor([1, 5, 8, 8])
    rowptr, colidx = synth.draw_corpus(4, 8, 1.0, nnz, seed=9)
    assert rowptr.tolist() == [0, 1, 6, 14, 22]
    assert colidx[6:14].tolist() == list(range(8))
    W = synth.make_codebook(16, 8, 1, kind="dupes")
    assert torch.equal(W[:, 0], W[:, 1]) and W.dtype == torch.float32 and W.shape == (16, 8)
    assert synth.make_codebook(4, 4, 1).max() < 1.0
