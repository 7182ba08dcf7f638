"""Seeded random cases: shapes, row-length mixes, codebook kinds and option settings drawn at
random, every kernel (and the half-precision and second-best entry points) held to the oracle
by the same rule as everywhere else.  A kernel may refuse a combination it documents as
unsupported (BMU_ERR_UNSUPPORTED); anything else it returns must be right."""
import random

import numpy as np
import pytest
import torch

import oracle
from tests import parity

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def bmu():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    import paper_2609_05138_b200 as lib
    lib.load()
    return lib


def draw_case(rng):
    D = rng.choice([1, 7, 63, 64, 100, 256, 700, 1024, 3000, 4096, 16384, 65024, 70000])
    M = rng.choice([1, 3, 4, 32, 36, 128, 256, 260, 512, 516, 768, 1024, 1536, 2048, 2052])
    while D * M > 3.5e7:
        M = max(256, M // 2)
    N = rng.choice([1, 2, 7, 8, 9, 127, 128, 129, 255, 257, 600])
    mode = rng.choice(["short", "mixed", "long", "empty-heavy", "repeats", "zipf"])
    g = torch.Generator().manual_seed(rng.randrange(1 << 30))
    if mode == "short":
        lens = torch.randint(0, 6, (N,), generator=g)
    elif mode == "mixed":
        lens = torch.randint(0, 120, (N,), generator=g)
    elif mode == "long":
        lens = torch.randint(0, 500, (N,), generator=g)
    elif mode == "empty-heavy":
        lens = torch.randint(0, 40, (N,), generator=g) * (torch.rand(N, generator=g) < 0.3)
    else:
        lens = torch.randint(1, 90, (N,), generator=g)
    lens = lens.to(torch.int64)
    if mode != "repeats":
        lens = lens.clamp(max=D)
    rows = []
    for n in lens.tolist():
        if mode == "repeats":
            r = torch.randint(0, D, (n,), generator=g)
        elif mode == "zipf":
            p = 1.0 / torch.arange(1, D + 1, dtype=torch.float64)
            r = torch.multinomial(p, min(n, D), replacement=False, generator=g)
        else:
            r = torch.randperm(D, generator=g)[:n]
        rows.append(torch.sort(r).values if rng.random() < 0.7 else r)
    rowptr = torch.zeros(N + 1, dtype=torch.int32)
    rowptr[1:] = torch.cumsum(torch.tensor([len(r) for r in rows]), 0).to(torch.int32)
    colidx = (torch.cat(rows) if int(rowptr[-1]) else torch.zeros(0)).to(torch.int32)
    kind = rng.choice(["uniform", "scaled", "signed", "sparse", "large"])
    W = torch.rand((D, M), generator=g)
    if kind == "scaled":
        W = W * 0.03
    elif kind == "signed":
        W = (W - 0.5) * 0.2
    elif kind == "sparse":
        W = W * (torch.rand((D, M), generator=g) < 0.05)
    elif kind == "large":
        W = W * 1e4
    return rowptr, colidx, W.float().contiguous(), (D, M, N, mode, kind)


def draw_opts(bmu, rng, kernel):
    o = bmu.Opts()
    o.kernel = kernel
    if rng.random() < 0.5:
        o.chunk_neurons = rng.choice([128, 256, 512, 1024])
    if kernel == 6 and rng.random() < 0.6:
        o.head_rows = rng.choice([64, 128, 256, 512, 768, 1024, 2048])
    if kernel == 6:
        o.relabel = rng.choice([0, 1, 2])
        o.repack = rng.choice([0, 2])
    if kernel in (4, 6):
        o.tile_order = rng.choice([0, 1, 2])
    if kernel in (3, 4, 6):
        o.cluster = rng.choice([0, 1, 3, 4])        # document order: by length / and content
    return o


@pytest.mark.parametrize("seed", range(10))
def test_random_cases_against_oracle(bmu, seed):
    rng = random.Random(1000 + seed)
    ran = refused = 0
    for case in range(12):
        rowptr, colidx, W, what = draw_case(rng)
        Wn, rp, ci = W.numpy(), rowptr.numpy(), colidx.numpy()
        nrm = oracle.norms(Wn)
        ref = (nrm,) + tuple(oracle.bmu(Wn, rp, ci, nrm))
        Wd, rpd, cid = W.cuda(), rowptr.cuda(), colidx.cuda()
        for kernel in (0, 1, 3, 4, 6):
            o = draw_opts(bmu, rng, kernel)
            try:
                ob, od = bmu.bmu_search_ws(Wd, rpd, cid, opts=o)
            except bmu.BmuError as e:
                assert e.status == 2, (what, kernel, str(e))
                refused += 1
                continue
            torch.cuda.synchronize()
            parity.compare(ob.cpu().numpy(), od.cpu().numpy(), Wn, rp, ci, cancel_floor=True, ref=ref)
            ran += 1
        D, M = W.shape
        if M >= 2:
            b1, d1, b2, d2 = bmu.bmu_search_top2_ws(Wd, rpd, cid)
            torch.cuda.synchronize()
            parity.compare(b1.cpu().numpy(), d1.cpu().numpy(), Wn, rp, ci, cancel_floor=True, ref=ref)
            assert bool((b2 != b1).all()) and bool((d2 >= d1 - 1e-5 * d1.abs() - 1e-3).all())
            ran += 1
        if M % 256 == 0 and D <= 65024:
            W16 = Wd.half()
            if bool(torch.isfinite(W16).all()):
                W16n = W16.float().cpu().numpy()
                n16 = oracle.norms(W16n)
                ref16 = (n16,) + tuple(oracle.bmu(W16n, rp, ci, n16))
                for kernel in (3, 6):
                    o = bmu.Opts()
                    o.kernel = kernel
                    if kernel == 6 and rng.random() < 0.5:
                        o.head_rows = rng.choice([64, 256, 512, 1024])
                    try:
                        ob, od = bmu.bmu_search_f16_ws(W16, rpd, cid, opts=o)
                    except bmu.BmuError as e:
                        assert e.status == 2, (what, "f16", kernel, str(e))
                        refused += 1
                        continue
                    torch.cuda.synchronize()
                    parity.compare(ob.cpu().numpy(), od.cpu().numpy(), W16n, rp, ci,
                                   cancel_floor=True, ref=ref16)
                    ran += 1
    assert ran >= 24                                   # the generic kernel alone guarantees twelve
