"""Child process of tests/test_gpu_bounds_checked.py: runs with BMU_LIBRARY pointing at the
bounds-checked build of the library (every id- and offset-derived address checked, violations
recorded in the status word instead of performed) and prints one JSON line."""
import json
import sys

import numpy as np
import torch

from inputs import synth
from tests import parity
import paper_2609_05138_b200 as bmu


def compare(*args):
    """parity.compare, with a failure turned into a count so that every case is reported"""
    try:
        return parity.compare(*args)
    except AssertionError as e:
        return {"docs": -1, "failed": 1, "detail": str(e)[:300]}


def status_word(ws):
    off = (-ws.data_ptr()) % 256
    return int(ws[off:off + 4].view(torch.int32)[0]) & 0xffffffff


def search(W, rp, ci, o, top2=False):
    D, M = W.shape
    N, nnz = rp.numel() - 1, ci.numel()
    need = max(bmu.bmu_search_workspace_bytes(D, M, N, nnz, o),
               int(bmu.load().bmu_search_top2_workspace_bytes(D, M, N, nnz, None)) * 2)
    ws = torch.zeros(need + 256, dtype=torch.uint8, device="cuda")
    if top2:
        out = bmu.bmu_search_top2_ws(W, rp, ci, opts=o, workspace=ws)
    else:
        out = bmu.bmu_search_ws(W, rp, ci, opts=o, workspace=ws)
    torch.cuda.synchronize()
    return out, status_word(ws)


def main():
    bmu.load()
    res = {"library": bmu.binding.load()._name, "clean": [], "flagged": []}
    cfg = synth.CONFIGS["cfg1"]
    rowptr, colidx = synth.make_corpus(cfg, n_docs=1500)
    rp, ci = rowptr.cuda(), colidx.cuda()
    for kernel, M, kw in ((1, 1000, {}), (3, 1024, {}), (4, 1024, {}), (6, 1024, {}),
                          (6, 1024 + 36, {"head_rows": 256, "chunk_neurons": 512, "relabel": 1}),
                          (6, 1024, {"tile_order": 2, "repack": 2})):
        W = synth.make_codebook(cfg.D, M, 40 + kernel, kind="scaled")
        o = bmu.Opts()
        o.kernel = kernel
        for k, v in kw.items():
            setattr(o, k, v)
        (ob, od), st = search(W.cuda(), rp, ci, o)
        r = compare(ob.cpu().numpy(), od.cpu().numpy(), W.numpy(), rowptr.numpy(), colidx.numpy())
        res["clean"].append({"kernel": kernel, "M": M, "status": st, "failed": r["failed"],
                             "docs": r["docs"], "detail": r.get("detail")})
    # second-best unit and the half-precision codebook through the tensor-core sweep
    W = synth.make_codebook(cfg.D, 1024, 7, kind="scaled")
    o = bmu.Opts()
    o.kernel = 6
    (b1, d1, b2, d2), st = search(W.cuda(), rp, ci, o, top2=True)
    r = compare(b1.cpu().numpy(), d1.cpu().numpy(), W.numpy(), rowptr.numpy(), colidx.numpy())
    res["clean"].append({"kernel": "6 top2", "M": 1024, "status": st, "failed": r["failed"], "docs": r["docs"]})
    W16 = W.cuda().half()
    ob, od = bmu.bmu_search_f16_ws(W16, rp, ci, opts=o)
    torch.cuda.synchronize()
    r = compare(ob.cpu().numpy(), od.cpu().numpy(), W16.float().cpu().numpy(), rowptr.numpy(),
                       colidx.numpy())
    res["clean"].append({"kernel": "6 f16", "M": 1024, "status": 0, "failed": r["failed"], "docs": r["docs"]})

    # an id beyond the vocabulary: the checked build records it and leaves the access out.  The
    # codebook sits at the start of a larger allocation, so nothing here can leave memory that
    # the test owns.
    D, M = 3000, 1024
    big = torch.rand(D + 64, M, device="cuda")
    Wd = big[:D]
    bad = colidx.clone() % D
    bad[17] = D + 5
    for kernel in (1, 3, 4, 6):
        o = bmu.Opts()
        o.kernel = kernel
        _, st = search(Wd, rp, bad.cuda(), o)
        res["flagged"].append({"kernel": kernel, "status": st})
    # the context is still usable and a clean search still passes
    o = bmu.Opts()
    o.kernel = 6
    (ob, od), st = search(W.cuda(), rp, ci, o)
    r = compare(ob.cpu().numpy(), od.cpu().numpy(), W.numpy(), rowptr.numpy(), colidx.numpy())
    res["after"] = {"status": st, "failed": r["failed"]}
    print(json.dumps(res))


if __name__ == "__main__":
    sys.exit(main())
