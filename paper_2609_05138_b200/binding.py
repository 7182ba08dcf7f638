"""ctypes binding of libbmu.so: argument marshalling only.

Every function takes torch tensors (device memory, or pinned host memory where
the name says host), checks dtype/contiguity/device, and passes raw pointers,
sizes and the current CUDA stream to the C entry point of the same name
(include/bmu.h).  No arithmetic happens here and there is no fallback: if the
library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libbmu.so")
_lib = None

STATUS_OK = 0


class BmuError(RuntimeError):
    def __init__(self, status: int, detail: str):
        super().__init__("bmu status %d (%s)" % (status, detail))
        self.status = status


class Opts(ctypes.Structure):
    """Mirror of `bmu_opts` (include/bmu.h); 0 = automatic."""
    _fields_ = [("kernel", ctypes.c_int32), ("chunk_neurons", ctypes.c_int32),
                ("vec", ctypes.c_int32), ("docs_per_warp", ctypes.c_int32),
                ("warps", ctypes.c_int32), ("cluster", ctypes.c_int32),
                ("stage_rows", ctypes.c_int32), ("stages", ctypes.c_int32),
                ("tile_order", ctypes.c_int32), ("tile_head", ctypes.c_int32),
                ("head_rows", ctypes.c_int32), ("repack", ctypes.c_int32),
                ("relabel", ctypes.c_int32), ("reserved", ctypes.c_int32 * 3)]


class SearchDesc(ctypes.Structure):
    """Mirror of `bmu_search_desc` (include/bmu.h)."""
    _fields_ = [("kernel", ctypes.c_int32), ("head_rows", ctypes.c_int32),
                ("slab", ctypes.c_int32), ("docs_per_block", ctypes.c_int32),
                ("repack", ctypes.c_int32), ("sweep_launches", ctypes.c_int32),
                ("ragged_neurons", ctypes.c_int32), ("reserved", ctypes.c_int32),
                ("chunk_neurons", ctypes.c_int64)]


EXPORTS = {
    # name: (restype, argtypes)
    "bmu_status_string": (ctypes.c_char_p, [ctypes.c_int]),
    "bmu_last_error": (ctypes.c_char_p, []),
    "bmu_version": (ctypes.c_int, []),
    "bmu_kernel_launches": (ctypes.c_uint64, []),
    "bmu_describe_search": (ctypes.c_int, [ctypes.c_int64, ctypes.c_int64, ctypes.c_int64,
                                           ctypes.c_int64, ctypes.c_void_p, ctypes.c_void_p]),
    "bmu_codebook_norms": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_int64, ctypes.c_int64,
                                          ctypes.c_void_p, ctypes.c_void_p]),
    "bmu_search_workspace_bytes": (ctypes.c_size_t, [ctypes.c_int64, ctypes.c_int64,
                                                     ctypes.c_int64, ctypes.c_int64,
                                                     ctypes.c_void_p]),
    "bmu_search_ws": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_int64, ctypes.c_int64,
                                     ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                                     ctypes.c_int64, ctypes.c_int64, ctypes.c_void_p,
                                     ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                                     ctypes.c_size_t, ctypes.c_void_p]),
    "bmu_search_top2_workspace_bytes": (ctypes.c_size_t, [ctypes.c_int64, ctypes.c_int64,
                                                          ctypes.c_int64, ctypes.c_int64,
                                                          ctypes.c_void_p]),
    "bmu_search_f16_workspace_bytes": (ctypes.c_size_t, [ctypes.c_int64, ctypes.c_int64,
                                                         ctypes.c_int64, ctypes.c_int64,
                                                         ctypes.c_void_p]),
    "bmu_search_top2_ws": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_int64, ctypes.c_int64,
                                          ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                                          ctypes.c_int64, ctypes.c_int64, ctypes.c_void_p,
                                          ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                                          ctypes.c_void_p, ctypes.c_void_p, ctypes.c_size_t,
                                          ctypes.c_void_p]),
    "bmu_codebook_norms_f16": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_int64, ctypes.c_int64,
                                              ctypes.c_void_p, ctypes.c_void_p]),
    "bmu_search_f16_ws": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_int64, ctypes.c_int64,
                                         ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                                         ctypes.c_int64, ctypes.c_int64, ctypes.c_void_p,
                                         ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                                         ctypes.c_void_p, ctypes.c_void_p, ctypes.c_size_t,
                                         ctypes.c_void_p]),
    "bmu_search": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_int64, ctypes.c_int64,
                                  ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64,
                                  ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]),
    "bmu_search_host": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_int64, ctypes.c_int64,
                                       ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64,
                                       ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]),
    "bmu_search_static": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_int64, ctypes.c_int64,
                                         ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64,
                                         ctypes.c_int64, ctypes.c_void_p, ctypes.c_void_p,
                                         ctypes.c_void_p]),
    "bmu_search_batches_host": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_int64, ctypes.c_int64,
                                               ctypes.c_int32, ctypes.c_void_p, ctypes.c_void_p,
                                               ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                                               ctypes.c_void_p]),
    "bmu_selftest_wait_timeout": (ctypes.c_int, [ctypes.c_void_p]),
    "bmu_status_of_word": (ctypes.c_int, [ctypes.c_uint32]),
    "bmu_last_status": (ctypes.c_int, [ctypes.POINTER(ctypes.c_uint32), ctypes.c_void_p]),
    "bmu_release_scratch": (ctypes.c_int, []),
    "bmu_validate_csr": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64,
                                        ctypes.c_int64, ctypes.c_int64, ctypes.c_void_p]),
    "bmu_plan_workspace_bytes": (ctypes.c_size_t, [ctypes.c_int64, ctypes.c_int64, ctypes.c_int64,
                                                   ctypes.c_int64, ctypes.c_void_p]),
    "bmu_plan_create": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64,
                                       ctypes.c_int64, ctypes.c_int64, ctypes.c_int64,
                                       ctypes.c_void_p, ctypes.c_void_p, ctypes.c_size_t,
                                       ctypes.POINTER(ctypes.c_void_p), ctypes.c_void_p]),
    "bmu_search_planned": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                                          ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]),
    "bmu_plan_order": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]),
    "bmu_plan_destroy": (None, [ctypes.c_void_p]),
    "bmu_update_scatter": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64,
                                          ctypes.c_int64, ctypes.c_void_p, ctypes.c_int64,
                                          ctypes.c_int64, ctypes.c_void_p, ctypes.c_void_p,
                                          ctypes.c_void_p]),
    "bmu_update_blur": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64,
                                       ctypes.c_int32, ctypes.c_int32, ctypes.c_float,
                                       ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]),
    "bmu_update_writeback": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64,
                                            ctypes.c_int64, ctypes.c_void_p, ctypes.c_void_p]),
    "bmu_map_errors_workspace_bytes": (ctypes.c_size_t, []),
    "bmu_map_errors": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                                      ctypes.c_int64, ctypes.c_int32, ctypes.c_int32,
                                      ctypes.c_int32, ctypes.c_void_p, ctypes.c_void_p,
                                      ctypes.c_size_t, ctypes.c_void_p]),
    "bmu_score_block_argmin": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64,
                                              ctypes.c_int64, ctypes.c_void_p, ctypes.c_void_p,
                                              ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]),
    "bmu_measure_roof": (ctypes.c_int, [ctypes.c_int, ctypes.c_void_p, ctypes.c_size_t,
                                        ctypes.c_int, ctypes.POINTER(ctypes.c_double),
                                        ctypes.c_void_p]),
}


def load(path: str | None = None):
    """Loads libbmu.so (raises if it has not been built).  `path` (or the environment
    variable BMU_LIBRARY) names another build of the same library, e.g. the bounds-checked
    one; it must be given on the first call, the library is loaded once per process."""
    global _lib
    if _lib is None:
        path = path or os.environ.get("BMU_LIBRARY") or LIB_PATH
        if not os.path.exists(path):
            raise ImportError(
                "%s is not built: run `python -m paper_2609_05138_b200.build` "
                "(there is no CPU fallback)" % path)
        lib = ctypes.CDLL(path)
        for name, (res, args) in EXPORTS.items():
            fn = getattr(lib, name)
            fn.restype, fn.argtypes = res, args
        _lib = lib
    return _lib


def _check(status: int):
    if status != STATUS_OK:
        lib = load()
        detail = lib.bmu_last_error().decode() or lib.bmu_status_string(status).decode()
        raise BmuError(status, detail)


def _dev(t: torch.Tensor, dtype, name: str):
    if not (isinstance(t, torch.Tensor) and t.is_cuda and t.dtype == dtype and t.is_contiguous()):
        raise TypeError("%s must be a contiguous CUDA tensor of dtype %s" % (name, dtype))
    return t.data_ptr()


def _host(t: torch.Tensor, dtype, name: str):
    if not (isinstance(t, torch.Tensor) and not t.is_cuda and t.dtype == dtype
            and t.is_contiguous()):
        raise TypeError("%s must be a contiguous host tensor of dtype %s" % (name, dtype))
    return t.data_ptr()


def _stream(t: torch.Tensor) -> int:
    return torch.cuda.current_stream(t.device).cuda_stream


def _codebook(W: torch.Tensor):
    if W.dim() != 2:
        raise TypeError("W must be [D, M] (feature-major)")
    return _dev(W, torch.float32, "W"), W.shape[0], W.shape[1]


def bmu_version() -> int:
    return load().bmu_version()


def bmu_codebook_norms(W: torch.Tensor, out: torch.Tensor | None = None) -> torch.Tensor:
    wp, D, M = _codebook(W)
    if out is None:
        out = torch.empty(M, dtype=torch.float32, device=W.device)
    with torch.cuda.device(W.device):
        _check(load().bmu_codebook_norms(wp, D, M, _dev(out, torch.float32, "norms"),
                                         _stream(W)))
    return out


def bmu_search_workspace_bytes(D: int, M: int, N: int, nnz: int, opts: Opts | None = None) -> int:
    return int(load().bmu_search_workspace_bytes(D, M, N, nnz,
                                                 ctypes.byref(opts) if opts else None))


def bmu_search_ws(W, rowptr, colidx, norms=None, opts: Opts | None = None, workspace=None,
                  out_bmu=None, out_dist=None):
    """Search with caller-owned scratch.  Returns (out_bmu int32 [N], out_dist float32 [N])."""
    wp, D, M = _codebook(W)
    N = rowptr.numel() - 1
    nnz = colidx.numel()
    if out_bmu is None:
        out_bmu = torch.empty(N, dtype=torch.int32, device=W.device)
    if out_dist is None:
        out_dist = torch.empty(N, dtype=torch.float32, device=W.device)
    need = bmu_search_workspace_bytes(D, M, N, nnz, opts)
    if workspace is None:
        workspace = torch.empty(need + 256, dtype=torch.uint8, device=W.device)
    ws_ptr = (workspace.data_ptr() + 255) // 256 * 256
    ws_bytes = workspace.numel() * workspace.element_size() - (ws_ptr - workspace.data_ptr())
    with torch.cuda.device(W.device):
        _check(load().bmu_search_ws(
            wp, D, M, _dev(norms, torch.float32, "norms") if norms is not None else None,
            _dev(rowptr, torch.int32, "rowptr"),
            _dev(colidx, torch.int32, "colidx") if nnz else None, N, nnz,
            _dev(out_bmu, torch.int32, "out_bmu"), _dev(out_dist, torch.float32, "out_dist"),
            ctypes.byref(opts) if opts else None, ws_ptr, ws_bytes, _stream(W)))
    return out_bmu, out_dist


def bmu_search_top2_ws(W, rowptr, colidx, norms=None, opts: Opts | None = None, workspace=None):
    """Best and second-best unit.  Returns (out_bmu, out_dist, out_bmu2, out_dist2)."""
    wp, D, M = _codebook(W)
    N = rowptr.numel() - 1
    nnz = colidx.numel()
    ob = torch.empty(N, dtype=torch.int32, device=W.device)
    od = torch.empty(N, dtype=torch.float32, device=W.device)
    ob2 = torch.empty(N, dtype=torch.int32, device=W.device)
    od2 = torch.empty(N, dtype=torch.float32, device=W.device)
    need = int(load().bmu_search_top2_workspace_bytes(D, M, N, nnz,
                                                      ctypes.byref(opts) if opts else None))
    ws = workspace if workspace is not None else torch.empty(need + 256, dtype=torch.uint8,
                                                             device=W.device)
    ws_ptr = (ws.data_ptr() + 255) // 256 * 256
    if ws_ptr + need > ws.data_ptr() + ws.numel():
        raise ValueError("workspace too small: need %d bytes after alignment" % need)
    with torch.cuda.device(W.device):
        _check(load().bmu_search_top2_ws(
            wp, D, M, _dev(norms, torch.float32, "norms") if norms is not None else None,
            _dev(rowptr, torch.int32, "rowptr"),
            _dev(colidx, torch.int32, "colidx") if nnz else None, N, nnz,
            ob.data_ptr(), od.data_ptr(), ob2.data_ptr(), od2.data_ptr(),
            ctypes.byref(opts) if opts else None, ws_ptr, need, _stream(W)))
    return ob, od, ob2, od2


def bmu_codebook_norms_f16(W16: torch.Tensor) -> torch.Tensor:
    D, M = W16.shape
    out = torch.empty(M, dtype=torch.float32, device=W16.device)
    with torch.cuda.device(W16.device):
        _check(load().bmu_codebook_norms_f16(_dev(W16, torch.float16, "W16"), D, M,
                                             out.data_ptr(), _stream(W16)))
    return out


def bmu_search_f16_ws(W16, rowptr, colidx, norms=None, opts: Opts | None = None, top2=False,
                      workspace=None):
    """Search against an fp16 codebook [D, M].  Returns (bmu, dist) or, with top2,
    (bmu, dist, bmu2, dist2)."""
    D, M = W16.shape
    N = rowptr.numel() - 1
    nnz = colidx.numel()
    dev = W16.device
    ob = torch.empty(N, dtype=torch.int32, device=dev)
    od = torch.empty(N, dtype=torch.float32, device=dev)
    ob2 = torch.empty(N, dtype=torch.int32, device=dev) if top2 else None
    od2 = torch.empty(N, dtype=torch.float32, device=dev) if top2 else None
    need = int(load().bmu_search_f16_workspace_bytes(D, M, N, nnz,
                                                     ctypes.byref(opts) if opts else None))
    ws = workspace if workspace is not None else torch.empty(need + 256, dtype=torch.uint8,
                                                             device=dev)
    ws_ptr = (ws.data_ptr() + 255) // 256 * 256
    with torch.cuda.device(dev):
        _check(load().bmu_search_f16_ws(
            _dev(W16, torch.float16, "W16"), D, M,
            _dev(norms, torch.float32, "norms") if norms is not None else None,
            _dev(rowptr, torch.int32, "rowptr"),
            _dev(colidx, torch.int32, "colidx") if nnz else None, N, nnz,
            ob.data_ptr(), od.data_ptr(), ob2.data_ptr() if top2 else None,
            od2.data_ptr() if top2 else None, ctypes.byref(opts) if opts else None,
            ws_ptr, ws.numel() - (ws_ptr - ws.data_ptr()), _stream(W16)))
    return (ob, od, ob2, od2) if top2 else (ob, od)


def bmu_search(W, rowptr, colidx, out_bmu=None, out_dist=None):
    """One-shot search (library-owned scratch).  Returns (out_bmu, out_dist)."""
    wp, D, M = _codebook(W)
    N = rowptr.numel() - 1
    if out_bmu is None:
        out_bmu = torch.empty(N, dtype=torch.int32, device=W.device)
    if out_dist is None:
        out_dist = torch.empty(N, dtype=torch.float32, device=W.device)
    with torch.cuda.device(W.device):
        _check(load().bmu_search(
            wp, D, M, _dev(rowptr, torch.int32, "rowptr"),
            _dev(colidx, torch.int32, "colidx") if colidx.numel() else None, N,
            _dev(out_bmu, torch.int32, "out_bmu"), _dev(out_dist, torch.float32, "out_dist"),
            _stream(W)))
    return out_bmu, out_dist


def bmu_search_static(W, rowptr, colidx, out_bmu, out_dist):
    """Search for callers that cannot allocate: the scratch is an 8 MiB array inside
    the library, so the sizes are limited (see include/bmu.h) and overlapping calls on
    one device race.  The caller passes the outputs; nothing is allocated here either."""
    wp, D, M = _codebook(W)
    N = rowptr.numel() - 1
    with torch.cuda.device(W.device):
        _check(load().bmu_search_static(
            wp, D, M, _dev(rowptr, torch.int32, "rowptr"),
            _dev(colidx, torch.int32, "colidx") if colidx.numel() else None, N, colidx.numel(),
            _dev(out_bmu, torch.int32, "out_bmu"), _dev(out_dist, torch.float32, "out_dist"),
            _stream(W)))
    return out_bmu, out_dist


def bmu_search_host(W, rowptr_host, colidx_host, out_bmu_host=None, out_dist_host=None):
    """End-to-end search of a host-resident CSR batch against a device codebook."""
    wp, D, M = _codebook(W)
    N = rowptr_host.numel() - 1
    if out_bmu_host is None:
        out_bmu_host = torch.empty(N, dtype=torch.int32).pin_memory()
    if out_dist_host is None:
        out_dist_host = torch.empty(N, dtype=torch.float32).pin_memory()
    with torch.cuda.device(W.device):
        _check(load().bmu_search_host(
            wp, D, M, _host(rowptr_host, torch.int32, "rowptr_host"),
            _host(colidx_host, torch.int32, "colidx_host") if colidx_host.numel() else None, N,
            _host(out_bmu_host, torch.int32, "out_bmu_host"),
            _host(out_dist_host, torch.float32, "out_dist_host"), _stream(W)))
    return out_bmu_host, out_dist_host


def bmu_search_batches_host(W, batches, outs=None):
    """Streams host-resident CSR batches [(rowptr_host, colidx_host), ...] through the
    search with copy/compute overlap.  Returns [(out_bmu_host, out_dist_host), ...]."""
    wp, D, M = _codebook(W)
    nb = len(batches)
    if outs is None:
        outs = [(torch.empty(rp.numel() - 1, dtype=torch.int32).pin_memory(),
                 torch.empty(rp.numel() - 1, dtype=torch.float32).pin_memory())
                for rp, _ in batches]
    PtrArr = ctypes.c_void_p * nb
    rps = PtrArr(*[_host(rp, torch.int32, "rowptr_host") for rp, _ in batches])
    cis = PtrArr(*[_host(ci, torch.int32, "colidx_host") if ci.numel() else None
                   for _, ci in batches])
    obs = PtrArr(*[_host(ob, torch.int32, "out_bmu_host") for ob, _ in outs])
    ods = PtrArr(*[_host(od, torch.float32, "out_dist_host") for _, od in outs])
    ns = (ctypes.c_int64 * nb)(*[rp.numel() - 1 for rp, _ in batches])
    with torch.cuda.device(W.device):
        _check(load().bmu_search_batches_host(wp, D, M, nb, rps, cis, ns, obs, ods, _stream(W)))
    return outs


def bmu_kernel_launches() -> int:
    return int(load().bmu_kernel_launches())


def bmu_describe_search(D: int, M: int, N: int, nnz: int, opts: Opts | None = None,
                        device=None) -> SearchDesc:
    """The kernel, chunking and launch count bmu_search_ws would use on `device`."""
    d = SearchDesc()
    with torch.cuda.device(torch.device("cuda" if device is None else device)):
        _check(load().bmu_describe_search(D, M, N, nnz, ctypes.byref(opts) if opts else None,
                                          ctypes.byref(d)))
    return d


def bmu_last_status(device=None):
    """(status, word): the status word of the last one-shot search on `device`."""
    device = torch.device("cuda" if device is None else device)
    w = ctypes.c_uint32(0)
    with torch.cuda.device(device):
        rc = int(load().bmu_last_status(ctypes.byref(w), torch.cuda.current_stream(device).cuda_stream))
    return rc, int(w.value)


def bmu_selftest_wait_timeout(device=None) -> int:
    """Runs the bounded-wait self-test; returns the status (5 = BMU_ERR_TIMEOUT expected)."""
    device = torch.device("cuda" if device is None else device)
    with torch.cuda.device(device):
        return int(load().bmu_selftest_wait_timeout(torch.cuda.current_stream(device).cuda_stream))


def bmu_release_scratch():
    _check(load().bmu_release_scratch())


def bmu_validate_csr(rowptr, colidx, D: int):
    N = rowptr.numel() - 1
    with torch.cuda.device(rowptr.device):
        _check(load().bmu_validate_csr(
            _dev(rowptr, torch.int32, "rowptr"),
            _dev(colidx, torch.int32, "colidx") if colidx.numel() else None, N, colidx.numel(),
            D, _stream(rowptr)))


class Plan:
    """A tiling plan of one corpus batch for a codebook shape (bmu_plan_create); keeps the
    tensors it refers to alive."""

    def __init__(self, rowptr, colidx, D: int, M: int, opts: Opts | None = None):
        self.rowptr, self.colidx, self.D, self.M, self.opts = rowptr, colidx, D, M, opts
        self.N = rowptr.numel() - 1
        nnz = colidx.numel()
        op = ctypes.byref(opts) if opts else None
        need = int(load().bmu_plan_workspace_bytes(self.N, nnz, D, M, op))
        self.workspace = torch.empty(need + 256, dtype=torch.uint8, device=rowptr.device)
        ws_ptr = (self.workspace.data_ptr() + 255) // 256 * 256
        handle = ctypes.c_void_p()
        with torch.cuda.device(rowptr.device):
            _check(load().bmu_plan_create(
                _dev(rowptr, torch.int32, "rowptr"),
                _dev(colidx, torch.int32, "colidx") if nnz else None, self.N, nnz, D, M, op,
                ws_ptr, need, ctypes.byref(handle), _stream(rowptr)))
        self.handle = handle

    def search(self, W, norms=None, out_bmu=None, out_dist=None):
        wp, D, M = _codebook(W)
        if (D, M) != (self.D, self.M):
            raise ValueError("codebook shape differs from the plan's")
        if out_bmu is None:
            out_bmu = torch.empty(self.N, dtype=torch.int32, device=W.device)
        if out_dist is None:
            out_dist = torch.empty(self.N, dtype=torch.float32, device=W.device)
        with torch.cuda.device(W.device):
            _check(load().bmu_search_planned(
                self.handle, wp, _dev(norms, torch.float32, "norms") if norms is not None else None,
                _dev(out_bmu, torch.int32, "out_bmu"), _dev(out_dist, torch.float32, "out_dist"),
                _stream(W)))
        return out_bmu, out_dist

    def order(self):
        """The planned order: int32 [N], the document at each planned position."""
        out = torch.empty(self.N, dtype=torch.int32, device=self.rowptr.device)
        with torch.cuda.device(self.rowptr.device):
            _check(load().bmu_plan_order(self.handle, out.data_ptr(), _stream(self.rowptr)))
        return out

    def close(self):
        if self.handle:
            load().bmu_plan_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


# ---- the rest of a batch epoch: scatter, blur, write-back (Table 4) ----------
def bmu_update_scatter(rowptr, colidx, bmu, num, cnt):
    """Adds this batch to the integer accumulators num uint32 [D, M] and cnt uint32 [M]."""
    D, M = num.shape
    N = rowptr.numel() - 1
    nnz = colidx.numel()
    for t, name in ((num, "num"), (cnt, "cnt")):
        if t.dtype not in (torch.uint32, torch.int32) or not t.is_cuda or not t.is_contiguous():
            raise ValueError("%s must be a contiguous CUDA uint32 (or int32) tensor" % name)
    with torch.cuda.device(num.device):
        _check(load().bmu_update_scatter(
            _dev(rowptr, torch.int32, "rowptr"),
            _dev(colidx, torch.int32, "colidx") if nnz else None, N, nnz,
            _dev(bmu, torch.int32, "bmu"), D, M, num.data_ptr(), cnt.data_ptr(), _stream(num)))


def bmu_update_blur(num, cnt, edge_x: int, edge_y: int, sigma: float):
    """Neighbourhood-weighted sums of the accumulators: (num_blur float32 [D, M], cnt_blur [M])."""
    D, M = num.shape
    if edge_x * edge_y != M:
        raise ValueError("edge_x * edge_y must equal M")
    nb = torch.empty((D, M), dtype=torch.float32, device=num.device)
    cb = torch.empty(M, dtype=torch.float32, device=num.device)
    with torch.cuda.device(num.device):
        _check(load().bmu_update_blur(num.data_ptr(), cnt.data_ptr(), D, edge_x, edge_y,
                                      float(sigma), nb.data_ptr(), cb.data_ptr(), _stream(num)))
    return nb, cb


def bmu_update_writeback(num_blur, cnt_blur, W):
    """W[f, j] = num_blur[f, j] / cnt_blur[j] where cnt_blur[j] > 0 (in place)."""
    wp, D, M = _codebook(W)
    with torch.cuda.device(W.device):
        _check(load().bmu_update_writeback(_dev(num_blur, torch.float32, "num_blur"),
                                           _dev(cnt_blur, torch.float32, "cnt_blur"), D, M, wp,
                                           _stream(W)))
    return W


def bmu_map_errors(bmu, bmu2, dist, edge_x: int, edge_y: int, adjacency: int = 4) -> torch.Tensor:
    """Device tensor of three float64: mean squared quantisation error, mean quantisation
    error, topographic error of a search with second-best units."""
    N = bmu.numel()
    dev = dist.device
    out = torch.empty(3, dtype=torch.float64, device=dev)
    need = int(load().bmu_map_errors_workspace_bytes())
    ws = torch.empty(need + 256, dtype=torch.uint8, device=dev)
    ws_ptr = (ws.data_ptr() + 255) // 256 * 256
    with torch.cuda.device(dev):
        _check(load().bmu_map_errors(_dev(bmu, torch.int32, "bmu") if N else None,
                                     _dev(bmu2, torch.int32, "bmu2") if N else None,
                                     _dev(dist, torch.float32, "dist") if N else None, N,
                                     int(edge_x), int(edge_y), int(adjacency), out.data_ptr(),
                                     ws_ptr, need, _stream(dist)))
    return out


def bmu_score_block_argmin(scores, norms, rowptr, out_bmu=None, out_dist=None):
    """Arg-min read-back over a materialised [n_rows, M] score block (fp32 or fp16)."""
    if scores.dim() != 2 or scores.dtype not in (torch.float32, torch.float16):
        raise TypeError("scores must be [n_rows, M] fp32 or fp16")
    n, M = scores.shape
    _dev(scores, scores.dtype, "scores")
    if rowptr.numel() != n + 1:
        raise ValueError("rowptr must have n_rows + 1 entries")
    if out_bmu is None:
        out_bmu = torch.empty(n, dtype=torch.int32, device=scores.device)
    if out_dist is None:
        out_dist = torch.empty(n, dtype=torch.float32, device=scores.device)
    with torch.cuda.device(scores.device):
        _check(load().bmu_score_block_argmin(
            scores.data_ptr(), int(scores.dtype == torch.float16), n, M,
            _dev(norms, torch.float32, "norms"), _dev(rowptr, torch.int32, "rowptr"),
            _dev(out_bmu, torch.int32, "out_bmu"), _dev(out_dist, torch.float32, "out_dist"),
            _stream(scores)))
    return out_bmu, out_dist


ROOFS = {"l2_ldg": 0, "l2_bulk": 1, "smem": 2, "l1": 3, "fadd": 4, "fadd2": 5, "l2_mixed": 6}


def bmu_measure_roof(which: str, footprint_bytes: int = 32 << 20, piece: int = 2048,
                     device=None) -> float:
    """One on-chip ceiling of the device, measured now (bytes/s or adds/s)."""
    device = torch.device("cuda" if device is None else device)
    buf = torch.empty(footprint_bytes + 512, dtype=torch.uint8, device=device)
    ptr = (buf.data_ptr() + 255) // 256 * 256
    out = ctypes.c_double(0.0)
    with torch.cuda.device(device):
        _check(load().bmu_measure_roof(ROOFS[which], ptr, footprint_bytes, piece,
                                       ctypes.byref(out),
                                       torch.cuda.current_stream(device).cuda_stream))
    return out.value
