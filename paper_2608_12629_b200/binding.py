"""ctypes binding of libcake_kmeans.so: argument marshalling only.

Each function has the name of the C entry point it calls (see include/cake_kmeans.h); every step
of the path runs in the library's CUDA kernels.  PyTorch supplies device memory and the stream.
There is no fallback of any kind: if the library is missing or the device is not a B200-class GPU
the call raises.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libcake_kmeans.so")

CAKE_OK = 0
CAKE_ERR_NULL, CAKE_ERR_SHAPE, CAKE_ERR_ALIGN, CAKE_ERR_UNSUPPORTED = -1, -2, -3, -4
CAKE_ERR_WORKSPACE, CAKE_ERR_CUDA, CAKE_ERR_BAD_INDEX, CAKE_ERR_TIMEOUT, CAKE_ERR_DEVICE = -5, -6, -7, -8, -9
CAKE_ASSIGN_AUTO, CAKE_ASSIGN_TCGEN05, CAKE_ASSIGN_SIMT, CAKE_ASSIGN_TCGEN05_EXACT = 0, 1, 2, 3
CAKE_ASSIGN_TCGEN05_PAIR, CAKE_ASSIGN_TCGEN05_PAIR_EXACT = 4, 5
CAKE_UPDATE_AUTO, CAKE_UPDATE_SMEM, CAKE_UPDATE_SORT = 0, 1 << 4, 2 << 4
CAKE_UPDATE_SLAB, CAKE_UPDATE_SLAB_F1, CAKE_UPDATE_SLAB_F2, CAKE_UPDATE_SLAB_F4 = 3 << 4, 4 << 4, 5 << 4, 6 << 4
CAKE_LLOYD_NO_FUSE = 1 << 8
CAKE_LLOYD_NO_RESIDENT = 1 << 9

EXPORTS = [
    "cake_version", "cake_kmeans_kernel_launches", "cake_strerror", "cake_kmeans_workspace_bytes", "cake_kmeans_assign",
    "cake_kmeans_assign_batched", "cake_kmeans_update", "cake_kmeans_update_batched", "cake_kmeans_lloyd",
    "cake_kmeans_lloyd_batched", "cake_kmeans_lloyd_host_device_bytes", "cake_kmeans_lloyd_host",
    "cake_kmeans_device_status", "cake_kmeans_selftest_bounded_wait", "cake_kmeans_assign_static",
    "cake_kmeans_update_partial_batched", "cake_kmeans_update_finish_batched", "cake_kmeans_inertia_batched",
    "cake_kmeans_assign_static_status", "cake_knn_workspace_bytes", "cake_knn_search",
    "cake_kmeans_lloyd_tol", "cake_kmeans_init_plusplus", "cake_kmeans_lloyd_sharded",
]

# int (*)(void* user, float* sums, long long n_sums, int* counts, long long n_counts, cake_stream_t stream)
ALLREDUCE_FN = ctypes.CFUNCTYPE(ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_longlong, ctypes.c_void_p,
                                ctypes.c_longlong, ctypes.c_void_p)

_lib = None


class CakeError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {strerror(code)} ({code})")


def lib() -> ctypes.CDLL:
    """The loaded C-ABI library. Raises if it has not been built (python -m paper_2608_12629_b200.build)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2608_12629_b200.build`; "
                               "there is no fallback path")
        L = ctypes.CDLL(LIB_PATH)
        vp, ll, i, u, sz = ctypes.c_void_p, ctypes.c_longlong, ctypes.c_int, ctypes.c_uint, ctypes.c_size_t
        L.cake_version.restype = i
        L.cake_strerror.restype = ctypes.c_char_p
        L.cake_strerror.argtypes = [i]
        L.cake_kmeans_workspace_bytes.argtypes = [ll, ll, i, i, ctypes.POINTER(sz)]
        L.cake_kmeans_assign.argtypes = [vp, vp, ll, i, i, vp, vp, vp, sz, vp, u]
        L.cake_kmeans_assign_batched.argtypes = [vp, vp, ll, ll, i, i, vp, vp, vp, sz, vp, u]
        L.cake_kmeans_update.argtypes = [vp, vp, ll, i, i, vp, vp, vp, vp, vp, sz, vp, u]
        L.cake_kmeans_update_batched.argtypes = [vp, vp, ll, ll, i, i, vp, vp, vp, vp, vp, sz, vp, u]
        L.cake_kmeans_lloyd.argtypes = [vp, vp, ll, i, i, i, vp, vp, vp, vp, vp, vp, vp, sz, vp, u]
        L.cake_kmeans_lloyd_batched.argtypes = [vp, vp, ll, ll, i, i, i, vp, vp, vp, vp, vp, vp, vp, sz, vp, u]
        L.cake_kmeans_lloyd_host_device_bytes.argtypes = [ll, ll, i, i, i, ctypes.POINTER(sz)]
        L.cake_kmeans_lloyd_host.argtypes = [vp, vp, ll, ll, i, i, i, vp, vp, vp, vp, vp, vp, vp, sz, vp, u]
        L.cake_kmeans_device_status.argtypes = [vp, vp, ctypes.POINTER(i)]
        L.cake_kmeans_selftest_bounded_wait.argtypes = [vp, sz, i, vp]
        L.cake_kmeans_assign_static.argtypes = [vp, vp, ll, i, i, vp, vp, vp]
        L.cake_kmeans_assign_static_status.argtypes = [vp, ctypes.POINTER(i)]
        L.cake_knn_workspace_bytes.argtypes = [ll, ll, i, i, ctypes.POINTER(sz)]
        L.cake_knn_search.argtypes = [vp, vp, ll, ll, i, i, vp, vp, vp, sz, vp]
        L.cake_kmeans_lloyd_tol.argtypes = [vp, vp, ll, i, i, i, ctypes.c_double, i, vp, vp, vp, vp, vp, vp,
                                            ctypes.POINTER(i), vp, sz, vp, u]
        L.cake_kmeans_init_plusplus.argtypes = [vp, ll, i, i, vp, vp, vp, vp, sz, vp]
        L.cake_kmeans_lloyd_sharded.argtypes = [vp, vp, ll, i, i, i, vp, vp, vp, vp, vp, vp, ALLREDUCE_FN, vp, vp, sz, vp, u]
        L.cake_kmeans_update_partial_batched.argtypes = [vp, vp, ll, ll, i, i, vp, vp, vp, sz, vp, u]
        L.cake_kmeans_update_finish_batched.argtypes = [vp, vp, vp, ll, i, i, vp, vp, vp]
        L.cake_kmeans_inertia_batched.argtypes = [vp, ll, ll, vp, i, vp]
        for name in EXPORTS:
            if name not in ("cake_strerror", "cake_kmeans_kernel_launches"):
                getattr(L, name).restype = i
        L.cake_kmeans_kernel_launches.restype = ctypes.c_ulonglong
        _lib = L
    return _lib


def strerror(code: int) -> str:
    return lib().cake_strerror(int(code)).decode()


def cake_version() -> int:
    return int(lib().cake_version())


def cake_kmeans_kernel_launches() -> int:
    return int(lib().cake_kmeans_kernel_launches())


def _check(rc: int, where: str):
    if rc != CAKE_OK:
        raise CakeError(rc, where)


def _ptr(t: torch.Tensor | None):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(stream, device):
    s = stream if stream is not None else torch.cuda.current_stream(device)
    return ctypes.c_void_p(s.cuda_stream)


def _want(t: torch.Tensor, dtype, name: str):
    if t.dtype != dtype or not t.is_contiguous():
        raise TypeError(f"{name} must be a contiguous {dtype} tensor")
    return t


def cake_kmeans_workspace_bytes(B: int, N: int, D: int, K: int) -> int:
    out = ctypes.c_size_t(0)
    _check(lib().cake_kmeans_workspace_bytes(B, N, D, K, ctypes.byref(out)), "cake_kmeans_workspace_bytes")
    return int(out.value)


def alloc_workspace(B: int, N: int, D: int, K: int, device) -> torch.Tensor:
    """A workspace tensor of the required size with its status header zeroed."""
    ws = torch.empty(cake_kmeans_workspace_bytes(B, N, D, K), dtype=torch.uint8, device=device)
    ws[:256].zero_()
    return ws


def _dims(X: torch.Tensor, C: torch.Tensor):
    if X.dim() == 2:
        X, C = X.unsqueeze(0), C.unsqueeze(0)
    if X.dim() != 3 or C.dim() != 3 or X.shape[0] != C.shape[0] or X.shape[2] != C.shape[2]:
        raise ValueError("X must be [N,D] or [B,N,D] and C [K,D] or [B,K,D] with matching B and D")
    return X.shape[0], X.shape[1], X.shape[2], C.shape[1]


def cake_kmeans_assign(X, C, out_idx=None, out_dist=None, ws=None, stream=None, flags=0, want_dist=True):
    """X bf16 [N,D] or [B,N,D], C bf16 [K,D] or [B,K,D] -> (idx int32, dist fp32 or None)."""
    _want(X, torch.bfloat16, "X"), _want(C, torch.bfloat16, "C")
    B, N, D, K = _dims(X, C)
    lead = X.shape[:-1]
    if out_idx is None:
        out_idx = torch.empty(lead, dtype=torch.int32, device=X.device)
    if out_dist is None and want_dist:
        out_dist = torch.empty(lead, dtype=torch.float32, device=X.device)
    if ws is None:
        ws = alloc_workspace(B, N, D, K, X.device)
    with torch.cuda.device(X.device):
        if X.dim() == 2:
            rc = lib().cake_kmeans_assign(_ptr(X), _ptr(C), N, D, K, _ptr(out_idx), _ptr(out_dist), _ptr(ws),
                                          ws.numel(), _stream(stream, X.device), flags)
        else:
            rc = lib().cake_kmeans_assign_batched(_ptr(X), _ptr(C), B, N, D, K, _ptr(out_idx), _ptr(out_dist),
                                                  _ptr(ws), ws.numel(), _stream(stream, X.device), flags)
    _check(rc, "cake_kmeans_assign")
    return out_idx, out_dist


def cake_kmeans_update(X, idx, K, C_prev=None, out_C=None, out_C_bf16=None, out_counts=None, ws=None,
                       stream=None, flags=0):
    """X bf16 [N,D] / [B,N,D], idx int32 [N] / [B,N] -> (C fp32, C bf16, counts int32)."""
    _want(X, torch.bfloat16, "X"), _want(idx, torch.int32, "idx")
    batched = X.dim() == 3
    B = X.shape[0] if batched else 1
    N, D = X.shape[-2], X.shape[-1]
    shape = (B, K, D) if batched else (K, D)
    if C_prev is not None:
        _want(C_prev, torch.bfloat16, "C_prev")
    if out_C is None:
        out_C = torch.empty(shape, dtype=torch.float32, device=X.device)
    if out_C_bf16 is None:
        out_C_bf16 = torch.empty(shape, dtype=torch.bfloat16, device=X.device)
    if out_counts is None:
        out_counts = torch.empty(shape[:-1], dtype=torch.int32, device=X.device)
    if ws is None:
        ws = alloc_workspace(B, N, D, K, X.device)
    with torch.cuda.device(X.device):
        if batched:
            rc = lib().cake_kmeans_update_batched(_ptr(X), _ptr(idx), B, N, D, K, _ptr(C_prev), _ptr(out_C),
                                                  _ptr(out_C_bf16), _ptr(out_counts), _ptr(ws), ws.numel(),
                                                  _stream(stream, X.device), flags)
        else:
            rc = lib().cake_kmeans_update(_ptr(X), _ptr(idx), N, D, K, _ptr(C_prev), _ptr(out_C), _ptr(out_C_bf16),
                                          _ptr(out_counts), _ptr(ws), ws.numel(), _stream(stream, X.device), flags)
    _check(rc, "cake_kmeans_update")
    return out_C, out_C_bf16, out_counts


def cake_kmeans_update_partial(X, idx, K, out_sums=None, out_counts=None, ws=None, stream=None, flags=0):
    """Sums and counts of the rows given: X bf16 [N,D] / [B,N,D], idx int32 -> (sums fp32 [..,K,D], counts int32 [..,K])."""
    _want(X, torch.bfloat16, "X"), _want(idx, torch.int32, "idx")
    batched = X.dim() == 3
    B = X.shape[0] if batched else 1
    N, D = X.shape[-2], X.shape[-1]
    shape = (B, K, D) if batched else (K, D)
    if out_sums is None:
        out_sums = torch.empty(shape, dtype=torch.float32, device=X.device)
    if out_counts is None:
        out_counts = torch.empty(shape[:-1], dtype=torch.int32, device=X.device)
    _want(out_sums, torch.float32, "out_sums"), _want(out_counts, torch.int32, "out_counts")
    if ws is None:
        ws = alloc_workspace(B, N, D, K, X.device)
    with torch.cuda.device(X.device):
        rc = lib().cake_kmeans_update_partial_batched(_ptr(X), _ptr(idx), B, N, D, K, _ptr(out_sums), _ptr(out_counts),
                                                      _ptr(ws), ws.numel(), _stream(stream, X.device), flags)
    _check(rc, "cake_kmeans_update_partial")
    return out_sums, out_counts


def cake_kmeans_update_finish(sums, counts, C_prev=None, out_C=None, out_C_bf16=None, stream=None):
    """Division: sums fp32 [..,K,D], counts int32 [..,K] -> (C fp32, C bf16); empty clusters keep C_prev."""
    _want(sums, torch.float32, "sums"), _want(counts, torch.int32, "counts")
    K, D = sums.shape[-2], sums.shape[-1]
    B = sums.shape[0] if sums.dim() == 3 else 1
    if C_prev is not None:
        _want(C_prev, torch.bfloat16, "C_prev")
    if out_C is None:
        out_C = torch.empty_like(sums)
    if out_C_bf16 is None:
        out_C_bf16 = torch.empty(sums.shape, dtype=torch.bfloat16, device=sums.device)
    with torch.cuda.device(sums.device):
        rc = lib().cake_kmeans_update_finish_batched(_ptr(sums), _ptr(counts), _ptr(C_prev), B, K, D, _ptr(out_C),
                                                     _ptr(out_C_bf16), _stream(stream, sums.device))
    _check(rc, "cake_kmeans_update_finish")
    return out_C, out_C_bf16


def cake_kmeans_inertia(dist, out_inertia=None, stride=1, stream=None):
    """Sum of the distances of an assignment in fp64: dist fp32 [N] / [B,N] -> out_inertia[b * stride] (fp64)."""
    _want(dist, torch.float32, "dist")
    B = dist.shape[0] if dist.dim() == 2 else 1
    N = dist.shape[-1]
    if out_inertia is None:
        out_inertia = torch.empty(B * stride, dtype=torch.float64, device=dist.device)
    if out_inertia.dtype != torch.float64:
        raise TypeError("out_inertia must be float64")
    with torch.cuda.device(dist.device):
        rc = lib().cake_kmeans_inertia_batched(_ptr(dist), B, N, _ptr(out_inertia), stride, _stream(stream, dist.device))
    _check(rc, "cake_kmeans_inertia")
    return out_inertia


@dataclass
class LloydOutput:
    C: torch.Tensor        # fp32 [.., K, D]
    C_bf16: torch.Tensor   # bf16 [.., K, D]
    idx: torch.Tensor      # int32 [.., N]   last assign
    dist: torch.Tensor     # fp32 [.., N]    last assign
    counts: torch.Tensor   # int32 [.., K]   last update
    inertia: torch.Tensor  # fp64 [.., iters]


def alloc_lloyd_outputs(X, C0, iters, pin_host: bool = False) -> LloydOutput:
    lead = X.shape[:-2]
    N, D, K = X.shape[-2], X.shape[-1], C0.shape[-2]
    kw = dict(device="cpu", pin_memory=True) if pin_host else dict(device=X.device)
    return LloydOutput(
        torch.empty(*lead, K, D, dtype=torch.float32, **kw), torch.empty(*lead, K, D, dtype=torch.bfloat16, **kw),
        torch.empty(*lead, N, dtype=torch.int32, **kw), torch.empty(*lead, N, dtype=torch.float32, **kw),
        torch.empty(*lead, K, dtype=torch.int32, **kw), torch.empty(*lead, iters, dtype=torch.float64, **kw))


def cake_kmeans_lloyd(X, C0, iters, out: LloydOutput | None = None, ws=None, stream=None, flags=0) -> LloydOutput:
    """iters Lloyd iterations from C0; X bf16 [N,D] / [B,N,D], C0 bf16 [K,D] / [B,K,D]."""
    _want(X, torch.bfloat16, "X"), _want(C0, torch.bfloat16, "C0")
    B, N, D, K = _dims(X, C0)
    if out is None:
        out = alloc_lloyd_outputs(X, C0, iters)
    if ws is None:
        ws = alloc_workspace(B, N, D, K, X.device)
    with torch.cuda.device(X.device):
        if X.dim() == 2:
            rc = lib().cake_kmeans_lloyd(_ptr(X), _ptr(C0), N, D, K, iters, _ptr(out.C), _ptr(out.C_bf16),
                                         _ptr(out.idx), _ptr(out.dist), _ptr(out.counts), _ptr(out.inertia),
                                         _ptr(ws), ws.numel(), _stream(stream, X.device), flags)
        else:
            rc = lib().cake_kmeans_lloyd_batched(_ptr(X), _ptr(C0), B, N, D, K, iters, _ptr(out.C), _ptr(out.C_bf16),
                                                 _ptr(out.idx), _ptr(out.dist), _ptr(out.counts), _ptr(out.inertia),
                                                 _ptr(ws), ws.numel(), _stream(stream, X.device), flags)
    _check(rc, "cake_kmeans_lloyd")
    return out


def cake_kmeans_lloyd_host_device_bytes(B, N, D, K, iters) -> int:
    out = ctypes.c_size_t(0)
    _check(lib().cake_kmeans_lloyd_host_device_bytes(B, N, D, K, iters, ctypes.byref(out)),
           "cake_kmeans_lloyd_host_device_bytes")
    return int(out.value)


def cake_kmeans_lloyd_host(X_host, C0_host, iters, out: LloydOutput, dev: torch.Tensor, stream=None, flags=0):
    """Host-buffer Lloyd: X_host / C0_host / `out` are CPU (ideally pinned) tensors, `dev` device scratch."""
    _want(X_host, torch.bfloat16, "X_host"), _want(C0_host, torch.bfloat16, "C0_host")
    if X_host.is_cuda or C0_host.is_cuda or out.C.is_cuda:
        raise TypeError("cake_kmeans_lloyd_host takes host tensors")
    B, N, D, K = _dims(X_host, C0_host)
    with torch.cuda.device(dev.device):
        rc = lib().cake_kmeans_lloyd_host(_ptr(X_host), _ptr(C0_host), B, N, D, K, iters, _ptr(out.C),
                                          _ptr(out.C_bf16), _ptr(out.idx), _ptr(out.dist), _ptr(out.counts),
                                          _ptr(out.inertia), _ptr(dev), dev.numel(), _stream(stream, dev.device),
                                          flags)
    _check(rc, "cake_kmeans_lloyd_host")
    return out


def cake_kmeans_device_status(ws: torch.Tensor, stream=None) -> int:
    v = ctypes.c_int(0)
    with torch.cuda.device(ws.device):
        _check(lib().cake_kmeans_device_status(_ptr(ws), _stream(stream, ws.device), ctypes.byref(v)),
               "cake_kmeans_device_status")
    return int(v.value)


def cake_kmeans_selftest_bounded_wait(ws: torch.Tensor, limit_ms: int, stream=None):
    with torch.cuda.device(ws.device):
        _check(lib().cake_kmeans_selftest_bounded_wait(_ptr(ws), ws.numel(), limit_ms, _stream(stream, ws.device)),
               "cake_kmeans_selftest_bounded_wait")


def cake_kmeans_assign_static(X, C, out_idx=None, out_dist=None, stream=None, want_dist=True):
    """Workspace-free assign for callers that cannot allocate: X bf16 [N,D], C bf16 [K,D], K <= 16384.

    The scratch is a fixed array inside the library, shared by every call on the device, so calls
    must not overlap on the GPU.  Output tensors are still the caller's (allocated here only as a
    convenience when not passed in).
    """
    _want(X, torch.bfloat16, "X"), _want(C, torch.bfloat16, "C")
    if X.dim() != 2 or C.dim() != 2 or X.shape[1] != C.shape[1]:
        raise ValueError("X must be [N,D] and C [K,D]")
    N, D, K = X.shape[0], X.shape[1], C.shape[0]
    if out_idx is None:
        out_idx = torch.empty(N, dtype=torch.int32, device=X.device)
    if out_dist is None and want_dist:
        out_dist = torch.empty(N, dtype=torch.float32, device=X.device)
    with torch.cuda.device(X.device):
        rc = lib().cake_kmeans_assign_static(_ptr(X), _ptr(C), N, D, K, _ptr(out_idx), _ptr(out_dist),
                                             _stream(stream, X.device))
    _check(rc, "cake_kmeans_assign_static")
    return out_idx, out_dist


def cake_kmeans_assign_static_status(device, stream=None) -> int:
    """Sticky device status of the workspace-free assign's fixed scratch on `device` (read and cleared)."""
    v = ctypes.c_int(0)
    with torch.cuda.device(device):
        _check(lib().cake_kmeans_assign_static_status(_stream(stream, device), ctypes.byref(v)),
               "cake_kmeans_assign_static_status")
    return int(v.value)


def cake_knn_workspace_bytes(N: int, M: int, D: int, k: int) -> int:
    out = ctypes.c_size_t(0)
    _check(lib().cake_knn_workspace_bytes(N, M, D, k, ctypes.byref(out)), "cake_knn_workspace_bytes")
    return int(out.value)


def cake_knn_search(Q, X, k, out_idx=None, out_dist=None, ws=None, stream=None, want_dist=True):
    """Q bf16 [N,D] queries, X bf16 [M,D] database -> (idx int32 [N,k], dist fp32 [N,k] or None), nearest first."""
    _want(Q, torch.bfloat16, "Q"), _want(X, torch.bfloat16, "X")
    if Q.dim() != 2 or X.dim() != 2 or Q.shape[1] != X.shape[1]:
        raise ValueError("Q must be [N,D] and X [M,D]")
    N, D, M = Q.shape[0], Q.shape[1], X.shape[0]
    if out_idx is None:
        out_idx = torch.empty(N, k, dtype=torch.int32, device=Q.device)
    if out_dist is None and want_dist:
        out_dist = torch.empty(N, k, dtype=torch.float32, device=Q.device)
    if ws is None:
        ws = torch.empty(cake_knn_workspace_bytes(N, M, D, k), dtype=torch.uint8, device=Q.device)
        ws[:256].zero_()
    with torch.cuda.device(Q.device):
        rc = lib().cake_knn_search(_ptr(Q), _ptr(X), N, M, D, k, _ptr(out_idx), _ptr(out_dist), _ptr(ws), ws.numel(),
                                   _stream(stream, Q.device))
    _check(rc, "cake_knn_search")
    return out_idx, out_dist


def cake_kmeans_lloyd_tol(X, C0, max_iters, tol, check_every=1, ws=None, stream=None, flags=0):
    """Lloyd iterations until the relative inertia decrease falls to `tol` (looked at every `check_every`
    iterations) or max_iters; X bf16 [N,D], C0 bf16 [K,D].  Returns (LloydOutput with inertia[:iters], iters)."""
    _want(X, torch.bfloat16, "X"), _want(C0, torch.bfloat16, "C0")
    if X.dim() != 2 or C0.dim() != 2:
        raise ValueError("one problem: X [N,D], C0 [K,D]")
    B, N, D, K = _dims(X, C0)
    out = alloc_lloyd_outputs(X, C0, max_iters)
    if ws is None:
        ws = alloc_workspace(1, N, D, K, X.device)
    n = ctypes.c_int(0)
    with torch.cuda.device(X.device):
        rc = lib().cake_kmeans_lloyd_tol(_ptr(X), _ptr(C0), N, D, K, max_iters, float(tol), check_every, _ptr(out.C),
                                         _ptr(out.C_bf16), _ptr(out.idx), _ptr(out.dist), _ptr(out.counts),
                                         _ptr(out.inertia), ctypes.byref(n), _ptr(ws), ws.numel(),
                                         _stream(stream, X.device), flags)
    _check(rc, "cake_kmeans_lloyd_tol")
    out.inertia = out.inertia[: n.value]
    return out, int(n.value)


def cake_kmeans_init_plusplus(X, K, u, ws=None, stream=None):
    """k-means++ seeding: X bf16 [N,D], u fp32 [K] uniforms in [0,1) on the device -> (C0 bf16 [K,D], rows int32 [K])."""
    _want(X, torch.bfloat16, "X"), _want(u, torch.float32, "u")
    if X.dim() != 2 or u.shape != (K,):
        raise ValueError("X must be [N,D] and u [K]")
    N, D = X.shape
    C0 = torch.empty(K, D, dtype=torch.bfloat16, device=X.device)
    rows = torch.empty(K, dtype=torch.int32, device=X.device)
    if ws is None:
        ws = alloc_workspace(1, N, D, K, X.device)
    with torch.cuda.device(X.device):
        rc = lib().cake_kmeans_init_plusplus(_ptr(X), N, D, K, _ptr(u), _ptr(C0), _ptr(rows), _ptr(ws), ws.numel(),
                                             _stream(stream, X.device))
    _check(rc, "cake_kmeans_init_plusplus")
    return C0, rows


def cake_kmeans_lloyd_sharded_call(X_local, C0, iters, out: LloydOutput, ws, reduce=None, stream=None, flags=0):
    """One rank's share of a row-sharded Lloyd run through the C entry point.  `reduce(sums, counts)` (or None for a
    single rank) is called once per iteration with the fp32 [K,D] sums and int32 [K] counts as tensors that alias the
    library's buffers and must add them up over all ranks in place, in stream order.  out.inertia holds the LOCAL sums."""
    _want(X_local, torch.bfloat16, "X_local"), _want(C0, torch.bfloat16, "C0")
    N, D = X_local.shape
    K = C0.shape[0]
    base = ws.data_ptr()

    def thunk(user, sums_ptr, n_sums, counts_ptr, n_counts, stream_ptr):
        try:
            off = sums_ptr - base
            sums = ws[off:off + 4 * n_sums].view(torch.float32).view(K, D)
            reduce(sums, out.counts)
            return 0
        except Exception:          # an exception must not cross the C frames
            import traceback
            traceback.print_exc()
            return 1

    cb = ALLREDUCE_FN(thunk) if reduce is not None else ctypes.cast(None, ALLREDUCE_FN)
    with torch.cuda.device(X_local.device):
        rc = lib().cake_kmeans_lloyd_sharded(_ptr(X_local), _ptr(C0), N, D, K, iters, _ptr(out.C), _ptr(out.C_bf16),
                                             _ptr(out.idx), _ptr(out.dist), _ptr(out.counts), _ptr(out.inertia), cb, None,
                                             _ptr(ws), ws.numel(), _stream(stream, X_local.device), flags)
    _check(rc, "cake_kmeans_lloyd_sharded")
    return out
