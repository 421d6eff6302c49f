"""Thin ctypes binding over the C ABI declared in ``include/patch.h``.

Argument marshalling only: every step of the path (mask selection, packing, the matmul, its
split-K reduction and the bf16 epilogue) runs in the CUDA library.  There is no CPU fallback:
if ``libpatch_b200.so`` is missing this module raises on first use.

Tensors are torch CUDA tensors used purely as device buffers (``data_ptr()``); weights,
activations and results are ``torch.bfloat16``; packed blobs and workspaces are ``torch.uint8``.
"""
from __future__ import annotations

import ctypes
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libpatch_b200.so")

TILE_DENSE, TILE_SPARSE_2_4, TILE_DENSE_Q4, TILE_SPARSE_2_4_Q4 = 0, 1, 2, 3
VARIANT_AUTO, VARIANT_GEMV, VARIANT_MMA, VARIANT_PAIR = 0, 1, 2, 3
WEIGHTS_STATIC = 0x100   # OR into `variant`: the packed weight is not produced by the preceding kernel
INPUT_STATIC = 0x200     # OR into `variant`: X is not produced by the preceding kernel
OUTPUT_STATIC = 0x400    # OR into `variant` (with the other two): nothing in the overlap window reads or writes Y
OK = 0
ERR_NULL, ERR_SHAPE, ERR_TILE, ERR_FLAG, ERR_ALIGN = -1, -2, -3, -4, -5
ERR_SIZE, ERR_FORMAT, ERR_ARCH, ERR_CUDA, ERR_TIMEOUT = -6, -7, -8, -9, -10

EXPORTS = ["patch_packed_size", "patch_pack", "patch_unpack", "patch_gemm_workspace_size",
           "patch_workspace_init", "patch_gemm", "patch_gemm_ex", "patch_gemm_gated", "patch_gemm_gated_workspace_size", "patch_gemm_host", "patch_gemm_host_batch", "patch_gemm_host_batch_pipelined",
           "patch_gemm_noalloc",
           "patch_hard_mask", "patch_pack_patterns", "patch_pack_dev", "patch_read_layout", "patch_soft_mask_workspace_size", "patch_soft_mask",
           "patch_mask_regularizers", "patch_mask_regularizer_coefficients", "patch_soft_mask_backward",
           "patch_strerror", "patch_version"]
MASK_NO_NOISE = 1


class Layout(ctypes.Structure):
    """Mirror of ``patch_layout_t``."""
    _fields_ = [("magic", ctypes.c_uint32), ("version", ctypes.c_uint32),
                ("N", ctypes.c_int64), ("K", ctypes.c_int64),
                ("tile_n", ctypes.c_int32), ("tile_k", ctypes.c_int32),
                ("n_dense", ctypes.c_int64), ("n_sparse", ctypes.c_int64),
                ("table_off", ctypes.c_uint64), ("payload_off", ctypes.c_uint64),
                ("payload_bytes", ctypes.c_uint64), ("total_bytes", ctypes.c_uint64),
                ("n_dense_q4", ctypes.c_int64), ("n_sparse_q4", ctypes.c_int64)]


class PatchError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {strerror(status)} (status {status})")


_lib = None


def load(path: str) -> ctypes.CDLL:
    """Load a build of the library from ``path`` and declare its argument types (``lib()`` is the product build;
    the tests also load the fault-injection build this way)."""
    if True:
        if not os.path.exists(path):
            raise RuntimeError(f"{path} is missing: run `python -m paper_2509_23410_b200.build` "
                               "(there is no CPU fallback)")
        L = ctypes.CDLL(path)
        vp, i64, sz = ctypes.c_void_p, ctypes.c_int64, ctypes.c_size_t
        L.patch_packed_size.argtypes = [i64, i64, ctypes.c_int, ctypes.c_int, vp, ctypes.POINTER(Layout)]
        L.patch_pack.argtypes = [vp, i64, vp, ctypes.POINTER(Layout), vp, sz, vp]
        L.patch_unpack.argtypes = [ctypes.POINTER(Layout), vp, vp, i64, vp]
        L.patch_gemm_workspace_size.argtypes = [ctypes.POINTER(Layout), i64, ctypes.POINTER(sz)]
        L.patch_workspace_init.argtypes = [vp, sz, vp]
        L.patch_gemm.argtypes = [vp, i64, i64, ctypes.POINTER(Layout), vp, vp, i64, vp, sz, vp, vp]
        L.patch_gemm_ex.argtypes = L.patch_gemm.argtypes + [ctypes.c_int]
        L.patch_gemm_gated.argtypes = [vp, i64, i64, ctypes.POINTER(Layout), vp, vp, i64, vp, sz, vp, vp, ctypes.c_int]
        L.patch_gemm_gated_workspace_size.argtypes = [ctypes.POINTER(Layout), i64, ctypes.POINTER(sz)]
        L.patch_gemm_host.argtypes = [vp, i64, ctypes.POINTER(Layout), vp, vp, vp, vp, vp, sz, vp]
        L.patch_gemm_noalloc.argtypes = [vp, i64, i64, ctypes.POINTER(Layout), vp, vp, i64, vp]
        L.patch_gemm_host_batch.argtypes = [vp, ctypes.c_int, ctypes.c_int, vp]
        L.patch_gemm_host_batch_pipelined.argtypes = [vp, ctypes.c_int, ctypes.c_int, ctypes.c_int, vp, vp, vp]
        L.patch_hard_mask.argtypes = [vp, vp, i64, i64, ctypes.c_int, ctypes.c_int, vp, vp, vp]
        L.patch_pack_patterns.argtypes = [vp, i64, vp, vp, ctypes.POINTER(Layout), vp, sz, vp, vp]
        L.patch_soft_mask_workspace_size.argtypes = [i64, i64, ctypes.c_int, ctypes.c_int, ctypes.POINTER(sz)]
        L.patch_soft_mask.argtypes = [vp, i64, vp, vp, i64, i64, ctypes.c_int, ctypes.c_int, ctypes.c_float,
                                      ctypes.c_float, ctypes.c_uint64, ctypes.c_int, vp, i64, vp, i64, vp, vp, sz, vp]
        L.patch_mask_regularizers.argtypes = [vp, ctypes.c_int, ctypes.c_double, ctypes.c_double, ctypes.c_double,
                                              ctypes.POINTER(ctypes.c_double)]
        L.patch_mask_regularizer_coefficients.argtypes = [vp, ctypes.c_int, ctypes.c_double, ctypes.c_double,
                                                          ctypes.c_double, ctypes.POINTER(ctypes.c_double),
                                                          ctypes.POINTER(ctypes.c_double)]
        L.patch_soft_mask_backward.argtypes = [vp, i64, vp, vp, i64, i64, ctypes.c_int, ctypes.c_int, ctypes.c_float,
                                               ctypes.c_float, ctypes.c_uint64, ctypes.c_int, vp, i64, ctypes.c_double,
                                               ctypes.c_double, vp, vp, vp]
        L.patch_pack_dev.argtypes = [vp, i64, vp, vp, i64, i64, ctypes.c_int, ctypes.c_int, vp, sz, vp, vp]
        L.patch_read_layout.argtypes = [vp, ctypes.POINTER(Layout), vp]
        L.patch_strerror.argtypes = [ctypes.c_int]
        L.patch_strerror.restype = ctypes.c_char_p
        for name in EXPORTS:
            if name != "patch_strerror":
                getattr(L, name).restype = ctypes.c_int
    return L


def lib() -> ctypes.CDLL:
    """The product build of the CUDA library; fails loudly if it has not been built."""
    global _lib
    if _lib is None:
        _lib = load(LIB_PATH)
    return _lib


def strerror(status: int) -> str:
    return lib().patch_strerror(status).decode()


def _check(status: int, where: str):
    if status != OK:
        raise PatchError(status, where)


def _ptr(t):
    return ctypes.c_void_p(t.data_ptr()) if t is not None else ctypes.c_void_p(0)


def _stream(stream=None):
    import torch
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def _flags_buf(flags):
    import numpy as np
    f = np.ascontiguousarray(flags, dtype=np.uint8).reshape(-1)
    return f, ctypes.c_void_p(f.ctypes.data)


def patch_packed_size(N: int, K: int, flags, tile_n: int = 128, tile_k: int = 128) -> Layout:
    L = Layout()
    f, fp = _flags_buf(flags)
    _check(lib().patch_packed_size(N, K, tile_n, tile_k, fp, ctypes.byref(L)), "patch_packed_size")
    return L


def patch_pack(W, flags, layout: Layout | None = None, out=None, stream=None):
    """Pack a bf16 CUDA weight [N x K]; returns (packed uint8 tensor, layout)."""
    import torch
    assert W.is_cuda and W.dtype == torch.bfloat16 and W.dim() == 2 and W.stride(1) == 1
    N, K = W.shape
    if layout is None:
        layout = patch_packed_size(N, K, flags)
    if out is None:
        out = torch.empty(layout.total_bytes, dtype=torch.uint8, device=W.device)
    f, fp = _flags_buf(flags)
    _check(lib().patch_pack(_ptr(W), W.stride(0), fp, ctypes.byref(layout), _ptr(out), out.numel(),
                            _stream(stream)), "patch_pack")
    return out, layout


def patch_unpack(layout: Layout, packed, out=None, stream=None):
    import torch
    if out is None:
        out = torch.empty((layout.N, layout.K), dtype=torch.bfloat16, device=packed.device)
    _check(lib().patch_unpack(ctypes.byref(layout), _ptr(packed), _ptr(out), out.stride(0), _stream(stream)),
           "patch_unpack")
    return out


def patch_gemm_workspace_size(layout: Layout, M: int) -> int:
    n = ctypes.c_size_t(0)
    _check(lib().patch_gemm_workspace_size(ctypes.byref(layout), M, ctypes.byref(n)), "patch_gemm_workspace_size")
    return int(n.value)


def patch_workspace_init(workspace, stream=None):
    if workspace is not None and workspace.numel():
        _check(lib().patch_workspace_init(_ptr(workspace), workspace.numel(), _stream(stream)), "patch_workspace_init")


def patch_gemm(X, layout: Layout, packed, Y=None, workspace=None, status=None, stream=None,
               variant: int = VARIANT_AUTO):
    """Y = X @ What^T.  X bf16 [M x K] (row stride >= K), returns Y bf16 [M x N]."""
    import torch
    assert X.is_cuda and X.dtype == torch.bfloat16 and X.dim() == 2 and (X.shape[0] == 0 or X.stride(1) == 1)
    M = X.shape[0]
    if Y is None:
        Y = torch.empty((M, layout.N), dtype=torch.bfloat16, device=X.device)
    ws_bytes = workspace.numel() if workspace is not None else 0
    _check(lib().patch_gemm_ex(_ptr(X), X.stride(0) if M else layout.K, M, ctypes.byref(layout), _ptr(packed),
                               _ptr(Y), Y.stride(0) if M else layout.N, _ptr(workspace), ws_bytes,
                               _ptr(status), _stream(stream), variant), "patch_gemm")
    return Y


def interleave_row_blocks(A, B_, block: int = 128):
    """Stack two [N x ...] arrays (torch or numpy) so that 128-row blocks alternate: A block 0, B block 0,
    A block 1, ...  With ``block=1`` the same for per-tile flag arrays.  Data movement only."""
    n = A.shape[0]
    assert A.shape == B_.shape and n % block == 0
    tail = tuple(A.shape[1:])
    if hasattr(A, "cpu"):
        import torch
        return torch.stack((A.reshape(n // block, block, *tail), B_.reshape(n // block, block, *tail)), dim=1).reshape(2 * n, *tail)
    import numpy as np
    return np.stack((A.reshape(n // block, block, *tail), B_.reshape(n // block, block, *tail)), axis=1).reshape(2 * n, *tail)


def patch_gemm_gated_workspace_size(layout: Layout, M: int) -> int:
    n = ctypes.c_size_t(0)
    _check(lib().patch_gemm_gated_workspace_size(ctypes.byref(layout), M, ctypes.byref(n)), "patch_gemm_gated_workspace_size")
    return int(n.value)


def patch_gemm_gated(X, layout: Layout, packed, Y=None, workspace=None, status=None, stream=None, flags: int = 0):
    """Y [M x N/2] = silu(X Wgate^T) * (X Wup^T) for a packed weight with interleaved gate/up row-blocks."""
    import torch
    M = X.shape[0]
    if Y is None:
        Y = torch.empty((M, layout.N // 2), dtype=torch.bfloat16, device=X.device)
    ws_bytes = workspace.numel() if workspace is not None else 0
    _check(lib().patch_gemm_gated(_ptr(X), X.stride(0) if M else layout.K, M, ctypes.byref(layout), _ptr(packed),
                                  _ptr(Y), Y.stride(0) if M else layout.N // 2, _ptr(workspace), ws_bytes,
                                  _ptr(status), _stream(stream), flags),
           "patch_gemm_gated")
    return Y


def patch_gemm_host(X_host, layout: Layout, packed, Y_host, X_stage, Y_stage, workspace=None, stream=None):
    """End-to-end call with host (pinned) X and Y; synchronises the stream."""
    M = X_host.shape[0]
    ws_bytes = workspace.numel() if workspace is not None else 0
    _check(lib().patch_gemm_host(_ptr(X_host), M, ctypes.byref(layout), _ptr(packed), _ptr(Y_host),
                                 _ptr(X_stage), _ptr(Y_stage), _ptr(workspace), ws_bytes, _stream(stream)),
           "patch_gemm_host")
    return Y_host


class HostJob(ctypes.Structure):
    """Mirror of ``patch_host_job_t``."""
    _fields_ = [("X_host", ctypes.c_void_p), ("M", ctypes.c_int64), ("layout", ctypes.POINTER(Layout)),
                ("packed_dev", ctypes.c_void_p), ("Y_host", ctypes.c_void_p), ("X_stage_dev", ctypes.c_void_p),
                ("Y_stage_dev", ctypes.c_void_p), ("workspace_dev", ctypes.c_void_p), ("workspace_bytes", ctypes.c_size_t)]


def make_host_batch(jobs):
    """Marshal a list of dicts (Xh, layout, packed, Yh, X, Y, ws) once; the arrays must outlive the result."""
    arr = (HostJob * len(jobs))()
    for a, j in zip(arr, jobs):
        a.X_host, a.M, a.layout = j["Xh"].data_ptr(), j["Xh"].shape[0], ctypes.pointer(j["layout"])
        a.packed_dev, a.Y_host = j["packed"].data_ptr(), j["Yh"].data_ptr()
        a.X_stage_dev, a.Y_stage_dev = j["X"].data_ptr(), j["Y"].data_ptr()
        ws = j.get("ws")
        a.workspace_dev, a.workspace_bytes = (ws.data_ptr(), ws.numel()) if ws is not None else (None, 0)
    return arr


def patch_gemm_host_batch(batch, weights_static: bool = False, stream=None):
    """One step of GEMMs with host X / Y: all copies in, all launches, all copies out, one synchronisation."""
    _check(lib().patch_gemm_host_batch(batch, len(batch), 1 if weights_static else 0, _stream(stream)),
           "patch_gemm_host_batch")


def patch_gemm_host_batch_pipelined(batch, copy_in_stream, copy_out_stream, n_chunks: int = 4,
                                    weights_static: bool = False, stream=None):
    """The same step with copies in, GEMMs and copies out overlapped over ``n_chunks`` runs of jobs (three streams)."""
    _check(lib().patch_gemm_host_batch_pipelined(batch, len(batch), 1 if weights_static else 0, int(n_chunks),
                                                 _stream(stream), _stream(copy_in_stream), _stream(copy_out_stream)),
           "patch_gemm_host_batch_pipelined")


def patch_gemm_noalloc(X, layout: Layout, packed, Y, stream=None):
    """Y = X @ What^T for callers that may not allocate: the library's own fixed scratch array is used.

    The caller passes every buffer, Y included; nothing is allocated here either.  M <= 16.
    """
    M = X.shape[0]
    _check(lib().patch_gemm_noalloc(_ptr(X), X.stride(0) if M else layout.K, M, ctypes.byref(layout), _ptr(packed),
                                    _ptr(Y), Y.stride(0) if M else layout.N, _stream(stream)), "patch_gemm_noalloc")
    return Y


def patch_version() -> int:
    return int(lib().patch_version())


# ---------------------------------------------------------------------------------------------
# Mask learning: hard masks from logits, packing with a given 2:4 mask, soft-mask forward.


def patch_hard_mask(P_tile, P24, N: int, K: int, flags_out=None, patterns_out=None, stream=None):
    """Tile flags (uint8 [N/128 * K/128]) and candidate index per group (uint8 [N * K/4]) from the logits."""
    import torch
    assert P_tile.is_cuda and P_tile.dtype == torch.float32 and P_tile.is_contiguous()
    assert P24.is_cuda and P24.dtype == torch.float32 and P24.is_contiguous() and tuple(P24.shape) == (6, N * K // 4)
    if flags_out is None:
        flags_out = torch.empty((N // 128) * (K // 128), dtype=torch.uint8, device=P24.device)
    if patterns_out is None:
        patterns_out = torch.empty(N * K // 4, dtype=torch.uint8, device=P24.device)
    _check(lib().patch_hard_mask(_ptr(P_tile), _ptr(P24), N, K, 128, 128, _ptr(flags_out), _ptr(patterns_out),
                                 _stream(stream)), "patch_hard_mask")
    return flags_out, patterns_out


def patch_pack_patterns(W, flags, patterns, layout: Layout | None = None, out=None, status=None, stream=None):
    """patch_pack with the 2:4 mask given as candidate indices (uint8 CUDA tensor [N * K/4])."""
    import torch
    assert W.is_cuda and W.dtype == torch.bfloat16 and W.dim() == 2 and W.stride(1) == 1
    assert patterns.is_cuda and patterns.dtype == torch.uint8 and patterns.is_contiguous()
    N, K = W.shape
    assert patterns.numel() == N * K // 4
    if layout is None:
        layout = patch_packed_size(N, K, flags)
    if out is None:
        out = torch.empty(layout.total_bytes, dtype=torch.uint8, device=W.device)
    f, fp = _flags_buf(flags)
    _check(lib().patch_pack_patterns(_ptr(W), W.stride(0), fp, _ptr(patterns), ctypes.byref(layout), _ptr(out),
                                     out.numel(), _ptr(status), _stream(stream)), "patch_pack_patterns")
    return out, layout


def patch_soft_mask_workspace_size(N: int, K: int) -> int:
    n = ctypes.c_size_t(0)
    _check(lib().patch_soft_mask_workspace_size(N, K, 128, 128, ctypes.byref(n)), "patch_soft_mask_workspace_size")
    return int(n.value)


def patch_soft_mask(W, P_tile, P24, tau: float, kappa: float, seed: int = 0, flags: int = 0, Wt=None, Mt=None,
                    sums=None, workspace=None, stream=None):
    """Soft-mask forward of one matrix: returns (Wt bf16 [N x K], sums float64 CUDA tensor [4]);
    pass a float32 ``Mt`` [N x K] to also get the soft mask itself."""
    import torch
    assert W.is_cuda and W.dtype == torch.bfloat16 and W.dim() == 2 and W.stride(1) == 1
    N, K = W.shape
    assert P_tile.is_cuda and P_tile.dtype == torch.float32 and P_tile.is_contiguous()
    assert P24.is_cuda and P24.dtype == torch.float32 and P24.is_contiguous() and tuple(P24.shape) == (6, N * K // 4)
    if Wt is None:
        Wt = torch.empty((N, K), dtype=torch.bfloat16, device=W.device)
    if sums is None:
        sums = torch.empty(4, dtype=torch.float64, device=W.device)
    if workspace is None:
        workspace = torch.empty(patch_soft_mask_workspace_size(N, K), dtype=torch.uint8, device=W.device)
    assert Mt is None or (Mt.is_cuda and Mt.dtype == torch.float32 and Mt.stride(1) == 1)
    _check(lib().patch_soft_mask(_ptr(W), W.stride(0), _ptr(P_tile), _ptr(P24), N, K, 128, 128, float(tau),
                                 float(kappa), int(seed) & 0xFFFFFFFFFFFFFFFF, int(flags), _ptr(Wt), Wt.stride(0),
                                 _ptr(Mt), Mt.stride(0) if Mt is not None else 0, _ptr(sums), _ptr(workspace),
                                 workspace.numel(), _stream(stream)), "patch_soft_mask")
    return Wt, sums


def patch_mask_regularizers(sums, rho: float, lambda1: float, lambda2: float) -> float:
    """The two regularisers of Eq. 5 from per-matrix sums (host array-like [n x 4])."""
    import numpy as np
    a = np.ascontiguousarray(sums, dtype=np.float64).reshape(-1, 4)
    out = ctypes.c_double(0.0)
    _check(lib().patch_mask_regularizers(ctypes.c_void_p(a.ctypes.data), int(a.shape[0]), float(rho), float(lambda1),
                                         float(lambda2), ctypes.byref(out)), "patch_mask_regularizers")
    return float(out.value)


def patch_mask_regularizer_coefficients(sums, rho: float, lambda1: float, lambda2: float):
    """(c1, c2) of the regularisers' gradient from per-matrix sums (host array-like [n x 4])."""
    import numpy as np
    a = np.ascontiguousarray(sums, dtype=np.float64).reshape(-1, 4)
    c1, c2 = ctypes.c_double(0.0), ctypes.c_double(0.0)
    _check(lib().patch_mask_regularizer_coefficients(ctypes.c_void_p(a.ctypes.data), int(a.shape[0]), float(rho),
                                                     float(lambda1), float(lambda2), ctypes.byref(c1), ctypes.byref(c2)),
           "patch_mask_regularizer_coefficients")
    return float(c1.value), float(c2.value)


def patch_soft_mask_backward(W, P_tile, P24, tau: float, kappa: float, Gw, c1: float, c2: float, seed: int = 0,
                             flags: int = 0, gP_tile=None, gP24=None, stream=None):
    """Gradient of the soft-mask objective w.r.t. the logits: returns (gP_tile float32, gP24 float32 [6 x G])."""
    import torch
    assert W.is_cuda and W.dtype == torch.bfloat16 and W.dim() == 2 and W.stride(1) == 1
    assert Gw.is_cuda and Gw.dtype == torch.bfloat16 and Gw.shape == W.shape and Gw.stride(1) == 1
    N, K = W.shape
    assert P_tile.is_cuda and P_tile.dtype == torch.float32 and P_tile.is_contiguous()
    assert P24.is_cuda and P24.dtype == torch.float32 and P24.is_contiguous() and tuple(P24.shape) == (6, N * K // 4)
    if gP_tile is None:
        gP_tile = torch.empty_like(P_tile)
    if gP24 is None:
        gP24 = torch.empty_like(P24)
    _check(lib().patch_soft_mask_backward(_ptr(W), W.stride(0), _ptr(P_tile), _ptr(P24), N, K, 128, 128, float(tau),
                                          float(kappa), int(seed) & 0xFFFFFFFFFFFFFFFF, int(flags), _ptr(Gw), Gw.stride(0),
                                          float(c1), float(c2), _ptr(gP_tile), _ptr(gP24), _stream(stream)),
           "patch_soft_mask_backward")
    return gP_tile, gP24


def patch_pack_dev(W, flags_dev, patterns=None, out=None, status=None, stream=None):
    """Pack with the tile flags in device memory (uint8 CUDA tensor); returns the packed uint8 tensor.
    ``out`` defaults to a buffer that fits any flags; get the layout with ``patch_read_layout``."""
    import torch
    assert W.is_cuda and W.dtype == torch.bfloat16 and W.dim() == 2 and W.stride(1) == 1
    assert flags_dev.is_cuda and flags_dev.dtype == torch.uint8 and flags_dev.is_contiguous()
    N, K = W.shape
    T = (N // 128) * (K // 128)
    assert flags_dev.numel() == T
    if out is None:
        out = torch.empty((256 + 16 * T + 1023) // 1024 * 1024 + T * 32768, dtype=torch.uint8, device=W.device)
    _check(lib().patch_pack_dev(_ptr(W), W.stride(0), _ptr(flags_dev), _ptr(patterns), N, K, 128, 128, _ptr(out),
                                out.numel(), _ptr(status), _stream(stream)), "patch_pack_dev")
    return out


def patch_read_layout(packed, stream=None) -> Layout:
    L = Layout()
    _check(lib().patch_read_layout(_ptr(packed), ctypes.byref(L), _stream(stream)), "patch_read_layout")
    return L
