"""ctypes binding of libmonarch: same names and argument order as include/monarch.h.

Tensors are torch CUDA tensors used as typed device buffers; the binding checks dtype,
contiguity and device, takes their pointers, and calls the C entry point on the current
CUDA stream (or the one given).  A non-zero status raises MonarchError.
"""
from __future__ import annotations

import ctypes
import os

F32, BF16 = 0, 1
OP_FWD, OP_BWD_DX, OP_BWD_DW, OP_MLP_FWD, OP_BWD, OP_MLP_BWD, OP_CPLX = 0, 1, 2, 3, 4, 5, 6
IMPL_AUTO, IMPL_STAGED, IMPL_FUSED = 0, 1, 2

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libmonarch.so")
_lib = None

_vp, _i64, _i32, _int, _sz = (ctypes.c_void_p, ctypes.c_int64, ctypes.c_int32, ctypes.c_int,
                              ctypes.c_size_t)
_SIGNATURES = {
    "monarch_fwd": (_int, [_vp, _vp, _vp, _vp, _i64, _i32, _i32, _int, _vp, _sz, _vp]),
    "monarch_bwd_dx": (_int, [_vp, _vp, _vp, _vp, _i64, _i32, _i32, _int, _vp, _sz, _vp]),
    "monarch_bwd_dw": (_int, [_vp, _vp, _vp, _vp, _vp, _vp, _int, _i64, _i32, _i32, _int, _vp,
                              _sz, _vp]),
    "monarch_mlp_fwd": (_int, [_vp] * 8 + [_i64, _i32, _i32, _int, _vp, _sz, _vp]),
    "monarch_bwd": (_int, [_vp] * 8 + [_int, _i64, _i32, _i32, _int, _vp, _sz, _vp]),
    "monarch_mlp_bwd": (_int, [_vp] * 14 + [_int, _i64, _i32, _i32, _int, _vp, _sz, _vp]),
    "monarch_rect_fwd": (_int, [_vp, _vp, _vp, _vp, _i64, _i32, _i32, _i32, _i32, _int, _vp, _sz, _vp]),
    "monarch_rect_workspace_bytes": (_sz, [_i64, _i32, _i32, _i32, _i32, _int]),
    "monarch_rect_bwd": (_int, [_vp] * 8 + [_int, _i64, _i32, _i32, _i32, _i32, _int, _vp, _sz, _vp]),
    "monarch_rect_bwd_workspace_bytes": (_sz, [_i64, _i32, _i32, _i32, _i32, _int]),
    "monarch_rectw_fwd": (_int, [_vp, _vp, _vp, _vp, _i64, _i32, _i32, _i32, _i32, _i32, _int, _vp, _sz, _vp]),
    "monarch_rectw_workspace_bytes": (_sz, [_i64, _i32, _i32, _i32, _i32, _i32, _int]),
    "monarch_rectw_bwd": (_int, [_vp, _vp, _vp, _vp, _vp, _vp, _vp, _int, _i64, _i32, _i32, _i32, _i32, _i32, _int, _vp, _sz,
                                 _vp]),
    "monarch_rectw_bwd_workspace_bytes": (_sz, [_i64, _i32, _i32, _i32, _i32, _i32, _int]),
    "monarch_cplx_fwd": (_int, [_vp, _vp, _vp, _vp, _int, _i64, _i32, _i32, _int, _vp, _sz, _vp]),
    "monarch_dense": (_int, [_vp, _vp, _vp, _i32, _i32, _int, _vp]),
    "monarch_project": (_int, [_vp, _vp, _vp, _i32, _i32, _int, _vp, _vp]),
    "monarch_workspace_bytes": (_sz, [_int, _i64, _i32, _i32, _int]),
    "monarch_workspace_init": (_int, [_vp, _sz, _vp]),
    "monarch_last_device_status": (_int, [_vp, _vp]),
    "monarch_debug_set_wait_limit": (_int, [_vp, ctypes.c_uint, _vp]),
    "monarch_debug_skip_load": (_int, [_i64]),
    "monarch_set_impl": (_int, [_int]),
    "monarch_set_deterministic": (_int, [_int]),
    "monarch_impl_name": (ctypes.c_char_p, [_int, _i32, _int]),
    "monarch_launch_count": (ctypes.c_uint64, []),
    "monarch_status_string": (ctypes.c_char_p, [_int]),
    "monarch_fwd_noalloc": (_int, [_vp, _vp, _vp, _vp, _i64, _i32, _i32, _int, _vp]),
    "monarch_host_create": (_int, [ctypes.POINTER(_vp), _i64, _i32, _i32, _int, _i64]),
    "monarch_host_destroy": (_int, [_vp]),
    "monarch_host_fwd": (_int, [_vp, _vp, _vp, _vp, _vp, _i64]),
    "monarch_host_fwd_bwd": (_int, [_vp] * 9 + [_i64]),
}


class MonarchError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: status {status} ({monarch_status_string(status)})")


def lib() -> ctypes.CDLL:
    """Load libmonarch.so (raises if it has not been built)."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise FileNotFoundError(
                f"{_LIB_PATH} not found: run `python -m paper_2204_00595_b200.build` first")
        handle = ctypes.CDLL(_LIB_PATH)
        for name, (res, args) in _SIGNATURES.items():
            fn = getattr(handle, name)
            fn.restype, fn.argtypes = res, args
        _lib = handle
    return _lib


def exported_symbols():
    """Names this binding expects the library to export."""
    return sorted(_SIGNATURES)


def _dtype_code(t) -> int:
    import torch
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    raise TypeError(f"unsupported tensor dtype {t.dtype}")


def _ptr(t, name, dtype=None):
    if t is None:
        return None
    if not t.is_cuda:
        raise ValueError(f"{name} must be a CUDA tensor")
    if not t.is_contiguous():
        raise ValueError(f"{name} must be contiguous")
    if dtype is not None and t.dtype != dtype:
        raise TypeError(f"{name} must have dtype {dtype}, got {t.dtype}")
    return t.data_ptr()


def _stream(stream):
    import torch
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    return getattr(stream, "cuda_stream", stream)


def _check(status: int, where: str):
    if status != 0:
        raise MonarchError(status, where)


class Workspace:
    """Caller-owned device scratch: a torch byte buffer plus its size."""

    def __init__(self, nbytes: int, device="cuda"):
        import torch
        nbytes = max(int(nbytes), 256)
        self.buf = torch.empty(nbytes + 256, dtype=torch.uint8, device=device)
        off = (-self.buf.data_ptr()) % 256
        self.ptr = self.buf.data_ptr() + off
        self.nbytes = nbytes
        monarch_workspace_init(self)

    @classmethod
    def for_op(cls, op: int, tokens: int, m: int, dtype: int, device="cuda"):
        need = monarch_workspace_bytes(op, tokens, m * m, m, dtype)
        if need == 0:
            raise MonarchError(2, "monarch_workspace_bytes")
        return cls(need, device)


def _ws(ws):
    if isinstance(ws, Workspace):
        return ws.ptr, ws.nbytes
    ptr, nbytes = ws
    return ptr, nbytes


def monarch_workspace_bytes(op: int, tokens: int, n: int, m: int, dtype: int) -> int:
    return int(lib().monarch_workspace_bytes(op, tokens, n, m, dtype))


def monarch_workspace_init(workspace, stream=None) -> None:
    p, b = _ws(workspace)
    _check(lib().monarch_workspace_init(p, b, _stream(stream)), "monarch_workspace_init")


def monarch_last_device_status(workspace, stream=None) -> int:
    p, _ = _ws(workspace)
    return int(lib().monarch_last_device_status(p, _stream(stream)))


def monarch_debug_set_wait_limit(workspace, microseconds: int, stream=None) -> None:
    p, _ = _ws(workspace)
    _check(lib().monarch_debug_set_wait_limit(p, int(microseconds), _stream(stream)), "monarch_debug_set_wait_limit")


def monarch_debug_skip_load(item: int) -> None:
    _check(lib().monarch_debug_skip_load(int(item)), "monarch_debug_skip_load")


def monarch_set_impl(impl: int) -> int:
    return int(lib().monarch_set_impl(impl))


def monarch_set_deterministic(on: bool) -> bool:
    """Fixed summation order for dL, dR of the bf16 m = 32 and m = 64 backward (the calls that split the tokens
    over thread blocks; their workspaces grow by 32 MiB while it is on); returns the previous setting."""
    return bool(lib().monarch_set_deterministic(1 if on else 0))


def monarch_impl_name(op: int, m: int, dtype: int) -> str:
    return lib().monarch_impl_name(op, m, dtype).decode()


def monarch_launch_count() -> int:
    return int(lib().monarch_launch_count())


def monarch_status_string(status: int) -> str:
    return lib().monarch_status_string(status).decode()


def monarch_fwd(x, L, R, y, tokens, n, m, workspace, stream=None) -> None:
    """y = P L P^T R x for ``tokens`` rows of x (see include/monarch.h)."""
    dt = x.dtype
    p, b = _ws(workspace)
    _check(lib().monarch_fwd(_ptr(x, "x"), _ptr(L, "L", dt), _ptr(R, "R", dt), _ptr(y, "y", dt),
                             tokens, n, m, _dtype_code(x), p, b, _stream(stream)), "monarch_fwd")


def monarch_bwd_dx(dy, L, R, dx, tokens, n, m, workspace, stream=None) -> None:
    """dx = M^T dy."""
    dt = dy.dtype
    p, b = _ws(workspace)
    _check(lib().monarch_bwd_dx(_ptr(dy, "dy"), _ptr(L, "L", dt), _ptr(R, "R", dt),
                                _ptr(dx, "dx", dt), tokens, n, m, _dtype_code(dy), p, b,
                                _stream(stream)), "monarch_bwd_dx")


def monarch_bwd_dw(x, dy, L, R, dL, dR, accumulate, tokens, n, m, workspace, stream=None) -> None:
    """dL, dR (float32) summed over tokens; accumulate=1 adds to their contents."""
    import torch
    dt = x.dtype
    p, b = _ws(workspace)
    _check(lib().monarch_bwd_dw(_ptr(x, "x"), _ptr(dy, "dy", dt), _ptr(L, "L", dt),
                                _ptr(R, "R", dt), _ptr(dL, "dL", torch.float32),
                                _ptr(dR, "dR", torch.float32), int(accumulate), tokens, n, m,
                                _dtype_code(x), p, b, _stream(stream)), "monarch_bwd_dw")


def monarch_bwd(x, dy, L, R, dx, dL, dR, accumulate, tokens, n, m, workspace, fwd_workspace=None,
                stream=None) -> None:
    """dx, dL, dR in one call; fwd_workspace = the Workspace monarch_fwd used for the same x, L, R."""
    import torch
    dt = x.dtype
    p, b = _ws(workspace)
    fp = _ws(fwd_workspace)[0] if fwd_workspace is not None else None
    _check(lib().monarch_bwd(_ptr(x, "x"), _ptr(dy, "dy", dt), _ptr(L, "L", dt), _ptr(R, "R", dt), fp,
                             _ptr(dx, "dx", dt), _ptr(dL, "dL", torch.float32),
                             _ptr(dR, "dR", torch.float32), int(accumulate), tokens, n, m,
                             _dtype_code(x), p, b, _stream(stream)), "monarch_bwd")


def monarch_mlp_fwd(x, L1, R1, b1, L2, R2, b2, y, tokens, n, m, workspace, stream=None) -> None:
    """y = M2 GELU(M1 x + b1) + b2."""
    dt = x.dtype
    p, b = _ws(workspace)
    _check(lib().monarch_mlp_fwd(_ptr(x, "x"), _ptr(L1, "L1", dt), _ptr(R1, "R1", dt),
                                 _ptr(b1, "b1", dt), _ptr(L2, "L2", dt), _ptr(R2, "R2", dt),
                                 _ptr(b2, "b2", dt), _ptr(y, "y", dt), tokens, n, m,
                                 _dtype_code(x), p, b, _stream(stream)), "monarch_mlp_fwd")


def monarch_mlp_bwd(x, dy, L1, R1, b1, L2, R2, dx, dL1, dR1, db1, dL2, dR2, db2, accumulate, tokens, n, m,
                    workspace, stream=None) -> None:
    """Gradients of <dy, y> for y = M2 GELU(M1 x + b1) + b2; weight and bias gradients are float32."""
    import torch
    dt, f32 = x.dtype, torch.float32
    p, b = _ws(workspace)
    _check(lib().monarch_mlp_bwd(_ptr(x, "x"), _ptr(dy, "dy", dt), _ptr(L1, "L1", dt), _ptr(R1, "R1", dt),
                                 _ptr(b1, "b1", dt), _ptr(L2, "L2", dt), _ptr(R2, "R2", dt),
                                 _ptr(dx, "dx", dt), _ptr(dL1, "dL1", f32), _ptr(dR1, "dR1", f32),
                                 _ptr(db1, "db1", f32), _ptr(dL2, "dL2", f32), _ptr(dR2, "dR2", f32),
                                 _ptr(db2, "db2", f32), int(accumulate), tokens, n, m, _dtype_code(x),
                                 p, b, _stream(stream)), "monarch_mlp_bwd")


def monarch_rect_workspace_bytes(tokens: int, q: int, b1: int, b: int, r: int, dtype: int) -> int:
    return int(lib().monarch_rect_workspace_bytes(tokens, q, b1, b, r, dtype))


def monarch_rect_fwd(x, L, R, y, tokens, q, b1, b, r, workspace, stream=None) -> None:
    """General (rectangular) Monarch multiply: x [tokens, q*b1], R [q, b, b1], L [b, r, q] -> y [tokens, r*b]."""
    dt = x.dtype
    p, nb = _ws(workspace)
    _check(lib().monarch_rect_fwd(_ptr(x, "x"), _ptr(L, "L", dt), _ptr(R, "R", dt), _ptr(y, "y", dt), tokens,
                                  q, b1, b, r, _dtype_code(x), p, nb, _stream(stream)), "monarch_rect_fwd")


def monarch_cplx_fwd(x, L, R, y, adjoint, tokens, n, m, workspace, stream=None) -> None:
    """Complex multiply on planar tensors: x, y [2, tokens, n]; L, R [2, m, m, m]; adjoint=1 applies M^H."""
    dt = x.dtype
    p, b = _ws(workspace)
    _check(lib().monarch_cplx_fwd(_ptr(x, "x"), _ptr(L, "L", dt), _ptr(R, "R", dt), _ptr(y, "y", dt), int(adjoint),
                                  tokens, n, m, _dtype_code(x), p, b, _stream(stream)), "monarch_cplx_fwd")


def monarch_dense(L, R, M, n, m, stream=None) -> None:
    """M[l*m+j, k*m+i] = L[j, l, k] * R[k, j, i] (Eq. 2); M is [n, n] in the dtype of L."""
    dt = L.dtype
    _check(lib().monarch_dense(_ptr(L, "L"), _ptr(R, "R", dt), _ptr(M, "M", dt), n, m, _dtype_code(L),
                               _stream(stream)), "monarch_dense")


def monarch_project(A, L, R, n, m, rotation_count=None, stream=None) -> None:
    """Algorithm 1: factors L, R of the Monarch matrix closest to the dense A in Frobenius norm.
    rotation_count: optional one-element int64 CUDA tensor, incremented by the number of Jacobi rotations."""
    import torch
    dt = A.dtype
    rc = _ptr(rotation_count, "rotation_count", torch.int64) if rotation_count is not None else None
    _check(lib().monarch_project(_ptr(A, "A"), _ptr(L, "L", dt), _ptr(R, "R", dt), n, m, _dtype_code(A), rc,
                                 _stream(stream)), "monarch_project")


def monarch_rect_bwd_workspace_bytes(tokens: int, q: int, b1: int, b: int, r: int, dtype: int) -> int:
    return int(lib().monarch_rect_bwd_workspace_bytes(tokens, q, b1, b, r, dtype))


def monarch_rect_bwd(x, dy, L, R, dx, dL, dR, accumulate, tokens, q, b1, b, r, workspace, fwd_workspace=None,
                     stream=None) -> None:
    """Gradients of <dy, L R x> for the general class: dx like x; dL [b, r, q] and dR [q, b, b1] in float32.
    fwd_workspace = the Workspace monarch_rect_fwd used for the same x, R (its intermediate is then reused)."""
    import torch
    dt, f32 = x.dtype, torch.float32
    p, nb = _ws(workspace)
    fp = _ws(fwd_workspace)[0] if fwd_workspace is not None else None
    _check(lib().monarch_rect_bwd(_ptr(x, "x"), _ptr(dy, "dy", dt), _ptr(L, "L", dt), _ptr(R, "R", dt), fp,
                                  _ptr(dx, "dx", dt), _ptr(dL, "dL", f32), _ptr(dR, "dR", f32), int(accumulate),
                                  tokens, q, b1, b, r, _dtype_code(x), p, nb, _stream(stream)), "monarch_rect_bwd")


def monarch_rectw_workspace_bytes(tokens: int, q: int, b1: int, b2: int, b3: int, r: int, dtype: int) -> int:
    return int(lib().monarch_rectw_workspace_bytes(tokens, q, b1, b2, b3, r, dtype))


def monarch_rectw_bwd_workspace_bytes(tokens: int, q: int, b1: int, b2: int, b3: int, r: int, dtype: int) -> int:
    return int(lib().monarch_rectw_bwd_workspace_bytes(tokens, q, b1, b2, b3, r, dtype))


def monarch_rectw_fwd(x, L, R, y, tokens, q, b1, b2, b3, r, workspace, stream=None) -> None:
    """y = L R x for the rectangular class with wrapped-diagonal blocks: R [q, b2, b1], L [r, q, max(b2, b3)]."""
    dt = x.dtype
    p, nb = _ws(workspace)
    _check(lib().monarch_rectw_fwd(_ptr(x, "x"), _ptr(L, "L", dt), _ptr(R, "R", dt), _ptr(y, "y", dt), tokens, q, b1, b2,
                                   b3, r, _dtype_code(x), p, nb, _stream(stream)), "monarch_rectw_fwd")


def monarch_rectw_bwd(x, dy, L, R, dx, dL, dR, accumulate, tokens, q, b1, b2, b3, r, workspace, stream=None) -> None:
    """Gradients of <dy, L R x> for the wrapped-diagonal class: dx like x; dL like L and dR like R, in float32."""
    import torch
    dt, f32 = x.dtype, torch.float32
    p, nb = _ws(workspace)
    _check(lib().monarch_rectw_bwd(_ptr(x, "x"), _ptr(dy, "dy", dt), _ptr(L, "L", dt), _ptr(R, "R", dt),
                                   _ptr(dx, "dx", dt), _ptr(dL, "dL", f32), _ptr(dR, "dR", f32), int(accumulate),
                                   tokens, q, b1, b2, b3, r, _dtype_code(x), p, nb, _stream(stream)), "monarch_rectw_bwd")


NOALLOC_SCRATCH_BYTES = 8 << 20


def monarch_fwd_noalloc(x, L, R, y, tokens, n, m, stream=None) -> None:
    """y = P L P^T R x without a workspace, for callers that cannot allocate device memory.

    The intermediate lives in an array built into the library, so the problem must satisfy
    tokens * n * element_size <= NOALLOC_SCRATCH_BYTES; calls share that array, so do not
    let two of them overlap on one GPU (see include/monarch.h).
    """
    dt = x.dtype
    _check(lib().monarch_fwd_noalloc(_ptr(x, "x"), _ptr(L, "L", dt), _ptr(R, "R", dt),
                                     _ptr(y, "y", dt), tokens, n, m, _dtype_code(x),
                                     _stream(stream)), "monarch_fwd_noalloc")


def _hptr(t, name, dtype=None):
    if t.is_cuda:
        raise ValueError(f"{name} must be a host tensor")
    if not t.is_contiguous():
        raise ValueError(f"{name} must be contiguous")
    if dtype is not None and t.dtype != dtype:
        raise TypeError(f"{name} must have dtype {dtype}, got {t.dtype}")
    return t.data_ptr()


class HostContext:
    """Device staging for the host-buffer calls (monarch_host_*): tensors are CPU tensors, ideally
    pinned; every call blocks until its outputs have arrived."""

    _h = None          # so that close() is safe when construction raised

    def __init__(self, max_tokens: int, n: int, m: int, dtype: int, chunk_tokens: int = 0):
        h = _vp()
        _check(lib().monarch_host_create(ctypes.byref(h), max_tokens, n, m, dtype, chunk_tokens),
               "monarch_host_create")
        self._h, self.n, self.m, self.dtype = h, n, m, dtype

    def close(self):
        if self._h:
            lib().monarch_host_destroy(self._h)
            self._h = None

    __del__ = close

    def fwd(self, x, L, R, y, tokens: int) -> None:
        dt = x.dtype
        _check(lib().monarch_host_fwd(self._h, _hptr(x, "x"), _hptr(L, "L", dt), _hptr(R, "R", dt),
                                      _hptr(y, "y", dt), tokens), "monarch_host_fwd")

    def fwd_bwd(self, x, dy, L, R, y, dx, dL, dR, tokens: int) -> None:
        import torch
        dt = x.dtype
        _check(lib().monarch_host_fwd_bwd(self._h, _hptr(x, "x"), _hptr(dy, "dy", dt),
                                          _hptr(L, "L", dt), _hptr(R, "R", dt), _hptr(y, "y", dt),
                                          _hptr(dx, "dx", dt), _hptr(dL, "dL", torch.float32),
                                          _hptr(dR, "dR", torch.float32), tokens),
               "monarch_host_fwd_bwd")
