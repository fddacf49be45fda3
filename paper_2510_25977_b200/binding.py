"""ctypes binding of libsvdmlp (argument marshalling only: every step runs in the CUDA library).

The functions carry the names of the C entry points declared in include/svdmlp.h.  Tensors are
torch CUDA tensors used purely as device memory; streams are torch streams.  There is no CPU
path: if the shared library is missing, or a call returns an error status, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libsvdmlp.so")

OK = 0
FLAG_Y_FP32 = 0x1
FLAG_PATH_SKINNY = 0x10
FLAG_PATH_TENSOR = 0x20
FLAG_DECODE_REGISTERS = 0x40
FLAG_NO_CTA_PAIRS = 0x80
FLAG_NO_TMEM_STRIP = 0x100
FLAG_NO_WIDE_GATEUP = 0x200
FLAG_NO_CLUSTER_SPLITK = 0x2000
FLAG_DECODE_COOPERATIVE = 0x400
FLAG_TOKEN_SLABS = 0x800
FLAG_NO_FUSED_DOWN1 = 0x1000

EXPORTS = ["svdmlp_create", "svdmlp_forward", "svdmlp_forward_host", "svdmlp_forward_prenorm_residual",
           "svdmlp_forward_partial", "svdmlp_forward_finish",
           "svdmlp_forward_partial_push", "svdmlp_forward_finish_gather", "svdmlp_tp_recv_bytes", "svdmlp_tp_wait_limit_ns",
           "svdlinear_forward", "svdlinear_workspace_bytes", "svdlinear_forward_noalloc",
           "svdlinear_create", "svdlinear_apply", "svdlinear_apply_layout", "svdlinear_destroy",
           "svdmlp_compress", "svdmlp_compress_workspace_bytes", "svdmlp_destroy", "svdmlp_strerror",
           "svdmlp_last_device_status", "svdmlp_launch_count", "svdmlp_path_name",
           "svdmlp_profile_enable", "svdmlp_profile_read", "svdmlp_profile_name", "svdmlp_stage_mask",
           "svdmlp_block_aligned_rank", "svdmlp_model", "svdmlp_selftest_timeout"]

_lib = None


class TpPeers(ctypes.Structure):
    """svdmlp_tp_peers_t: the receive buffers and flag words of all ranks, as addressed from this rank."""
    _fields_ = [("world", ctypes.c_int), ("rank", ctypes.c_int), ("recv", ctypes.c_void_p * 8), ("flags", ctypes.c_void_p * 8)]


class Model(ctypes.Structure):
    """svdmlp_model_t: the capacity / intensity model of one shape (field meanings: include/svdmlp.h)."""
    _fields_ = [(n, ctypes.c_int) for n in ("d", "ffn", "r", "T", "path", "strip_rows", "z_in_tmem", "tmem_cols_strip",
                                            "tmem_cols_acc", "tmem_cols_zd", "tmem_cols_total")] + \
               [("smem_bytes", ctypes.c_long)] + \
               [(n, ctypes.c_double) for n in ("flops", "hbm_bytes", "sm_bytes", "intensity_hbm", "intensity_sm", "ridge_hbm",
                                               "t_tensor_us", "t_hbm_us", "t_floor_us")]

    def as_dict(self):
        return {n: getattr(self, n) for n, _ in self._fields_}


class SvdMlpError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {strerror(status)} (status {status})")


def lib() -> ctypes.CDLL:
    """Load the library; raises OSError if it has not been built (python -m paper_2510_25977_b200.build)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise OSError(f"{LIB_PATH} not found: build it first (paper_2510_25977_b200/build.py); there is no fallback")
        L = ctypes.CDLL(LIB_PATH)
        vp, ci, cu = ctypes.c_void_p, ctypes.c_int, ctypes.c_uint
        L.svdmlp_create.restype = ci
        L.svdmlp_create.argtypes = [ctypes.POINTER(vp), ci, ci, ci, ci, ci, vp, vp, vp, vp, vp, vp, ci, cu, vp]
        L.svdmlp_forward.restype = ci
        L.svdmlp_forward.argtypes = [vp, vp, ci, vp, vp]
        L.svdmlp_forward_partial.restype = ci
        L.svdmlp_forward_partial.argtypes = [vp, vp, ci, vp, vp]
        L.svdmlp_forward_finish.restype = ci
        L.svdmlp_forward_finish.argtypes = [vp, vp, ci, vp, vp]
        L.svdmlp_forward_host.restype = ci
        L.svdmlp_forward_host.argtypes = [vp, vp, ci, vp, vp]
        L.svdmlp_forward_prenorm_residual.restype = ci
        L.svdmlp_forward_prenorm_residual.argtypes = [vp, vp, vp, ci, ctypes.c_float, vp]
        L.svdlinear_forward.restype = ci
        L.svdlinear_forward.argtypes = [vp, ci, ci, ci, ci, vp, vp, vp, vp, ctypes.c_size_t, vp]
        L.svdlinear_forward_noalloc.restype = ci
        L.svdlinear_forward_noalloc.argtypes = [vp, ci, ci, ci, ci, vp, vp, vp, vp]
        L.svdmlp_compress.restype = ci
        L.svdmlp_compress.argtypes = [vp, ci, ci, ci, vp, vp, ctypes.POINTER(ctypes.c_float), vp, ctypes.c_size_t, cu, vp]
        L.svdmlp_compress_workspace_bytes.restype = ctypes.c_size_t
        L.svdmlp_compress_workspace_bytes.argtypes = [ci, ci]
        L.svdlinear_create.restype = ci
        L.svdlinear_create.argtypes = [ctypes.POINTER(vp), ci, ci, ci, vp, vp, ci, vp]
        L.svdlinear_apply.restype = ci
        L.svdlinear_apply.argtypes = [vp, vp, ci, vp, vp]
        L.svdlinear_apply_layout.restype = ci
        L.svdlinear_apply_layout.argtypes = [vp, vp, ci, vp, cu, vp]
        L.svdlinear_destroy.restype = ci
        L.svdlinear_destroy.argtypes = [vp]
        L.svdlinear_workspace_bytes.restype = ctypes.c_size_t
        L.svdlinear_workspace_bytes.argtypes = [ci, ci, ci, ci]
        L.svdmlp_destroy.restype = ci
        L.svdmlp_destroy.argtypes = [vp]
        L.svdmlp_strerror.restype = ctypes.c_char_p
        L.svdmlp_strerror.argtypes = [ci]
        L.svdmlp_last_device_status.restype = ci
        L.svdmlp_last_device_status.argtypes = [vp]
        L.svdmlp_launch_count.restype = ctypes.c_ulonglong
        L.svdmlp_launch_count.argtypes = [vp]
        L.svdmlp_path_name.restype = ctypes.c_char_p
        L.svdmlp_path_name.argtypes = [vp, ci]
        L.svdmlp_block_aligned_rank.restype = ci
        L.svdmlp_block_aligned_rank.argtypes = [ci, ci, ctypes.c_double, ci, ctypes.c_double]
        L.svdmlp_tp_recv_bytes.restype = ctypes.c_size_t
        L.svdmlp_tp_recv_bytes.argtypes = [ci, ci, ci]
        L.svdmlp_forward_partial_push.restype = ci
        L.svdmlp_forward_partial_push.argtypes = [vp, vp, ci, ctypes.POINTER(TpPeers), ctypes.c_ulonglong, vp]
        L.svdmlp_forward_finish_gather.restype = ci
        L.svdmlp_forward_finish_gather.argtypes = [vp, vp, vp, ci, ctypes.c_ulonglong, ci, vp, vp]
        L.svdmlp_tp_wait_limit_ns.restype = ci
        L.svdmlp_tp_wait_limit_ns.argtypes = [vp, ctypes.c_ulonglong]
        L.svdmlp_model.restype = ci
        L.svdmlp_model.argtypes = [ci, ci, ci, ci, ctypes.c_double, ctypes.c_double, ctypes.c_double, ctypes.POINTER(Model)]
        L.svdmlp_selftest_timeout.restype = ci
        L.svdmlp_selftest_timeout.argtypes = [vp, cu, vp]
        L.svdmlp_stage_mask.restype = ci
        L.svdmlp_stage_mask.argtypes = [vp, cu]
        L.svdmlp_profile_enable.restype = ci
        L.svdmlp_profile_enable.argtypes = [vp, ci]
        L.svdmlp_profile_read.restype = ci
        L.svdmlp_profile_read.argtypes = [vp, ctypes.POINTER(ctypes.c_float), ci]
        L.svdmlp_profile_name.restype = ctypes.c_char_p
        L.svdmlp_profile_name.argtypes = [vp, ci]
        _lib = L
    return _lib


def strerror(status: int) -> str:
    return lib().svdmlp_strerror(int(status)).decode()


def _stream(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return int(stream.cuda_stream) if hasattr(stream, "cuda_stream") else int(stream)


def _ptr(t) -> int:
    return int(t.data_ptr()) if hasattr(t, "data_ptr") else int(t)


def _check(status: int, where: str):
    if status != OK:
        raise SvdMlpError(status, where)


def svdmlp_create_raw(d, ffn, r_gate, r_up, r_down, Ug, Vg, Uu, Vu, Ud, Vd, max_T, flags=0, stream=0):
    """Direct call with integer pointers; returns (status, handle).  Usable without a GPU to
    exercise host-side validation."""
    h = ctypes.c_void_p()
    st = lib().svdmlp_create(ctypes.byref(h), d, ffn, r_gate, r_up, r_down, Ug, Vg, Uu, Vu, Ud, Vd, max_T, flags, stream)
    return st, h


class Handle:
    """Owns one svdmlp_t and keeps the factor tensors alive (the library borrows their memory)."""

    def __init__(self, ptr, keep, d, ffn, flags, max_T):
        self.ptr, self._keep, self.d, self.ffn, self.flags, self.max_T = ptr, keep, d, ffn, flags, max_T

    def close(self):
        if self.ptr:
            lib().svdmlp_destroy(self.ptr)
            self.ptr = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def svdmlp_create(Ug, Vg, Uu, Vu, Ud, Vd, max_T: int, flags: int = 0, stream=None) -> Handle:
    for t in (Ug, Vg, Uu, Vu, Ud, Vd):
        if not (t.is_cuda and t.dtype == torch.bfloat16 and t.is_contiguous()):
            raise ValueError("factor tensors must be contiguous bf16 CUDA tensors")
    ffn, rg = Ug.shape
    ru, d = Vu.shape
    rd = Ud.shape[1]
    if Vg.shape != (rg, d) or Uu.shape != (ffn, ru) or Ud.shape != (d, rd) or Vd.shape != (rd, ffn):
        raise ValueError("inconsistent factor shapes")
    st, h = svdmlp_create_raw(d, ffn, rg, ru, rd, _ptr(Ug), _ptr(Vg), _ptr(Uu), _ptr(Vu), _ptr(Ud), _ptr(Vd),
                              max_T, flags, _stream(stream))
    _check(st, "svdmlp_create")
    return Handle(h, (Ug, Vg, Uu, Vu, Ud, Vd), d, ffn, flags, max_T)


def svdmlp_forward(h: Handle, X: torch.Tensor, Y: torch.Tensor | None = None, stream=None) -> torch.Tensor:
    T = X.shape[0]
    if Y is None:
        Y = torch.empty((T, h.d), dtype=torch.float32 if h.flags & FLAG_Y_FP32 else torch.bfloat16, device=X.device)
    _check(lib().svdmlp_forward(h.ptr, _ptr(X), T, _ptr(Y), _stream(stream)), "svdmlp_forward")
    return Y


def svdmlp_forward_partial(h: Handle, X: torch.Tensor, Zd: torch.Tensor | None = None, stream=None) -> torch.Tensor:
    """This handle's (shard's) fp32 Zd[T, r_down]; the caller sums it over the shards."""
    T = X.shape[0]
    if Zd is None:
        Zd = torch.empty((T, h._keep[4].shape[1]), dtype=torch.float32, device=X.device)
    _check(lib().svdmlp_forward_partial(h.ptr, _ptr(X), T, _ptr(Zd), _stream(stream)), "svdmlp_forward_partial")
    return Zd


def svdmlp_forward_finish(h: Handle, Zd: torch.Tensor, Y: torch.Tensor | None = None, stream=None) -> torch.Tensor:
    T = Zd.shape[0]
    if Y is None:
        Y = torch.empty((T, h.d), dtype=torch.float32 if h.flags & FLAG_Y_FP32 else torch.bfloat16, device=Zd.device)
    _check(lib().svdmlp_forward_finish(h.ptr, _ptr(Zd), T, _ptr(Y), _stream(stream)), "svdmlp_forward_finish")
    return Y


def svdmlp_forward_host(h: Handle, X_host: torch.Tensor, Y_host: torch.Tensor, stream=None) -> torch.Tensor:
    _check(lib().svdmlp_forward_host(h.ptr, _ptr(X_host), X_host.shape[0], _ptr(Y_host), _stream(stream)),
           "svdmlp_forward_host")
    return Y_host


def svdmlp_forward_prenorm_residual(h: Handle, h_in: torch.Tensor, h_out: torch.Tensor | None = None,
                                    eps: float = 1e-5, stream=None) -> torch.Tensor:
    if h_out is None:
        h_out = torch.empty_like(h_in)
    _check(lib().svdmlp_forward_prenorm_residual(h.ptr, _ptr(h_in), _ptr(h_out), h_in.shape[0], eps, _stream(stream)),
           "svdmlp_forward_prenorm_residual")
    return h_out


def svdmlp_tp_recv_bytes(world: int, max_T: int, r_down: int) -> int:
    return int(lib().svdmlp_tp_recv_bytes(world, max_T, r_down))


def tp_peers(rank: int, recv_ptrs, flag_ptrs) -> TpPeers:
    p = TpPeers()
    p.world, p.rank = len(recv_ptrs), rank
    for i, (r, f) in enumerate(zip(recv_ptrs, flag_ptrs)):
        p.recv[i], p.flags[i] = r, f
    return p


def svdmlp_forward_partial_push(h: Handle, X, peers: TpPeers, step: int, stream=None):
    _check(lib().svdmlp_forward_partial_push(h.ptr, _ptr(X), X.shape[0], ctypes.byref(peers), step, _stream(stream)),
           "svdmlp_forward_partial_push")


def svdmlp_forward_finish_gather(h: Handle, recv, flags, world: int, step: int, T: int, Y=None, stream=None):
    if Y is None:
        Y = torch.empty((T, h.d), dtype=torch.float32 if h.flags & FLAG_Y_FP32 else torch.bfloat16, device=recv.device)
    _check(lib().svdmlp_forward_finish_gather(h.ptr, _ptr(recv), _ptr(flags), world, step, T, _ptr(Y), _stream(stream)),
           "svdmlp_forward_finish_gather")
    return Y


def svdmlp_tp_wait_limit_ns(h: Handle, ns: int):
    _check(lib().svdmlp_tp_wait_limit_ns(h.ptr, ns), "svdmlp_tp_wait_limit_ns")


def svdmlp_block_aligned_rank(k: int, n: int, ratio: float, block: int, alpha: float = 0.5) -> int:
    r = int(lib().svdmlp_block_aligned_rank(k, n, ratio, block, alpha))
    if r < 0:
        raise SvdMlpError(r, "svdmlp_block_aligned_rank")
    return r


def svdmlp_model(d: int, ffn: int, r: int, T: int, tensor_tflops: float = 0.0, hbm_gbs: float = 0.0, l2_bytes: float = 0.0) -> dict:
    m = Model()
    _check(lib().svdmlp_model(d, ffn, r, T, tensor_tflops, hbm_gbs, l2_bytes, ctypes.byref(m)), "svdmlp_model")
    return m.as_dict()


def svdlinear_workspace_bytes(T: int, n_in: int, n_out: int, r: int) -> int:
    return int(lib().svdlinear_workspace_bytes(T, n_in, n_out, r))


def svdlinear_forward(X, U, V, Y=None, workspace=None, stream=None) -> torch.Tensor:
    T, n_in = X.shape
    n_out, r = U.shape
    if Y is None:
        Y = torch.empty((T, n_out), dtype=torch.bfloat16, device=X.device)
    need = svdlinear_workspace_bytes(T, n_in, n_out, r)
    if workspace is None:
        workspace = torch.empty(need, dtype=torch.uint8, device=X.device)
    _check(lib().svdlinear_forward(_ptr(X), T, n_in, n_out, r, _ptr(U), _ptr(V), _ptr(Y), _ptr(workspace),
                                   workspace.numel(), _stream(stream)), "svdlinear_forward")
    return Y


class LinearHandle:
    """Owns one svdlinear_t and keeps U and V alive (the library borrows their memory)."""

    def __init__(self, ptr, keep, n_out):
        self.ptr, self._keep, self.n_out = ptr, keep, n_out

    def close(self):
        if self.ptr:
            lib().svdlinear_destroy(self.ptr)
            self.ptr = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def svdlinear_create(U, V, max_T: int, stream=None) -> LinearHandle:
    n_out, r = U.shape
    n_in = V.shape[1]
    h = ctypes.c_void_p()
    _check(lib().svdlinear_create(ctypes.byref(h), n_in, n_out, r, _ptr(U), _ptr(V), max_T, _stream(stream)), "svdlinear_create")
    return LinearHandle(h, (U, V), n_out)


def svdlinear_apply(h: LinearHandle, X, Y=None, stream=None) -> torch.Tensor:
    if Y is None:
        Y = torch.empty((X.shape[0], h.n_out), dtype=torch.bfloat16, device=X.device)
    _check(lib().svdlinear_apply(h.ptr, _ptr(X), X.shape[0], _ptr(Y), _stream(stream)), "svdlinear_apply")
    return Y


X_TRANSPOSED, Y_TRANSPOSED = 0x1, 0x2


def svdlinear_apply_layout(h: LinearHandle, X, layout: int, Y=None, stream=None) -> torch.Tensor:
    """svdlinear_apply with Algorithm 2's layout flags: X_TRANSPOSED: X is X^T[in, T]; Y_TRANSPOSED: the result is
    Y^T[out, T]."""
    T = X.shape[1] if layout & X_TRANSPOSED else X.shape[0]
    if Y is None:
        shape = (h.n_out, T) if layout & Y_TRANSPOSED else (T, h.n_out)
        Y = torch.empty(shape, dtype=torch.bfloat16, device=X.device)
    _check(lib().svdlinear_apply_layout(h.ptr, _ptr(X), T, _ptr(Y), layout, _stream(stream)), "svdlinear_apply_layout")
    return Y


def svdlinear_destroy(h: LinearHandle):
    h.close()


COMPRESS_SPLIT_SQRT = 0x1


def svdmlp_compress(W: torch.Tensor, r: int, flags: int = 0, stream=None):
    """Rank-r factors of a dense fp32 CUDA weight W[out, in]: (U[out, r], V[r, in]) bf16 and all singular values
    (a CPU float tensor, descending)."""
    if not (W.is_cuda and W.dtype == torch.float32 and W.is_contiguous()):
        raise ValueError("W must be a contiguous fp32 CUDA tensor")
    n_out, n_in = W.shape
    U = torch.empty((n_out, r), dtype=torch.bfloat16, device=W.device)
    V = torch.empty((r, n_in), dtype=torch.bfloat16, device=W.device)
    sigma = (ctypes.c_float * min(n_out, n_in))()
    ws = torch.empty(int(lib().svdmlp_compress_workspace_bytes(n_out, n_in)), dtype=torch.uint8, device=W.device)
    _check(lib().svdmlp_compress(_ptr(W), n_out, n_in, r, _ptr(U), _ptr(V), sigma, _ptr(ws), ws.numel(), flags, _stream(stream)),
           "svdmlp_compress")
    return U, V, torch.tensor(list(sigma), dtype=torch.float32)


NOALLOC_MAX_T = 32
NOALLOC_MAX_ELEMS = 32768
NOALLOC_MAX_R = 7232


def svdlinear_forward_noalloc(X, U, V, Y, stream=None) -> torch.Tensor:
    """XUV operator for callers that must not allocate: Y is caller-provided and the library's
    built-in 128 KiB scratch array holds the intermediate (T <= 32, T * r <= 32768, r <= 7232).  Calls that
    may overlap on the GPU race on that array; the first call per device should precede any
    stream capture."""
    T, n_in = X.shape
    n_out, r = U.shape
    _check(lib().svdlinear_forward_noalloc(_ptr(X), T, n_in, n_out, r, _ptr(U), _ptr(V), _ptr(Y), _stream(stream)),
           "svdlinear_forward_noalloc")
    return Y


def svdmlp_selftest_timeout(h: Handle, limit_us: int = 1000, stream=None) -> None:
    _check(lib().svdmlp_selftest_timeout(h.ptr, limit_us, _stream(stream)), "svdmlp_selftest_timeout")


def svdmlp_destroy(h: Handle):
    h.close()


def svdmlp_last_device_status(h: Handle) -> int:
    return int(lib().svdmlp_last_device_status(h.ptr))


def svdmlp_launch_count(h: Handle) -> int:
    return int(lib().svdmlp_launch_count(h.ptr))


def svdmlp_path_name(h: Handle, T: int) -> str:
    return lib().svdmlp_path_name(h.ptr, T).decode()


def svdmlp_profile_enable(h: Handle, enable: bool = True):
    _check(lib().svdmlp_profile_enable(h.ptr, 1 if enable else 0), "svdmlp_profile_enable")


def svdmlp_profile_read(h: Handle) -> list[tuple[str, float]]:
    """(kernel label, milliseconds) for each kernel of the most recent forward call."""
    buf = (ctypes.c_float * 16)()
    n = lib().svdmlp_profile_read(h.ptr, buf, 16)
    if n < 0:
        raise SvdMlpError(n, "svdmlp_profile_read")
    return [(lib().svdmlp_profile_name(h.ptr, i).decode(), float(buf[i])) for i in range(min(n, 16))]


def svdmlp_stage_mask(h: Handle, mask: int):
    """Measurement aid: launch only the selected kernels of the path in later forwards."""
    _check(lib().svdmlp_stage_mask(h.ptr, mask & 0xFFFFFFFF), "svdmlp_stage_mask")
