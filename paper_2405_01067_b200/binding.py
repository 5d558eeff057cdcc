"""ctypes binding of libab.so: same names as the C entry points (include/ab.h), argument
marshalling only.  Tensors are torch CUDA tensors (torch supplies device memory and streams);
every step of the computation runs in the library's kernels.  There is no CPU path: loading
fails loudly when the library has not been built, and every call raises on a negative status.
"""
from __future__ import annotations

import ctypes
import os
from ctypes import c_char_p, c_float, c_int, c_int64, c_size_t, c_void_p

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libab.so")

AB_F32, AB_BF16 = 0, 1
AB_OP_LAYER_FORWARD, AB_OP_LAYER_BACKWARD, AB_OP_GROUP_AVERAGE, AB_OP_RECOMBINE, AB_OP_SVD_SPLIT = range(5)
AB_OP_DENSE_FORWARD, AB_OP_DENSE_BACKWARD = 5, 6
AB_OK = 0
AB_ERR_INVALID_ARG, AB_ERR_UNSUPPORTED, AB_ERR_WORKSPACE = -1, -2, -3
AB_ERR_NOT_CONVERGED, AB_ERR_TIMEOUT, AB_ERR_CUDA, AB_ERR_ACCURACY = -4, -5, -6, -7
AB_SYNC_AUTO, AB_SYNC_DENSE, AB_SYNC_FACTORED = 0, 1, 2

EXPORTS = ["ab_status_string", "ab_version", "ab_launch_count", "ab_workspace_bytes", "ab_layer_forward", "ab_layer_backward",
           "ab_group_average", "ab_recombine", "ab_svd_split", "ab_group_sync", "ab_sync_workspace_bytes",
           "ab_layer_forward_static", "ab_static_scratch_elems", "ab_adamw_step", "ab_lr_rebound_factor", "ab_selftest_bounded_wait",
           "ab_selftest_chain_stall", "ab_selftest_chain_stall_workspace_bytes",
           "ab_dense_forward", "ab_dense_backward", "ab_conv3x3_forward", "ab_conv3x3_backward",
           "ab_conv3x3_workspace_bytes", "ab_recombine_mean"]


class AbError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} ({status})")


class ab_sync_desc(ctypes.Structure):
    _fields_ = [("A_copies", c_void_p), ("B_copies", c_void_p), ("strideA", c_int64), ("strideB", c_int64),
                ("m", c_int), ("n", c_int), ("r", c_int), ("A_out", c_void_p), ("B_out", c_void_p),
                ("sigma", c_void_p), ("r_out", c_void_p), ("W_out", c_void_p)]


_lib = None


def lib() -> ctypes.CDLL:
    """The loaded library.  Raises if it has not been built (python -m paper_2405_01067_b200.build)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: build it with `python paper_2405_01067_b200/build.py`; "
                           "there is no fallback path")
    L = ctypes.CDLL(LIB_PATH)
    L.ab_status_string.restype = c_char_p
    L.ab_status_string.argtypes = [c_int]
    L.ab_version.restype = c_char_p
    L.ab_launch_count.restype = ctypes.c_longlong
    L.ab_workspace_bytes.restype = c_size_t
    L.ab_workspace_bytes.argtypes = [c_int, c_int64, c_int, c_int, c_int, c_int, c_int]
    L.ab_layer_forward.restype = c_int
    L.ab_layer_forward.argtypes = [c_void_p] * 5 + [c_int64] + [c_int] * 6 + [c_void_p, c_size_t, c_void_p]
    L.ab_layer_backward.restype = c_int
    L.ab_layer_backward.argtypes = [c_void_p] * 8 + [c_int64] + [c_int] * 6 + [c_void_p, c_size_t, c_void_p]
    L.ab_group_average.restype = c_int
    L.ab_group_average.argtypes = [c_void_p, c_int64, c_int, c_int64, c_int, c_int, c_void_p, c_void_p]
    L.ab_recombine.restype = c_int
    L.ab_recombine.argtypes = [c_void_p, c_void_p, c_void_p] + [c_int] * 6 + [c_void_p, c_size_t, c_void_p]
    L.ab_svd_split.restype = c_int
    L.ab_svd_split.argtypes = [c_void_p, c_int, c_int, c_int, c_float] + [c_void_p] * 5 + [c_int, c_int,
                                                                                         c_void_p, c_size_t, c_void_p]
    L.ab_group_sync.restype = c_int
    L.ab_group_sync.argtypes = [ctypes.POINTER(ab_sync_desc), c_int, c_int, c_float, c_int, c_void_p, c_void_p,
                                c_size_t, c_void_p, c_int]
    L.ab_sync_workspace_bytes.restype = c_size_t
    L.ab_sync_workspace_bytes.argtypes = [ctypes.POINTER(ab_sync_desc), c_int, c_int, c_int]
    L.ab_layer_forward_static.restype = c_int
    L.ab_layer_forward_static.argtypes = [c_void_p] * 4 + [c_int64] + [c_int] * 6 + [c_void_p]
    L.ab_static_scratch_elems.restype = c_size_t
    L.ab_adamw_step.restype = c_int
    L.ab_adamw_step.argtypes = [c_void_p] * 5 + [c_int64] + [c_float] * 5 + [c_int, c_void_p]
    L.ab_lr_rebound_factor.restype = c_float
    L.ab_lr_rebound_factor.argtypes = [c_int, c_int, c_float]
    L.ab_selftest_bounded_wait.restype = c_int
    L.ab_selftest_bounded_wait.argtypes = [c_void_p, ctypes.c_uint, c_void_p]
    L.ab_selftest_chain_stall.restype = c_int
    L.ab_selftest_chain_stall.argtypes = [c_void_p, c_size_t, ctypes.c_uint, c_void_p]
    L.ab_selftest_chain_stall_workspace_bytes.restype = c_size_t
    L.ab_dense_forward.restype = c_int
    L.ab_dense_forward.argtypes = [c_void_p] * 3 + [c_int64, c_int, c_int, c_int, c_void_p, c_size_t, c_void_p]
    L.ab_dense_backward.restype = c_int
    L.ab_dense_backward.argtypes = [c_void_p] * 5 + [c_int64, c_int, c_int, c_int, c_void_p, c_size_t, c_void_p]
    L.ab_conv3x3_forward.restype = c_int
    L.ab_conv3x3_forward.argtypes = [c_void_p] * 5 + [c_int] * 9 + [c_void_p, c_size_t, c_void_p]
    L.ab_conv3x3_backward.restype = c_int
    L.ab_conv3x3_backward.argtypes = [c_void_p] * 8 + [c_int] * 9 + [c_void_p, c_size_t, c_void_p]
    L.ab_conv3x3_workspace_bytes.restype = c_size_t
    L.ab_conv3x3_workspace_bytes.argtypes = [c_int] * 6
    L.ab_recombine_mean.restype = c_int
    L.ab_recombine_mean.argtypes = [c_void_p, c_int64, c_void_p, c_int64, c_int, c_void_p, c_void_p, c_void_p,
                                    c_int, c_int, c_int, c_int, c_void_p]
    _lib = L
    return L


def ab_selftest_bounded_wait(limit_us: int = 1000, stream=None) -> int:
    """Runs the bounded-wait self-test and returns the device status it left (AB_ERR_TIMEOUT when the wait
    gave up as designed).  Synchronises."""
    status = torch.zeros((1,), dtype=torch.int32, device="cuda")
    _check(lib().ab_selftest_bounded_wait(_ptr(status), int(limit_us), _stream(stream)), "ab_selftest_bounded_wait")
    return int(status.item())


def ab_selftest_chain_stall(limit_us: int = 1000, stream=None) -> int:
    """Runs the fused chain kernel with its loader switched off and returns the device status its unwinding
    left (AB_ERR_TIMEOUT).  Synchronises."""
    ws = workspace(int(lib().ab_selftest_chain_stall_workspace_bytes()), "cuda")
    _check(lib().ab_selftest_chain_stall(_ptr(ws), ws.numel(), int(limit_us), _stream(stream)), "ab_selftest_chain_stall")
    return workspace_status(ws)


def ab_launch_count() -> int:
    return int(lib().ab_launch_count())


def status_string(status: int) -> str:
    return lib().ab_status_string(int(status)).decode()


def _dt(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return AB_F32
    if t.dtype == torch.bfloat16:
        return AB_BF16
    raise TypeError(f"unsupported dtype {t.dtype}")


def _ptr(t):
    return None if t is None else c_void_p(t.data_ptr())


def _stream(stream):
    s = torch.cuda.current_stream() if stream is None else stream
    return c_void_p(s.cuda_stream)


def _check(status: int, where: str):
    if status != AB_OK:
        raise AbError(status, where)


def _dev_ok(*ts):
    for t in ts:
        if t is not None and (not t.is_cuda or not t.is_contiguous()):
            raise ValueError("tensors must be contiguous CUDA tensors")


def workspace(nbytes: int, device) -> torch.Tensor:
    """A 256-byte aligned scratch buffer of at least nbytes (torch's allocator aligns to 512)."""
    return torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=device)


def workspace_status(ws: torch.Tensor) -> int:
    """Device status word a layer call left at the head of its workspace (synchronises)."""
    return int(ws[:4].view(torch.int32).item())


def ab_workspace_bytes(op: int, N: int, m: int, n: int, r: int, K: int = 1, dt: int = AB_F32) -> int:
    return int(lib().ab_workspace_bytes(op, N, m, n, r, K, dt))


def ab_layer_forward(x, A, B, y=None, T_save=None, ws=None, stream=None, save_T=False):
    """y = (x B^T) A^T.  Returns (y, T_save or None)."""
    _dev_ok(x, A, B, y, T_save)
    N, n = x.shape
    m, r = A.shape
    dt = _dt(x)
    if y is None:
        y = torch.empty((N, m), dtype=x.dtype, device=x.device)
    if save_T and T_save is None:
        T_save = torch.empty((N, r), dtype=x.dtype, device=x.device)
    if ws is None:
        ws = workspace(ab_workspace_bytes(AB_OP_LAYER_FORWARD, N, m, n, r, 1, dt), x.device)
    st = lib().ab_layer_forward(_ptr(x), _ptr(A), _ptr(B), _ptr(y), _ptr(T_save), N, m, n, r,
                                A.stride(0), B.stride(0), dt, _ptr(ws), ws.numel(), _stream(stream))
    _check(st, "ab_layer_forward")
    return y, T_save


def ab_layer_forward_static(x, A, B, y, stream=None):
    """y = (x B^T) A^T with the intermediate in the library's built-in scratch array: for callers that
    cannot allocate a workspace.  `y` must be supplied (this call allocates nothing); N*r is limited to
    ab_static_scratch_elems().  Calls that may overlap on the GPU race on the shared array."""
    _dev_ok(x, A, B, y)
    N, n = x.shape
    m, r = A.shape
    st = lib().ab_layer_forward_static(_ptr(x), _ptr(A), _ptr(B), _ptr(y), N, m, n, r, A.stride(0), B.stride(0),
                                       _dt(x), _stream(stream))
    _check(st, "ab_layer_forward_static")
    return y


def ab_layer_backward(x, dY, A, B, T_saved=None, want=("dX", "dA", "dB"), dX=None, dA=None, dB=None,
                      ws=None, stream=None):
    """dX = (dY A) B, dA = dY^T T, dB = (dY A)^T x.  Returns (dX, dA, dB); entries not in `want` are None."""
    _dev_ok(x, dY, A, B, T_saved, dX, dA, dB)
    N, n = x.shape
    m, r = A.shape
    dt = _dt(x)
    if "dX" in want and dX is None:
        dX = torch.empty((N, n), dtype=x.dtype, device=x.device)
    if "dA" in want and dA is None:
        dA = torch.empty((m, r), dtype=torch.float32, device=x.device)
    if "dB" in want and dB is None:
        dB = torch.empty((r, n), dtype=torch.float32, device=x.device)
    if ws is None:
        ws = workspace(ab_workspace_bytes(AB_OP_LAYER_BACKWARD, N, m, n, r, 1, dt), x.device)
    st = lib().ab_layer_backward(_ptr(x), _ptr(dY), _ptr(A), _ptr(B), _ptr(T_saved), _ptr(dX), _ptr(dA), _ptr(dB),
                                 N, m, n, r, A.stride(0), B.stride(0), dt, _ptr(ws), ws.numel(), _stream(stream))
    _check(st, "ab_layer_backward")
    return dX, dA, dB


def ab_conv3x3_workspace_bytes(batch, H, W, C, m, r) -> int:
    return int(lib().ab_conv3x3_workspace_bytes(batch, H, W, C, m, r))


def ab_conv3x3_forward(x, A, B, y=None, T_save=None, ws=None, stream=None, save_T=False):
    """Factorised 3 x 3 convolution on an NHWC activation x [batch, H, W, C].  Returns (y [batch,H,W,m], T or None)."""
    _dev_ok(x, A, B, y, T_save)
    batch, H, W, C = x.shape
    m, r = A.shape
    if y is None:
        y = torch.empty((batch, H, W, m), dtype=x.dtype, device=x.device)
    if save_T and T_save is None:
        T_save = torch.empty((batch * H * W, r), dtype=x.dtype, device=x.device)
    if ws is None:
        ws = workspace(ab_conv3x3_workspace_bytes(batch, H, W, C, m, r), x.device)
    st = lib().ab_conv3x3_forward(_ptr(x), _ptr(A), _ptr(B), _ptr(y), _ptr(T_save), batch, H, W, C, m, r,
                                  A.stride(0), B.stride(0), _dt(x), _ptr(ws), ws.numel(), _stream(stream))
    _check(st, "ab_conv3x3_forward")
    return y, T_save


def ab_conv3x3_backward(x, dY, A, B, T_saved=None, want=("dX", "dA", "dB"), dX=None, dA=None, dB=None, ws=None,
                        stream=None):
    """dX [batch,H,W,C], dA [m,r], dB [r,9C] of the factorised convolution; dY is [batch,H,W,m]."""
    _dev_ok(x, dY, A, B, T_saved, dX, dA, dB)
    batch, H, W, C = x.shape
    m, r = A.shape
    if "dX" in want and dX is None:
        dX = torch.empty_like(x)
    if "dA" in want and dA is None:
        dA = torch.empty((m, r), dtype=torch.float32, device=x.device)
    if "dB" in want and dB is None:
        dB = torch.empty((r, 9 * C), dtype=torch.float32, device=x.device)
    if ws is None:
        ws = workspace(ab_conv3x3_workspace_bytes(batch, H, W, C, m, r), x.device)
    st = lib().ab_conv3x3_backward(_ptr(x), _ptr(dY), _ptr(A), _ptr(B), _ptr(T_saved), _ptr(dX), _ptr(dA), _ptr(dB),
                                   batch, H, W, C, m, r, A.stride(0), B.stride(0), _dt(x), _ptr(ws), ws.numel(),
                                   _stream(stream))
    _check(st, "ab_conv3x3_backward")
    return dX, dA, dB


def ab_dense_forward(x, W, y=None, ws=None, stream=None):
    """y = x W^T with W held dense (the full-rank phases of a cycle)."""
    _dev_ok(x, W, y)
    N, n = x.shape
    m = W.shape[0]
    dt = _dt(x)
    if y is None:
        y = torch.empty((N, m), dtype=x.dtype, device=x.device)
    if ws is None:
        ws = workspace(ab_workspace_bytes(AB_OP_DENSE_FORWARD, N, m, n, 0, 1, dt), x.device)
    st = lib().ab_dense_forward(_ptr(x), _ptr(W), _ptr(y), N, m, n, dt, _ptr(ws), ws.numel(), _stream(stream))
    _check(st, "ab_dense_forward")
    return y


def ab_dense_backward(x, dY, W, want=("dX", "dW"), dX=None, dW=None, ws=None, stream=None):
    """dX = dY W, dW = dY^T x (fp32).  Returns (dX, dW); entries not in `want` are None."""
    _dev_ok(x, dY, W, dX, dW)
    N, n = x.shape
    m = W.shape[0]
    dt = _dt(x)
    if "dX" in want and dX is None:
        dX = torch.empty((N, n), dtype=x.dtype, device=x.device)
    if "dW" in want and dW is None:
        dW = torch.empty((m, n), dtype=torch.float32, device=x.device)
    if ws is None:
        ws = workspace(ab_workspace_bytes(AB_OP_DENSE_BACKWARD, N, m, n, 0, 1, dt), x.device)
    st = lib().ab_dense_backward(_ptr(x), _ptr(dY), _ptr(W), _ptr(dX), _ptr(dW), N, m, n, dt, _ptr(ws), ws.numel(),
                                 _stream(stream))
    _check(st, "ab_dense_backward")
    return dX, dW


def ab_adamw_step(param, grad, m, v, lr, step, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=1e-2, param_bf16=None,
                  stream=None):
    """One AdamW update in place (param, m, v fp32; grad fp32); param_bf16 optionally receives the rounded copy."""
    _dev_ok(param, grad, m, v, param_bf16)
    for t in (param, grad, m, v):
        if t.dtype != torch.float32 or not t.is_contiguous():
            raise ValueError("ab_adamw_step takes contiguous fp32 tensors")
    if param_bf16 is not None and (param_bf16.dtype != torch.bfloat16 or param_bf16.numel() != param.numel()):
        raise ValueError("param_bf16 must be a bf16 tensor of the same size")
    st = lib().ab_adamw_step(_ptr(param), _ptr(grad), _ptr(m), _ptr(v), _ptr(param_bf16), param.numel(), lr, beta1, beta2,
                             eps, weight_decay, step, _stream(stream))
    _check(st, "ab_adamw_step")
    return param


def ab_lr_rebound_factor(steps_since_change: int, rebound_steps: int, floor: float = 0.0) -> float:
    return float(lib().ab_lr_rebound_factor(steps_since_change, rebound_steps, floor))


def ab_group_average(copies, out=None, out_dtype=None, stream=None):
    """Mean over the leading axis of a (K, ...) tensor, fp32 sum in ascending k."""
    _dev_ok(copies, out)
    K = copies.shape[0]
    count = copies[0].numel()
    if out is None:
        out = torch.empty(copies.shape[1:], dtype=out_dtype or torch.float32, device=copies.device)
    st = lib().ab_group_average(_ptr(copies), copies.stride(0) if K > 1 else count, K, count, _dt(copies), _dt(out),
                                _ptr(out), _stream(stream))
    _check(st, "ab_group_average")
    return out


def ab_recombine(Abar, Bbar, W=None, ws=None, stream=None):
    """W = Abar Bbar in fp32."""
    _dev_ok(Abar, Bbar, W)
    m, r = Abar.shape
    n = Bbar.shape[1]
    if W is None:
        W = torch.empty((m, n), dtype=torch.float32, device=Abar.device)
    if ws is None:
        ws = workspace(ab_workspace_bytes(AB_OP_RECOMBINE, 0, m, n, r, 1, _dt(Abar)), Abar.device)
    st = lib().ab_recombine(_ptr(Abar), _ptr(Bbar), _ptr(W), m, n, r, Abar.stride(0), Bbar.stride(0), _dt(Abar),
                            _ptr(ws), ws.numel(), _stream(stream))
    _check(st, "ab_recombine")
    return W


def ab_recombine_mean(A_copies, B_copies, W=None, Abar=None, Bbar=None, want_means=True, stream=None):
    """W = mean_k(A_k) mean_k(B_k) in one kernel; A_copies (K, m, r), B_copies (K, r, n), fp32.
    Returns (W, Abar, Bbar) (the means are None when want_means is False and none were passed)."""
    _dev_ok(A_copies, B_copies, W, Abar, Bbar)
    K, m, r = A_copies.shape
    n = B_copies.shape[2]
    dev = A_copies.device
    if W is None:
        W = torch.empty((m, n), dtype=torch.float32, device=dev)
    if want_means and Abar is None:
        Abar = torch.empty((m, r), dtype=torch.float32, device=dev)
    if want_means and Bbar is None:
        Bbar = torch.empty((r, n), dtype=torch.float32, device=dev)
    st = lib().ab_recombine_mean(_ptr(A_copies), A_copies.stride(0) if K > 1 else m * r, _ptr(B_copies),
                                 B_copies.stride(0) if K > 1 else r * n, K, _ptr(W), _ptr(Abar), _ptr(Bbar), m, n, r,
                                 _dt(A_copies), _stream(stream))
    _check(st, "ab_recombine_mean")
    return W, Abar, Bbar


def ab_svd_split(W, r_max, sigma_cutoff=0.0, out_dtype=None, ws=None, stream=None):
    """A = U_r' S^(1/2), B = S^(1/2) V_r'^T under the rank rule.  Returns (A, B, sigma, r_out, dev_status);
    r_out and dev_status are device int tensors (read them after synchronising)."""
    _dev_ok(W)
    m, n = W.shape
    od = out_dtype or W.dtype
    r_cap = min(r_max, m, n)
    A = torch.empty((m, r_max), dtype=od, device=W.device)
    B = torch.empty((r_max, n), dtype=od, device=W.device)
    sigma = torch.empty((r_cap,), dtype=torch.float32, device=W.device)
    r_out = torch.zeros((1,), dtype=torch.int32, device=W.device)
    status = torch.zeros((1,), dtype=torch.int32, device=W.device)
    if ws is None:
        ws = workspace(ab_workspace_bytes(AB_OP_SVD_SPLIT, 0, m, n, r_max, 1, _dt(W)), W.device)
    st = lib().ab_svd_split(_ptr(W), m, n, r_max, float(sigma_cutoff), _ptr(A), _ptr(B), _ptr(sigma), _ptr(r_out),
                            _ptr(status), _dt(W), AB_BF16 if od == torch.bfloat16 else AB_F32, _ptr(ws), ws.numel(),
                            _stream(stream))
    _check(st, "ab_svd_split")
    return A, B, sigma, r_out, status


class SyncPlan:
    """Buffers and descriptors of one model's group synchronisation (ab_group_sync)."""

    def __init__(self, A_copies, B_copies, sigma_cutoff, want_W=False, strided=False):
        """A_copies[i]: (K, m, r), B_copies[i]: (K, r, n).  strided=True accepts views whose copies are
        each contiguous but spaced by any stride along the leading axis (e.g. slices of a packed arena)."""
        self.A_copies, self.B_copies = list(A_copies), list(B_copies)
        self.L = len(self.A_copies)
        self.K = self.A_copies[0].shape[0]
        self.cutoff = float(sigma_cutoff)
        dev = self.A_copies[0].device
        self.dt = _dt(self.A_copies[0])
        self.A_out, self.B_out, self.sigma, self.W_out = [], [], [], []
        self.r_out = torch.zeros((self.L,), dtype=torch.int32, device=dev)
        self.status = torch.zeros((self.L,), dtype=torch.int32, device=dev)
        self.descs = (ab_sync_desc * self.L)()
        for i, (Ak, Bk) in enumerate(zip(self.A_copies, self.B_copies)):
            if strided:
                if not (Ak.is_cuda and Bk.is_cuda and Ak[0].is_contiguous() and Bk[0].is_contiguous()):
                    raise ValueError("each copy must be a contiguous CUDA tensor")
            else:
                _dev_ok(Ak, Bk)
            K, m, r = Ak.shape
            n = Bk.shape[2]
            self.A_out.append(torch.empty((m, r), dtype=Ak.dtype, device=dev))
            self.B_out.append(torch.empty((r, n), dtype=Ak.dtype, device=dev))
            self.sigma.append(torch.empty((min(r, m, n),), dtype=torch.float32, device=dev))
            d = self.descs[i]
            d.A_copies, d.B_copies = Ak.data_ptr(), Bk.data_ptr()
            d.strideA, d.strideB = (Ak.stride(0), Bk.stride(0)) if K > 1 else (m * r, r * n)
            d.m, d.n, d.r = m, n, r
            d.A_out, d.B_out = self.A_out[i].data_ptr(), self.B_out[i].data_ptr()
            d.sigma = self.sigma[i].data_ptr()
            d.r_out = self.r_out.data_ptr() + 4 * i
            if want_W:
                self.W_out.append(torch.empty((m, n), dtype=torch.float32, device=dev))
                d.W_out = self.W_out[i].data_ptr()
            else:
                d.W_out = None
        self.ws = workspace(lib().ab_sync_workspace_bytes(self.descs, self.L, self.K, self.dt), dev)


def ab_group_sync(plan: SyncPlan, stream=None, path=AB_SYNC_AUTO):
    """Mean of K copies -> W = Abar Bbar -> split under the rank rule, for every matrix of the plan.
    path: AB_SYNC_AUTO / AB_SYNC_DENSE (forms W, dense split) / AB_SYNC_FACTORED (r x r problems only)."""
    st = lib().ab_group_sync(plan.descs, plan.L, plan.K, plan.cutoff, plan.dt, _ptr(plan.status), _ptr(plan.ws),
                             plan.ws.numel(), _stream(stream), int(path))
    _check(st, "ab_group_sync")
    return plan.A_out, plan.B_out, plan.sigma, plan.r_out, plan.status
