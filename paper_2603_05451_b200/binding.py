"""ctypes binding of the C-ABI attention library: argument marshalling only.

Function names and argument order follow `include/fa.h`.  Tensors are torch CUDA tensors
(used purely as device memory); every step of the computation runs in the CUDA kernels of
`libfa_b200.so`.  There is no fallback: a missing library or a failing call raises.
"""

import ctypes
import os

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libfa_b200.so")

FA_OK = 0
FA_ERR_INVALID_ARGUMENT = 1
FA_ERR_UNSUPPORTED = 2
FA_ERR_CUDA = 3
FA_ERR_WORKSPACE = 4
FA_ERR_DEVICE_TIMEOUT = 5

_lib = None


class FaError(RuntimeError):
    def __init__(self, status, where):
        self.status = status
        super().__init__(f"{where}: status {status} ({status_string(status)})")


def lib():
    """Loads libfa_b200.so (built by `build.py`); raises if it is not there."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: run __graft_entry__.build() (there is no CPU fallback)")
        l = ctypes.CDLL(LIB_PATH)
        vp, i, f, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_float, ctypes.c_size_t
        l.fa_fwd.argtypes = [vp, vp, vp, vp, vp, i, i, i, i, i, i, f, i, vp]
        l.fa_fwd.restype = i
        l.fa_fwd_f16.argtypes = l.fa_fwd.argtypes
        l.fa_fwd_f16.restype = i
        l.fa_fwd_hdim.argtypes = [vp, vp, vp, vp, vp, i, i, i, i, i, i, i, f, i, vp]
        l.fa_fwd_hdim.restype = i
        l.fa_fwd_varlen.argtypes = [vp] * 8 + [i] * 7 + [f, i, vp]
        l.fa_fwd_varlen.restype = i
        l.fa_varlen_lpt_order.argtypes = [vp, vp, i, i, vp, vp]
        l.fa_varlen_lpt_order.restype = i
        l.fa_bwd_varlen_workspace_bytes.argtypes = [i, i, i, i]
        l.fa_bwd_varlen_workspace_bytes.restype = sz
        l.fa_bwd_varlen.argtypes = [vp] * 11 + [i] * 8 + [f, i, vp, sz, vp]
        l.fa_bwd_varlen.restype = i
        l.fa_bwd_workspace_bytes.argtypes = [i, i, i, i, i, i]
        l.fa_bwd_workspace_bytes.restype = sz
        l.fa_bwd.argtypes = [vp] * 9 + [i, i, i, i, i, i, f, i, vp, sz, vp]
        l.fa_bwd.restype = i
        l.fa_bwd_deterministic.argtypes = l.fa_bwd.argtypes
        l.fa_bwd_f16.argtypes = l.fa_bwd.argtypes
        l.fa_bwd_f16.restype = i
        l.fa_bwd_deterministic.restype = i
        l.fa_bwd_deterministic_f16.argtypes = l.fa_bwd.argtypes
        l.fa_bwd_deterministic_f16.restype = i
        l.fa_status_string.argtypes = [i]
        l.fa_status_string.restype = ctypes.c_char_p
        l.fa_last_device_status.argtypes = [vp]
        l.fa_last_device_status.restype = i
        l.fa_exp2_emulated.argtypes = [vp, vp, sz, vp]
        l.fa_exp2_emulated.restype = i
        l.fa_selftest_per_device_flags.argtypes = []
        l.fa_selftest_per_device_flags.restype = i
        l.fa_selftest_unsatisfied_wait.argtypes = [vp]
        l.fa_selftest_unsatisfied_wait.restype = i
        _lib = l
    return _lib


def status_string(status):
    return lib().fa_status_string(int(status)).decode()


def _stream_ptr(stream):
    import torch

    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream)


def _check_bf16(t, shape, name, dtype=None):
    import torch

    if t.dtype != (dtype or torch.bfloat16) or not t.is_cuda or not t.is_contiguous() or tuple(t.shape) != tuple(shape):
        raise ValueError(f"{name}: expected contiguous CUDA bfloat16 (or, where supported, float16) tensor of shape {tuple(shape)}, "
                         f"got {t.dtype} {tuple(t.shape)} cuda={t.is_cuda} contiguous={t.is_contiguous()}")


def fa_fwd_raw(q_ptr, k_ptr, v_ptr, o_ptr, lse_ptr, B, H, Hkv, Sq, Sk, D, scale, causal, stream_ptr=None):
    """Direct call with integer device addresses; returns the status code."""
    return lib().fa_fwd(q_ptr, k_ptr, v_ptr, o_ptr, lse_ptr, B, H, Hkv, Sq, Sk, D, float(scale), int(causal),
                        stream_ptr)


def fa_fwd(q, k, v, scale=None, causal=False, o=None, lse=None, stream=None):
    """q [B,Sq,H,D], k/v [B,Sk,Hkv,D] bfloat16 -> (o [B,Sq,H,D] bfloat16, lse [B,H,Sq] float32).

    float16 tensors select fa_fwd_f16 (all of q, k, v, o must then be float16)."""
    import torch

    B, Sq, H, D = q.shape
    _, Sk, Hkv, _ = k.shape
    dt = torch.float16 if q.dtype == torch.float16 else torch.bfloat16
    _check_bf16(q, (B, Sq, H, D), "q", dt)
    _check_bf16(k, (B, Sk, Hkv, D), "k", dt)
    _check_bf16(v, (B, Sk, Hkv, D), "v", dt)
    if scale is None:
        scale = D ** -0.5
    if o is None:
        o = torch.empty_like(q)
    if lse is None:
        lse = torch.empty((B, H, Sq), dtype=torch.float32, device=q.device)
    _check_bf16(o, (B, Sq, H, D), "o", dt)
    entry = lib().fa_fwd_f16 if dt == torch.float16 else lib().fa_fwd
    st = entry(q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(), lse.data_ptr(),
               B, H, Hkv, Sq, Sk, D, float(scale), int(bool(causal)), _stream_ptr(stream))
    if st != FA_OK:
        raise FaError(st, "fa_fwd_f16" if dt == torch.float16 else "fa_fwd")
    return o, lse


def fa_fwd_hdim(q, k, v, scale=None, causal=False, o=None, lse=None, stream=None):
    """q [B,Sq,H,Dqk], k [B,Sk,Hkv,Dqk], v [B,Sk,Hkv,Dv] bfloat16 -> (o [B,Sq,H,Dv], lse [B,H,Sq] float32)."""
    import torch

    B, Sq, H, Dqk = q.shape
    _, Sk, Hkv, Dv = v.shape
    _check_bf16(q, (B, Sq, H, Dqk), "q")
    _check_bf16(k, (B, Sk, Hkv, Dqk), "k")
    _check_bf16(v, (B, Sk, Hkv, Dv), "v")
    if scale is None:
        scale = Dqk ** -0.5
    if o is None:
        o = torch.empty((B, Sq, H, Dv), dtype=torch.bfloat16, device=q.device)
    if lse is None:
        lse = torch.empty((B, H, Sq), dtype=torch.float32, device=q.device)
    _check_bf16(o, (B, Sq, H, Dv), "o")
    st = lib().fa_fwd_hdim(q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(), lse.data_ptr(),
                           B, H, Hkv, Sq, Sk, Dqk, Dv, float(scale), int(bool(causal)), _stream_ptr(stream))
    if st != FA_OK:
        raise FaError(st, "fa_fwd_hdim")
    return o, lse


def fa_varlen_lpt_order(cu_seqlens_q, cu_seqlens_k, causal=False, stream=None):
    """int32 CUDA tensors [batch + 1] -> int32 CUDA tensor [batch]: sequence indices, most work first."""
    import torch

    batch = cu_seqlens_q.numel() - 1
    order = torch.empty(batch, dtype=torch.int32, device=cu_seqlens_q.device)
    st = lib().fa_varlen_lpt_order(cu_seqlens_q.data_ptr(), cu_seqlens_k.data_ptr(), batch, int(bool(causal)),
                                   order.data_ptr(), _stream_ptr(stream))
    if st != FA_OK:
        raise FaError(st, "fa_varlen_lpt_order")
    return order


def fa_fwd_varlen(q, k, v, cu_seqlens_q, cu_seqlens_k, max_seqlen_q, scale=None, causal=False, order=None, stream=None):
    """Packed q [total_q,H,D], k/v [total_k,Hkv,D] bfloat16 -> (o [total_q,H,D], lse [H,total_q] float32)."""
    import torch

    total_q, H, D = q.shape
    total_k, Hkv, _ = k.shape
    _check_bf16(q, (total_q, H, D), "q")
    _check_bf16(k, (total_k, Hkv, D), "k")
    _check_bf16(v, (total_k, Hkv, D), "v")
    for t, name in ((cu_seqlens_q, "cu_seqlens_q"), (cu_seqlens_k, "cu_seqlens_k")):
        if t.dtype != torch.int32 or not t.is_cuda or not t.is_contiguous() or t.dim() != 1:
            raise ValueError(f"{name}: expected contiguous 1-D CUDA int32 tensor")
    batch = cu_seqlens_q.numel() - 1
    if cu_seqlens_k.numel() != batch + 1 or (order is not None and (order.numel() != batch or order.dtype != torch.int32)):
        raise ValueError("cu_seqlens_k / order do not match the batch size")
    if scale is None:
        scale = D ** -0.5
    o = torch.empty_like(q)
    lse = torch.empty((H, total_q), dtype=torch.float32, device=q.device)
    st = lib().fa_fwd_varlen(q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(), lse.data_ptr(),
                             cu_seqlens_q.data_ptr(), cu_seqlens_k.data_ptr(),
                             order.data_ptr() if order is not None else None, batch, total_q, total_k,
                             int(max_seqlen_q), H, Hkv, D, float(scale), int(bool(causal)), _stream_ptr(stream))
    if st != FA_OK:
        raise FaError(st, "fa_fwd_varlen")
    return o, lse


def fa_bwd_varlen(q, k, v, o, lse, d_o, cu_seqlens_q, cu_seqlens_k, max_seqlen_q, max_seqlen_k, scale=None, causal=False,
                  stream=None):
    """Gradients (dq, dk, dv) of fa_fwd_varlen's packed batch (bfloat16, D = 128)."""
    import torch

    total_q, H, D = q.shape
    total_k, Hkv, _ = k.shape
    for t, shp, name in ((q, (total_q, H, D), "q"), (k, (total_k, Hkv, D), "k"), (v, (total_k, Hkv, D), "v"),
                         (o, (total_q, H, D), "o"), (d_o, (total_q, H, D), "d_o")):
        _check_bf16(t, shp, name)
    batch = cu_seqlens_q.numel() - 1
    if scale is None:
        scale = D ** -0.5
    dq, dk, dv = torch.empty_like(q), torch.empty_like(k), torch.empty_like(v)
    need = int(lib().fa_bwd_varlen_workspace_bytes(batch, total_q, H, D))
    ws = torch.empty(max(need, 256), dtype=torch.uint8, device=q.device)
    st = lib().fa_bwd_varlen(q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(), lse.data_ptr(), d_o.data_ptr(),
                             dq.data_ptr(), dk.data_ptr(), dv.data_ptr(), cu_seqlens_q.data_ptr(),
                             cu_seqlens_k.data_ptr(), batch, total_q, total_k, int(max_seqlen_q), int(max_seqlen_k),
                             H, Hkv, D, float(scale), int(bool(causal)), ws.data_ptr(), ws.numel(),
                             _stream_ptr(stream))
    if st != FA_OK:
        raise FaError(st, "fa_bwd_varlen")
    return dq, dk, dv


def fa_bwd_workspace_bytes(B, H, Hkv, Sq, Sk, D):
    return int(lib().fa_bwd_workspace_bytes(B, H, Hkv, Sq, Sk, D))


def fa_bwd(q, k, v, o, lse, d_o, scale=None, causal=False, dq=None, dk=None, dv=None, workspace=None, stream=None,
           deterministic=False):
    """Gradients (dq, dk, dv) in bfloat16 for the same layouts as fa_fwd.

    float16 tensors select the _f16 entry points; deterministic=True calls fa_bwd_deterministic[_f16]
    (bit-reproducible dq, dk, dv)."""
    import torch

    B, Sq, H, D = q.shape
    _, Sk, Hkv, _ = k.shape
    dt = torch.float16 if q.dtype == torch.float16 else torch.bfloat16
    for t, shp, name in ((q, (B, Sq, H, D), "q"), (k, (B, Sk, Hkv, D), "k"), (v, (B, Sk, Hkv, D), "v"),
                         (o, (B, Sq, H, D), "o"), (d_o, (B, Sq, H, D), "d_o")):
        _check_bf16(t, shp, name, dt)
    if scale is None:
        scale = D ** -0.5
    dq = torch.empty_like(q) if dq is None else dq
    dk = torch.empty_like(k) if dk is None else dk
    dv = torch.empty_like(v) if dv is None else dv
    need = fa_bwd_workspace_bytes(B, H, Hkv, Sq, Sk, D)
    if workspace is None:
        workspace = torch.empty(need, dtype=torch.uint8, device=q.device)
    name = "fa_bwd" + ("_deterministic" if deterministic else "") + ("_f16" if dt == torch.float16 else "")
    entry = getattr(lib(), name)
    st = entry(q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(), lse.data_ptr(), d_o.data_ptr(),
               dq.data_ptr(), dk.data_ptr(), dv.data_ptr(), B, H, Hkv, Sq, Sk, D, float(scale),
               int(bool(causal)), workspace.data_ptr(), workspace.numel() * workspace.element_size(),
               _stream_ptr(stream))
    if st != FA_OK:
        raise FaError(st, name)
    return dq, dk, dv


def fa_last_device_status(stream=None):
    return int(lib().fa_last_device_status(_stream_ptr(stream)))


def fa_selftest_unsatisfied_wait(stream=None):
    """Launches a wait that cannot be satisfied; fa_last_device_status() then reports the timeout once."""
    st = lib().fa_selftest_unsatisfied_wait(_stream_ptr(stream))
    if st != FA_OK:
        raise FaError(st, "fa_selftest_unsatisfied_wait")


def fa_exp2_emulated(x, stream=None):
    """float32 CUDA tensor -> emulated 2^x (test hook for the kernel's software exponential)."""
    import torch

    y = torch.empty_like(x)
    st = lib().fa_exp2_emulated(x.data_ptr(), y.data_ptr(), x.numel(), _stream_ptr(stream))
    if st != FA_OK:
        raise FaError(st, "fa_exp2_emulated")
    return y


BWD_LAUNCHES = 3  # kernels fa_bwd enqueues: preprocess, main, dQ conversion


BWD_NOALLOC_MAX_BYTES = 40 * 1024 * 1024


def fa_bwd_noalloc(q, k, v, o, lse, d_o, scale=None, causal=False, dq=None, dk=None, dv=None, stream=None):
    """fa_bwd for callers that may not allocate device memory: the scratch lives in a fixed
    array inside the library (at most BWD_NOALLOC_MAX_BYTES; larger problems raise
    FaError with FA_ERR_WORKSPACE).  dq/dk/dv must be passed by such callers; when they are
    omitted here they are created with torch for convenience in tests.  Calls that overlap on
    the GPU share the array and race: keep them ordered."""
    import torch

    B, Sq, H, D = q.shape
    _, Sk, Hkv, _ = k.shape
    dt = torch.float16 if q.dtype == torch.float16 else torch.bfloat16
    for t, shp, name in ((q, (B, Sq, H, D), "q"), (k, (B, Sk, Hkv, D), "k"), (v, (B, Sk, Hkv, D), "v"),
                         (o, (B, Sq, H, D), "o"), (d_o, (B, Sq, H, D), "d_o")):
        _check_bf16(t, shp, name, dt)
    if scale is None:
        scale = D ** -0.5
    dq = torch.empty_like(q) if dq is None else dq
    dk = torch.empty_like(k) if dk is None else dk
    dv = torch.empty_like(v) if dv is None else dv
    f = lib().fa_bwd_noalloc
    f.argtypes = [ctypes.c_void_p] * 9 + [ctypes.c_int] * 6 + [ctypes.c_float, ctypes.c_int, ctypes.c_void_p]
    f.restype = ctypes.c_int
    st = f(q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(), lse.data_ptr(), d_o.data_ptr(), dq.data_ptr(),
           dk.data_ptr(), dv.data_ptr(), B, H, Hkv, Sq, Sk, D, float(scale), int(bool(causal)), _stream_ptr(stream))
    if st != FA_OK:
        raise FaError(st, "fa_bwd_noalloc")
    return dq, dk, dv
