"""Python binding of the C-ABI library `libgdnprep.so` (argument marshalling only).

Every function has the name and the argument order of its C entry point in
`include/gdnprep.h`; tensors are passed as raw device pointers on torch's
current CUDA stream. All arithmetic runs inside the library's CUDA kernels; if
the library is missing the import of a function raises, there is no fallback.
"""
from __future__ import annotations

import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libgdnprep.so")

GDN_OK = 0
GDN_ERR_INVALID_ARG = -1
GDN_ERR_UNSUPPORTED = -2
GDN_ERR_NULL = -3
GDN_ERR_ALIGN = -4
GDN_ERR_LAUNCH = -5
GDN_ERR_TIMEOUT = -6
GDN_ERR_ARCH = -7
GDN_ERR_SCRATCH = -8
GDN_DTYPE_FP32 = 0
GDN_DTYPE_BF16 = 1
GDN_FLAG_G_RAW = 1
GDN_FLAG_K_L2NORM = 2
GDN_FLAG_OUT_FP32 = 4
GDN_FLAG_LAYOUT_BTHD = 8
GDN_FLAG_W_GATED = 16
GDN_FWDSUBST_ROWS = 0
GDN_FWDSUBST_BLOCKED = 1
GDN_FWDSUBST_BLOCKED_TC = 2

EXPORTS = (
    "gdn_chunk_prepare", "gdn_chunk_prepare_gqa", "gdn_chunk_prepare_ex", "gdn_chunk_prepare_varlen",
    "gdn_chunk_prepare_fwdsubst",
    "gdn_chunk_prepare_int8", "gdn_chunk_prepare_int16", "gdn_chunk_state_output", "gdn_chunk_state_output_varlen", "gdn_chunk_state_output_segmented",
    "gdn_chunk_state_output_segmented_noalloc",
    "gdn_chunk_state_segments", "gdn_chunk_state_segmented_workspace", "gdn_selftest_bounded_wait",
    "gdn_int8_lut_checksum",
    "gdn_device_status", "gdn_default_order", "gdn_default_residual_steps",
    "gdn_status_string", "gdn_launch_count",
)

_lib = None


class GdnError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} (status {status})")


def load_library() -> ctypes.CDLL:
    """Loads the shared library (built in-tree by `paper_2606_06034_b200.build`)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise FileNotFoundError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2606_06034_b200.build` "
            "(the CUDA path has no fallback)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, ip = ctypes.c_void_p, ctypes.c_int
    lib.gdn_chunk_prepare.restype = ip
    lib.gdn_chunk_prepare.argtypes = [vp, vp, vp, vp, ip, ip, ip, ip, ip, ip, ip, ip, ip, vp, vp, vp, vp]
    lib.gdn_chunk_prepare_gqa.restype = ip
    lib.gdn_chunk_prepare_gqa.argtypes = [vp, vp, vp, vp, ip, ip, ip, ip, ip, ip, ip, ip, ip, ip, vp, vp, vp, vp]
    lib.gdn_chunk_prepare_ex.restype = ip
    lib.gdn_chunk_prepare_ex.argtypes = [vp, vp, vp, vp, ip, ip, ip, ip, ip, ip, ip, ip, ip, ip, vp, vp, vp, ctypes.c_uint, vp]
    lib.gdn_chunk_prepare_varlen.restype = ip
    lib.gdn_chunk_prepare_varlen.argtypes = [vp, vp, vp, vp, vp, vp, ip, ip, ip, ip, ip, ip, ip, ip, ip, vp, vp, vp, ctypes.c_uint, vp]
    lib.gdn_chunk_prepare_fwdsubst.restype = ip
    lib.gdn_chunk_prepare_fwdsubst.argtypes = [vp, vp, vp, vp, ip, ip, ip, ip, ip, ip, ip, ip, ip, vp, vp, vp, vp]
    lib.gdn_chunk_prepare_int8.restype = ip
    lib.gdn_chunk_prepare_int8.argtypes = [vp, vp, vp, vp, vp, vp, ip, ip, ip, ip, ip, ip, ip, ip, ip, vp, vp, vp, vp, vp, vp, vp, vp]
    lib.gdn_chunk_prepare_int16.restype = ip
    lib.gdn_chunk_prepare_int16.argtypes = [vp, vp, vp, vp, vp, vp, ip, ip, ip, ip, ip, ip, ip, ip, ip, vp, vp, vp, vp, vp, vp, vp, vp]
    lib.gdn_int8_lut_checksum.restype = ctypes.c_uint
    lib.gdn_chunk_state_output.argtypes = [vp, vp, vp, vp, vp, ip, ip, ip, ip, ip, ip, ip, ctypes.c_float, vp, vp, vp,
                                           ctypes.c_uint, vp]
    lib.gdn_chunk_state_output.restype = ip
    lib.gdn_chunk_state_output_varlen.argtypes = [vp, vp, vp, vp, vp, vp, ip, ip, ip, ip, ip, ip, ip, ctypes.c_float, vp, vp, vp,
                                                  ctypes.c_uint, vp]
    lib.gdn_chunk_state_output_varlen.restype = ip
    lib.gdn_chunk_state_segments.argtypes = [ip]
    lib.gdn_chunk_state_segments.restype = ip
    lib.gdn_chunk_state_segmented_workspace.argtypes = [ip, ip]
    lib.gdn_chunk_state_segmented_workspace.restype = ctypes.c_size_t
    lib.gdn_chunk_state_output_segmented.argtypes = [vp, vp, vp, vp, vp, ip, ip, ip, ip, ip, ip, ctypes.c_float, vp, vp, vp, ip,
                                                     vp, ctypes.c_size_t, ctypes.c_uint, vp]
    lib.gdn_chunk_state_output_segmented.restype = ip
    lib.gdn_chunk_state_output_segmented_noalloc.argtypes = [vp, vp, vp, vp, vp, ip, ip, ip, ip, ip, ip, ctypes.c_float, vp, vp, vp,
                                                             ip, ctypes.c_uint, vp]
    lib.gdn_chunk_state_output_segmented_noalloc.restype = ip
    lib.gdn_selftest_bounded_wait.argtypes = [vp]
    lib.gdn_selftest_bounded_wait.restype = ip
    lib.gdn_int8_lut_checksum.argtypes = []
    lib.gdn_device_status.restype = ip
    lib.gdn_device_status.argtypes = [vp]
    lib.gdn_default_order.restype = ip
    lib.gdn_default_order.argtypes = [ip]
    lib.gdn_default_residual_steps.restype = ip
    lib.gdn_default_residual_steps.argtypes = [ip]
    lib.gdn_status_string.restype = ctypes.c_char_p
    lib.gdn_status_string.argtypes = [ip]
    lib.gdn_launch_count.restype = ctypes.c_longlong
    lib.gdn_launch_count.argtypes = []
    _lib = lib
    return lib


def status_string(status: int) -> str:
    return load_library().gdn_status_string(int(status)).decode()


def gdn_default_order(C: int) -> int:
    return load_library().gdn_default_order(int(C))


def gdn_default_residual_steps(C: int) -> int:
    return load_library().gdn_default_residual_steps(int(C))


def gdn_launch_count() -> int:
    return int(load_library().gdn_launch_count())


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return GDN_DTYPE_FP32
    if t.dtype == torch.bfloat16:
        return GDN_DTYPE_BF16
    raise TypeError(f"unsupported dtype {t.dtype}")


_EMPTY = {}  # per device: a small allocation whose address stands in for tensors without elements


def _ptr(t):
    """Address of a tensor's data. torch gives tensors without elements a null data pointer, which the library would
    report as a missing argument; an empty batch or zero tokens is a valid (empty) problem, so such tensors are passed
    as the address of a small allocation that is never read or written."""
    if t is None:
        return None
    if t.numel() == 0 and t.is_cuda:
        key = t.device.index
        if key not in _EMPTY:
            _EMPTY[key] = torch.zeros(64, dtype=torch.float32, device=t.device)
        return ctypes.c_void_p(_EMPTY[key].data_ptr())
    return ctypes.c_void_p(t.data_ptr())


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _check_inputs(K, V, beta, g, outs):
    for t in (K, V, beta, g, *[o for o in outs if o is not None]):
        if not t.is_cuda:
            raise ValueError("all tensors must live on a CUDA device (there is no CPU path)")
        if not t.is_contiguous():
            raise ValueError("all tensors must be contiguous")
    if V.dtype != K.dtype or beta.dtype != torch.float32 or g.dtype != torch.float32:
        raise TypeError("K and V share a dtype; beta and g are fp32")


def alloc_outputs(K, V, C, want_tinv=True, token_major=False):
    """Allocates W [B,H_v,T,d_k], U [B,H_v,T,d_v], Tinv [B,H_v,T/C,C,C] with torch
    (token_major: K, V are [B,T,H,d] and so are W, U; Tinv keeps its layout)."""
    if token_major:
        B, T, H_v, d_v = V.shape
    else:
        B, H_v, T, d_v = V.shape
    d_k = K.shape[-1]
    W = torch.empty((B, T, H_v, d_k) if token_major else (B, H_v, T, d_k), dtype=K.dtype, device=K.device)
    U = torch.empty((B, T, H_v, d_v) if token_major else (B, H_v, T, d_v), dtype=K.dtype, device=K.device)
    Tinv = torch.empty(B, H_v, T // C, C, C, dtype=K.dtype, device=K.device) if want_tinv else None
    return W, U, Tinv


def gdn_chunk_prepare(K, V, beta, g, B, H, T, C, d_k, d_v, order, residual_steps, dtype, W_out, U_out, Tinv_out,
                      *, check=True):
    """Raw call (same argument list as the C function, tensors instead of pointers)."""
    _check_inputs(K, V, beta, g, (W_out, U_out, Tinv_out))
    rc = load_library().gdn_chunk_prepare(_ptr(K), _ptr(V), _ptr(beta), _ptr(g), B, H, T, C, d_k, d_v, order,
                                          residual_steps, dtype, _ptr(W_out), _ptr(U_out), _ptr(Tinv_out), _stream())
    if check and rc != GDN_OK:
        raise GdnError(rc, "gdn_chunk_prepare")
    return rc


def gdn_chunk_prepare_gqa(K, V, beta, g, B, H_k, H_v, T, C, d_k, d_v, order, residual_steps, dtype, W_out, U_out,
                          Tinv_out, *, check=True):
    _check_inputs(K, V, beta, g, (W_out, U_out, Tinv_out))
    rc = load_library().gdn_chunk_prepare_gqa(_ptr(K), _ptr(V), _ptr(beta), _ptr(g), B, H_k, H_v, T, C, d_k, d_v,
                                              order, residual_steps, dtype, _ptr(W_out), _ptr(U_out), _ptr(Tinv_out),
                                              _stream())
    if check and rc != GDN_OK:
        raise GdnError(rc, "gdn_chunk_prepare_gqa")
    return rc


def gdn_chunk_prepare_ex(K, V, beta, g, B, H_k, H_v, T, C, d_k, d_v, order, residual_steps, dtype, W_out, U_out,
                         Tinv_out, flags, *, check=True):
    _check_inputs(K, V, beta, g, ())
    rc = load_library().gdn_chunk_prepare_ex(_ptr(K), _ptr(V), _ptr(beta), _ptr(g), B, H_k, H_v, T, C, d_k, d_v, order,
                                             residual_steps, dtype, _ptr(W_out), _ptr(U_out), _ptr(Tinv_out), int(flags),
                                             _stream())
    if check and rc != GDN_OK:
        raise GdnError(rc, "gdn_chunk_prepare_ex")
    return rc


def gdn_chunk_prepare_varlen(K, V, beta, g, chunk_start, chunk_len, n_chunks, T_total, H_k, H_v, C, d_k, d_v, order,
                             residual_steps, W_out, U_out, Tinv_out, flags, *, check=True):
    _check_inputs(K, V, beta, g, (W_out, U_out, Tinv_out))
    for t in (chunk_start, chunk_len):
        if t is not None and (not t.is_cuda or not t.is_contiguous() or t.dtype != torch.int32):
            raise TypeError("chunk_start and chunk_len are contiguous int32 CUDA tensors")
    rc = load_library().gdn_chunk_prepare_varlen(_ptr(K), _ptr(V), _ptr(beta), _ptr(g), _ptr(chunk_start), _ptr(chunk_len),
                                                 n_chunks, T_total, H_k, H_v, C, d_k, d_v, order, residual_steps,
                                                 _ptr(W_out), _ptr(U_out), _ptr(Tinv_out), int(flags), _stream())
    if check and rc != GDN_OK:
        raise GdnError(rc, "gdn_chunk_prepare_varlen")
    return rc


def chunk_table(cu_seqlens, C):
    """First token and length of every chunk of packed sequences (host lists): sequence s holds the tokens
    [cu_seqlens[s], cu_seqlens[s + 1]) and is cut into chunks of C tokens from its own start."""
    bounds = [int(x) for x in cu_seqlens]
    start, length = [], []
    for a, b in zip(bounds[:-1], bounds[1:]):
        if b < a:
            raise ValueError("cu_seqlens must be non-decreasing")
        n_full, rest = divmod(b - a, C)
        start += [a + i * C for i in range(n_full + (1 if rest else 0))]
        length += [C] * n_full + ([rest] if rest else [])
    return start, length


def chunk_prepare_varlen(K, V, beta, g, cu_seqlens, C, order=-1, residual_steps=-1, *, want_tinv=True, flags=0):
    """Packed variable-length sequences: K [H_k,T,d_k], V [H_v,T,d_v], beta, g [H_v,T] (with GDN_FLAG_LAYOUT_BTHD:
    [T,H,d] and [T,H_v]), cu_seqlens = the sequence boundaries on the host. Returns (W, U, Tinv [H_v,n_chunks,C,C] or
    None, chunk_start, chunk_len) with the chunk table as int32 CUDA tensors."""
    token_major = bool(flags & GDN_FLAG_LAYOUT_BTHD)
    if token_major:
        T, H_k, d_k = K.shape
        _, H_v, d_v = V.shape
    else:
        H_k, T, d_k = K.shape
        H_v, _, d_v = V.shape
    start, length = chunk_table(cu_seqlens, C)
    n = len(start)
    cs = torch.tensor(start, dtype=torch.int32, device=K.device)
    cl = torch.tensor(length, dtype=torch.int32, device=K.device)
    per_tile = max(1, 128 // C)
    padded = -(-n // per_tile) * per_tile
    W = torch.zeros((T, H_v, d_k) if token_major else (H_v, T, d_k), dtype=K.dtype, device=K.device)
    U = torch.zeros_like(V)
    Tinv = torch.empty(H_v, padded, C, C, dtype=K.dtype, device=K.device) if want_tinv else None
    gdn_chunk_prepare_varlen(K, V, beta, g, cs, cl, n, T, H_k, H_v, C, d_k, d_v, order, residual_steps, W, U, Tinv, flags)
    return W, U, (Tinv[:, :n] if want_tinv else None), cs, cl


def gdn_chunk_prepare_fwdsubst(K, V, beta, g, B, H_k, H_v, T, C, d_k, d_v, dtype, variant, W_out, U_out, Tinv_out,
                               *, check=True):
    _check_inputs(K, V, beta, g, (W_out, U_out, Tinv_out))
    rc = load_library().gdn_chunk_prepare_fwdsubst(_ptr(K), _ptr(V), _ptr(beta), _ptr(g), B, H_k, H_v, T, C, d_k,
                                                   d_v, dtype, variant, _ptr(W_out), _ptr(U_out), _ptr(Tinv_out),
                                                   _stream())
    if check and rc != GDN_OK:
        raise GdnError(rc, "gdn_chunk_prepare_fwdsubst")
    return rc


def gdn_int8_lut_checksum() -> int:
    return int(load_library().gdn_int8_lut_checksum())


def gdn_chunk_prepare_int8(Kq, Vq, k_exp, v_exp, beta_q, decay_q, B, H_k, H_v, T, C, d_k, d_v, order, residual_steps,
                           Wq_out, Uq_out, w_exp_out, u_exp_out, Toff_q_out, t_exp_out, dbg_acc_out=None, *, check=True):
    """Raw call of the INT8 entry point (tensors instead of pointers, torch's current stream)."""
    for t in (Kq, Vq, k_exp, v_exp, beta_q, decay_q, Wq_out, Uq_out, w_exp_out, u_exp_out, t_exp_out):
        if not t.is_cuda or not t.is_contiguous():
            raise ValueError("all tensors must be contiguous CUDA tensors (there is no CPU path)")
    rc = load_library().gdn_chunk_prepare_int8(_ptr(Kq), _ptr(Vq), _ptr(k_exp), _ptr(v_exp), _ptr(beta_q), _ptr(decay_q),
                                               B, H_k, H_v, T, C, d_k, d_v, order, residual_steps, _ptr(Wq_out),
                                               _ptr(Uq_out), _ptr(w_exp_out), _ptr(u_exp_out), _ptr(Toff_q_out),
                                               _ptr(t_exp_out), _ptr(dbg_acc_out), _stream())
    if check and rc != GDN_OK:
        raise GdnError(rc, "gdn_chunk_prepare_int8")
    return rc


def chunk_prepare_int8(q, order=-1, residual_steps=-1, *, want_toff=True, outputs=None, dbg_acc=None):
    """Convenience wrapper over integer inputs (an `inputs.Int8Inputs` whose tensors live on the GPU).

    Returns (Wq, Uq, w_exp, u_exp, Toff_q, t_exp). `dbg_acc`: optional zeroed int32 tensor
    [B, H_v, T/C, C, 8*C + d_k + d_v] that receives the tensor-core accumulators (small cases, C = 64).
    With C = 128 (two 64-blocks per chunk) w_exp, u_exp are [B, H_v, T/128, 2] (rows 0..63, rows 64..127) and t_exp is
    [B, H_v, T/128, 3] (blocks 11, 21, 22); Toff_q is always produced.
    """
    dev = q.Kq.device
    n_c = q.T // q.C
    if outputs is None:
        Wq = torch.empty(q.B, q.H_v, q.T, q.d_k, dtype=torch.int8, device=dev)
        Uq = torch.empty(q.B, q.H_v, q.T, q.d_v, dtype=torch.int8, device=dev)
        if q.C == 128:
            w_exp = torch.empty(q.B, q.H_v, n_c, 2, dtype=torch.int32, device=dev)
            u_exp = torch.empty_like(w_exp)
            t_exp = torch.empty(q.B, q.H_v, n_c, 3, dtype=torch.int32, device=dev)
            want_toff = True
        else:
            w_exp = torch.empty(q.B, q.H_v, n_c, dtype=torch.int32, device=dev)
            u_exp = torch.empty_like(w_exp)
            t_exp = torch.empty_like(w_exp)
        Toff = torch.empty(q.B, q.H_v, n_c, q.C, q.C, dtype=torch.int8, device=dev) if want_toff else None
        outputs = (Wq, Uq, w_exp, u_exp, Toff, t_exp)
    Wq, Uq, w_exp, u_exp, Toff, t_exp = outputs
    gdn_chunk_prepare_int8(q.Kq, q.Vq, q.k_exp, q.v_exp, q.beta_q, q.decay_q, q.B, q.H_k, q.H_v, q.T, q.C, q.d_k, q.d_v,
                           order, residual_steps, Wq, Uq, w_exp, u_exp, Toff, t_exp, dbg_acc)
    return outputs


def gdn_chunk_prepare_int16(Kq, Vq, k_exp, v_exp, beta_q, decay_q, B, H_k, H_v, T, C, d_k, d_v, order, residual_steps,
                            Wq_out, Uq_out, w_exp_out, u_exp_out, Toff_q_out, t_exp_out, dbg_acc_out=None, *, check=True):
    """Raw call of the INT16 entry point (tensors instead of pointers, torch's current stream)."""
    for t in (Kq, Vq, k_exp, v_exp, beta_q, decay_q, Wq_out, Uq_out, w_exp_out, u_exp_out, t_exp_out):
        if not t.is_cuda or not t.is_contiguous():
            raise ValueError("all tensors must be contiguous CUDA tensors (there is no CPU path)")
    rc = load_library().gdn_chunk_prepare_int16(_ptr(Kq), _ptr(Vq), _ptr(k_exp), _ptr(v_exp), _ptr(beta_q), _ptr(decay_q),
                                                B, H_k, H_v, T, C, d_k, d_v, order, residual_steps, _ptr(Wq_out),
                                                _ptr(Uq_out), _ptr(w_exp_out), _ptr(u_exp_out), _ptr(Toff_q_out),
                                                _ptr(t_exp_out), _ptr(dbg_acc_out), _stream())
    if check and rc != GDN_OK:
        raise GdnError(rc, "gdn_chunk_prepare_int16")
    return rc


def chunk_prepare_int16(q, order=-1, residual_steps=-1, *, want_toff=True, outputs=None, dbg_acc=None):
    """Convenience wrapper over 16-bit integer inputs (`inputs.make_int16_inputs`, tensors on the GPU).

    Returns (Wq, Uq, w_exp, u_exp, Toff_q, t_exp), mantissas int16. `dbg_acc`: optional zeroed int64 tensor
    [B, H_v, T/C, C, 8*C + d_k + d_v] that receives the exact matrix products (small cases).
    """
    dev = q.Kq.device
    n_c = q.T // q.C
    if outputs is None:
        Wq = torch.empty(q.B, q.H_v, q.T, q.d_k, dtype=torch.int16, device=dev)
        Uq = torch.empty(q.B, q.H_v, q.T, q.d_v, dtype=torch.int16, device=dev)
        w_exp = torch.empty(q.B, q.H_v, n_c, dtype=torch.int32, device=dev)
        u_exp = torch.empty_like(w_exp)
        t_exp = torch.empty_like(w_exp)
        Toff = torch.empty(q.B, q.H_v, n_c, q.C, q.C, dtype=torch.int16, device=dev) if want_toff else None
        outputs = (Wq, Uq, w_exp, u_exp, Toff, t_exp)
    Wq, Uq, w_exp, u_exp, Toff, t_exp = outputs
    gdn_chunk_prepare_int16(q.Kq, q.Vq, q.k_exp, q.v_exp, q.beta_q, q.decay_q, q.B, q.H_k, q.H_v, q.T, q.C, q.d_k, q.d_v,
                            order, residual_steps, Wq, Uq, w_exp, u_exp, Toff, t_exp, dbg_acc)
    return outputs


def gdn_chunk_state_output(Q, K, W_gated, U, g, B, H_k, H_v, T, C, d_k, d_v, scale, S_in, O_out, S_out, flags=0, *,
                           check=True):
    """Raw call of the state-passing / output entry point (tensors instead of pointers, torch's current stream)."""
    for t in (Q, K, W_gated, U, g, S_in, O_out, S_out):
        if t is not None and (not t.is_cuda or not t.is_contiguous()):
            raise ValueError("all tensors must be contiguous CUDA tensors (there is no CPU path)")
    rc = load_library().gdn_chunk_state_output(_ptr(Q), _ptr(K), _ptr(W_gated), _ptr(U), _ptr(g), B, H_k, H_v, T, C, d_k, d_v,
                                               ctypes.c_float(scale), _ptr(S_in), _ptr(O_out), _ptr(S_out), flags,
                                               _stream())
    if check and rc != GDN_OK:
        raise GdnError(rc, "gdn_chunk_state_output")
    return rc


def gdn_chunk_state_output_varlen(Q, K, W_gated, U, g, cu_seqlens, n_seq, T_total, H_k, H_v, C, d_k, d_v, scale, S_in, O_out,
                                  S_out, flags=0, *, check=True):
    """Raw call of the packed-sequence form (cu_seqlens: int32 CUDA tensor of n_seq + 1 boundaries)."""
    for t in (Q, K, W_gated, U, g, cu_seqlens, S_in, O_out, S_out):
        if t is not None and (not t.is_cuda or not t.is_contiguous()):
            raise ValueError("all tensors must be contiguous CUDA tensors (there is no CPU path)")
    if cu_seqlens is not None and cu_seqlens.dtype != torch.int32:
        raise TypeError("cu_seqlens is an int32 tensor")
    rc = load_library().gdn_chunk_state_output_varlen(_ptr(Q), _ptr(K), _ptr(W_gated), _ptr(U), _ptr(g), _ptr(cu_seqlens), n_seq,
                                                      T_total, H_k, H_v, C, d_k, d_v, ctypes.c_float(scale), _ptr(S_in),
                                                      _ptr(O_out), _ptr(S_out), flags, _stream())
    if check and rc != GDN_OK:
        raise GdnError(rc, "gdn_chunk_state_output_varlen")
    return rc


def chunk_state_output_segmented(Q, K, W_gated, U, g, C, scale=1.0, S_in=None, *, segments=0, want_state=True, flags=0,
                                 workspace=None):
    """Few long sequences (B = 1; Q, K [H_k,T,d_k], W_gated, U [H_v,T,d], g [H_v,T], or token-major with
    GDN_FLAG_LAYOUT_BTHD): the segmented form of the state passing. segments = 0: the library's proposal.
    Returns (O, S_out [H_v,d_v,d_k] or None)."""
    if flags & GDN_FLAG_LAYOUT_BTHD:
        T, H_k, d_k = K.shape
        _, H_v, d_v = U.shape
    else:
        H_k, T, d_k = K.shape
        H_v, _, d_v = U.shape
    lib = load_library()
    if segments <= 0:
        segments = int(lib.gdn_chunk_state_segments(H_v))
    need = int(lib.gdn_chunk_state_segmented_workspace(H_v, segments))
    if workspace is None and need > 0:
        workspace = torch.empty(need, dtype=torch.uint8, device=U.device)
    for t in (Q, K, W_gated, U, g, S_in):
        if t is not None and (not t.is_cuda or not t.is_contiguous()):
            raise ValueError("all tensors must be contiguous CUDA tensors (there is no CPU path)")
    O = torch.empty_like(U)
    S_out = torch.empty(H_v, d_v, d_k, dtype=torch.float32, device=U.device) if want_state else None
    rc = lib.gdn_chunk_state_output_segmented(_ptr(Q), _ptr(K), _ptr(W_gated), _ptr(U), _ptr(g), H_k, H_v, T, C, d_k, d_v,
                                              ctypes.c_float(scale), _ptr(S_in), _ptr(O), _ptr(S_out), segments,
                                              _ptr(workspace), need, flags, _stream())
    if rc != GDN_OK:
        raise GdnError(rc, "gdn_chunk_state_output_segmented")
    return O, S_out


def gdn_chunk_state_output_segmented_noalloc(Q, K, W_gated, U, g, H_k, H_v, T, C, d_k, d_v, scale, S_in, O_out, S_out, segments,
                                             flags=0, *, check=True):
    """Raw call of the segmented state passing on the library's built-in scratch array: for callers that cannot
    allocate device memory around the call. The caller passes every input and output tensor; this wrapper and the
    entry point allocate nothing. Returns the status (GDN_ERR_SCRATCH when H_v * (6 * segments - 6) > 128)."""
    for t in (Q, K, W_gated, U, g, S_in, O_out, S_out):
        if t is not None and (not t.is_cuda or not t.is_contiguous()):
            raise ValueError("all tensors must be contiguous CUDA tensors (there is no CPU path)")
    rc = load_library().gdn_chunk_state_output_segmented_noalloc(_ptr(Q), _ptr(K), _ptr(W_gated), _ptr(U), _ptr(g), H_k, H_v, T, C,
                                                                 d_k, d_v, ctypes.c_float(scale), _ptr(S_in), _ptr(O_out),
                                                                 _ptr(S_out), segments, flags, _stream())
    if check and rc != GDN_OK:
        raise GdnError(rc, "gdn_chunk_state_output_segmented_noalloc")
    return rc


def chunk_state_output_varlen(Q, K, W_gated, U, g, cu_seqlens, C, scale=1.0, S_in=None, *, want_state=True, flags=0):
    """Packed sequences: Q, K [H_k,T,d_k], W_gated [H_v,T,d_k], U [H_v,T,d_v], g [H_v,T]; cu_seqlens on the host.
    Returns (O [H_v,T,d_v], S_out [n_seq,H_v,d_v,d_k] fp32 or None); rows of O that no sequence covers stay zero."""
    if flags & GDN_FLAG_LAYOUT_BTHD:  # token-major: [T, H, d]
        T, H_k, d_k = K.shape
        _, H_v, d_v = U.shape
    else:
        H_k, T, d_k = K.shape
        H_v, _, d_v = U.shape
    cu = torch.tensor([int(x) for x in cu_seqlens], dtype=torch.int32, device=U.device)
    n_seq = cu.numel() - 1
    O = torch.zeros_like(U)
    S_out = torch.empty(n_seq, H_v, d_v, d_k, dtype=torch.float32, device=U.device) if want_state else None
    gdn_chunk_state_output_varlen(Q, K, W_gated, U, g, cu, n_seq, T, H_k, H_v, C, d_k, d_v, scale, S_in, O, S_out, flags)
    return O, S_out


def chunk_state_output(Q, K, W_gated, U, g, C, scale=1.0, S_in=None, *, want_state=True, outputs=None, flags=0):
    """Convenience wrapper: Q, K [B,H_k,T,d_k], W_gated [B,H_v,T,d_k], U [B,H_v,T,d_v], g [B,H_v,T] (chunk-local
    cumulative log-gate). Returns (O [B,H_v,T,d_v], S_out [B,H_v,d_v,d_k] fp32 or None)."""
    if flags & GDN_FLAG_LAYOUT_BTHD:  # token-major: [B, T, H, d]
        B, T, H_k, d_k = K.shape
        _, _, H_v, d_v = U.shape
    else:
        B, H_k, T, d_k = K.shape
        _, H_v, _, d_v = U.shape
    if outputs is None:
        O = torch.empty_like(U)
        S_out = torch.empty(B, H_v, d_v, d_k, dtype=torch.float32, device=U.device) if want_state else None
    else:
        O, S_out = outputs
    gdn_chunk_state_output(Q, K, W_gated, U, g, B, H_k, H_v, T, C, d_k, d_v, scale, S_in, O, S_out, flags)
    return O, S_out


def gated_delta_layer(Q, K, V, beta, g_raw, C=64, scale=None, S_in=None, *, cu_seqlens=None, token_major=True,
                      qk_l2norm=True, want_state=True):
    """The chunk-wise layer as model code calls it: the two library calls back to back (chunk-prepare with the gated W,
    then state passing and output) on raw per-token log-gates and, with qk_l2norm, raw key / query projections.
    Dense: Q, K [B,T,H_k,d], V [B,T,H_v,d], beta, g_raw [B,T,H_v] (token_major) or the head-major forms. Packed
    sequences (cu_seqlens on the host): the same tensors without the batch axis. Returns (O, S_out or None)."""
    flags = GDN_FLAG_G_RAW | (GDN_FLAG_LAYOUT_BTHD if token_major else 0) | (GDN_FLAG_K_L2NORM if qk_l2norm else 0)
    if scale is None:
        scale = float(K.shape[-1]) ** -0.5
    if cu_seqlens is not None:
        W, U, _, _, _ = chunk_prepare_varlen(K, V, beta, g_raw, cu_seqlens, C, flags=flags | GDN_FLAG_W_GATED, want_tinv=False)
        return chunk_state_output_varlen(Q, K, W, U, g_raw, cu_seqlens, C, scale, S_in, want_state=want_state, flags=flags)
    W, U, _ = chunk_prepare(K, V, beta, g_raw, C, flags=flags | GDN_FLAG_W_GATED, want_tinv=False)
    H_v = V.shape[2] if token_major else V.shape[1]
    if K.shape[0] == 1 and int(load_library().gdn_chunk_state_segments(H_v)) > 1:
        # one long sequence per head and fewer heads than SMs: the segments of a sequence run in parallel
        O, S = chunk_state_output_segmented(Q[0], K[0], W[0], U[0], g_raw[0], C, scale, None if S_in is None else S_in[0],
                                            want_state=want_state, flags=flags)
        return O[None], (None if S is None else S[None])
    return chunk_state_output(Q, K, W, U, g_raw, C, scale, S_in, want_state=want_state, flags=flags)


def gdn_selftest_bounded_wait() -> int:
    """Enqueues the bounded-wait self-test on torch's current stream (see the header)."""
    return load_library().gdn_selftest_bounded_wait(_stream())


def gdn_device_status() -> int:
    """Synchronises torch's current stream and returns (and clears) the kernels' status word."""
    return load_library().gdn_device_status(_stream())


def chunk_prepare(K, V, beta, g, C, order=-1, residual_steps=-1, *, want_tinv=True, outputs=None,
                  method="neumann", variant=GDN_FWDSUBST_ROWS, flags=0):
    """Convenience wrapper: shapes from the tensors, outputs allocated with torch.

    K [B,H_k,T,d_k], V [B,H_v,T,d_v], beta, g [B,H_v,T]. Returns (W, U, Tinv).
    With GDN_FLAG_LAYOUT_BTHD in `flags` the tensors are token-major: K [B,T,H_k,d_k], V [B,T,H_v,d_v],
    beta, g [B,T,H_v], W [B,T,H_v,d_k], U [B,T,H_v,d_v] (Tinv keeps [B,H_v,T/C,C,C]).
    """
    token_major = bool(flags & GDN_FLAG_LAYOUT_BTHD)
    if token_major:
        B, T, H_k, d_k = K.shape
        _, _, H_v, d_v = V.shape
    else:
        B, H_k, T, d_k = K.shape
        _, H_v, _, d_v = V.shape
    if outputs is None:
        outputs = alloc_outputs(K, V, C, want_tinv, token_major)
        if flags & GDN_FLAG_OUT_FP32:
            outputs = tuple(None if o is None else torch.empty(o.shape, dtype=torch.float32, device=o.device) for o in outputs)
    W, U, Tinv = outputs
    dt = _dtype_code(K)
    if method == "neumann" and flags:
        gdn_chunk_prepare_ex(K, V, beta, g, B, H_k, H_v, T, C, d_k, d_v, order, residual_steps, dt, W, U, Tinv, flags)
    elif method == "neumann":
        gdn_chunk_prepare_gqa(K, V, beta, g, B, H_k, H_v, T, C, d_k, d_v, order, residual_steps, dt, W, U, Tinv)
    elif method == "fwdsubst":
        gdn_chunk_prepare_fwdsubst(K, V, beta, g, B, H_k, H_v, T, C, d_k, d_v, dt, variant, W, U, Tinv)
    else:
        raise ValueError(method)
    return W, U, Tinv
