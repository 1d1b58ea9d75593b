"""ctypes binding of libbsp.so: the same names as the C ABI (include/bsp.h), argument marshalling
only -- every step of the path runs in the CUDA kernels.  Tensors are torch CUDA tensors (or
None for optional pointers); torch is used for device memory and streams, nothing else.

There is no CPU fallback: loading fails loudly when the library has not been built.
"""
from __future__ import annotations

import ctypes as C
import os

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libbsp.so")

OK, ERR_ARG, ERR_ALIGN, ERR_UNSUPPORTED, ERR_WORKSPACE, ERR_NONFINITE, ERR_TIMEOUT, ERR_CUDA, ERR_TOO_LARGE = range(9)
NORM_BWD_NOALLOC_CAPACITY_BYTES = 20 << 20
E4M3, E5M2 = 0, 1
ROUND_NEAREST, ROUND_STOCHASTIC = 0, 1
READ_ORIGINAL, READ_FORWARD, READ_FRESH, READ_FORWARD_PLUS_FRESH_ERROR = 0, 1, 2, 3
F32, BF16 = 0, 1
RMSNORM, LAYERNORM = 0, 1
HOLDS, FAILS, UNDECIDED = 0, 1, 2
STREAM_FORWARD, STREAM_GAIN, STREAM_WGRAD, STREAM_DX, STREAM_ATTN_D, STREAM_SHARED = 0, 1, 2, 3, 4, 255
OUT_DGAMMA, OUT_DBETA, OUT_DW, OUT_DX, OUT_D, OUT_DQ, OUT_DK, OUT_DV = range(8)


class Key(C.Structure):
    _fields_ = [("seed", C.c_uint64), ("tensor_id", C.c_uint32), ("stream", C.c_uint32),
                ("draw", C.c_uint32), ("reserved", C.c_uint32)]


class Quant(C.Structure):
    _fields_ = [("fmt", C.c_int32), ("mode", C.c_int32), ("scale", C.c_float), ("scale_dev", C.c_void_p)]


class Diag(C.Structure):
    _fields_ = [("n_saturated", C.c_ulonglong), ("n_nonfinite", C.c_ulonglong),
                ("amax_bits", C.c_uint32), ("status", C.c_int32)]


class UseResult(C.Structure):
    _fields_ = [("use_id", C.c_int32), ("output_id", C.c_int32), ("policy", C.c_int32), ("K", C.c_int32),
                ("n_elements", C.c_int64), ("rel_l2_mean_err", C.c_double), ("R", C.c_double),
                ("Qprime", C.c_double), ("mean_z", C.c_double), ("rms_z", C.c_double),
                ("max_abs_z", C.c_double), ("frac_abs_z_gt3", C.c_double), ("verdict", C.c_int32),
                ("informational", C.c_int32)]

    def as_dict(self):
        return {n: getattr(self, n) for n, _ in self._fields_}


class VerdictRule(C.Structure):
    _fields_ = [("rel_tol_deterministic", C.c_double), ("qprime_hold", C.c_double), ("r_hold", C.c_double),
                ("qprime_fail", C.c_double), ("r_fail", C.c_double), ("rel_hold", C.c_double)]


class McLayout(C.Structure):
    _fields_ = [(n, C.c_size_t) for n in (
        "dgamma_ref", "dbeta_ref", "dgamma_forward", "dgamma_S1", "dgamma_S2", "dW_ref", "dW_S1", "dW_S2", "dx",
        "rstd", "mean", "u_codes", "scale_u", "scale_dy", "du")]


class NormLinearDesc(C.Structure):
    _fields_ = [("norm_kind", C.c_int32), ("dtype", C.c_int32), ("T", C.c_int64), ("C", C.c_int64),
                ("O", C.c_int64), ("x", C.c_void_p), ("gamma", C.c_void_p), ("beta", C.c_void_p),
                ("W", C.c_void_p), ("dY", C.c_void_p), ("eps", C.c_float), ("store_fmt", C.c_int32),
                ("grad_fmt", C.c_int32), ("forward_mode", C.c_int32), ("seed", C.c_uint64),
                ("tensor_id", C.c_uint32), ("policy_mask", C.c_uint32), ("side_stream", C.c_void_p),
                ("draw_buffer_bytes", C.c_size_t)]


class AttnDesc(C.Structure):
    _fields_ = [("B", C.c_int32), ("H", C.c_int32), ("S", C.c_int32), ("Dh", C.c_int32), ("causal", C.c_int32),
                ("softmax_scale", C.c_float), ("dtype", C.c_int32), ("q", C.c_void_p), ("k", C.c_void_p),
                ("v", C.c_void_p), ("dO", C.c_void_p), ("store_fmt", C.c_int32), ("forward_mode", C.c_int32),
                ("seed", C.c_uint64), ("tensor_id", C.c_uint32), ("policy_mask", C.c_uint32),
                ("fp8_operands", C.c_int32), ("p_scale", C.c_float), ("ds_scale", C.c_float)]


class StoreDesc(C.Structure):
    _fields_ = [("norm_kind", C.c_int32), ("dtype", C.c_int32), ("T", C.c_int64), ("C", C.c_int64),
                ("O", C.c_int64), ("x", C.c_void_p), ("gamma", C.c_void_p), ("beta", C.c_void_p),
                ("W", C.c_void_p), ("dY", C.c_void_p), ("eps", C.c_float), ("bits", C.c_int32),
                ("grad_fmt", C.c_int32), ("seed", C.c_uint64), ("tensor_id", C.c_uint32), ("policy_mask", C.c_uint32)]


class CouplingDesc(C.Structure):
    _fields_ = [("norm_kind", C.c_int32), ("dtype", C.c_int32), ("T", C.c_int64), ("C", C.c_int64), ("O", C.c_int64),
                ("x", C.c_void_p), ("gamma", C.c_void_p), ("beta", C.c_void_p), ("W", C.c_void_p), ("eps", C.c_float),
                ("store_fmt", C.c_int32), ("forward_mode", C.c_int32), ("seed", C.c_uint64), ("tensor_id", C.c_uint32),
                ("reserved", C.c_uint32)]


class CouplingLayout(C.Structure):
    _fields_ = [(n, C.c_size_t) for n in ("gain_total", "gain_mean_part", "gain_fresh", "X", "X_sq")]


class LsmStat(C.Structure):
    _fields_ = [("mean", C.c_double), ("se", C.c_double), ("z", C.c_double)]


class AttnFp8(C.Structure):
    _fields_ = [("q_scale", C.c_void_p), ("k_scale", C.c_void_p), ("v_scale", C.c_void_p),
                ("do_scale", C.c_void_p), ("p_scale", C.c_float), ("ds_scale", C.c_float),
                ("q_codes", C.c_void_p), ("k_codes", C.c_void_p), ("v_codes", C.c_void_p), ("do_codes", C.c_void_p)]


class BspError(RuntimeError):
    def __init__(self, status, where):
        self.status = status
        super().__init__("%s: %s (status %d)" % (where, status_string(status), status))


_lib = None

_P, _SZ, _I, _I64, _U64, _F = C.c_void_p, C.c_size_t, C.c_int, C.c_int64, C.c_uint64, C.c_float

_SIGNATURES = {
    "bsp_status_string": (C.c_char_p, [_I]),
    "bsp_launch_count": (C.c_ulonglong, []),
    "bsp_d2h_byte_count": (C.c_ulonglong, []),
    "bsp_diag_clear": (_I, [_P, _P]),
    "bsp_philox_fill": (_I, [Key, _SZ, _P, _P]),
    "bsp_amax": (_I, [_P, _I, _SZ, _SZ, _P, _P, _P]),
    "bsp_scale_from_amax": (_I, [_P, _SZ, _I, _P, _P]),
    "bsp_round": (_I, [_P, _I, _SZ, Quant, Key, _U64, _P, _P, _P]),
    "bsp_round_grouped": (_I, [_P, _I, _SZ, _SZ, _I, _I, _P, Key, _P, _P, _P]),
    "bsp_round_2d": (_I, [_P, _I, _I64, _I64, Quant, Key, _P, _P, _I64, _P, _P]),
    "bsp_norm_stats": (_I, [_I, _P, _I, _I64, _I64, _P, _P, _F, _P, _P, _P, _P, _P]),
    "bsp_norm_fwd": (_I, [_I, _P, _I, _I64, _I64, _P, _P, _P, _P, Quant, Key, _P, _P, _I64, _P, _P, _P, _P]),
    "bsp_norm_fwd_draws": (_I, [_I, _P, _I, _I64, _I64, _P, _P, _P, _P, Quant, Key, _I, _I, _P, _I64, _P]),
    "bsp_gemm": (_I, [_I64, _I64, _I64, _I, _P, _I64, _I, _I, _P, _I64, _I, _I, _F, _P, _I64, _P, _P]),
    "bsp_linear_wgrad_mc": (_I, [_I64, _I64, _I64, _P, Quant, _P, Quant, _I64, _I, _P, _P, _P, _P, _P]),
    "bsp_norm_bwd_workspace_bytes": (_SZ, [_I64, _I64]),
    "bsp_norm_bwd": (_I, [_I, _P, _I, _I64, _I64, _P, _P, _P, _P, _P, _I, _I, _I, _P, Quant, Key, _P, _P, _P,
                          _P, _SZ, _P, _P]),
    "bsp_norm_bwd_noalloc": (_I, [_I, _P, _I, _I64, _I64, _P, _P, _P, _P, _P, _I, _I, _I, _P, Quant, Key, _P, _P, _P,
                                  _P, _P]),
    "bsp_norm_gain_mc_workspace_bytes": (_SZ, [_I64, _I64, _I]),
    "bsp_norm_gain_mc": (_I, [_I, _P, _I, _I64, _I64, _P, _P, _P, _P, _P, _I, Quant, Key, _I, _I, _P, _P, _P,
                              _P, _SZ, _P, _P]),
    "bsp_linear_wgrad_workspace_bytes": (_SZ, [_I64, _I64, _I64, _I]),
    "bsp_linear_wgrad": (_I, [_I64, _I64, _I64, _P, Quant, _I, _P, Quant, _I64, _P, _P, _P, _P, _P, _SZ, _P, _P]),
    "bsp_linear_dgrad_workspace_bytes": (_SZ, [_I64, _I64, _I64]),
    "bsp_linear_dgrad": (_I, [_I64, _I64, _I64, _P, Quant, _P, _I, _P, _I, _P, _SZ, _P, _P]),
    "bsp_attn_fwd_stats": (_I, [_I, _I, _I, _I, _I, _F, _P, _P, _P, _I, C.POINTER(AttnFp8), _P, _P, _P, _P]),
    "bsp_attn_dterm": (_I, [_I, _I, _I, _I, _P, _I, _P, _P, _P, _P, _I, _I, Key, _I, _I, _P, _P, _P]),
    "bsp_attn_bwd_dterm": (_I, [_I, _I, _I, _I, _I, _F, _P, _P, _P, _P, _I, C.POINTER(AttnFp8), _P, _P, _P, _P, _P,
                                _P, _P]),
    "bsp_attn_bwd_dterm_fused": (_I, [_I, _I, _I, _I, _I, _F, _P, _P, _P, _P, _I, _P, _P, _P, _P, _P, _P, _P]),
    "bsp_attn_bwd": (_I, [_I, _I, _I, _I, _I, _F, _I, _P, _P, _P, _P, _I, C.POINTER(AttnFp8), _P, _P, _P, _P, _I, _I,
                          Key, _P, _P, _P, _P, _P, _P]),
    "bsp_attn_quantize": (_I, [_P, _I, _SZ, _I, _P, _P, _P, _P, _P, _P]),
    "bsp_mc_accumulate": (_I, [_P, _P, _P, _P, _SZ, _P]),
    "bsp_mc_moments": (_I, [_P, _P, _P, _SZ, _I, _P, _P, _P, _P]),
    "bsp_mc_check_attn_workspace_bytes": (_SZ, [C.POINTER(AttnDesc), _I]),
    "bsp_mc_check_attn": (_I, [C.POINTER(AttnDesc), _I, C.POINTER(VerdictRule), C.POINTER(UseResult), C.POINTER(_I),
                               _P, _SZ, _P, _P]),
    "bsp_mc_stats_workspace_bytes": (_SZ, [_I64]),
    "bsp_mc_stats": (_I, [_P, _P, _P, _I64, _I, _I, C.POINTER(VerdictRule), C.POINTER(UseResult), _P, _SZ, _P]),
    "bsp_mc_check_workspace_bytes": (_SZ, [C.POINTER(NormLinearDesc), _I]),
    "bsp_mc_check_layout": (_I, [C.POINTER(NormLinearDesc), _I, C.POINTER(McLayout)]),
    "bsp_mc_check": (_I, [C.POINTER(NormLinearDesc), _I, C.POINTER(VerdictRule), C.POINTER(UseResult), C.POINTER(_I),
                          _P, _SZ, _P, _P]),
    "bsp_selftest_bounded_wait": (_I, [_U64, _P, _P]),
    "bsp_lsm_check_workspace_bytes": (_SZ, [_I, _I, _I]),
    "bsp_lsm_check": (_I, [_P, _P, _I, _I, _F, _I, _U64, C.c_uint32, _P, C.POINTER(LsmStat), _P, _SZ, _P]),
    "bsp_probs_mc": (_I, [_P, _P, _I64, _I, _I, _I, _F, _U64, C.c_uint32, _I, _I, _P, _P, _P, _P]),
    "bsp_coupling_check_workspace_bytes": (_SZ, [C.POINTER(CouplingDesc), _I]),
    "bsp_coupling_layout": (_I, [C.POINTER(CouplingDesc), _I, C.POINTER(CouplingLayout)]),
    "bsp_coupling_check": (_I, [C.POINTER(CouplingDesc), _I, C.POINTER(C.c_double), C.POINTER(C.c_double), _P, _SZ, _P, _P]),
    "bsp_store_fwd": (_I, [_I, _P, _I, _I64, _I64, _P, _P, _P, _P, _I, Key, _P, _P, _P]),
    "bsp_store_read": (_I, [_I, _P, _I, _I64, _I64, _P, _P, _P, _P, _P, _P, _I, Key, _P, _P, _I64, _P]),
    "bsp_store_wgrad_workspace_bytes": (_SZ, [_I64, _I64]),
    "bsp_store_wgrad": (_I, [_I64, _I64, _I64, _P, Quant, _P, _I64, _P, _P, _SZ, _P, _P]),
    "bsp_mc_check_store_workspace_bytes": (_SZ, [C.POINTER(StoreDesc), _I]),
    "bsp_mc_check_store": (_I, [C.POINTER(StoreDesc), _I, C.POINTER(VerdictRule), C.POINTER(UseResult), C.POINTER(_I),
                                _P, _SZ, _P, _P]),
}


def exported_names():
    """Every symbol include/bsp.h declares."""
    return sorted(_SIGNATURES)


def lib():
    """The loaded library.  Raises if it has not been built: there is no other path."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                "libbsp.so is missing (%s): build it with `python -m paper_2609_39813_b200.build`; "
                "this package has no CPU or PyTorch fallback" % LIB_PATH)
        l = C.CDLL(LIB_PATH)
        for name, (res, args) in _SIGNATURES.items():
            fn = getattr(l, name)
            fn.restype = res
            fn.argtypes = args
        _lib = l
    return _lib


def status_string(status: int) -> str:
    return lib().bsp_status_string(int(status)).decode()


def check(status: int, where: str = "bsp"):
    if status != OK:
        raise BspError(status, where)


def ptr(t):
    """Device pointer of a torch tensor (must be contiguous), or NULL for None; ints pass through."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    if not t.is_contiguous():
        raise ValueError("tensor must be contiguous")
    return t.data_ptr()


def dtype_code(t) -> int:
    import torch
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    raise ValueError("unsupported dtype %s" % t.dtype)


def cur_stream():
    import torch
    return torch.cuda.current_stream().cuda_stream


def key(seed, tensor_id, stream, draw=0) -> Key:
    return Key(int(seed) & 0xFFFFFFFFFFFFFFFF, int(tensor_id), int(stream), int(draw), 0)


def quant(fmt, mode, scale=1.0, scale_dev=None) -> Quant:
    return Quant(int(fmt), int(mode), float(scale), ptr(scale_dev))


def new_diag():
    """A zeroed device bsp_diag_t as a uint8 tensor."""
    import torch
    return torch.zeros(C.sizeof(Diag), dtype=torch.uint8, device="cuda")


def read_diag(d) -> dict:
    import torch
    torch.cuda.synchronize()
    raw = bytes(d.cpu().numpy().tobytes())
    s = Diag.from_buffer_copy(raw)
    import struct
    amax = struct.unpack("<f", struct.pack("<I", s.amax_bits))[0]
    return dict(n_saturated=s.n_saturated, n_nonfinite=s.n_nonfinite, amax=amax, status=s.status)


def workspace(nbytes: int):
    import torch
    return torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device="cuda")


# ----------------------------------------------------------------------------- entry points


def bsp_launch_count() -> int:
    return int(lib().bsp_launch_count())


def bsp_d2h_byte_count() -> int:
    return int(lib().bsp_d2h_byte_count())


def bsp_diag_clear(diag, stream=None):
    check(lib().bsp_diag_clear(ptr(diag), stream if stream is not None else cur_stream()), "bsp_diag_clear")


def bsp_philox_fill(k: Key, n, out, stream=None):
    check(lib().bsp_philox_fill(k, n, ptr(out), stream if stream is not None else cur_stream()), "bsp_philox_fill")


def bsp_amax(x, n_groups, group_size, amax, diag=None, stream=None):
    check(lib().bsp_amax(ptr(x), dtype_code(x), n_groups, group_size, ptr(amax), ptr(diag),
                         stream if stream is not None else cur_stream()), "bsp_amax")


def bsp_scale_from_amax(amax, n, fmt, scale, stream=None):
    check(lib().bsp_scale_from_amax(ptr(amax), n, fmt, ptr(scale), stream if stream is not None else cur_stream()),
          "bsp_scale_from_amax")


def bsp_round(x, n, q: Quant, k: Key, elem_offset, codes, diag=None, stream=None):
    check(lib().bsp_round(ptr(x), dtype_code(x), n, q, k, elem_offset, ptr(codes), ptr(diag),
                          stream if stream is not None else cur_stream()), "bsp_round")


def bsp_round_grouped(x, n_groups, group_size, fmt, mode, scales, k: Key, codes, diag=None, stream=None):
    check(lib().bsp_round_grouped(ptr(x), dtype_code(x), n_groups, group_size, fmt, mode, ptr(scales), k,
                                  ptr(codes), ptr(diag), stream if stream is not None else cur_stream()),
          "bsp_round_grouped")


def bsp_round_2d(x, rows, cols, q: Quant, k: Key, codes, codes_t, ld_t, diag=None, stream=None):
    check(lib().bsp_round_2d(ptr(x), dtype_code(x), rows, cols, q, k, ptr(codes), ptr(codes_t), ld_t, ptr(diag),
                             stream if stream is not None else cur_stream()), "bsp_round_2d")


def bsp_norm_stats(kind, x, T, Cc, gamma, beta, eps, rstd, mean, amax, diag=None, stream=None):
    check(lib().bsp_norm_stats(kind, ptr(x), dtype_code(x), T, Cc, ptr(gamma), ptr(beta), eps, ptr(rstd),
                               ptr(mean), ptr(amax), ptr(diag), stream if stream is not None else cur_stream()),
          "bsp_norm_stats")


def bsp_norm_fwd(kind, x, T, Cc, gamma, beta, rstd, mean, q: Quant, k: Key, u_codes, u_codes_t, ld_t,
                 u_f32=None, u_bf16_t=None, diag=None, stream=None):
    check(lib().bsp_norm_fwd(kind, ptr(x), dtype_code(x), T, Cc, ptr(gamma), ptr(beta), ptr(rstd), ptr(mean), q, k,
                             ptr(u_codes), ptr(u_codes_t), ld_t, ptr(u_f32), ptr(u_bf16_t), ptr(diag),
                             stream if stream is not None else cur_stream()), "bsp_norm_fwd")


def bsp_norm_fwd_draws(kind, x, T, Cc, gamma, beta, rstd, mean, q: Quant, k: Key, draw0, n_draws,
                       u_codes_t_draws, ld_t, stream=None):
    check(lib().bsp_norm_fwd_draws(kind, ptr(x), dtype_code(x), T, Cc, ptr(gamma), ptr(beta), ptr(rstd), ptr(mean),
                                   q, k, draw0, n_draws, ptr(u_codes_t_draws), ld_t,
                                   stream if stream is not None else cur_stream()), "bsp_norm_fwd_draws")


def bsp_gemm(M, N, K, elem, A, lda, a_mn, a_fmt, B, ldb, b_mn, b_fmt, alpha, Cout, ldc, diag=None, stream=None):
    check(lib().bsp_gemm(M, N, K, elem, ptr(A), lda, int(a_mn), a_fmt, ptr(B), ldb, int(b_mn), b_fmt, alpha,
                         ptr(Cout), ldc, ptr(diag), stream if stream is not None else cur_stream()), "bsp_gemm")


def bsp_linear_wgrad_mc(T, O, Cc, dy_codes_t, q_dy: Quant, x_t_draws, q_x: Quant, ld_t, n_draws, g_ref, S1, S2,
                        diag=None, stream=None):
    check(lib().bsp_linear_wgrad_mc(T, O, Cc, ptr(dy_codes_t), q_dy, ptr(x_t_draws), q_x, ld_t, n_draws,
                                    ptr(g_ref), ptr(S1), ptr(S2), ptr(diag),
                                    stream if stream is not None else cur_stream()), "bsp_linear_wgrad_mc")


def bsp_norm_bwd_workspace_bytes(T, Cc):
    return lib().bsp_norm_bwd_workspace_bytes(T, Cc)


def bsp_norm_bwd(kind, x, T, Cc, gamma, beta, rstd, mean, du, gain_read, u_codes, q: Quant, k: Key,
                 dgamma, dbeta, dx, ws, diag=None, stream=None, dx_read=READ_ORIGINAL):
    check(lib().bsp_norm_bwd(kind, ptr(x), dtype_code(x), T, Cc, ptr(gamma), ptr(beta), ptr(rstd), ptr(mean),
                             ptr(du), dtype_code(du), gain_read, dx_read, ptr(u_codes), q, k, ptr(dgamma), ptr(dbeta),
                             ptr(dx), ptr(ws), ws.numel() if ws is not None else 0, ptr(diag),
                             stream if stream is not None else cur_stream()), "bsp_norm_bwd")


def bsp_norm_bwd_noalloc(kind, x, T, Cc, gamma, beta, rstd, mean, du, gain_read, u_codes, q: Quant, k: Key,
                         dgamma, dbeta, dx, diag=None, stream=None, dx_read=READ_ORIGINAL):
    """bsp_norm_bwd without a workspace argument: scratch is the library's own fixed device array
    (for callers that may not allocate device memory).  Raises BspError(ERR_TOO_LARGE) when the
    problem does not fit NORM_BWD_NOALLOC_CAPACITY_BYTES.  Calls that overlap on the GPU race."""
    check(lib().bsp_norm_bwd_noalloc(kind, ptr(x), dtype_code(x), T, Cc, ptr(gamma), ptr(beta), ptr(rstd),
                                     ptr(mean), ptr(du), dtype_code(du), gain_read, dx_read, ptr(u_codes), q, k,
                                     ptr(dgamma), ptr(dbeta), ptr(dx), ptr(diag),
                                     stream if stream is not None else cur_stream()), "bsp_norm_bwd_noalloc")


def bsp_norm_gain_mc_workspace_bytes(T, Cc, K):
    return lib().bsp_norm_gain_mc_workspace_bytes(T, Cc, K)


def bsp_norm_gain_mc(kind, x, T, Cc, gamma, beta, rstd, mean, du, q: Quant, k: Key, draw0, K, g_ref, S1, S2,
                     ws, diag=None, stream=None):
    check(lib().bsp_norm_gain_mc(kind, ptr(x), dtype_code(x), T, Cc, ptr(gamma), ptr(beta), ptr(rstd), ptr(mean),
                                 ptr(du), dtype_code(du), q, k, draw0, K, ptr(g_ref), ptr(S1), ptr(S2), ptr(ws),
                                 ws.numel() if ws is not None else 0, ptr(diag),
                                 stream if stream is not None else cur_stream()), "bsp_norm_gain_mc")


def bsp_linear_wgrad_workspace_bytes(T, O, Cc, x_read):
    return lib().bsp_linear_wgrad_workspace_bytes(T, O, Cc, x_read)


def bsp_linear_wgrad(T, O, Cc, dy_codes_t, q_dy: Quant, x_read, x_t, q_x: Quant, ld_t, dW, mc_ref=None,
                     mc_S1=None, mc_S2=None, ws=None, diag=None, stream=None):
    check(lib().bsp_linear_wgrad(T, O, Cc, ptr(dy_codes_t), q_dy, x_read, ptr(x_t), q_x, ld_t, ptr(dW),
                                 ptr(mc_ref), ptr(mc_S1), ptr(mc_S2), ptr(ws), ws.numel() if ws is not None else 0,
                                 ptr(diag), stream if stream is not None else cur_stream()), "bsp_linear_wgrad")


def bsp_linear_dgrad_workspace_bytes(T, O, Cc):
    return lib().bsp_linear_dgrad_workspace_bytes(T, O, Cc)


def bsp_linear_dgrad(T, O, Cc, dy_codes, q_dy: Quant, W, du, ws, diag=None, stream=None):
    check(lib().bsp_linear_dgrad(T, O, Cc, ptr(dy_codes), q_dy, ptr(W), dtype_code(W), ptr(du), dtype_code(du),
                                 ptr(ws), ws.numel() if ws is not None else 0, ptr(diag),
                                 stream if stream is not None else cur_stream()), "bsp_linear_dgrad")


def _st(stream):
    return stream if stream is not None else cur_stream()


def _fp8ref(f):
    return C.byref(f) if f is not None else None


def bsp_attn_fwd_stats(B, H, S, Dh, causal, softmax_scale, q, k, v, o, lse, diag=None, stream=None, fp8=None):
    check(lib().bsp_attn_fwd_stats(B, H, S, Dh, int(causal), softmax_scale, ptr(q), ptr(k), ptr(v), dtype_code(q),
                                   _fp8ref(fp8), ptr(o), ptr(lse), ptr(diag), _st(stream)), "bsp_attn_fwd_stats")


def bsp_attn_dterm(B, H, S, Dh, dO, o_orig, o_codes, o_scales, o_fmt, d_read, k: Key, draw0, n_draws, d_out,
                   diag=None, stream=None, do_scales=None):
    check(lib().bsp_attn_dterm(B, H, S, Dh, ptr(dO), dtype_code(dO), ptr(do_scales), ptr(o_orig), ptr(o_codes),
                               ptr(o_scales), o_fmt, d_read, k, draw0, n_draws, ptr(d_out), ptr(diag), _st(stream)),
          "bsp_attn_dterm")


def bsp_attn_bwd_dterm(B, H, S, Dh, causal, softmax_scale, q, k, v, dO, lse, dterm, dq, dk, dv, diag=None,
                       stream=None, fp8=None):
    check(lib().bsp_attn_bwd_dterm(B, H, S, Dh, int(causal), softmax_scale, ptr(q), ptr(k), ptr(v), ptr(dO),
                                   dtype_code(q), _fp8ref(fp8), ptr(lse), ptr(dterm), ptr(dq), ptr(dk), ptr(dv),
                                   ptr(diag), _st(stream)), "bsp_attn_bwd_dterm")


def bsp_attn_bwd_dterm_fused(B, H, S, Dh, causal, softmax_scale, q, k, v, dO, lse, dterm, dq, dk, dv, diag=None,
                             stream=None):
    check(lib().bsp_attn_bwd_dterm_fused(B, H, S, Dh, int(causal), softmax_scale, ptr(q), ptr(k), ptr(v), ptr(dO),
                                         dtype_code(q), ptr(lse), ptr(dterm), ptr(dq), ptr(dk), ptr(dv), ptr(diag),
                                         _st(stream)), "bsp_attn_bwd_dterm_fused")


def bsp_attn_bwd(B, H, S, Dh, causal, softmax_scale, fp8_operands, q, k, v, dO, lse, o_orig, o_codes, o_scales,
                 o_fmt, d_read, key_: Key, dq, dk, dv, d_out, diag=None, stream=None, fp8=None):
    """fp8_operands = 1 needs `fp8` (an AttnFp8 with the operand scales) and q, k, v, dO as written by
    bsp_attn_quantize."""
    check(lib().bsp_attn_bwd(B, H, S, Dh, int(causal), softmax_scale, int(fp8_operands), ptr(q), ptr(k), ptr(v),
                             ptr(dO), dtype_code(q), _fp8ref(fp8), ptr(lse), ptr(o_orig), ptr(o_codes), ptr(o_scales),
                             o_fmt, d_read, key_, ptr(dq), ptr(dk), ptr(dv), ptr(d_out), ptr(diag), _st(stream)),
          "bsp_attn_bwd")


def bsp_attn_quantize(x, n_groups, group_size, fmt, xq, amax, scales, diag=None, stream=None, codes=None):
    check(lib().bsp_attn_quantize(ptr(x), n_groups, group_size, fmt, ptr(xq), ptr(codes), ptr(amax), ptr(scales),
                                  ptr(diag), _st(stream)), "bsp_attn_quantize")


def attn_fp8(q_scale, k_scale, v_scale, do_scale, p_scale=256.0, ds_scale=1.0, q_codes=None, k_codes=None,
             v_codes=None, do_codes=None) -> AttnFp8:
    return AttnFp8(ptr(q_scale), ptr(k_scale), ptr(v_scale), ptr(do_scale), float(p_scale), float(ds_scale),
                   ptr(q_codes), ptr(k_codes), ptr(v_codes), ptr(do_codes))


def rule(rel_tol_deterministic=1e-4, qprime_hold=2.0, r_hold=3.0, qprime_fail=4.0, r_fail=6.0, rel_hold=0.0):
    return VerdictRule(rel_tol_deterministic, qprime_hold, r_hold, qprime_fail, r_fail, rel_hold)


def _ruleref(r):
    return C.byref(r) if r is not None else None


def bsp_mc_accumulate(g, g_ref, S1, S2, n, stream=None):
    check(lib().bsp_mc_accumulate(ptr(g), ptr(g_ref), ptr(S1), ptr(S2), n, _st(stream)), "bsp_mc_accumulate")


def bsp_mc_moments(g_ref, S1, S2, n, K, mean=None, var=None, z=None, stream=None):
    check(lib().bsp_mc_moments(ptr(g_ref), ptr(S1), ptr(S2), n, K, ptr(mean), ptr(var), ptr(z), _st(stream)),
          "bsp_mc_moments")


def bsp_selftest_bounded_wait(limit_ns, diag, stream=None):
    check(lib().bsp_selftest_bounded_wait(int(limit_ns), ptr(diag), _st(stream)), "bsp_selftest_bounded_wait")


def bsp_mc_check_attn_workspace_bytes(desc: AttnDesc, K):
    return lib().bsp_mc_check_attn_workspace_bytes(C.byref(desc), K)


def bsp_mc_check_attn(desc: AttnDesc, K, ws, diag=None, stream=None, rule=None):
    """Returns the list of UseResult: per selected policy (U, R, N) the four outputs D, dQ, dK, dV."""
    res = (UseResult * 12)()
    n = C.c_int(0)
    check(lib().bsp_mc_check_attn(C.byref(desc), K, _ruleref(rule), res, C.byref(n), ptr(ws), ws.numel(), ptr(diag),
                                  _st(stream)), "bsp_mc_check_attn")
    return [res[i] for i in range(n.value)]


def bsp_mc_stats_workspace_bytes(n):
    return lib().bsp_mc_stats_workspace_bytes(n)


def bsp_mc_stats(g_ref, g, S2, n, K, fresh, ws, stream=None, rule=None) -> UseResult:
    r = UseResult()
    check(lib().bsp_mc_stats(ptr(g_ref), ptr(g), ptr(S2), n, K, fresh, _ruleref(rule), C.byref(r), ptr(ws),
                             ws.numel(), _st(stream)), "bsp_mc_stats")
    return r


def bsp_mc_check_workspace_bytes(desc: NormLinearDesc, K):
    return lib().bsp_mc_check_workspace_bytes(C.byref(desc), K)


def bsp_mc_check_layout(desc: NormLinearDesc, K) -> McLayout:
    lay = McLayout()
    check(lib().bsp_mc_check_layout(C.byref(desc), K, C.byref(lay)), "bsp_mc_check_layout")
    return lay


def bsp_mc_check(desc: NormLinearDesc, K, ws, diag=None, stream=None, rule=None):
    """Returns the list of UseResult: gain U (dgamma, dbeta), R, N, then weight U, R, N; selected ones only."""
    res = (UseResult * 12)()
    n = C.c_int(0)
    check(lib().bsp_mc_check(C.byref(desc), K, _ruleref(rule), res, C.byref(n), ptr(ws), ws.numel(), ptr(diag),
                             _st(stream)), "bsp_mc_check")
    return [res[i] for i in range(n.value)]


def bsp_store_fwd(kind, x, T, Cc, gamma, beta, rstd, mean, bits, k: Key, codes, steps, stream=None):
    check(lib().bsp_store_fwd(kind, ptr(x), dtype_code(x), T, Cc, ptr(gamma), ptr(beta), ptr(rstd), ptr(mean), bits, k,
                              ptr(codes), ptr(steps), _st(stream)), "bsp_store_fwd")


def bsp_store_read(kind, x, T, Cc, gamma, beta, rstd, mean, codes, steps, read, k: Key, copy_f32, copy_split_t, ld_t,
                   stream=None):
    check(lib().bsp_store_read(kind, ptr(x), dtype_code(x), T, Cc, ptr(gamma), ptr(beta), ptr(rstd), ptr(mean),
                               ptr(codes), ptr(steps), read, k, ptr(copy_f32), ptr(copy_split_t), ld_t, _st(stream)),
          "bsp_store_read")


def bsp_store_wgrad_workspace_bytes(T, O):
    return lib().bsp_store_wgrad_workspace_bytes(T, O)


def bsp_store_wgrad(T, O, Cc, dy_codes_t, q_dy: Quant, copy_split_t, ld_t, dW, ws, diag=None, stream=None):
    check(lib().bsp_store_wgrad(T, O, Cc, ptr(dy_codes_t), q_dy, ptr(copy_split_t), ld_t, ptr(dW), ptr(ws), ws.numel(),
                                ptr(diag), _st(stream)), "bsp_store_wgrad")


def bsp_mc_check_store_workspace_bytes(desc: StoreDesc, K):
    return lib().bsp_mc_check_store_workspace_bytes(C.byref(desc), K)


def bsp_mc_check_store(desc: StoreDesc, K, ws, diag=None, stream=None, rule=None):
    """Returns the list of UseResult: gain U, R, N then weight U, R, N, U/R+eps; selected ones only."""
    res = (UseResult * 8)()
    n = C.c_int(0)
    check(lib().bsp_mc_check_store(C.byref(desc), K, _ruleref(rule), res, C.byref(n), ptr(ws), ws.numel(), ptr(diag),
                                   _st(stream)), "bsp_mc_check_store")
    return [res[i] for i in range(n.value)]


def bsp_lsm_check_workspace_bytes(rows, classes, trials):
    return lib().bsp_lsm_check_workspace_bytes(rows, classes, trials)


def bsp_lsm_check(logits, target, rows, classes, eps, trials, seed, tensor_id, per_trial, ws, stream=None):
    """Returns the eight LsmStat (mean, se, z) of the log-softmax test."""
    out = (LsmStat * 8)()
    check(lib().bsp_lsm_check(ptr(logits), ptr(target), rows, classes, eps, trials, int(seed), tensor_id, ptr(per_trial),
                              out, ptr(ws), ws.numel(), _st(stream)), "bsp_lsm_check")
    return [out[i] for i in range(8)]


def bsp_probs_mc(p, V, rows, n, d, law, param, seed, tensor_id, draw0, K, ds_sum, ds_sq, dV_sum, stream=None):
    check(lib().bsp_probs_mc(ptr(p), ptr(V), rows, n, d, law, param, int(seed), tensor_id, draw0, K, ptr(ds_sum),
                             ptr(ds_sq), ptr(dV_sum), _st(stream)), "bsp_probs_mc")


def bsp_coupling_check_workspace_bytes(desc: CouplingDesc, pairs):
    return lib().bsp_coupling_check_workspace_bytes(C.byref(desc), pairs)


def bsp_coupling_layout(desc: CouplingDesc, pairs) -> CouplingLayout:
    lay = CouplingLayout()
    check(lib().bsp_coupling_layout(C.byref(desc), pairs, C.byref(lay)), "bsp_coupling_layout")
    return lay


def bsp_coupling_check(desc: CouplingDesc, pairs, ws, diag=None, stream=None):
    """Returns (T[pairs], control[pairs]) as lists of floats; the averaged tensors stay in `ws`."""
    T = (C.c_double * pairs)()
    ctl = (C.c_double * pairs)()
    check(lib().bsp_coupling_check(C.byref(desc), pairs, T, ctl, ptr(ws), ws.numel(), ptr(diag), _st(stream)),
          "bsp_coupling_check")
    return list(T), list(ctl)


def ws_view(ws, offset, count, dtype=None):
    """A typed view of `count` elements at byte `offset` of a workspace tensor (float32 by default)."""
    import torch
    dtype = dtype or torch.float32
    nbytes = count * torch.empty((), dtype=dtype).element_size()
    return ws[offset:offset + nbytes].view(dtype)
