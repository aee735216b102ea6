"""Thin Python binding of the iptq C-ABI library (``include/iptq.h``).

Argument marshalling only: torch is used for device memory and streams; every step of the
path runs in the library's CUDA kernels.  The binding fails loudly when ``libiptq.so`` is
missing -- there is no CPU or eager fallback.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libiptq.so")

SM_BITEXP, SM_SHIFTMAX, SM_POLY, SM_LOG2 = 0, 1, 2, 3
LOG2_ZERO = 255          # SM_LOG2 output: code c <= 15 means probability 2^-c, LOG2_ZERO means 0
PROBS_LOG2 = 0           # out_bits value that tells metric_softmax the bytes are SM_LOG2 codes
GELU_POLY4, GELU_POLY2, GELU_SHIFT = 0, 1, 2
LN_SHIFT, LN_NEWTON, LN_PTF = 0, 1, 2

BLOCK_STAGES = ("ln1", "qkv", "attention", "proj", "ln2", "fc1_gelu", "fc2")

OK, ERR_NULL, ERR_SHAPE, ERR_ALIGN, ERR_BITS, ERR_SCALE_RANGE, ERR_VARIANT, ERR_WORKSPACE, ERR_TIMEOUT, ERR_CUDA = range(10)


class Requant(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("mult", "shift", "zp", "qmin", "qmax")]


class SoftmaxConsts(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("variant", "out_bits", "row_len", "x0", "nsh", "M", "dcap",
                                         "qln2", "qb", "qc", "norm_l", "norm_r")] + \
               [("div_mul", C.c_uint32), ("div_shift", C.c_int32), ("f_shl", C.c_int32), ("p_shr", C.c_int32),
                ("table", C.c_void_p), ("table_n", C.c_int32)]


class GeluConsts(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("variant", "in_bits", "Bq", "sh2", "C", "gs", "x0", "nsh", "dcap")] + \
               [("div_mul", C.c_uint32), ("div_shift", C.c_int32), ("out", Requant), ("table", C.c_void_p)]


class LnConsts(C.Structure):
    _fields_ = [("variant", C.c_int32), ("dim", C.c_int32), ("out", Requant)]


class VariantTable(C.Structure):
    _fields_ = [("sm", C.c_int), ("gelu", C.c_int), ("ln1", C.c_int), ("ln2", C.c_int)]


class BlockParams(C.Structure):
    _fields_ = [
        ("B", C.c_int64), ("N", C.c_int32), ("D", C.c_int32), ("H", C.c_int32), ("dh", C.c_int32),
        ("Dh", C.c_int32), ("w_bits", C.c_int32),
        ("table", VariantTable),
        ("ln1_gamma", C.c_void_p), ("ln1_beta", C.c_void_p), ("ln1_ptf", C.c_void_p), ("ln1", C.c_void_p),
        ("w_qkv", C.c_void_p), ("b_qkv", C.c_void_p), ("m_qkv", C.c_void_p), ("s_qkv", C.c_void_p),
        ("attn_bias", C.c_void_p), ("mask_id", C.c_void_p),
        ("sm", C.c_void_p), ("pv_rq", C.c_void_p),
        ("w_proj", C.c_void_p), ("b_proj", C.c_void_p), ("m_proj", C.c_void_p), ("s_proj", C.c_void_p),
        ("proj_zp", C.c_int32),
        ("res1_rq", C.c_void_p),
        ("ln2_gamma", C.c_void_p), ("ln2_beta", C.c_void_p), ("ln2_ptf", C.c_void_p), ("ln2", C.c_void_p),
        ("w_fc1", C.c_void_p), ("b_fc1", C.c_void_p), ("m_fc1", C.c_void_p), ("s_fc1", C.c_void_p),
        ("gelu", C.c_void_p),
        ("w_fc2", C.c_void_p), ("b_fc2", C.c_void_p), ("m_fc2", C.c_void_p), ("s_fc2", C.c_void_p),
        ("fc2_zp", C.c_int32),
        ("res2_rq", C.c_void_p),
        ("act_bits", C.c_int32),
        ("attn_bias_t", C.c_void_p),
    ]


class LinearPlan(C.Structure):
    _fields_ = [("tile_tokens", C.c_int32), ("stages", C.c_int32), ("cta_pairs", C.c_int32), ("smem_bytes", C.c_int32),
                ("grid", C.c_int32), ("channel_tiles", C.c_int32), ("token_tiles", C.c_int32),
                ("staging_buffers", C.c_int32)]


class IptqError(RuntimeError):
    def __init__(self, status, what):
        self.status = status
        msg = lib().iptq_strerror(status).decode() if _lib is not None else "?"
        super().__init__("%s: iptq status %d (%s)" % (what, status, msg))


_lib = None
_vp = C.c_void_p


def lib():
    """Load ``libiptq.so`` (built in-tree by ``paper_2511_15369_b200.build``)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError("libiptq.so is missing: run `python -m paper_2511_15369_b200.build` "
                              "(the library has no CPU fallback)")
        L = C.CDLL(LIB_PATH)
        L.iptq_strerror.restype = C.c_char_p
        L.iptq_strerror.argtypes = [C.c_int]
        L.iptq_launch_count.restype = C.c_int64
        L.iptq_requant_prepare.argtypes = [C.c_double, C.c_int32, C.c_int32, C.c_int32, C.POINTER(Requant)]
        L.iptq_channel_requant_prepare.argtypes = [_vp, C.c_int, _vp, _vp]
        L.iptq_softmax_prepare.argtypes = [C.c_double, C.c_int, C.c_int, C.c_int, C.POINTER(SoftmaxConsts)]
        L.iptq_softmax.argtypes = [_vp, _vp, C.c_int64, C.c_int, _vp, C.c_int64, C.POINTER(SoftmaxConsts), _vp]
        L.iptq_softmax_table.argtypes = [C.POINTER(SoftmaxConsts), _vp, C.c_int32, _vp]
        L.iptq_gelu_prepare.argtypes = [C.c_double, C.c_int, C.c_double, C.c_int, C.c_int, C.c_int,
                                        C.POINTER(GeluConsts)]
        L.iptq_gelu.argtypes = [_vp, _vp, C.c_int64, C.POINTER(GeluConsts), _vp]
        L.iptq_gelu_fit.argtypes = [C.c_double, C.c_double, C.c_int, C.POINTER(C.c_double), C.POINTER(C.c_double),
                                    C.POINTER(C.c_double)]
        L.iptq_gelu_prepare_coeffs.argtypes = [C.c_double, C.c_int, C.c_double, C.c_int, C.c_int, C.c_double,
                                               C.c_double, C.POINTER(GeluConsts)]
        L.iptq_gelu_table.argtypes = [C.POINTER(GeluConsts), _vp, _vp]
        L.iptq_layernorm_prepare.argtypes = [C.c_int, _vp, _vp, C.c_double, C.c_int, C.c_int, C.c_int, _vp, _vp,
                                             C.POINTER(LnConsts)]
        L.iptq_layernorm.argtypes = [_vp, _vp, C.c_int64, C.c_int, _vp, _vp, _vp, C.POINTER(LnConsts), _vp]
        L.iptq_linear_workspace_bytes.restype = C.c_size_t
        L.iptq_linear_workspace_bytes.argtypes = [C.c_int64, C.c_int, C.c_int, C.c_int]
        L.iptq_linear_plan.argtypes = [C.c_int64, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, C.POINTER(LinearPlan)]
        L.iptq_linear.argtypes = [_vp, _vp, C.c_int, _vp, _vp, _vp, C.c_int32, _vp, C.POINTER(Requant), _vp,
                                  C.c_int64, C.c_int, C.c_int, _vp, C.c_size_t, _vp]
        L.iptq_linear_bits.argtypes = [_vp, _vp, C.c_int, _vp, _vp, _vp, C.c_int32, _vp, C.POINTER(Requant), _vp,
                                       C.c_int64, C.c_int, C.c_int, C.c_int, _vp, C.c_size_t, _vp]
        L.iptq_linear_w4_static.argtypes = [_vp, _vp, _vp, _vp, _vp, C.c_int32, _vp, C.POINTER(Requant), _vp,
                                            C.c_int64, C.c_int, C.c_int, _vp, _vp]
        L.iptq_unpack_int4.argtypes = [_vp, _vp, C.c_int64, _vp]
        L.iptq_gather_rows.argtypes = [_vp, _vp, _vp, C.c_int64, C.c_int, C.c_int, _vp]
        L.iptq_patchify.argtypes = [_vp, _vp, C.c_int64, C.c_int, C.c_int, C.c_int, C.c_int, _vp]
        L.iptq_attention_workspace_bytes.restype = C.c_size_t
        L.iptq_attention_workspace_bytes.argtypes = [C.c_int64, C.c_int, C.c_int, C.c_int]
        L.iptq_attention_bias_bytes.restype = C.c_size_t
        L.iptq_attention_bias_bytes.argtypes = [C.c_int, C.c_int]
        L.iptq_attention_bias_prepare.argtypes = [_vp, _vp, C.c_int, C.c_int, _vp]
        L.iptq_attention_block.argtypes = [_vp, _vp, _vp, _vp, C.c_int64, C.c_int, C.c_int, C.c_int, _vp, _vp, _vp,
                                           C.POINTER(SoftmaxConsts), C.POINTER(Requant), _vp, C.c_size_t, _vp]
        L.iptq_mlp_workspace_bytes.restype = C.c_size_t
        L.iptq_mlp_workspace_bytes.argtypes = [C.c_int64, C.c_int, C.c_int, C.c_int]
        L.iptq_mlp_block.argtypes = [_vp, _vp, _vp, _vp, _vp, C.POINTER(GeluConsts), _vp, _vp, _vp, _vp, C.c_int32,
                                     _vp, C.POINTER(Requant), _vp, C.c_int64, C.c_int, C.c_int, C.c_int, _vp,
                                     C.c_size_t, _vp]
        L.iptq_encoder_block_workspace_bytes.restype = C.c_size_t
        L.iptq_encoder_block_workspace_bytes.argtypes = [C.POINTER(BlockParams)]
        L.iptq_encoder_block.argtypes = [_vp, _vp, C.POINTER(BlockParams), _vp, C.c_size_t, _vp]
        L.iptq_encoder_block_profiled.argtypes = [_vp, _vp, C.POINTER(BlockParams), _vp, C.c_size_t, _vp,
                                                  C.POINTER(C.c_void_p), C.c_int]
        L.iptq_workspace_init.argtypes = [_vp, C.c_size_t, _vp]
        L.iptq_check.argtypes = [_vp, _vp]
        L.iptq_workspace_set_wait_limit.argtypes = [_vp, C.c_size_t, C.c_int32, _vp]
        L.iptq_selftest_wait_timeout.argtypes = [_vp, C.c_size_t, _vp]
        L.iptq_metric_softmax.argtypes = [_vp, _vp, C.c_int64, C.c_int, C.c_double, C.c_int, _vp, _vp, _vp]
        L.iptq_metric_gelu.argtypes = [_vp, _vp, C.c_int64, C.c_double, C.c_double, C.c_int, _vp, _vp, _vp]
        L.iptq_metric_layernorm.argtypes = [_vp, _vp, C.c_int64, C.c_int, _vp, _vp, _vp, C.c_double, C.c_int, _vp,
                                            _vp, _vp]
        for f in (L.iptq_softplus, L.iptq_sqnr_db, L.iptq_metric_term, L.iptq_op_count):
            f.restype = C.c_double
        L.iptq_softplus.argtypes = [C.c_double]
        L.iptq_sqnr_db.argtypes = [C.c_double, C.c_double]
        L.iptq_metric_term.argtypes = [C.c_double, C.c_double, C.c_double, C.c_double]
        L.iptq_op_count.argtypes = [C.c_int, C.c_int, C.c_int64, C.c_int]
        L.iptq_metric_select.argtypes = [C.POINTER(C.c_double), C.c_int]
        _lib = L
    return _lib


def exported_symbols():
    """Names declared in include/iptq.h (used by the CPU-side load test)."""
    return ["iptq_requant_prepare", "iptq_channel_requant_prepare", "iptq_softmax_prepare", "iptq_softmax", "iptq_softmax_table",
            "iptq_gelu_prepare", "iptq_gelu", "iptq_gelu_table", "iptq_gelu_fit", "iptq_gelu_prepare_coeffs", "iptq_layernorm_prepare", "iptq_layernorm",
            "iptq_unpack_int4", "iptq_linear_workspace_bytes", "iptq_linear_plan", "iptq_linear", "iptq_linear_bits", "iptq_linear_w4_static", "iptq_gather_rows", "iptq_patchify", "iptq_attention_workspace_bytes", "iptq_attention_bias_bytes", "iptq_attention_bias_prepare", "iptq_attention_block",
            "iptq_mlp_workspace_bytes", "iptq_mlp_block", "iptq_encoder_block_workspace_bytes",
            "iptq_encoder_block", "iptq_encoder_block_profiled", "iptq_workspace_init", "iptq_check", "iptq_workspace_set_wait_limit", "iptq_selftest_wait_timeout", "iptq_strerror", "iptq_launch_count",
            "iptq_metric_softmax", "iptq_metric_gelu", "iptq_metric_layernorm", "iptq_softplus", "iptq_sqnr_db",
            "iptq_metric_term", "iptq_op_count", "iptq_metric_select"]


def _chk(rc, what):
    if rc != 0:
        raise IptqError(rc, what)


def _dp(t):
    """Device pointer of a contiguous CUDA tensor (None -> NULL)."""
    if t is None:
        return None
    assert isinstance(t, torch.Tensor) and t.is_cuda and t.is_contiguous(), "expected a contiguous CUDA tensor"
    return t.data_ptr()


def _stream():
    return torch.cuda.current_stream().cuda_stream


def _ref(s):
    return None if s is None else C.byref(s)


def launch_count() -> int:
    return int(lib().iptq_launch_count())


# ------------------------------------------------------------------ host-side prepare

def requant_prepare(ratio, zp=0, qmin=-128, qmax=127) -> Requant:
    r = Requant()
    _chk(lib().iptq_requant_prepare(float(ratio), zp, qmin, qmax, C.byref(r)), "iptq_requant_prepare")
    return r


def channel_requant_prepare(ratios):
    ratios = np.ascontiguousarray(ratios, dtype=np.float64)
    mult = np.empty(ratios.shape[0], dtype=np.int32)
    shift = np.empty(ratios.shape[0], dtype=np.int8)
    _chk(lib().iptq_channel_requant_prepare(ratios.ctypes.data, ratios.shape[0], mult.ctypes.data,
                                            shift.ctypes.data), "iptq_channel_requant_prepare")
    return mult, shift


def softmax_prepare(in_scale, row_len, out_bits=8, variant=SM_BITEXP) -> SoftmaxConsts:
    c = SoftmaxConsts()
    _chk(lib().iptq_softmax_prepare(float(in_scale), row_len, out_bits, variant, C.byref(c)), "iptq_softmax_prepare")
    return c


def gelu_prepare(in_scale, in_bits, out_scale, out_zp=0, out_bits=8, variant=GELU_POLY4) -> GeluConsts:
    c = GeluConsts()
    _chk(lib().iptq_gelu_prepare(float(in_scale), in_bits, float(out_scale), out_zp, out_bits, variant,
                                 C.byref(c)), "iptq_gelu_prepare")
    return c


def layernorm_prepare(gamma, beta, out_scale, out_zp=0, out_bits=8, variant=LN_SHIFT):
    g = np.ascontiguousarray(gamma, dtype=np.float32)
    b = np.ascontiguousarray(beta, dtype=np.float32)
    gq = np.empty(g.shape[0], dtype=np.int32)
    bq = np.empty(g.shape[0], dtype=np.int32)
    c = LnConsts()
    _chk(lib().iptq_layernorm_prepare(g.shape[0], g.ctypes.data, b.ctypes.data, float(out_scale), out_zp, out_bits,
                                      variant, gq.ctypes.data, bq.ctypes.data, C.byref(c)), "iptq_layernorm_prepare")
    return gq, bq, c


# ------------------------------------------------------------------ workspace

class Workspace:
    """A caller-owned device scratch buffer whose first 256 bytes are the status block."""

    def __init__(self, nbytes: int, device="cuda"):
        nbytes = max(int(nbytes), 256)
        self.buf = torch.empty(nbytes + 256, dtype=torch.uint8, device=device)
        off = (-self.buf.data_ptr()) % 256
        self.ptr = self.buf.data_ptr() + off
        self.nbytes = nbytes
        _chk(lib().iptq_workspace_init(self.ptr, self.nbytes, _stream()), "iptq_workspace_init")

    def check(self):
        _chk(lib().iptq_check(_stream(), self.ptr), "iptq_check")

    def reset(self):
        """Clears the status block (after a reported time-out the workspace is usable again)."""
        _chk(lib().iptq_workspace_init(self.ptr, self.nbytes, _stream()), "iptq_workspace_init")

    def set_wait_limit(self, microseconds: int):
        _chk(lib().iptq_workspace_set_wait_limit(self.ptr, self.nbytes, int(microseconds), _stream()),
             "iptq_workspace_set_wait_limit")

    def status_words(self):
        """The first int32 fields of the status block: (flag, wait id, block, work_next, work_done, wait limit)."""
        torch.cuda.synchronize()
        off = self.ptr - self.buf.data_ptr()
        return self.buf[off:off + 24].cpu().view(torch.int32).tolist()


# ------------------------------------------------------------------ device entry points

def softmax(scores, consts: SoftmaxConsts, bias=None, out=None):
    rows, n = scores.shape
    if out is None:
        out = torch.empty((rows, n), dtype=torch.uint8, device=scores.device)
    period = bias.shape[0] if bias is not None else 1
    _chk(lib().iptq_softmax(_dp(scores), _dp(out), rows, n, _dp(bias), period, C.byref(consts), _stream()),
         "iptq_softmax")
    return out


SOFTMAX_TABLE_MAX = 51200


def softmax_table(consts: SoftmaxConsts, device="cuda"):
    """Writes the exponential table of ``consts`` to device memory once and attaches it to ``consts`` (the Softmax
    and attention kernels then copy it to shared memory instead of rebuilding it in every CTA).  Returns the table
    tensor, which the caller must keep alive as long as ``consts`` is used, or None where the variant or scale has
    no table."""
    t = torch.empty(SOFTMAX_TABLE_MAX, dtype=torch.int16, device=device)
    _chk(lib().iptq_softmax_table(C.byref(consts), _dp(t), SOFTMAX_TABLE_MAX, _stream()), "iptq_softmax_table")
    if not consts.table:
        return None
    return t


def gelu(x, consts: GeluConsts, out=None):
    if out is None:
        out = torch.empty(x.shape, dtype=torch.int8, device=x.device)
    _chk(lib().iptq_gelu(_dp(x), _dp(out), x.numel(), C.byref(consts), _stream()), "iptq_gelu")
    return out


GELU_TABLE_SIZE = 65536


def gelu_fit(lo, hi, points=4001):
    """Data-aware coefficients of the quartic erf polynomial for inputs in [lo, hi] (Sec. 3.3, Eq. (4)).
    Returns (a, b, rms residual)."""
    a, b, r = C.c_double(), C.c_double(), C.c_double()
    _chk(lib().iptq_gelu_fit(float(lo), float(hi), int(points), C.byref(a), C.byref(b), C.byref(r)), "iptq_gelu_fit")
    return a.value, b.value, r.value


def gelu_prepare_coeffs(in_scale, in_bits, out_scale, out_zp, out_bits, a, b) -> GeluConsts:
    c = GeluConsts()
    _chk(lib().iptq_gelu_prepare_coeffs(float(in_scale), in_bits, float(out_scale), out_zp, out_bits, float(a),
                                        float(b), C.byref(c)), "iptq_gelu_prepare_coeffs")
    return c


def gelu_table(consts: GeluConsts, device="cuda"):
    """Tabulates the integer GELU of ``consts`` over all 16-bit inputs on the device and attaches the table to
    ``consts`` (the FC1 epilogue then reads it instead of evaluating the polynomial).  Returns the table tensor,
    which the caller must keep alive as long as ``consts`` is used."""
    t = torch.empty(GELU_TABLE_SIZE, dtype=torch.int8, device=device)
    _chk(lib().iptq_gelu_table(C.byref(consts), _dp(t), _stream()), "iptq_gelu_table")
    consts.table = t.data_ptr()
    return t


# ------------------------------------------------------------------ Unified Metric (Sec. 3.5)

LAYER_SOFTMAX, LAYER_GELU, LAYER_LAYERNORM = 0, 1, 2
METRIC_WORK_BYTES = 32768


class MetricScratch:
    """Device scratch of the metric reductions: the partial sums and the [sum X^2, sum (X - Q)^2] result."""

    def __init__(self, device="cuda"):
        self.work = torch.empty(METRIC_WORK_BYTES // 8, dtype=torch.float64, device=device)
        self.sums = torch.empty(2, dtype=torch.float64, device=device)


def metric_softmax(scores, probs, in_scale, out_bits=8, scratch: MetricScratch | None = None):
    """Enqueues the reduction; returns the device tensor [sum X^2, sum (X - Q)^2] (scratch.sums)."""
    sc = scratch or MetricScratch(scores.device)
    rows, n = scores.shape
    _chk(lib().iptq_metric_softmax(_dp(scores), _dp(probs), rows, n, float(in_scale), out_bits, _dp(sc.sums),
                                   _dp(sc.work), _stream()), "iptq_metric_softmax")
    return sc.sums


def metric_gelu(x, y, in_scale, out_scale, out_zp, scratch: MetricScratch | None = None):
    sc = scratch or MetricScratch(x.device)
    _chk(lib().iptq_metric_gelu(_dp(x), _dp(y), x.numel(), float(in_scale), float(out_scale), int(out_zp),
                                _dp(sc.sums), _dp(sc.work), _stream()), "iptq_metric_gelu")
    return sc.sums


def metric_layernorm(x, y, gamma, beta, out_scale, out_zp, ptf_shift=None, scratch: MetricScratch | None = None):
    """gamma, beta: device float32 [dim] (the float parameters, not the quantised ones)."""
    sc = scratch or MetricScratch(x.device)
    rows, dim = x.shape
    _chk(lib().iptq_metric_layernorm(_dp(x), _dp(y), rows, dim, _dp(gamma), _dp(beta), _dp(ptf_shift),
                                     float(out_scale), int(out_zp), _dp(sc.sums), _dp(sc.work), _stream()),
         "iptq_metric_layernorm")
    return sc.sums


def softplus(v):
    return float(lib().iptq_softplus(float(v)))


def sqnr_db(sum_x2, sum_err2):
    return float(lib().iptq_sqnr_db(float(sum_x2), float(sum_err2)))


def metric_term(q_db, p, c_ops, c_unit=1.0e6):
    return float(lib().iptq_metric_term(float(q_db), float(p), float(c_ops), float(c_unit)))


def op_count(kind, variant, rows, row_len):
    return float(lib().iptq_op_count(int(kind), int(variant), int(rows), int(row_len)))


def metric_select(terms):
    arr = (C.c_double * len(terms))(*[float(t) for t in terms])
    return int(lib().iptq_metric_select(arr, len(terms)))


def layernorm(x, gamma_q, beta_q, consts: LnConsts, ptf_shift=None, out=None):
    rows, dim = x.shape
    if out is None:
        out = torch.empty((rows, dim), dtype=torch.int8, device=x.device)
    _chk(lib().iptq_layernorm(_dp(x), _dp(out), rows, dim, _dp(gamma_q), _dp(beta_q), _dp(ptf_shift),
                              C.byref(consts), _stream()), "iptq_layernorm")
    return out


def unpack_int4(w_packed):
    """Packed int4 weights [N, K/2] -> int8 [N, K] on the device (what ``w_bits=8`` takes), once at load time."""
    n, k2 = w_packed.shape
    out = torch.empty((n, 2 * k2), dtype=torch.int8, device=w_packed.device)
    _chk(lib().iptq_unpack_int4(_dp(w_packed), _dp(out), n * 2 * k2, _stream()), "iptq_unpack_int4")
    return out


def linear_plan(M, N, K, residual=False, gelu_table=False, sm_count=0) -> LinearPlan:
    """How ``linear`` would tile the product (host arithmetic; ``sm_count=0`` asks the current device)."""
    out = LinearPlan()
    _chk(lib().iptq_linear_plan(M, N, K, int(residual), int(gelu_table), sm_count, C.byref(out)), "iptq_linear_plan")
    return out


def linear_workspace_bytes(M, N, K, w_bits=8):
    return int(lib().iptq_linear_workspace_bytes(M, N, K, w_bits))


def linear(x, w, bias, mult, shift, ws: Workspace, out_zp=0, residual=None, residual_rq=None, w_bits=8, out=None,
           out_bits=8):
    M, K = x.shape
    N = w.shape[0]
    if out is None:
        out = torch.empty((M, N), dtype=torch.int8, device=x.device)
    _chk(lib().iptq_linear_bits(_dp(x), _dp(w), w_bits, _dp(bias), _dp(mult), _dp(shift), out_zp, _dp(residual),
                                _ref(residual_rq), _dp(out), M, N, K, out_bits, ws.ptr, ws.nbytes, _stream()),
         "iptq_linear")
    return out


STATIC_SCRATCH_BYTES = 4 << 20


def linear_w4_static(x, w_packed, bias, mult, shift, out_zp=0, residual=None, residual_rq=None, status=None, out=None):
    """``linear(..., w_bits=4)`` for callers that cannot hand over a workspace: the unpacked weights go to a
    device array the library owns (N*K <= STATIC_SCRATCH_BYTES).  Nothing is allocated by the call itself, so
    ``out`` should be passed in by such callers; it is created here only as a convenience.  Calls on one
    device share the array: keep them on one stream."""
    M, K = x.shape
    N = w_packed.shape[0]
    if out is None:
        out = torch.empty((M, N), dtype=torch.int8, device=x.device)
    _chk(lib().iptq_linear_w4_static(_dp(x), _dp(w_packed), _dp(bias), _dp(mult), _dp(shift), out_zp, _dp(residual),
                                     _ref(residual_rq), _dp(out), M, N, K, status, _stream()),
         "iptq_linear_w4_static")
    return out


def gather_rows(src, index, out=None):
    """dst row i = concatenation of the src rows index[i, :] (negative -> zeros); src [n_src, C] int8, index [n_dst, parts] int32."""
    n_dst, parts = index.shape
    C_ = src.shape[1]
    if out is None:
        out = torch.empty((n_dst, parts * C_), dtype=torch.int8, device=src.device)
    _chk(lib().iptq_gather_rows(_dp(src), _dp(out), _dp(index), n_dst, parts, C_, _stream()), "iptq_gather_rows")
    return out


def patchify(img, patch=16, out=None):
    """img: int8 [B, C, H, W] -> patch rows int8 [B * (H/patch) * (W/patch), C * patch * patch]."""
    B, C_, H, W = img.shape
    if out is None:
        out = torch.empty((B * (H // patch) * (W // patch), C_ * patch * patch), dtype=torch.int8, device=img.device)
    _chk(lib().iptq_patchify(_dp(img), _dp(out), B, C_, H, W, patch, _stream()), "iptq_patchify")
    return out


def attention_workspace_bytes(B, H, N, dh):
    return int(lib().iptq_attention_workspace_bytes(B, H, N, dh))


def attention_bias_prepare(bias):
    """The relative-position bias [H, N, N] (N <= 64) in the layout the window kernel reads fastest, written once at
    load time; returns the device tensor to pass as ``bias_t`` (None for N > 64, where there is no such layout)."""
    H, N, _ = bias.shape
    nbytes = int(lib().iptq_attention_bias_bytes(H, N))
    if nbytes == 0:
        return None
    t = torch.empty(nbytes // 4, dtype=torch.int32, device=bias.device)
    _chk(lib().iptq_attention_bias_prepare(_dp(bias), _dp(t), H, N, _stream()), "iptq_attention_bias_prepare")
    return t


def attention_block(q, k, v, sm: SoftmaxConsts, out_rq: Requant, ws: Workspace, bias=None, mask_id=None, out=None,
                    bias_t=None):
    B, H, N, dh = q.shape
    if out is None:
        out = torch.empty((B, N, H * dh), dtype=torch.int8, device=q.device)
    _chk(lib().iptq_attention_block(_dp(q), _dp(k), _dp(v), _dp(out), B, H, N, dh, _dp(bias), _dp(bias_t),
                                    _dp(mask_id), C.byref(sm), C.byref(out_rq), ws.ptr, ws.nbytes, _stream()),
         "iptq_attention_block")
    return out


def mlp_workspace_bytes(M, D, Dh, w_bits=8):
    return int(lib().iptq_mlp_workspace_bytes(M, D, Dh, w_bits))


def mlp_block(x, w1, b1, m1, s1, gelu_c: GeluConsts, ws: Workspace, w2=None, b2=None, m2=None, s2=None, out_zp=0,
              residual=None, residual_rq=None, w_bits=8, out=None):
    M, D = x.shape
    Dh = w1.shape[0]
    if out is None:
        out = torch.empty((M, D if w2 is not None else Dh), dtype=torch.int8, device=x.device)
    _chk(lib().iptq_mlp_block(_dp(x), _dp(w1), _dp(b1), _dp(m1), _dp(s1), C.byref(gelu_c), _dp(w2), _dp(b2),
                              _dp(m2), _dp(s2), out_zp, _dp(residual), _ref(residual_rq), _dp(out), M, D, Dh,
                              w_bits, ws.ptr, ws.nbytes, _stream()), "iptq_mlp_block")
    return out


class EncoderBlock:
    """Device-resident parameters of one integer encoder block, prepared from a ``synth.BlockSpec``
    (or any object with the same fields) with the library's own ``*_prepare`` functions."""

    def __init__(self, spec, table=(SM_BITEXP, GELU_POLY4, LN_SHIFT, LN_SHIFT), device="cuda", gelu_table_on=True,
                 softmax_table_on=True, unpack_w4_once=False):
        sh = spec.shape
        self.shape = sh
        self.keep = []          # host structs and device tensors referenced by raw pointers
        p = BlockParams()
        # W4 weights may be unpacked here, once, instead of by four kernels at every call (same values, same results)
        w_bits = 8 if (spec.w_bits == 4 and unpack_w4_once) or spec.w_bits == 6 else spec.w_bits   # 6-bit weights are int8 values
        ab = getattr(spec, "a_bits", 8)                # activation width: 8, or 6 for the W6A6 setting
        p.B, p.N, p.D, p.H, p.dh, p.Dh, p.w_bits = sh.B, sh.N, sh.D, sh.H, sh.dh, sh.Dh, w_bits
        p.table = VariantTable(*table)
        p.act_bits = ab
        sm_v, gelu_v, ln1_v, ln2_v = table

        def dev(a):
            if a is None:
                return None
            t = torch.from_numpy(np.ascontiguousarray(a)).to(device)
            self.keep.append(t)
            return t.data_ptr()

        def host(s):
            self.keep.append(s)
            return C.addressof(s)

        for name, lnspec, var in (("ln1", spec.ln1, ln1_v), ("ln2", spec.ln2, ln2_v)):
            gq, bq, c = layernorm_prepare(lnspec["gamma"], lnspec["beta"], lnspec["out_scale"], lnspec["out_zp"], ab, var)
            setattr(p, name + "_gamma", dev(gq))
            setattr(p, name + "_beta", dev(bq))
            setattr(p, name + "_ptf", dev(lnspec.get("ptf")))
            setattr(p, name, host(c))
        for name, ls in (("qkv", spec.qkv), ("proj", spec.proj), ("fc1", spec.fc1), ("fc2", spec.fc2)):
            m, s = channel_requant_prepare(ls.ratio)
            if spec.w_bits == 4 and unpack_w4_once:
                wt = unpack_int4(torch.from_numpy(np.ascontiguousarray(ls.w_packed)).to(device))
                self.keep.append(wt)
                setattr(p, "w_" + name, wt.data_ptr())
            else:
                setattr(p, "w_" + name, dev(ls.w_packed))
            setattr(p, "b_" + name, dev(ls.bias))
            setattr(p, "m_" + name, dev(m))
            setattr(p, "s_" + name, dev(s))
        p.attn_bias = dev(spec.attn_bias)
        if spec.attn_bias is not None:
            bt = attention_bias_prepare(self.keep[-1])      # a weight: laid out once, here
            if bt is not None:
                self.keep.append(bt)
                p.attn_bias_t = bt.data_ptr()
        p.mask_id = dev(spec.mask_id)
        # the logarithm candidate writes 4-bit codes and its P V product is at scale 2^-15 instead of 2^-7
        log2 = sm_v == SM_LOG2
        sc = softmax_prepare(spec.softmax_scale, sh.N, 4 if log2 else ab, sm_v)
        if softmax_table_on:
            self.keep.append(softmax_table(sc, device))
        p.sm = host(sc)
        qa = 1 << (ab - 1)
        p.pv_rq = host(requant_prepare(spec.pv_ratio * qa / 32768 if log2 else spec.pv_ratio, 0, -qa, qa - 1))
        p.proj_zp, p.fc2_zp = spec.proj.out_zp, spec.fc2.out_zp
        p.res1_rq = host(requant_prepare(spec.proj.res_ratio / 65536.0, zp=spec.proj.res_zp))
        p.res2_rq = host(requant_prepare(spec.fc2.res_ratio / 65536.0, zp=spec.fc2.res_zp))
        gl = spec.gelu
        gc = gelu_prepare(gl["in_scale"], gl["in_bits"], gl["out_scale"], gl["out_zp"], ab, gelu_v)
        if gelu_table_on:
            self.keep.append(gelu_table(gc, device))
        p.gelu = host(gc)
        self.params = p
        self.ws = Workspace(int(lib().iptq_encoder_block_workspace_bytes(C.byref(p))), device)

    def __call__(self, x, out=None):
        T, D = x.shape
        if out is None:
            out = torch.empty((T, D), dtype=torch.int8, device=x.device)
        _chk(lib().iptq_encoder_block(_dp(x), _dp(out), C.byref(self.params), self.ws.ptr, self.ws.nbytes,
                                      _stream()), "iptq_encoder_block")
        return out

    def profiled(self, x, out, events):
        """Same launches as ``__call__`` with ``events[0]`` recorded before the first kernel and ``events[i]``
        after stage i of ``BLOCK_STAGES`` (``torch.cuda.Event(enable_timing=True)``, each recorded once before)."""
        assert len(events) == len(BLOCK_STAGES) + 1
        arr = (C.c_void_p * len(events))(*[e.cuda_event for e in events])
        _chk(lib().iptq_encoder_block_profiled(_dp(x), _dp(out), C.byref(self.params), self.ws.ptr, self.ws.nbytes,
                                               _stream(), arr, len(events)), "iptq_encoder_block_profiled")
        return out

    def run_host(self, x_host, y_host, x_dev, y_dev):
        """One step from HOST buffers: pinned ``x_host`` -> device, the block, device -> pinned ``y_host``;
        all three are enqueued on the current stream (the caller synchronises)."""
        x_dev.copy_(x_host, non_blocking=True)
        self(x_dev, y_dev)
        y_host.copy_(y_dev, non_blocking=True)
        return y_host
