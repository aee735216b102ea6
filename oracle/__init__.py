"""ctypes front end of the CPU oracle (``iptq_oracle.c``).

TEST INFRASTRUCTURE ONLY.  The oracle is a plain C restatement of the integer
Softmax / GELU / LayerNorm / fused-block arithmetic; it is built with gcc and
called through ctypes with numpy arrays.  Nothing in the CUDA package imports
this module, and this module imports nothing from the CUDA package.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "iptq_oracle.c")
_HDR = os.path.join(_HERE, "iptq_oracle.h")
_LIB = os.path.join(_HERE, "liboracle_iptq.so")

SM_BITEXP, SM_SHIFTMAX, SM_POLY, SM_LOG2 = 0, 1, 2, 3
LOG2_ZERO = 255          # SM_LOG2 writes codes: probability 2^-code for 0..15, LOG2_ZERO for probability 0
GELU_POLY4, GELU_POLY2, GELU_SHIFT = 0, 1, 2
LN_SHIFT, LN_NEWTON, LN_PTF = 0, 1, 2


class Requant(C.Structure):
    _fields_ = [("mult", C.c_int32), ("shift", C.c_int32), ("zp", C.c_int32),
                ("qmin", C.c_int32), ("qmax", C.c_int32)]


class SoftmaxConsts(C.Structure):
    _fields_ = [(n, C.c_int32) for n in
                ("variant", "out_bits", "row_len", "x0", "nsh", "M", "dcap",
                 "qln2", "qb", "qc", "norm_l", "norm_r")]


class GeluConsts(C.Structure):
    _fields_ = [(n, C.c_int32) for n in
                ("variant", "in_bits", "Bq", "sh2", "C", "gs", "x0", "nsh", "dcap")] + [("out", Requant)]


class LnConsts(C.Structure):
    _fields_ = [("variant", C.c_int32), ("dim", C.c_int32), ("out", Requant)]


class BlockParams(C.Structure):
    _fields_ = [
        ("B", C.c_int64), ("N", C.c_int32), ("D", C.c_int32), ("H", C.c_int32), ("dh", C.c_int32),
        ("Dh", C.c_int32), ("w_bits", C.c_int32),
        ("sm_variant", C.c_int32), ("gelu_variant", C.c_int32), ("ln1_variant", C.c_int32), ("ln2_variant", C.c_int32),
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
    ]


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (``-O2 -fopenmp``) if the library is stale."""
    stale = force or not os.path.exists(_LIB) or any(
        os.path.getmtime(p) > os.path.getmtime(_LIB) for p in (_SRC, _HDR))
    if stale:
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-Wall",
                               "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        L = _lib
        L.oracle_requant.restype = C.c_int32
        L.oracle_requant.argtypes = [C.c_int32, C.POINTER(Requant)]
        L.oracle_requant_prepare.argtypes = [C.c_double, C.c_int32, C.c_int32, C.c_int32, C.POINTER(Requant)]
        L.oracle_softmax_prepare.argtypes = [C.c_double, C.c_int, C.c_int, C.c_int, C.POINTER(SoftmaxConsts)]
        L.oracle_softmax_exp.restype = C.c_int64
        L.oracle_softmax_exp.argtypes = [C.c_int64, C.POINTER(SoftmaxConsts)]
        L.oracle_softmax.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_int, C.c_void_p, C.c_int64,
                                     C.POINTER(SoftmaxConsts)]
        L.oracle_softmax_row.restype = None
        L.oracle_softmax_row.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.POINTER(SoftmaxConsts), C.c_void_p]
        L.oracle_gelu_prepare.argtypes = [C.c_double, C.c_int, C.c_double, C.c_int, C.c_int, C.c_int,
                                          C.POINTER(GeluConsts)]
        L.oracle_gelu_prepare_coeffs.argtypes = [C.c_double, C.c_int, C.c_double, C.c_int, C.c_int, C.c_double,
                                                 C.c_double, C.POINTER(GeluConsts)]
        L.oracle_gelu_core.restype = C.c_int64
        L.oracle_gelu_core.argtypes = [C.c_int64, C.POINTER(GeluConsts)]
        L.oracle_gelu_core_scale.restype = C.c_double
        L.oracle_gelu_core_scale.argtypes = [C.c_double, C.POINTER(GeluConsts)]
        L.oracle_gelu.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.POINTER(GeluConsts)]
        L.oracle_layernorm_prepare.argtypes = [C.c_int, C.c_void_p, C.c_void_p, C.c_double, C.c_int, C.c_int,
                                               C.c_int, C.c_void_p, C.c_void_p, C.POINTER(LnConsts)]
        L.oracle_isqrt.restype = C.c_uint64
        L.oracle_isqrt.argtypes = [C.c_uint64, C.c_int]
        L.oracle_layernorm.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_int, C.c_void_p, C.c_void_p,
                                       C.c_void_p, C.POINTER(LnConsts)]
        L.oracle_linear.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32,
                                    C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64, C.c_int, C.c_int]
        L.oracle_linear_bits.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32,
                                         C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64, C.c_int, C.c_int, C.c_int]
        L.oracle_attention_block.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64, C.c_int,
                                             C.c_int, C.c_int, C.c_void_p, C.c_void_p, C.POINTER(SoftmaxConsts),
                                             C.POINTER(Requant)]
        L.oracle_mlp_block.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                       C.POINTER(GeluConsts), C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                       C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64, C.c_int, C.c_int,
                                       C.c_int]
        L.oracle_encoder_block.argtypes = [C.c_void_p, C.c_void_p, C.POINTER(BlockParams)]
        L.oracle_num_threads.restype = C.c_int
    return _lib


class OracleError(RuntimeError):
    pass


def _chk(rc, what):
    if rc != 0:
        raise OracleError("%s failed with oracle status %d" % (what, rc))


def _p(a):
    """Host pointer of a C-contiguous numpy array (None -> NULL)."""
    if a is None:
        return None
    assert isinstance(a, np.ndarray) and a.flags["C_CONTIGUOUS"], "oracle wants C-contiguous numpy arrays"
    return a.ctypes.data


def _ref(s):
    return None if s is None else C.addressof(s)


# ---------------------------------------------------------------- requant
def requant_prepare(ratio, zp=0, qmin=-128, qmax=127) -> Requant:
    rq = Requant()
    _chk(lib().oracle_requant_prepare(float(ratio), zp, qmin, qmax, C.byref(rq)), "requant_prepare")
    return rq


def requant(y: int, rq: Requant) -> int:
    return int(lib().oracle_requant(int(y), C.byref(rq)))


# ---------------------------------------------------------------- softmax
def softmax_prepare(in_scale, row_len, out_bits=8, variant=SM_BITEXP) -> SoftmaxConsts:
    c = SoftmaxConsts()
    _chk(lib().oracle_softmax_prepare(float(in_scale), row_len, out_bits, variant, C.byref(c)), "softmax_prepare")
    return c


def softmax_exp(d: int, c: SoftmaxConsts) -> int:
    return int(lib().oracle_softmax_exp(int(d), C.byref(c)))


def softmax(scores: np.ndarray, c: SoftmaxConsts, bias: np.ndarray | None = None, bias_period: int = 1) -> np.ndarray:
    assert scores.dtype == np.int32 and scores.ndim == 2
    rows, n = scores.shape
    out = np.empty((rows, n), dtype=np.uint8)
    if bias is not None:
        assert bias.dtype == np.int32 and bias.shape == (bias_period, n)
    _chk(lib().oracle_softmax(_p(scores), _p(out), rows, n, _p(bias), bias_period, C.byref(c)), "softmax")
    return out


def softmax_row(s: np.ndarray, c: SoftmaxConsts, mask: np.ndarray | None = None) -> np.ndarray:
    s = np.ascontiguousarray(s, dtype=np.int64)
    out = np.empty(s.shape[0], dtype=np.uint8)
    if mask is not None:
        mask = np.ascontiguousarray(mask, dtype=np.uint8)
    lib().oracle_softmax_row(_p(s), _p(mask), s.shape[0], C.byref(c), _p(out))
    return out


# ---------------------------------------------------------------- GELU
def gelu_prepare(in_scale, in_bits, out_scale, out_zp=0, out_bits=8, variant=GELU_POLY4) -> GeluConsts:
    c = GeluConsts()
    _chk(lib().oracle_gelu_prepare(float(in_scale), in_bits, float(out_scale), out_zp, out_bits, variant,
                                   C.byref(c)), "gelu_prepare")
    return c


def gelu_prepare_coeffs(in_scale, in_bits, out_scale, out_zp, out_bits, a, b) -> GeluConsts:
    """Quartic GELU with refitted erf coefficients (a, b) (Sec. 3.3, Eq. (4))."""
    c = GeluConsts()
    _chk(lib().oracle_gelu_prepare_coeffs(float(in_scale), in_bits, float(out_scale), out_zp, out_bits, float(a),
                                          float(b), C.byref(c)), "gelu_prepare_coeffs")
    return c


def gelu_core(x: int, c: GeluConsts) -> int:
    return int(lib().oracle_gelu_core(int(x), C.byref(c)))


def gelu_core_scale(in_scale, c: GeluConsts) -> float:
    return float(lib().oracle_gelu_core_scale(float(in_scale), C.byref(c)))


def gelu(x: np.ndarray, c: GeluConsts) -> np.ndarray:
    assert x.dtype == np.int32
    out = np.empty(x.shape, dtype=np.int8)
    _chk(lib().oracle_gelu(_p(np.ascontiguousarray(x)), _p(out), x.size, C.byref(c)), "gelu")
    return out


# ---------------------------------------------------------------- LayerNorm
def layernorm_prepare(gamma: np.ndarray, beta: np.ndarray, out_scale, out_zp=0, out_bits=8, variant=LN_SHIFT):
    g = np.ascontiguousarray(gamma, dtype=np.float32)
    b = np.ascontiguousarray(beta, dtype=np.float32)
    dim = g.shape[0]
    gq = np.empty(dim, dtype=np.int32)
    bq = np.empty(dim, dtype=np.int32)
    c = LnConsts()
    _chk(lib().oracle_layernorm_prepare(dim, _p(g), _p(b), float(out_scale), out_zp, out_bits, variant,
                                        _p(gq), _p(bq), C.byref(c)), "layernorm_prepare")
    return gq, bq, c


def isqrt(V: int, variant: int) -> int:
    return int(lib().oracle_isqrt(int(V), variant))


def layernorm(x: np.ndarray, gq: np.ndarray, bq: np.ndarray, c: LnConsts, ptf_shift: np.ndarray | None = None):
    assert x.dtype == np.int8 and x.ndim == 2
    rows, dim = x.shape
    out = np.empty((rows, dim), dtype=np.int8)
    _chk(lib().oracle_layernorm(_p(x), _p(out), rows, dim, _p(gq), _p(bq), _p(ptf_shift), C.byref(c)), "layernorm")
    return out


# ---------------------------------------------------------------- GEMM carriers and blocks
def linear(x, w, bias, mult, shift, out_zp=0, residual=None, residual_rq=None, w_bits=8, out_bits=8):
    M, K = x.shape
    N = w.shape[0]
    y = np.empty((M, N), dtype=np.int8)
    _chk(lib().oracle_linear_bits(_p(x), _p(w), w_bits, _p(bias), _p(mult), _p(shift), out_zp, _p(residual),
                                  _ref(residual_rq), _p(y), M, N, K, out_bits), "linear")
    return y


def attention_block(q, k, v, sc: SoftmaxConsts, out_rq: Requant, bias=None, mask_id=None):
    B, H, N, dh = q.shape
    out = np.empty((B, N, H * dh), dtype=np.int8)
    _chk(lib().oracle_attention_block(_p(q), _p(k), _p(v), _p(out), B, H, N, dh, _p(bias), _p(mask_id),
                                      C.byref(sc), C.byref(out_rq)), "attention_block")
    return out


def mlp_block(x, w1, b1, m1, s1, gc: GeluConsts, w2=None, b2=None, m2=None, s2=None, out_zp=0,
              residual=None, residual_rq=None, w_bits=8):
    M, D = x.shape
    Dh = w1.shape[0]
    y = np.empty((M, D if w2 is not None else Dh), dtype=np.int8)
    _chk(lib().oracle_mlp_block(_p(x), _p(w1), _p(b1), _p(m1), _p(s1), C.byref(gc), _p(w2), _p(b2), _p(m2), _p(s2),
                                out_zp, _p(residual), _ref(residual_rq), _p(y), M, D, Dh, w_bits), "mlp_block")
    return y


def encoder_block(x: np.ndarray, blk: dict) -> np.ndarray:
    """Run one integer encoder block.  ``blk`` maps the field names of
    ``oracle_block_params_t`` to numpy arrays / consts structs / ints."""
    p = BlockParams()
    keep = []
    for name, ctype in BlockParams._fields_:
        v = blk.get(name)
        if ctype is C.c_void_p:
            if v is None:
                setattr(p, name, None)
            elif isinstance(v, np.ndarray):
                keep.append(v)
                setattr(p, name, _p(v))
            else:
                keep.append(v)
                setattr(p, name, C.addressof(v))
        else:
            setattr(p, name, int(v if v is not None else 0))
    T = p.B * p.N
    assert x.dtype == np.int8 and x.shape == (T, p.D)
    y = np.empty((T, p.D), dtype=np.int8)
    _chk(lib().oracle_encoder_block(_p(x), _p(y), C.byref(p)), "encoder_block")
    return y


def num_threads() -> int:
    return int(lib().oracle_num_threads())
