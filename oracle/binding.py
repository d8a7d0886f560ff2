"""ctypes front end of the C oracle (numpy in, numpy out).

TEST INFRASTRUCTURE ONLY.  bf16 tensors are passed as ``uint16`` bit patterns
with ``dtype="bf16"``.
"""
import ctypes as C

import numpy as np

from . import build as _build

OK, INVALID, CAPACITY, NONFINITE = 0, 1, 4, 7
STAT_MAXABS, STAT_L2 = 0, 1
_DT = {"f32": 0, "bf16": 1, "f64": 2}


class OracleError(RuntimeError):
    def __init__(self, status):
        super().__init__(f"oracle status {status}")
        self.status = status


class Format(C.Structure):
    _fields_ = [("batch", C.c_int32), ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32),
                ("max_seq", C.c_int32), ("block", C.c_int32), ("mant_bits", C.c_int32)]

    @property
    def row_m(self):
        return self.head_dim * self.mant_bits // 8

    @property
    def row_e(self):
        return self.head_dim // self.block


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(_build.build())
        L.oracle_bfp_value.restype = C.c_double
        L.oracle_bfp_value.argtypes = [C.c_int, C.c_int, C.c_int]
        L.oracle_row_mant_bytes.restype = C.c_size_t
        L.oracle_row_exp_bytes.restype = C.c_size_t
        L.oracle_channel_stat.argtypes = [C.c_void_p, C.c_int, C.c_int64, C.c_int, C.c_int, C.c_int,
                                          C.c_void_p]
        L.oracle_calibrate.argtypes = [C.c_void_p, C.c_int, C.c_int64, C.c_int, C.c_int, C.c_int,
                                       C.c_void_p, C.c_void_p, C.c_void_p]
        L.oracle_fold_perm.restype = None
        L.oracle_fold_perm.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_int64, C.c_void_p, C.c_void_p]
        L.oracle_append.argtypes = [C.c_void_p] * 7 + [C.c_int, C.c_int] + [C.c_void_p] * 3
        L.oracle_dequant.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int,
                                     C.c_int, C.c_void_p, C.c_void_p]
        L.oracle_decode_attn.argtypes = [C.c_void_p] * 6 + [C.c_int, C.c_int] + [C.c_void_p] * 3 + \
            [C.c_double, C.c_int, C.c_void_p]
        L.oracle_decode_attn_rope.argtypes = [C.c_void_p] * 6 + [C.c_int, C.c_int] + [C.c_void_p] * 3 + \
            [C.c_double] + [C.c_void_p] * 4
        L.oracle_rope_tables.restype = None
        L.oracle_rope_tables.argtypes = [C.c_int, C.c_double, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p]
        L.oracle_rope_permute_tables.restype = None
        L.oracle_rope_permute_tables.argtypes = [C.c_int] + [C.c_void_p] * 8
        L.oracle_rope_apply.restype = None
        L.oracle_rope_apply.argtypes = [C.c_int, C.c_double] + [C.c_void_p] * 5
        _lib = L
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _c(a, dtype):
    return np.ascontiguousarray(a, dtype=dtype)


def _check(rc):
    if rc != OK:
        raise OracleError(rc)


def _as_input(x, dtype):
    if dtype == "bf16":
        return _c(x, np.uint16)
    return _c(x, np.float32 if dtype == "f32" else np.float64)


def bfp_value(M, e8, p):
    return lib().oracle_bfp_value(int(M), int(e8), int(p))


def bfp_cast_block(x, p):
    """Cast one block (all of ``x``) -> (e8, mantissas[int32])."""
    x = _c(x, np.float64)
    M = np.zeros(x.size, dtype=np.int32)
    e8 = C.c_int(0)
    _check(lib().oracle_bfp_cast_block(_p(x), C.c_int(x.size), C.c_int(p), C.byref(e8), _p(M)))
    return e8.value, M


def pack_mantissas(M, p):
    M = _c(M, np.int32)
    out = np.zeros((M.size * p + 7) // 8, dtype=np.uint8)
    lib().oracle_pack_mantissas(_p(M), C.c_int(M.size), C.c_int(p), _p(out))
    return out


def unpack_mantissas(b, count, p):
    b = _c(b, np.uint8)
    M = np.zeros(count, dtype=np.int32)
    lib().oracle_unpack_mantissas(_p(b), C.c_int(count), C.c_int(p), _p(M))
    return M


def channel_stat(x, dtype, n_heads, head_dim, stat=STAT_MAXABS):
    x = _as_input(x, dtype)
    T = x.size // (n_heads * head_dim)
    out = np.zeros(n_heads * head_dim, dtype=np.float64)
    _check(lib().oracle_channel_stat(_p(x), _DT[dtype], T, n_heads, head_dim, stat, _p(out)))
    return out.reshape(n_heads, head_dim)


def argsort_stable(stat):
    stat = _c(stat, np.float64)
    perm = np.zeros(stat.size, dtype=np.int32)
    inv = np.zeros(stat.size, dtype=np.int32)
    lib().oracle_argsort_stable(_p(stat), C.c_int(stat.size), _p(perm), _p(inv))
    return perm, inv


def calibrate(x, dtype, n_heads, head_dim, stat=STAT_MAXABS):
    """-> (stat[H,d] f64, perm[H,d] i32, inv_perm[H,d] i32)"""
    x = _as_input(x, dtype)
    T = x.size // (n_heads * head_dim)
    st = np.zeros(n_heads * head_dim, dtype=np.float64)
    perm = np.zeros(n_heads * head_dim, dtype=np.int32)
    inv = np.zeros(n_heads * head_dim, dtype=np.int32)
    _check(lib().oracle_calibrate(_p(x), _DT[dtype], T, n_heads, head_dim, stat, _p(st), _p(perm), _p(inv)))
    shp = (n_heads, head_dim)
    return st.reshape(shp), perm.reshape(shp), inv.reshape(shp)


def fold_perm(w, perm):
    """w[H, d, d_in] -> rows gathered by perm[H, d]."""
    w = _c(w, np.float64)
    H, d, d_in = w.shape
    perm = _c(perm, np.int32)
    out = np.zeros_like(w)
    lib().oracle_fold_perm(_p(w), H, d, d_in, _p(perm), _p(out))
    return out


class Cache:
    """Four caller-owned byte planes, token-major per (batch, kv head)."""

    def __init__(self, batch, n_kv_heads, head_dim, max_seq, block, mant_bits):
        self.fmt = Format(batch, n_kv_heads, head_dim, max_seq, block, mant_bits)
        f = self.fmt
        self.k_mant = np.zeros((batch, n_kv_heads, max_seq, f.row_m), dtype=np.uint8)
        self.k_exp = np.zeros((batch, n_kv_heads, max_seq, f.row_e), dtype=np.uint8)
        self.v_mant = np.zeros_like(self.k_mant)
        self.v_exp = np.zeros_like(self.k_exp)


def append(cache, k_new, v_new, dtype, start_pos, perm_k=None, perm_v=None):
    f = cache.fmt
    k = None if k_new is None else _as_input(k_new, dtype)
    v = None if v_new is None else _as_input(v_new, dtype)
    ref = k if k is not None else v
    n_new = ref.size // (f.batch * f.n_kv_heads * f.head_dim)
    sp = _c(start_pos, np.int32)
    pk = None if perm_k is None else _c(perm_k, np.int32)
    pv = None if perm_v is None else _c(perm_v, np.int32)
    _check(lib().oracle_append(C.byref(f), _p(cache.k_mant), _p(cache.k_exp), _p(cache.v_mant),
                               _p(cache.v_exp), _p(k), _p(v), _DT[dtype], n_new, _p(sp), _p(pk), _p(pv)))


def dequant(cache, which, b, h, t0, n_tok, perm=None):
    f = cache.fmt
    mant, exp8 = (cache.k_mant, cache.k_exp) if which == "k" else (cache.v_mant, cache.v_exp)
    out = np.zeros((n_tok, f.head_dim), dtype=np.float64)
    pp = None if perm is None else _c(perm, np.int32)
    _check(lib().oracle_dequant(C.byref(f), _p(mant), _p(exp8), b, h, t0, n_tok, _p(pp), _p(out)))
    return out


def decode_attn(cache, q, q_dtype, n_q_heads, seq_lens, perm_k=None, inv_perm_v=None,
                softmax_scale=0.0, q_mant_bits=0):
    f = cache.fmt
    qq = _as_input(q, q_dtype)
    sl = _c(seq_lens, np.int32)
    pk = None if perm_k is None else _c(perm_k, np.int32)
    ipv = None if inv_perm_v is None else _c(inv_perm_v, np.int32)
    out = np.zeros((f.batch, n_q_heads, f.head_dim), dtype=np.float64)
    _check(lib().oracle_decode_attn(C.byref(f), _p(cache.k_mant), _p(cache.k_exp), _p(cache.v_mant),
                                    _p(cache.v_exp), _p(qq), _DT[q_dtype], n_q_heads, _p(sl), _p(pk),
                                    _p(ipv), float(softmax_scale), int(q_mant_bits), _p(out)))
    return out


def decode_attn_rope(cache, q, q_dtype, n_q_heads, seq_lens, theta, partner, sign, perm_k=None, inv_perm_v=None,
                     softmax_scale=0.0):
    """Attention over a cache of pre-rotation keys; theta/partner/sign: [n_kv_heads * head_dim] in stored order."""
    f = cache.fmt
    qq = _as_input(q, q_dtype)
    sl = _c(seq_lens, np.int32)
    pk = None if perm_k is None else _c(perm_k, np.int32)
    ipv = None if inv_perm_v is None else _c(inv_perm_v, np.int32)
    th, pa, sg = _c(theta, np.float64), _c(partner, np.int32), _c(sign, np.float64)
    assert th.size == pa.size == sg.size == f.n_kv_heads * f.head_dim
    out = np.zeros((f.batch, n_q_heads, f.head_dim), dtype=np.float64)
    _check(lib().oracle_decode_attn_rope(C.byref(f), _p(cache.k_mant), _p(cache.k_exp), _p(cache.v_mant),
                                         _p(cache.v_exp), _p(qq), _DT[q_dtype], n_q_heads, _p(sl), _p(pk),
                                         _p(ipv), float(softmax_scale), _p(th), _p(pa), _p(sg), _p(out)))
    return out


def rope_tables(d, base=10000.0, half_split=False):
    theta = np.zeros(d, dtype=np.float64)
    partner = np.zeros(d, dtype=np.int32)
    sign = np.zeros(d, dtype=np.float64)
    lib().oracle_rope_tables(d, float(base), int(half_split), _p(theta), _p(partner), _p(sign))
    return theta, partner, sign


def rope_permute_tables(perm, inv_perm, theta, partner, sign):
    d = theta.size
    perm, inv_perm = _c(perm, np.int32), _c(inv_perm, np.int32)
    theta, partner, sign = _c(theta, np.float64), _c(partner, np.int32), _c(sign, np.float64)
    tp, pp, sp = np.zeros(d), np.zeros(d, dtype=np.int32), np.zeros(d)
    lib().oracle_rope_permute_tables(d, _p(perm), _p(inv_perm), _p(theta), _p(partner), _p(sign),
                                     _p(tp), _p(pp), _p(sp))
    return tp, pp, sp


def rope_apply(x, m, theta, partner, sign):
    x = _c(x, np.float64)
    theta, partner, sign = _c(theta, np.float64), _c(partner, np.int32), _c(sign, np.float64)
    y = np.zeros_like(x)
    lib().oracle_rope_apply(x.size, float(m), _p(theta), _p(partner), _p(sign), _p(x), _p(y))
    return y
