"""Thin ctypes binding of ``libkvbfp.so``: argument marshalling only.

Every function takes ``torch`` CUDA tensors (used here for device memory and
streams, nothing else), passes their data pointers through the C ABI declared
in ``include/kvbfp.h`` and returns/raises on the status code.  There is no CPU
fallback: if the CUDA library cannot be loaded the first call raises.
"""
import ctypes as C
import os

import torch

from . import build as _build

OK = 0
ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_ALIGNMENT, ERR_CAPACITY, ERR_WORKSPACE, ERR_CUDA = 1, 2, 3, 4, 5, 6
F32, BF16 = 0, 1
STAT_MAXABS, STAT_L2 = 0, 1
FLAG_NONFINITE, FLAG_POSITION, FLAG_LEN_HINT, FLAG_WAIT_TIMEOUT = 1, 2, 4, 8
DECODE_AUTO, DECODE_SIMT, DECODE_MMA, DECODE_MMA_BF16 = 0, 1, 2, 3

EXPORTS = ["kvbfp_version", "kvbfp_status_string", "kvbfp_last_cuda_error", "kvbfp_plane_bytes",
           "kvbfp_calibrate", "kvbfp_fold_perm", "kvbfp_append", "kvbfp_dequant",
           "kvbfp_decode_workspace_bytes", "kvbfp_decode_attn", "kvbfp_device_status",
           "kvbfp_launch_count", "kvbfp_step_staging_bytes", "kvbfp_decode_step_host",
           "kvbfp_profile_decode_events", "kvbfp_static_scratch_bytes", "kvbfp_decode_attn_static",
           "kvbfp_rope_tables", "kvbfp_rope_apply", "kvbfp_decode_attn_rope", "kvbfp_split_plan",
           "kvbfp_split_range_start", "kvbfp_split_range_of", "kvbfp_split_partial_slot",
           "kvbfp_selftest_wait_timeout"]


class KvbfpError(RuntimeError):
    def __init__(self, status, text):
        super().__init__(f"kvbfp status {status}: {text}")
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


class CacheStruct(C.Structure):
    _fields_ = [("fmt", Format), ("k_mant", C.c_void_p), ("k_exp", C.c_void_p),
                ("v_mant", C.c_void_p), ("v_exp", C.c_void_p)]


_lib = None


def lib_path():
    return _build.LIB


def lib():
    """Load the CUDA library, first rebuilding it in-tree unless it was built from the sources as they
    are now (a hash of the sources is kept beside the binary); raises if that is impossible."""
    global _lib
    if _lib is None:
        path = os.environ.get("KVBFP_LIB") or _build.LIB      # KVBFP_LIB: another build of the same library
        if path == _build.LIB:
            path = _build.build()                             # returns at once when the binary is current
        L = C.CDLL(path)
        L.kvbfp_version.restype = C.c_int32
        L.kvbfp_status_string.restype = C.c_char_p
        L.kvbfp_status_string.argtypes = [C.c_int]
        L.kvbfp_last_cuda_error.restype = C.c_char_p
        L.kvbfp_launch_count.restype = C.c_uint64
        L.kvbfp_plane_bytes.argtypes = [C.c_void_p, C.POINTER(C.c_size_t), C.POINTER(C.c_size_t)]
        L.kvbfp_calibrate.argtypes = [C.c_void_p, C.c_int, C.c_int64, C.c_int32, C.c_int32, C.c_int,
                                      C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
        L.kvbfp_fold_perm.argtypes = [C.c_void_p, C.c_int, C.c_int32, C.c_int32, C.c_int64, C.c_void_p,
                                      C.c_void_p, C.c_void_p]
        L.kvbfp_append.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_int32, C.c_void_p,
                                   C.c_void_p, C.c_void_p, C.c_void_p]
        L.kvbfp_dequant.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_int32,
                                    C.c_int32, C.c_void_p, C.c_void_p, C.c_int, C.c_void_p]
        L.kvbfp_decode_workspace_bytes.restype = C.c_size_t
        L.kvbfp_decode_workspace_bytes.argtypes = [C.c_void_p, C.c_int32]
        L.kvbfp_decode_attn.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int32, C.c_void_p, C.c_int32,
                                        C.c_void_p, C.c_void_p, C.c_float, C.c_int32, C.c_void_p,
                                        C.c_void_p, C.c_size_t, C.c_uint32, C.c_void_p]
        L.kvbfp_device_status.argtypes = [C.POINTER(C.c_uint32), C.c_void_p]
        L.kvbfp_step_staging_bytes.restype = C.c_size_t
        L.kvbfp_step_staging_bytes.argtypes = [C.c_void_p, C.c_int32, C.c_int]
        L.kvbfp_decode_step_host.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_int32,
                                             C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p,
                                             C.c_void_p, C.c_float, C.c_void_p, C.c_void_p, C.c_size_t,
                                             C.c_void_p, C.c_size_t, C.c_uint32, C.c_void_p]
        L.kvbfp_profile_decode_events.argtypes = [C.c_void_p, C.c_void_p]
        L.kvbfp_static_scratch_bytes.restype = C.c_size_t
        L.kvbfp_decode_attn_static.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int32, C.c_void_p, C.c_int32,
                                               C.c_void_p, C.c_void_p, C.c_float, C.c_int32, C.c_void_p,
                                               C.c_uint32, C.c_void_p]
        L.kvbfp_decode_attn_rope.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int32, C.c_void_p, C.c_int32,
                                             C.c_void_p, C.c_void_p, C.c_float, C.c_void_p, C.c_void_p, C.c_void_p,
                                             C.c_void_p, C.c_void_p, C.c_size_t, C.c_uint32, C.c_void_p]
        L.kvbfp_rope_tables.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_double, C.c_int32,
                                        C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        L.kvbfp_rope_apply.argtypes = [C.c_void_p, C.c_int, C.c_int64, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p,
                                       C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        L.kvbfp_split_plan.argtypes = [C.c_int32] * 6 + [C.POINTER(C.c_int32)]
        for name in ("kvbfp_split_range_start", "kvbfp_split_range_of"):
            getattr(L, name).argtypes = [C.c_int32] * 3
            getattr(L, name).restype = C.c_int32
        L.kvbfp_selftest_wait_timeout.argtypes = [C.c_uint32, C.c_uint32, C.c_void_p]
        L.kvbfp_split_partial_slot.argtypes = [C.c_int32] * 4
        L.kvbfp_split_partial_slot.restype = C.c_int32
        _lib = L
    return _lib


def _check(rc):
    if rc != OK:
        L = lib()
        text = L.kvbfp_status_string(rc).decode()
        if rc == ERR_CUDA:
            text += " (" + L.kvbfp_last_cuda_error().decode() + ")"
        raise KvbfpError(rc, text)


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream(stream=None):
    s = torch.cuda.current_stream() if stream is None else stream
    return C.c_void_p(s.cuda_stream)


def _dt(t):
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    raise TypeError(f"unsupported dtype {t.dtype}")


def _dev(t, dtype=None):
    if t is None:
        return None
    if not t.is_cuda or not t.is_contiguous():
        raise ValueError("expected a contiguous CUDA tensor")
    if dtype is not None and t.dtype != dtype:
        raise TypeError(f"expected {dtype}, got {t.dtype}")
    return t


def version():
    return lib().kvbfp_version()


def launch_count():
    return int(lib().kvbfp_launch_count())


def plane_bytes(fmt):
    m, e = C.c_size_t(0), C.c_size_t(0)
    _check(lib().kvbfp_plane_bytes(C.byref(fmt), C.byref(m), C.byref(e)))
    return m.value, e.value


class Cache:
    """Four caller-owned planes on the device plus the format (kvbfp_cache)."""

    def __init__(self, batch, n_kv_heads, head_dim, max_seq, block, mant_bits, device="cuda", fill=None):
        self.fmt = Format(batch, n_kv_heads, head_dim, max_seq, block, mant_bits)
        mb, eb = plane_bytes(self.fmt)
        shape_m = (batch, n_kv_heads, max_seq, self.fmt.row_m)
        shape_e = (batch, n_kv_heads, max_seq, self.fmt.row_e)
        assert mb == batch * n_kv_heads * max_seq * self.fmt.row_m and eb == batch * n_kv_heads * max_seq * self.fmt.row_e
        mk = (lambda s: torch.empty(s, dtype=torch.uint8, device=device)) if fill is None else \
             (lambda s: torch.full(s, fill, dtype=torch.uint8, device=device))
        self.k_mant, self.k_exp, self.v_mant, self.v_exp = mk(shape_m), mk(shape_e), mk(shape_m), mk(shape_e)

    def struct(self):
        return CacheStruct(self.fmt, self.k_mant.data_ptr(), self.k_exp.data_ptr(),
                           self.v_mant.data_ptr(), self.v_exp.data_ptr())


def calibrate(x, n_heads, head_dim, stat=STAT_MAXABS, stream=None):
    """kvbfp_calibrate -> (stat f32 [H, d], perm i32 [H, d], inv_perm i32 [H, d])."""
    x = _dev(x)
    n_tokens = x.numel() // (n_heads * head_dim)
    dev = x.device
    st = torch.empty(n_heads, head_dim, dtype=torch.float32, device=dev)
    perm = torch.empty(n_heads, head_dim, dtype=torch.int32, device=dev)
    inv = torch.empty(n_heads, head_dim, dtype=torch.int32, device=dev)
    ws = torch.empty(n_heads * head_dim, dtype=torch.float64, device=dev) if stat == STAT_L2 else None
    _check(lib().kvbfp_calibrate(_ptr(x), _dt(x), n_tokens, n_heads, head_dim, stat, _ptr(st), _ptr(perm),
                                 _ptr(inv), _ptr(ws), 0 if ws is None else ws.numel() * 8, _stream(stream)))
    return st, perm, inv


def fold_perm(w, perm, n_heads, head_dim, stream=None):
    """kvbfp_fold_perm: rows of w [H*d, d_in] gathered per head by perm."""
    w, perm = _dev(w), _dev(perm, torch.int32)
    out = torch.empty_like(w)
    _check(lib().kvbfp_fold_perm(_ptr(w), _dt(w), n_heads, head_dim, w.shape[-1], _ptr(perm), _ptr(out),
                                 _stream(stream)))
    return out


def append(cache, k_new, v_new, start_pos, perm_k=None, perm_v=None, stream=None):
    """kvbfp_append: k_new, v_new [B, n_new, H_kv, d]."""
    k_new, v_new = _dev(k_new), _dev(v_new)
    ref = k_new if k_new is not None else v_new
    f = cache.fmt
    n_new = ref.numel() // (f.batch * f.n_kv_heads * f.head_dim)
    cs = cache.struct()
    _check(lib().kvbfp_append(C.byref(cs), _ptr(k_new), _ptr(v_new), _dt(ref), n_new,
                              _ptr(_dev(start_pos, torch.int32)), _ptr(_dev(perm_k, torch.int32)),
                              _ptr(_dev(perm_v, torch.int32)), _stream(stream)))


def dequant(cache, which, b, h, t0, n_tok, perm=None, out_dtype=torch.float32, stream=None):
    """kvbfp_dequant -> [n_tok, d] of out_dtype."""
    mant, exp8 = (cache.k_mant, cache.k_exp) if which == "k" else (cache.v_mant, cache.v_exp)
    out = torch.empty(n_tok, cache.fmt.head_dim, dtype=out_dtype, device=mant.device)
    _check(lib().kvbfp_dequant(C.byref(cache.fmt), _ptr(mant), _ptr(exp8), b, h, t0, n_tok,
                               _ptr(_dev(perm, torch.int32)), _ptr(out), _dt(out), _stream(stream)))
    return out


def dequant_all(cache, which, n_tok, perm=None, t0=0, out_dtype=torch.float32, stream=None):
    """kvbfp_dequant with b = h = -1: every sequence and head in one launch -> [B, n_tok, H_kv, d] of out_dtype
    (the layout append() takes)."""
    mant, exp8 = (cache.k_mant, cache.k_exp) if which == "k" else (cache.v_mant, cache.v_exp)
    f = cache.fmt
    out = torch.empty(f.batch, n_tok, f.n_kv_heads, f.head_dim, dtype=out_dtype, device=mant.device)
    _check(lib().kvbfp_dequant(C.byref(f), _ptr(mant), _ptr(exp8), -1, -1, t0, n_tok,
                               _ptr(_dev(perm, torch.int32)), _ptr(out), _dt(out), _stream(stream)))
    return out


def decode_workspace_bytes(fmt, n_q_heads):
    return int(lib().kvbfp_decode_workspace_bytes(C.byref(fmt), n_q_heads))


def decode_attn(cache, q, seq_lens, perm_k=None, inv_perm_v=None, softmax_scale=0.0, max_len_hint=0,
                q_mant_bits=0, impl=DECODE_AUTO, chunk_tokens=0, out=None, workspace=None, stream=None):
    """kvbfp_decode_attn: q [B, H_q, d] -> out f32 [B, H_q, d]."""
    q = _dev(q)
    n_q_heads = q.shape[1]
    if out is None:
        out = torch.empty(q.shape, dtype=torch.float32, device=q.device)
    if workspace is None:
        workspace = torch.empty(decode_workspace_bytes(cache.fmt, n_q_heads), dtype=torch.uint8, device=q.device)
    flags = impl | ((chunk_tokens // 128) << 8)
    cs = cache.struct()
    _check(lib().kvbfp_decode_attn(C.byref(cs), _ptr(q), _dt(q), n_q_heads, _ptr(_dev(seq_lens, torch.int32)),
                                   max_len_hint, _ptr(_dev(perm_k, torch.int32)),
                                   _ptr(_dev(inv_perm_v, torch.int32)), float(softmax_scale), q_mant_bits,
                                   _ptr(_dev(out, torch.float32)), _ptr(workspace), workspace.numel(), flags,
                                   _stream(stream)))
    return out


def decode_attn_rope(cache, q, seq_lens, theta, partner, sign, perm_k=None, inv_perm_v=None, softmax_scale=0.0,
                     max_len_hint=0, impl=DECODE_AUTO, chunk_tokens=0, out=None, workspace=None, stream=None):
    """kvbfp_decode_attn_rope: as decode_attn over keys cached before the rotary embedding; theta (f64), partner
    (i32), sign (f32) are the [H_kv, d] tables of rope_tables()."""
    q = _dev(q)
    n_q_heads = q.shape[1]
    if out is None:
        out = torch.empty(q.shape, dtype=torch.float32, device=q.device)
    if workspace is None:
        workspace = torch.empty(decode_workspace_bytes(cache.fmt, n_q_heads), dtype=torch.uint8, device=q.device)
    flags = impl | ((chunk_tokens // 128) << 8)
    cs = cache.struct()
    _check(lib().kvbfp_decode_attn_rope(C.byref(cs), _ptr(q), _dt(q), n_q_heads, _ptr(_dev(seq_lens, torch.int32)),
                                        max_len_hint, _ptr(_dev(perm_k, torch.int32)),
                                        _ptr(_dev(inv_perm_v, torch.int32)), float(softmax_scale),
                                        _ptr(_dev(theta, torch.float64)), _ptr(_dev(partner, torch.int32)),
                                        _ptr(_dev(sign, torch.float32)), _ptr(_dev(out, torch.float32)),
                                        _ptr(workspace), workspace.numel(), flags, _stream(stream)))
    return out


def device_status(stream=None):
    """kvbfp_device_status: synchronises the stream, returns and clears the status flags."""
    flags = C.c_uint32(0)
    _check(lib().kvbfp_device_status(C.byref(flags), _stream(stream)))
    return flags.value


def step_staging_bytes(fmt, n_q_heads, dtype):
    return int(lib().kvbfp_step_staging_bytes(C.byref(fmt), n_q_heads, BF16 if dtype == torch.bfloat16 else F32))


class HostStep:
    """kvbfp_decode_step_host with its arguments marshalled once, for a decode loop that keeps its buffers: host
    tensors k_new, v_new [B,1,H_kv,d], q [B,H_q,d] and the f32 output are refilled / read in place between calls,
    start_pos and seq_lens are device tensors updated in place.  Calling the object runs one step and returns the
    output tensor after the stream has been synchronised."""

    def __init__(self, cache, k_new_host, v_new_host, q_host, start_pos, seq_lens, out_host, staging, workspace,
                 perm_k=None, perm_v=None, inv_perm_v=None, softmax_scale=0.0, max_len_hint=0, impl=DECODE_AUTO,
                 stream=None):
        for t in (k_new_host, v_new_host, q_host, out_host):
            if t.is_cuda or not t.is_contiguous():
                raise ValueError("expected contiguous host tensors")
        self.out_host = out_host
        self._cs = cache.struct()
        self._keep = (cache, k_new_host, v_new_host, q_host, start_pos, seq_lens, out_host, staging, workspace, perm_k,
                      perm_v, inv_perm_v, stream)
        self._fn = lib().kvbfp_decode_step_host
        self._args = (C.byref(self._cs), _ptr(k_new_host), _ptr(v_new_host), _ptr(q_host), _dt(q_host), q_host.shape[1],
                      _ptr(_dev(start_pos, torch.int32)), _ptr(_dev(seq_lens, torch.int32)), max_len_hint,
                      _ptr(_dev(perm_k, torch.int32)), _ptr(_dev(perm_v, torch.int32)),
                      _ptr(_dev(inv_perm_v, torch.int32)), float(softmax_scale), _ptr(out_host), _ptr(staging),
                      staging.numel(), _ptr(workspace), workspace.numel(), impl, _stream(stream))

    def __call__(self):
        rc = self._fn(*self._args)
        if rc != OK:
            _check(rc)
        return self.out_host


def decode_step_host(cache, k_new_host, v_new_host, q_host, start_pos, seq_lens, out_host, staging, workspace,
                     perm_k=None, perm_v=None, inv_perm_v=None, softmax_scale=0.0, max_len_hint=0,
                     impl=DECODE_AUTO, stream=None):
    """kvbfp_decode_step_host: host tensors in (k_new, v_new [B,1,H_kv,d]; q [B,H_q,d]), host f32 out;
    returns after the stream has been synchronised.  (One call; a loop over fixed buffers keeps a HostStep.)"""
    return HostStep(cache, k_new_host, v_new_host, q_host, start_pos, seq_lens, out_host, staging, workspace,
                    perm_k=perm_k, perm_v=perm_v, inv_perm_v=inv_perm_v, softmax_scale=softmax_scale,
                    max_len_hint=max_len_hint, impl=impl, stream=stream)()


def profile_decode_events(start=None, stop=None):
    """kvbfp_profile_decode_events with torch.cuda.Event objects (already recorded once or created with
    enable_timing=True); (None, None) switches the hook off."""
    a = None if start is None else C.c_void_p(start.cuda_event)
    b = None if stop is None else C.c_void_p(stop.cuda_event)
    _check(lib().kvbfp_profile_decode_events(a, b))


def selftest_wait_timeout(tries=8, hint_ns=1000, stream=None):
    """kvbfp_selftest_wait_timeout: a bounded barrier wait that must run out; raises FLAG_WAIT_TIMEOUT."""
    _check(lib().kvbfp_selftest_wait_timeout(tries, hint_ns, _stream(stream)))


def static_scratch_bytes():
    return int(lib().kvbfp_static_scratch_bytes())


def decode_attn_static(cache, q, seq_lens, perm_k=None, inv_perm_v=None, softmax_scale=0.0, max_len_hint=0,
                       q_mant_bits=0, impl=DECODE_AUTO, chunk_tokens=0, out=None, stream=None):
    """kvbfp_decode_attn_static: the same decode step for callers that cannot allocate device memory
    (frozen memory pools, plug-ins without an allocator).  Its workspace is a fixed 32 MiB array inside
    the library; larger geometries are refused.  Calls that overlap on the GPU race on that array.
    ``out`` should be passed in by such callers; it is allocated here only as a convenience."""
    q = _dev(q)
    if out is None:
        out = torch.empty(q.shape, dtype=torch.float32, device=q.device)
    flags = impl | ((chunk_tokens // 128) << 8)
    cs = cache.struct()
    _check(lib().kvbfp_decode_attn_static(C.byref(cs), _ptr(q), _dt(q), q.shape[1],
                                          _ptr(_dev(seq_lens, torch.int32)), max_len_hint,
                                          _ptr(_dev(perm_k, torch.int32)), _ptr(_dev(inv_perm_v, torch.int32)),
                                          float(softmax_scale), q_mant_bits, _ptr(_dev(out, torch.float32)), flags,
                                          _stream(stream)))
    return out


def rope_tables(perm, inv_perm, n_heads, head_dim, base=10000.0, half_split=False, device="cuda", stream=None):
    """kvbfp_rope_tables -> (theta f64 [H, d], partner i32 [H, d], sign f32 [H, d]) in slot order."""
    theta = torch.empty(n_heads, head_dim, dtype=torch.float64, device=device)
    partner = torch.empty(n_heads, head_dim, dtype=torch.int32, device=device)
    sign = torch.empty(n_heads, head_dim, dtype=torch.float32, device=device)
    _check(lib().kvbfp_rope_tables(_ptr(_dev(perm, torch.int32)), _ptr(_dev(inv_perm, torch.int32)), n_heads, head_dim,
                                   float(base), int(half_split), _ptr(theta), _ptr(partner), _ptr(sign), _stream(stream)))
    return theta, partner, sign


def rope_apply(x, positions, theta, partner, sign, stream=None):
    """kvbfp_rope_apply: x [rows, H, d] in slot order, positions i32 [rows] -> rotated rows of the same dtype."""
    x = _dev(x)
    y = torch.empty_like(x)
    n_heads, head_dim = x.shape[-2], x.shape[-1]
    n_rows = x.numel() // (n_heads * head_dim)
    _check(lib().kvbfp_rope_apply(_ptr(x), _dt(x), n_rows, n_heads, head_dim, _ptr(_dev(positions, torch.int32)),
                                  _ptr(_dev(theta, torch.float64)), _ptr(_dev(partner, torch.int32)),
                                  _ptr(_dev(sign, torch.float32)), _ptr(y), _stream(stream)))
    return y
