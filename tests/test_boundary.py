"""CPU-side checks of the C-ABI boundary: the library loads, exports every symbol the header
declares, and rejects bad arguments on the host before anything is enqueued (no GPU needed)."""
import ctypes as C
import os
import re

import pytest

from paper_2403_20137_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "kvbfp.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(kvbfp_[a-z_0-9]+)\s*\(", text)))


def test_header_and_library_agree():
    names = declared_functions()
    assert "kvbfp_calibrate" in names and "kvbfp_append" in names
    assert "kvbfp_dequant" in names and "kvbfp_decode_attn" in names
    L = B.lib()
    for n in names:
        assert hasattr(L, n), f"{n} declared in include/kvbfp.h but not exported"
    assert sorted(B.EXPORTS) == [n for n in names if n in B.EXPORTS]
    assert set(names) <= set(B.EXPORTS) | {"kvbfp_decode_attn_static"}
    assert B.version() >= 100


def test_status_strings():
    L = B.lib()
    texts = [L.kvbfp_status_string(i).decode() for i in range(7)]
    assert texts[0] == "ok" and len(set(texts)) == 7
    assert L.kvbfp_status_string(99).decode() == "unknown status"


@pytest.mark.parametrize("n,p", [(16, 4), (32, 4), (64, 6), (128, 8)])
def test_plane_bytes(n, p):
    f = B.Format(2, 3, 128, 64, n, p)
    m, e = B.plane_bytes(f)
    assert m == 2 * 3 * 64 * 128 * p // 8 and e == 2 * 3 * 64 * 128 // n
    assert 8.0 * (m + e) / (2 * 3 * 64 * 128) == p + 8.0 / n      # bits per element


@pytest.mark.parametrize("bad", [dict(head_dim=64), dict(block=8), dict(block=48), dict(mant_bits=5),
                                 dict(mant_bits=2), dict(max_seq=40), dict(batch=0), dict(n_kv_heads=0)])
def test_format_validation(bad):
    kw = dict(batch=1, n_kv_heads=1, head_dim=128, max_seq=32, block=32, mant_bits=4)
    kw.update(bad)
    f = B.Format(**kw)
    with pytest.raises(B.KvbfpError) as e:
        B.plane_bytes(f)
    assert e.value.status in (B.ERR_INVALID_ARG, B.ERR_UNSUPPORTED)
    assert B.decode_workspace_bytes(f, 1) == 0


def test_host_side_argument_errors():
    """Null, misaligned and inconsistent arguments come back as a status; nothing is launched."""
    L = B.lib()
    before = B.launch_count()
    f = B.Format(1, 2, 128, 32, 32, 4)
    cs = B.CacheStruct(f, 0x1000, 0x2000, 0x3000, 0x4000)
    vp = C.c_void_p
    assert L.kvbfp_append(None, vp(16), vp(16), 0, 1, vp(16), None, None, None) == B.ERR_INVALID_ARG
    assert L.kvbfp_append(C.byref(cs), None, None, 0, 1, vp(16), None, None, None) == B.ERR_INVALID_ARG
    assert L.kvbfp_append(C.byref(cs), vp(16), None, 0, 1, None, None, None, None) == B.ERR_INVALID_ARG
    assert L.kvbfp_append(C.byref(cs), vp(16), None, 7, 1, vp(16), None, None, None) == B.ERR_INVALID_ARG
    assert L.kvbfp_append(C.byref(cs), vp(24), None, 0, 1, vp(16), None, None, None) == B.ERR_ALIGNMENT
    assert L.kvbfp_append(C.byref(cs), vp(16), None, 0, 33, vp(16), None, None, None) == B.ERR_CAPACITY
    assert L.kvbfp_dequant(C.byref(f), vp(16), vp(16), 0, 2, 0, 1, None, vp(16), 0, None) == B.ERR_INVALID_ARG
    assert L.kvbfp_dequant(C.byref(f), vp(16), vp(16), 0, 0, 30, 4, None, vp(16), 0, None) == B.ERR_CAPACITY
    assert L.kvbfp_dequant(C.byref(f), vp(16), vp(20), 0, 0, 0, 4, None, vp(16), 0, None) == B.ERR_ALIGNMENT
    assert L.kvbfp_calibrate(vp(16), 0, 4, 1, 64, 0, vp(16), vp(16), None, None, 0, None) == B.ERR_UNSUPPORTED
    assert L.kvbfp_calibrate(vp(16), 0, 4, 1, 128, 1, vp(16), vp(16), None, None, 0, None) == B.ERR_WORKSPACE
    assert L.kvbfp_calibrate(vp(16), 0, 4, 1, 128, 0, None, vp(16), None, None, 0, None) == B.ERR_INVALID_ARG
    assert L.kvbfp_fold_perm(vp(16), 0, 1, 128, 8, vp(16), vp(16), None) == B.ERR_INVALID_ARG   # out == w
    need = B.decode_workspace_bytes(f, 4)
    assert need > 0
    args = lambda **k: [C.byref(cs), vp(16), k.get("dt", 0), k.get("hq", 4), vp(16), k.get("hint", 0), None, None,
                        k.get("scale", 0.0), k.get("qb", 0), vp(16), vp(k.get("ws", 16)), k.get("wsb", need),
                        k.get("flags", 0), None]
    assert L.kvbfp_decode_attn(*args(hq=3)) == B.ERR_INVALID_ARG          # not a multiple of kv heads
    assert L.kvbfp_decode_attn(*args(hq=32)) == B.ERR_UNSUPPORTED         # group of 16
    assert L.kvbfp_decode_attn(*args(wsb=need - 1)) == B.ERR_WORKSPACE
    assert L.kvbfp_decode_attn(*args(ws=8)) == B.ERR_ALIGNMENT
    assert L.kvbfp_decode_attn(*args(qb=4)) == B.ERR_UNSUPPORTED
    assert L.kvbfp_decode_attn(*args(flags=4)) == B.ERR_INVALID_ARG
    assert L.kvbfp_decode_attn(*args(scale=-1.0)) == B.ERR_INVALID_ARG
    rope = lambda **k: [C.byref(cs), vp(16), 0, 4, vp(16), 0, None, None, 0.0, k.get("th", vp(16)), vp(16), vp(16), vp(16),
                        vp(16), need, k.get("flags", 0), None]
    assert L.kvbfp_decode_attn_rope(*rope(th=None)) == B.ERR_INVALID_ARG
    assert L.kvbfp_decode_attn_rope(*rope(th=vp(8))) == B.ERR_ALIGNMENT
    assert L.kvbfp_decode_attn_rope(*rope(flags=2)) == B.ERR_UNSUPPORTED    # tensor-core kernels do not rotate
    assert L.kvbfp_rope_tables(vp(16), None, 1, 128, 10000.0, 0, vp(16), vp(16), vp(16), None) == B.ERR_INVALID_ARG
    assert L.kvbfp_rope_tables(None, None, 1, 64, 10000.0, 0, vp(16), vp(16), vp(16), None) == B.ERR_UNSUPPORTED
    assert L.kvbfp_rope_apply(vp(16), 0, 4, 1, 128, vp(16), vp(16), vp(16), vp(16), vp(16), None) == B.ERR_INVALID_ARG   # y == x
    assert L.kvbfp_device_status(None, None) == B.ERR_INVALID_ARG
    assert B.launch_count() == before
