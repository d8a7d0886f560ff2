"""The allocation-free decode entry point (collected last on purpose: if it fails, a run that stops
at the first failure has already run every other test).

kvbfp_decode_attn_static serves callers that cannot call cudaMalloc -- a serving loop with a frozen
memory pool, a plug-in that receives tensors but no allocator.  Its workspace is a fixed array inside
the library, shared by all calls and never cleared, so the test makes two different calls in a row
and checks each against the ordinary entry point, which gets a fresh workspace every time.
"""
import numpy as np
import pytest
import torch

from paper_2403_20137_b200 import binding as B
from paper_2403_20137_b200 import workloads as W

pytestmark = pytest.mark.gpu
ATTN_TOL = 2e-3


def rel_err(got, ref):
    num = (got - ref).abs().amax(dim=-1)
    den = ref.abs().amax(dim=-1).clamp_min(1e-30)
    return float((num / den).max())


def test_static_scratch_matches_regular_entry_point_twice():
    w = W.CONFIGS[4]                       # grouped queries: 32 query heads on 8 KV heads
    Bn, S = 2, 900
    k, v = W.make_kv(w, n_tokens=S, batch=Bn)
    cache = B.Cache(Bn, w.n_kv_heads, 128, 912, w.block, w.mant_bits, fill=0x5A)
    kd, vd = k.cuda(), v.cuda()
    _, perm, _ = B.calibrate(kd.reshape(-1, w.n_kv_heads, 128), w.n_kv_heads, 128)
    B.append(cache, kd, vd, torch.zeros(Bn, dtype=torch.int32, device="cuda"), perm_k=perm)
    assert B.decode_workspace_bytes(cache.fmt, w.n_q_heads) <= B.static_scratch_bytes()

    q1 = W.make_q(w, batch=Bn).cuda()
    q2 = (q1.float() * -0.5 + 0.25).to(q1.dtype)                 # a different query for the second call
    # the third call is much shorter than the ones before it: the array still holds their partial results in
    # slots that this call's merge must not read
    cases = [(q1, [S, 301], B.DECODE_AUTO), (q2, [17, S], B.DECODE_SIMT), (q1, [40, 0], B.DECODE_AUTO)]
    out = torch.empty(Bn, w.n_q_heads, 128, dtype=torch.float32, device="cuda")     # caller-owned output
    lens_dev = [torch.tensor(lens, dtype=torch.int32, device="cuda") for _, lens, _ in cases]
    refs = [B.decode_attn(cache, q, sl, perm_k=perm, impl=impl) for (q, _, impl), sl in zip(cases, lens_dev)]
    B.decode_attn_static(cache, q1, lens_dev[0], perm_k=perm, out=out)     # first call on the device: address look-up
    torch.cuda.synchronize()
    free0 = torch.cuda.mem_get_info()[0]
    reserved0, allocated0 = torch.cuda.memory_reserved(), torch.cuda.memory_allocated()
    for (q, lens, impl), sl, ref in zip(cases, lens_dev, refs):
        got = B.decode_attn_static(cache, q, sl, perm_k=perm, impl=impl, out=out)
        torch.cuda.synchronize()
        assert got.data_ptr() == out.data_ptr()
        assert rel_err(got, ref) <= ATTN_TOL
        assert torch.equal(got, ref)       # same kernels, same arithmetic: in fact identical
    # nothing was allocated on the device by those calls, neither by the library nor through torch
    assert torch.cuda.mem_get_info()[0] == free0
    assert (torch.cuda.memory_reserved(), torch.cuda.memory_allocated()) == (reserved0, allocated0)
    assert B.device_status() == 0


def test_static_scratch_refuses_large_geometry():
    big = B.Format(64, 32, 128, 1 << 16, 32, 4)                  # needs far more than the fixed array
    assert B.decode_workspace_bytes(big, 32) > B.static_scratch_bytes()
    cs = B.CacheStruct(big, 0x1000, 0x2000, 0x3000, 0x4000)      # never dereferenced: refused on the host
    import ctypes as C
    before = B.launch_count()
    rc = B.lib().kvbfp_decode_attn_static(C.byref(cs), C.c_void_p(16), 0, 32, C.c_void_p(16), 0, None, None, 0.0, 0,
                                          C.c_void_p(16), 0, None)
    assert rc == B.ERR_WORKSPACE and B.launch_count() == before
