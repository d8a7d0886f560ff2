"""GPU parity: the CUDA library (through its C ABI) against the CPU oracle on the same seeded inputs.

Bit-exact for permutations, exponent planes, mantissa planes, statistics and dequantised values;
attention within 2e-3 of fp64 attention over the oracle's own cache, measured per (batch, query head)
row as max_c |o_gpu - o_ref| / max_c |o_ref|.
"""
import math

import numpy as np
import pytest
import torch

from paper_2403_20137_b200 import binding as B
from paper_2403_20137_b200 import workloads as W

pytestmark = pytest.mark.gpu

ATTN_TOL = 2e-3
P_GRID = [4, 6, 8]
N_GRID = [16, 32, 64, 128]


def dev(x):
    return x.cuda().contiguous()


def host(x):
    return x.detach().cpu().numpy()


def adversarial_rows(dtype, rows=96, seed=0):
    """[1, rows, 2, 128] with the cases that break casts: exact .5 ties, clamp-zone values, zeros,
    subnormals, +-max finite, a huge dynamic range between rows."""
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((1, rows, 2, 128)).astype(np.float32)
    x *= np.exp2(rng.integers(-30, 30, size=(1, rows, 2, 1))).astype(np.float32)
    x[0, 0] = 0.0                                             # all-zero rows
    x[0, 1, :, :] = 0.0
    x[0, 1, 0, 5] = 1.0                                       # a lone power of two
    x[0, 2, 0, :] = np.arange(128) * 0.125 - 8.0              # dense dyadic grid: many exact ties
    x[0, 2, 1, :] = np.arange(128) * 0.5 - 32.0
    x[0, 3, 0, :] = np.float32(1e-40)                         # subnormal block
    x[0, 3, 0, 7] = np.float32(3e-39)
    x[0, 3, 1, :] = np.float32(3.0e38) * rng.choice([-1, 1], 128)   # near the largest finite value
    x[0, 4, 0, :] = 1.0
    x[0, 4, 0, ::16] = 1.96875                                # rounds up into the clamp zone (p=4: 7.875)
    x[0, 4, 1, :] = -1.0
    x[0, 4, 1, 1::16] = -1.9921875
    x[0, 5, 0, :] = np.float32(2.0 ** -126)                   # smallest normal and below
    x[0, 5, 0, 1::2] = np.float32(2.0 ** -127)
    x[0, 5, 1, :] = np.float32(2.0 ** -149)
    x[0, 6, :, :] = rng.integers(-7, 8, size=(2, 128)) * 0.25  # already on a coarse grid
    t = torch.from_numpy(x)
    return t.to(W.torch_dtype(dtype))


def oracle_cache(oracle, k, v, dtype, block, p, max_seq, start=None, perm_k=None, perm_v=None):
    Bn, T, H, d = k.shape
    c = oracle.Cache(Bn, H, d, max_seq, block, p)
    sp = np.zeros(Bn, dtype=np.int32) if start is None else np.asarray(start, dtype=np.int32)
    oracle.append(c, W.to_oracle(k), None if v is None else W.to_oracle(v), dtype, sp, perm_k, perm_v)
    return c


def assert_planes_equal(gc, oc, lens, start=None):
    """Compare the rows that were written; everything else is unspecified."""
    Bn = gc.fmt.batch
    for b in range(Bn):
        s0 = 0 if start is None else int(start[b])
        sl = slice(s0, s0 + int(lens[b]))
        for name in ("k_mant", "k_exp", "v_mant", "v_exp"):
            g = host(getattr(gc, name)[b, :, sl])
            o = getattr(oc, name)[b, :, sl]
            assert np.array_equal(g, o), f"{name} differs for batch {b}"


# ------------------------------------------------------------------------------- append
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("p", P_GRID)
@pytest.mark.parametrize("n", N_GRID)
def test_append_bit_exact_format_grid(oracle, dtype, p, n):
    k = adversarial_rows(dtype, seed=1)
    v = adversarial_rows(dtype, seed=2)
    rng = np.random.default_rng(3)
    perm_k = np.stack([rng.permutation(128) for _ in range(2)]).astype(np.int32)
    perm_v = np.stack([rng.permutation(128) for _ in range(2)]).astype(np.int32)
    T = k.shape[1]
    gc = B.Cache(1, 2, 128, 112, n, p, fill=0xA5)
    start = torch.tensor([16], dtype=torch.int32)
    B.append(gc, dev(k), dev(v), dev(start), dev(torch.from_numpy(perm_k)), dev(torch.from_numpy(perm_v)))
    assert B.device_status() == 0
    oc = oracle_cache(oracle, k, v, dtype, n, p, 112, start=[16], perm_k=perm_k, perm_v=perm_v)
    assert_planes_equal(gc, oc, [T], start=[16])
    # rows outside [16, 16+T) keep their fill
    assert bool((gc.k_mant[0, :, :16] == 0xA5).all()) and bool((gc.k_exp[0, :, 16 + T:] == 0xA5).all())
    # dequant parity (Eq. (1)), original channel order, both output types
    for which, perm in (("k", perm_k), ("v", perm_v)):
        for h in range(2):
            ref = oracle.dequant(oc, which, 0, h, 16, T, perm=perm)
            pd = dev(torch.from_numpy(perm))
            got = host(B.dequant(gc, which, 0, h, 16, T, perm=pd))
            assert np.array_equal(got.astype(np.float64), ref)
            got16 = B.dequant(gc, which, 0, h, 16, T, perm=pd, out_dtype=torch.bfloat16)
            assert np.array_equal(host(got16.float()).astype(np.float64), ref)
    ref = oracle.dequant(oc, "k", 0, 1, 20, 7)
    assert np.array_equal(host(B.dequant(gc, "k", 0, 1, 20, 7)).astype(np.float64), ref)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("p", P_GRID)
@pytest.mark.parametrize("n", N_GRID)
@pytest.mark.parametrize("heads", [3, 8])
def test_append_many_tokens_bit_exact(oracle, dtype, p, n, heads):
    """The cache write on many tokens (many thread blocks, each walking the heads; the token stride of the grid is
    taken by test_append_config5_sampled): the adversarial rows tiled to a few thousand tokens over three sequences,
    two head counts, K permuted, V not, ragged start positions, one sequence that does not fit."""
    base_k, base_v = adversarial_rows(dtype, seed=4), adversarial_rows(dtype, seed=5)      # [1, 96, 2, 128]
    reps = 9
    k = base_k.repeat(3, reps, (heads + 1) // 2, 1)[:, :, :heads].contiguous()               # [3, 864, heads, 128]
    v = base_v.repeat(3, reps, (heads + 1) // 2, 1)[:, :, :heads].contiguous()
    k[1] = k[1].flip(0)                                                                      # sequences differ
    v[2] = v[2].flip(1)
    T = k.shape[1]
    rng = np.random.default_rng(6)
    perm_k = np.stack([rng.permutation(128) for _ in range(heads)]).astype(np.int32)
    S_max = 1024
    start = [0, 160, 512]                                                                    # 512 + 864 > 1024: skipped whole
    gc = B.Cache(3, heads, 128, S_max, n, p, fill=0x5A)
    B.append(gc, dev(k), dev(v), dev(torch.tensor(start, dtype=torch.int32)), dev(torch.from_numpy(perm_k)))
    assert B.device_status() == B.FLAG_POSITION
    assert bool((gc.k_mant[2] == 0x5A).all()) and bool((gc.v_exp[2] == 0x5A).all())
    oc = oracle.Cache(2, heads, 128, S_max, n, p)
    oracle.append(oc, W.to_oracle(k[:2]), W.to_oracle(v[:2]), dtype, np.array(start[:2], np.int32), perm_k)
    for b in range(2):
        sl = slice(start[b], start[b] + T)
        for name in ("k_mant", "k_exp", "v_mant", "v_exp"):
            assert np.array_equal(host(getattr(gc, name)[b, :, sl]), getattr(oc, name)[b, :, sl]), f"{name} differs for batch {b}"
    assert bool((gc.k_mant[1, :, :160] == 0x5A).all()) and bool((gc.v_mant[0, :, T:] == 0x5A).all())


def test_append_identity_and_single_plane(oracle):
    w = W.CONFIGS[2]
    k, v = W.make_kv(w, n_tokens=50)
    gc = B.Cache(1, 32, 128, 64, 32, 4, fill=0)
    B.append(gc, dev(k), None, dev(torch.zeros(1, dtype=torch.int32)))
    oc = oracle_cache(oracle, k, None, "bf16", 32, 4, 64)
    assert np.array_equal(host(gc.k_mant[0, :, :50]), oc.k_mant[0, :, :50])
    assert np.array_equal(host(gc.k_exp[0, :, :50]), oc.k_exp[0, :, :50])
    assert not bool(gc.v_mant.any())          # V untouched (the cache was created filled with zero bytes)
    B.append(gc, None, dev(v), dev(torch.zeros(1, dtype=torch.int32)))
    oc2 = oracle_cache(oracle, v, None, "bf16", 32, 4, 64)
    assert np.array_equal(host(gc.v_mant[0, :, :50]), oc2.k_mant[0, :, :50])


def test_append_ragged_positions_and_flags(oracle):
    """Per-sequence start positions; a sequence that would overflow is skipped whole and flagged."""
    w = W.CONFIGS[3]
    k, v = W.make_kv(w, n_tokens=3, batch=4)
    gc = B.Cache(4, 32, 128, 32, 32, 4, fill=0x11)
    start = [0, 29, 30, 7]
    B.append(gc, dev(k), dev(v), dev(torch.tensor(start, dtype=torch.int32)))
    assert B.device_status() == B.FLAG_POSITION
    assert B.device_status() == 0                    # cleared by the read
    assert bool((gc.k_mant[2] == 0x11).all()) and bool((gc.v_exp[2] == 0x11).all())
    oc = oracle.Cache(4, 32, 128, 32, 32, 4)
    ok = [0, 1, 3]
    for b in ok:     # the oracle refuses an overflowing call, so feed it the sequences that fit
        sub = oracle.Cache(1, 32, 128, 32, 32, 4)
        oracle.append(sub, W.to_oracle(k[b:b + 1]), W.to_oracle(v[b:b + 1]), "bf16", np.array([start[b]], np.int32))
        sl = slice(start[b], start[b] + 3)
        assert np.array_equal(host(gc.k_mant[b, :, sl]), sub.k_mant[0, :, sl])
        assert np.array_equal(host(gc.v_exp[b, :, sl]), sub.v_exp[0, :, sl])
    del oc
    bad = k.clone()
    bad[0, 1, 3, 9] = float("inf")
    B.append(gc, dev(bad), None, dev(torch.zeros(4, dtype=torch.int32)))
    assert B.device_status() & B.FLAG_NONFINITE


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("p", P_GRID)
def test_append_runs_ragged_tiles_and_nonfinite(oracle, dtype, p):
    """Runs of tokens (16 and more per sequence: the kernel that stages rows in shared memory) whose length leaves a
    tile with one row, with three rows and with a full tile less one; two sequences at different positions, both
    sides permuted.  Then an Inf and a NaN in two rows: flagged, every row without them unchanged."""
    rng = np.random.default_rng(21)
    H = 3
    perm_k = np.stack([rng.permutation(128) for _ in range(H)]).astype(np.int32)
    perm_v = np.stack([rng.permutation(128) for _ in range(H)]).astype(np.int32)
    base_k, base_v = adversarial_rows(dtype, seed=22), adversarial_rows(dtype, seed=23)      # [1, 96, 2, 128]
    for T in (16, 17, 19, 47, 96):
        k = base_k.repeat(2, 1, 2, 1)[:, :T, :H].contiguous()
        v = base_v.repeat(2, 1, 2, 1)[:, :T, :H].contiguous()
        k[1] = k[1].flip(0)
        start = [5, 0]
        gc = B.Cache(2, H, 128, 112, 32, p, fill=0xC3)
        B.append(gc, dev(k), dev(v), dev(torch.tensor(start, dtype=torch.int32)), dev(torch.from_numpy(perm_k)),
                 dev(torch.from_numpy(perm_v)))
        assert B.device_status() == 0
        oc = oracle_cache(oracle, k, v, dtype, 32, p, 112, start=start, perm_k=perm_k, perm_v=perm_v)
        assert_planes_equal(gc, oc, [T, T], start=start)
        assert bool((gc.k_mant[0, :, :5] == 0xC3).all()) and bool((gc.v_exp[1, :, T:] == 0xC3).all())
        assert bool((gc.v_mant[0, :, 5 + T:] == 0xC3).all()) and bool((gc.k_exp[0, :, :5] == 0xC3).all())
    bad = k.clone()
    bad[0, 18, 1, 9] = float("inf")
    bad[1, 95, 2, 127] = float("nan")
    gb = B.Cache(2, H, 128, 112, 32, p, fill=0xC3)
    B.append(gb, dev(bad), dev(v), dev(torch.tensor(start, dtype=torch.int32)), dev(torch.from_numpy(perm_k)),
             dev(torch.from_numpy(perm_v)))
    assert B.device_status() == B.FLAG_NONFINITE
    same = torch.ones(2, H, 112, dtype=torch.bool)
    same[0, 1, 5 + 18] = False
    same[1, 2, 95] = False
    assert bool((gb.k_mant.cpu()[same] == gc.k_mant.cpu()[same]).all()) and bool((gb.k_exp.cpu()[same] == gc.k_exp.cpu()[same]).all())
    assert bool((gb.v_mant == gc.v_mant).all())


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("p,n", [(4, 32), (6, 16), (8, 128), (4, 64)])
def test_append_few_tokens_permuted_bit_exact(oracle, dtype, p, n):
    """One, five and fifteen tokens per sequence (the kernel of the decode step's cache write), K and V permuted,
    several sequences at different positions and more heads than one pass of a thread block takes: planes bit for bit."""
    rng = np.random.default_rng(41)
    H, Bn = 5, 3
    perm_k = np.stack([rng.permutation(128) for _ in range(H)]).astype(np.int32)
    perm_v = np.stack([rng.permutation(128) for _ in range(H)]).astype(np.int32)
    base_k, base_v = adversarial_rows(dtype, seed=42), adversarial_rows(dtype, seed=43)      # [1, 96, 2, 128]
    for T in (1, 5, 15):
        k = base_k.reshape(3, 32, 2, 128).repeat(1, 1, 3, 1)[:, 7:7 + T, :H].contiguous()   # [3, T, H, 128]
        v = base_v.reshape(3, 32, 2, 128).repeat(1, 1, 3, 1)[:, 11:11 + T, :H].contiguous()
        start = [0, 9, 33]
        gc = B.Cache(Bn, H, 128, 48, n, p, fill=0x3C)
        B.append(gc, dev(k), dev(v), dev(torch.tensor(start, dtype=torch.int32)), dev(torch.from_numpy(perm_k)),
                 dev(torch.from_numpy(perm_v)))
        assert B.device_status() == 0
        oc = oracle_cache(oracle, k, v, dtype, n, p, 48, start=start, perm_k=perm_k, perm_v=perm_v)
        assert_planes_equal(gc, oc, [T] * Bn, start=start)
        assert bool((gc.k_mant[1, :, :9] == 0x3C).all()) and bool((gc.v_exp[2, :, 33 + T:] == 0x3C).all())


# ------------------------------------------------------------------------------- calibrate
@pytest.mark.parametrize("cfg,T", [(1, 256), (2, 1000), (4, 777)])
def test_calibrate_matches_oracle(oracle, cfg, T):
    w = W.CONFIGS[cfg]
    x = W.make_calibration(w, n_tokens=T)
    st, perm, inv = B.calibrate(dev(x), w.n_kv_heads, 128)
    assert B.device_status() == 0
    st_o, perm_o, inv_o = oracle.calibrate(W.to_oracle(x), w.dtype, w.n_kv_heads, 128)
    assert np.array_equal(host(st).astype(np.float64), st_o)
    assert np.array_equal(host(perm), perm_o) and np.array_equal(host(inv), inv_o)


def test_calibrate_ties_and_edge_cases(oracle):
    """Duplicate statistics decide real outputs (bf16 magnitudes repeat): the order must be stable."""
    rng = np.random.default_rng(4)
    x = rng.integers(-3, 4, size=(40, 3, 128)).astype(np.float32)     # only 4 distinct magnitudes
    xt = torch.from_numpy(x).to(torch.bfloat16)
    st, perm, inv = B.calibrate(dev(xt), 3, 128)
    st_o, perm_o, inv_o = oracle.calibrate(W.to_oracle(xt), "bf16", 3, 128)
    assert np.array_equal(host(perm), perm_o) and np.array_equal(host(inv), inv_o)
    # one token, and zero tokens (all statistics 0 -> identity order)
    st, perm, _ = B.calibrate(dev(xt[:1]), 3, 128)
    _, perm_o, _ = oracle.calibrate(W.to_oracle(xt[:1]), "bf16", 3, 128)
    assert np.array_equal(host(perm), perm_o)
    st, perm, _ = B.calibrate(dev(torch.zeros(1, 3, 128))[:0], 3, 128)
    assert np.array_equal(host(perm), np.tile(np.arange(128, dtype=np.int32), (3, 1)))
    assert not bool(st.any())


def test_calibrate_l2_and_fold(oracle):
    """Algorithm 1 verbatim: Euclidean row norms of W_k (given transposed), argsort, row gather."""
    rng = np.random.default_rng(5)
    H, d, d_in = 4, 128, 320
    wk = rng.standard_normal((H * d, d_in)).astype(np.float32)
    wk[rng.integers(0, H * d, size=20)] *= 15.0
    x = torch.from_numpy(np.ascontiguousarray(wk.T))                  # [d_in, H, d]
    st, perm, inv = B.calibrate(dev(x), H, d, stat=B.STAT_L2)
    st_o, perm_o, inv_o = oracle.calibrate(x.numpy(), "f32", H, d, stat=oracle.STAT_L2)
    assert np.allclose(host(st), st_o, rtol=1e-6, atol=0)
    gp, go = host(perm), perm_o
    for h in range(H):      # identical, or differing only between channels whose norms agree to 1e-12
        for j in np.nonzero(gp[h] != go[h])[0]:
            assert abs(st_o[h, gp[h, j]] - st_o[h, go[h, j]]) <= 1e-12 * st_o[h, go[h, j]]
    folded = B.fold_perm(dev(torch.from_numpy(wk)), perm, H, d)
    ref = oracle.fold_perm(wk.reshape(H, d, d_in).astype(np.float64), gp)
    assert np.array_equal(host(folded).reshape(H, d, d_in).astype(np.float64), ref)
    # Eq. (2): with both weights folded the products agree with the unfolded ones
    wq = rng.standard_normal((H * d, d_in)).astype(np.float32)
    fq = host(B.fold_perm(dev(torch.from_numpy(wq)), perm, H, d)).astype(np.float64)
    fk = host(folded).astype(np.float64)
    a = wq[:d].astype(np.float64).T @ wk[:d].astype(np.float64)
    b = fq[:d].T @ fk[:d]
    assert np.allclose(a, b, rtol=1e-12, atol=1e-12)


@pytest.mark.parametrize("dtype,T,H", [("bf16", 8192, 32), ("f32", 8192, 32), ("bf16", 1 << 20, 8)])
def test_calibrate_long_inputs_match_oracle(oracle, dtype, T, H):
    """Token counts at which every thread of the reduction walks its unrolled main loop several times (a thread
    block covers a few hundred rows per grid stride): config 3's head count in both input types, and config 5's
    2^20 calibration tokens.  Statistic, permutation and inverse are bit-exact."""
    import dataclasses
    w = dataclasses.replace(W.CONFIGS[5 if H == 8 else 3], dtype=dtype)
    x = W.make_calibration(w, n_tokens=T, device="cuda")
    st, perm, inv = B.calibrate(x, H, 128)
    assert B.device_status() == 0
    st_o, perm_o, inv_o = oracle.calibrate(W.to_oracle(x), dtype, H, 128)
    assert np.array_equal(host(st).astype(np.float64), st_o)
    assert np.array_equal(host(perm), perm_o) and np.array_equal(host(inv), inv_o)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_calibrate_l2_long_input(oracle, dtype):
    """Euclidean-norm statistic over 8192 rows (several grid strides of the fp64 sum kernel)."""
    rng = np.random.default_rng(15)
    H, d, rows = 8, 128, 8192
    x = torch.from_numpy(rng.standard_normal((rows, H, d)).astype(np.float32)).to(W.torch_dtype(dtype))
    x[:, 3, 17] *= 9.0
    st, perm, inv = B.calibrate(dev(x), H, d, stat=B.STAT_L2)
    st_o, perm_o, inv_o = oracle.calibrate(W.to_oracle(x), dtype, H, d, stat=oracle.STAT_L2)
    assert np.allclose(host(st), st_o, rtol=1e-6, atol=0)
    gp = host(perm)
    for h in range(H):      # identical, or differing only between channels whose norms agree to 1e-12
        for j in np.nonzero(gp[h] != perm_o[h])[0]:
            assert abs(st_o[h, gp[h, j]] - st_o[h, perm_o[h, j]]) <= 1e-12 * st_o[h, perm_o[h, j]]
    assert np.array_equal(np.argsort(gp, axis=1), host(inv))


@pytest.mark.parametrize("dtype,p,n", [("bf16", 4, 32), ("f32", 8, 16), ("bf16", 6, 64)])
def test_append_config5_sampled(oracle, dtype, p, n):
    """The prefill of config 5: 65536 new tokens x 8 KV heads in one call (more tokens than one pass of the grid
    takes, so thread blocks stride over the tokens), K permuted.  Two sampled heads are compared with the oracle
    bit for bit over all 65536 rows, K and V planes."""
    import dataclasses
    w = dataclasses.replace(W.CONFIGS[5], dtype=dtype)
    T, H, d = w.seq, w.n_kv_heads, 128
    dv = torch.device("cuda")
    k, v = W.make_kv(w, n_tokens=T, device=dv, batch=1)
    _, perm, _ = B.calibrate(k.reshape(-1, H, d), H, d)
    cache = B.Cache(1, H, d, T, n, p, device=dv)
    B.append(cache, k, v, torch.zeros(1, dtype=torch.int32, device=dv), perm_k=perm)
    assert B.device_status() == 0
    perm_h = host(perm)
    for h in (1, H - 1):
        oc = oracle.Cache(1, 1, d, T, n, p)
        oracle.append(oc, W.to_oracle(k[:, :, h:h + 1]), W.to_oracle(v[:, :, h:h + 1]), dtype, np.zeros(1, np.int32),
                      perm_k=perm_h[h:h + 1])
        for name in ("k_mant", "k_exp", "v_mant", "v_exp"):
            assert np.array_equal(host(getattr(cache, name)[0, h]), getattr(oc, name)[0, 0]), f"{name} differs, head {h}"


@pytest.mark.parametrize("p,n", [(4, 32), (6, 16), (8, 64), (6, 128)])
@pytest.mark.parametrize("out_dtype", [torch.float32, torch.bfloat16])
def test_dequant_rectangles_exact(oracle, p, n, out_dtype):
    """Eq. (1) read-back: one (sequence, head), all heads, and all sequences and heads in one launch, with and
    without the permutation, at a token offset and with a ragged last tile -- equal to the oracle's numbers."""
    w = W.CONFIGS[4]
    Bn, H, T = 2, 8, 203
    k, v = W.make_kv(w, n_tokens=T, batch=Bn)
    _, perm, _ = oracle.calibrate(W.to_oracle(k.reshape(-1, H, 128)), w.dtype, H, 128)
    oc = oracle_cache(oracle, k, v, w.dtype, n, p, 208, perm_k=perm)
    gc = B.Cache(Bn, H, 128, 208, n, p)
    pd = dev(torch.from_numpy(perm))
    B.append(gc, dev(k), dev(v), dev(torch.zeros(Bn, dtype=torch.int32)), pd)
    ref = np.stack([np.stack([oracle.dequant(oc, "k", b, h, 0, T, perm=perm) for h in range(H)], axis=1) for b in range(Bn)])
    ref_v = np.stack([np.stack([oracle.dequant(oc, "v", b, h, 0, T) for h in range(H)], axis=1) for b in range(Bn)])
    f = lambda x: host(x.float()).astype(np.float64)
    assert np.array_equal(f(B.dequant_all(gc, "k", T, perm=pd, out_dtype=out_dtype)), ref)
    assert np.array_equal(f(B.dequant_all(gc, "v", T, out_dtype=out_dtype)), ref_v)
    t0, nt = 37, 150                                                      # offset that is no multiple of 16
    assert np.array_equal(f(B.dequant_all(gc, "k", nt, perm=pd, t0=t0, out_dtype=out_dtype)), ref[:, t0:t0 + nt])
    assert np.array_equal(f(B.dequant(gc, "k", 1, 5, t0, nt, perm=pd, out_dtype=out_dtype)), ref[1, t0:t0 + nt, 5])
    assert np.array_equal(f(B.dequant(gc, "v", 0, 7, 0, T, out_dtype=out_dtype)), ref_v[0, :, 7])
    assert B.device_status() == 0


# ------------------------------------------------------------------------------- decode attention
def rel_err(got, ref):
    """Per (batch, head) row: max |diff| / max |ref|."""
    num = np.abs(got - ref).max(axis=-1)
    den = np.abs(ref).max(axis=-1)
    return float((num / np.maximum(den, 1e-30)).max())


def run_decode_case(oracle, w, Bn, S, lens, block, p, impl, use_perm=True, perm_v=False, max_seq=None,
                    chunk_tokens=0, q_mant_bits=0, scale=0.0, hint=0, v_token_log2=None):
    max_seq = max_seq or ((S + 15) // 16) * 16
    k, v = W.make_kv(w, n_tokens=S, batch=Bn)
    if v_token_log2 is not None:          # token t of V times 2^v_token_log2[t] (exact in bf16 and fp32)
        v = (v.float() * torch.exp2(torch.as_tensor(v_token_log2, dtype=torch.float32)).view(1, S, 1, 1)).to(v.dtype)
    q = W.make_q(w, batch=Bn)
    pk = pv = ipv = None
    if use_perm:
        _, pk, _ = oracle.calibrate(W.to_oracle(k.reshape(-1, w.n_kv_heads, 128)), w.dtype, w.n_kv_heads, 128)
    if perm_v:
        _, pv, ipv = oracle.calibrate(W.to_oracle(v.reshape(-1, w.n_kv_heads, 128)), w.dtype, w.n_kv_heads, 128)
    oc = oracle_cache(oracle, k, v, w.dtype, block, p, max_seq, perm_k=pk, perm_v=pv)
    ref = oracle.decode_attn(oc, W.to_oracle(q), w.dtype, w.n_q_heads, lens, perm_k=pk, inv_perm_v=ipv,
                             softmax_scale=scale, q_mant_bits=q_mant_bits)
    t = lambda a: None if a is None else dev(torch.from_numpy(a))
    gc = B.Cache(Bn, w.n_kv_heads, 128, max_seq, block, p, fill=0xFF)    # unwritten rows: worst-case bytes
    B.append(gc, dev(k), dev(v), dev(torch.zeros(Bn, dtype=torch.int32)), t(pk), t(pv))
    out = B.decode_attn(gc, dev(q), dev(torch.tensor(lens, dtype=torch.int32)), perm_k=t(pk), inv_perm_v=t(ipv),
                        softmax_scale=scale, impl=impl, chunk_tokens=chunk_tokens, q_mant_bits=q_mant_bits,
                        max_len_hint=hint)
    assert B.device_status() == 0
    return host(out).astype(np.float64), ref


IMPLS = [B.DECODE_SIMT, B.DECODE_MMA, B.DECODE_MMA_BF16]


@pytest.mark.parametrize("impl", IMPLS)
def test_decode_config1(oracle, impl):
    """Single head, fp32, block 16, 4-bit, four x20 outlier channels, 256 tokens."""
    w = W.CONFIGS[1]
    got, ref = run_decode_case(oracle, w, 1, 256, [256], 16, 4, impl)
    assert rel_err(got, ref) <= ATTN_TOL


@pytest.mark.parametrize("impl", IMPLS)
@pytest.mark.parametrize("p", P_GRID)
@pytest.mark.parametrize("n", N_GRID)
def test_decode_format_grid_ragged(oracle, impl, p, n):
    """Llama-2-shaped heads, ragged lengths spanning several stages, tiles and a ragged tail."""
    w = W.CONFIGS[2]
    lens = [333, 1, 16, 200]
    got, ref = run_decode_case(oracle, w, 4, 333, lens, n, p, impl, max_seq=400)
    assert rel_err(got, ref) <= ATTN_TOL


@pytest.mark.parametrize("impl", IMPLS)
def test_decode_gqa(oracle, impl):
    w = W.CONFIGS[4]
    lens = [700, 129]
    got, ref = run_decode_case(oracle, w, 2, 700, lens, 32, 4, impl, perm_v=True)
    assert rel_err(got, ref) <= ATTN_TOL


@pytest.mark.parametrize("impl", IMPLS)
@pytest.mark.parametrize("p,n", [(4, 32), (6, 32), (8, 64), (4, 16)])
def test_decode_weights_folded_and_vsort(oracle, impl, p, n):
    """One query head per kv head with the key permutation folded into the weights (perm_k = NULL: the paper's own
    inference-time setting) and with V-sort (values stored permuted, the output scattered back), ragged lengths."""
    w = W.CONFIGS[2]
    lens = [401, 64, 1]
    got, ref = run_decode_case(oracle, w, 3, 401, lens, n, p, impl, use_perm=False, perm_v=True)
    assert rel_err(got, ref) <= ATTN_TOL
    got, ref = run_decode_case(oracle, w, 3, 401, lens, n, p, impl, use_perm=False)
    assert rel_err(got, ref) <= ATTN_TOL


@pytest.mark.parametrize("impl", IMPLS)
@pytest.mark.parametrize("p,n", [(4, 32), (8, 32), (8, 128), (6, 64)])
def test_decode_group_of_8_and_2(oracle, impl, p, n):
    import dataclasses
    for hq, hkv in ((16, 2), (4, 2)):
        w = dataclasses.replace(W.CONFIGS[4], n_q_heads=hq, n_kv_heads=hkv)
        got, ref = run_decode_case(oracle, w, 1, 150, [150], n, p, impl)
        assert rel_err(got, ref) <= ATTN_TOL


@pytest.mark.parametrize("impl", IMPLS)
@pytest.mark.parametrize("p", P_GRID)
def test_decode_empty_and_capacity_edges(oracle, impl, p):
    w = W.CONFIGS[2]
    got, ref = run_decode_case(oracle, w, 3, 128, [0, 128, 5], 32, p, impl, max_seq=128)
    assert not got[0].any() and not ref[0].any()          # empty sequence -> zeros
    assert rel_err(got[1:], ref[1:]) <= ATTN_TOL


@pytest.mark.parametrize("p", P_GRID)
@pytest.mark.parametrize("max_seq,lens", [(16, [16]), (16, [3]), (48, [33]), (80, [80])])
def test_decode_tiny_caches(oracle, p, max_seq, lens):
    """Caches smaller than one staged tile (one head, 16 to 80 rows in a plane): the tiled copies of the 4-bit kernel
    read past the plane's end (zeros arrive) and the kernels must not care."""
    w = W.CONFIGS[1]
    got, ref = run_decode_case(oracle, w, 1, lens[0], lens, 32, p, B.DECODE_AUTO, max_seq=max_seq)
    assert rel_err(got, ref) <= ATTN_TOL


@pytest.mark.parametrize("impl", IMPLS)
@pytest.mark.parametrize("p", [4, 6, 8])
def test_decode_split_invariance(oracle, impl, p):
    """The chunk count must not matter: 1, 2, 7 and 52 chunks agree with each other.  The fp32 kernel
    agrees to 1e-5; the tensor-core kernel carries q and the softmax weights as two bf16 terms
    (2^-16 relative each), and a different chunking moves the softmax reference point, so its runs
    may differ from each other by a few 2^-16."""
    w = W.CONFIGS[2]
    S = 6600
    outs = []
    for chunk in (6656, 3328, 1024, 128):
        got, ref = run_decode_case(oracle, w, 1, S, [S], 32, p, impl, chunk_tokens=chunk)
        assert rel_err(got, ref) <= ATTN_TOL
        outs.append(got)
    # The 6-bit single-head kernel feeds the stored V bytes, excess-32 offsets included, to fp16 MMAs whose fp32
    # accumulation truncates; the offsets are several times the signal, so the bias of a run (about 2^-24 per
    # accumulation step of what the accumulator holds) shows more, and it changes with the number of steps per run.
    bound = 1e-5 if impl == B.DECODE_SIMT else (3e-4 if (p == 6 and impl == B.DECODE_MMA) else 1e-4)
    for o in outs[1:]:
        assert rel_err(o, outs[0]) <= bound


@pytest.mark.parametrize("impl", IMPLS)
@pytest.mark.parametrize("p,n", [(4, 16), (4, 32), (4, 128), (8, 32), (8, 64), (6, 32), (6, 128)])
def test_decode_value_exponents_drift(oracle, impl, p, n):
    """V magnitudes that climb and fall along the sequence, and that jump by 2^60 and up to the top of the
    exponent range for a few tokens: the 4-bit and 8-bit kernels raise the reference exponent of their fp16 V weights
    while they walk a run and rescale their sums, so every step of the way has to stay exact.  The softmax is
    made nearly flat (small scale) so that every token carries weight and a wrong step shows in the result."""
    w = W.CONFIGS[2]
    S = 1500
    t = np.arange(S)
    flat = dict(scale=0.004)
    climb = np.where(t < 750, t // 24, (1499 - t) // 24)               # +1 binade per 24 tokens, up to 2^31, and back
    for chunk in (0, 1536):                                             # library's split; one run over all 24 stages
        got, ref = run_decode_case(oracle, w, 1, S, [S], n, p, impl, v_token_log2=climb, chunk_tokens=chunk, **flat)
        assert np.isfinite(got).all() and rel_err(got, ref) <= ATTN_TOL
    jump = np.zeros(S, dtype=np.int64)
    jump[:200] = -20
    jump[700:703] = 60
    got, ref = run_decode_case(oracle, w, 1, S, [S], n, p, impl, v_token_log2=jump, chunk_tokens=1536, **flat)
    assert np.isfinite(got).all() and rel_err(got, ref) <= ATTN_TOL
    # exponent bytes next to the largest one; the bf16 kernel's conversion (136 times the block's power of two
    # as an intermediate) leaves the bf16 range above 2^120, which its header states as its limit
    jump[1301] = 110 if impl == B.DECODE_MMA_BF16 else 122
    got, ref = run_decode_case(oracle, w, 1, S, [S], n, p, impl, v_token_log2=jump, **flat)
    assert np.isfinite(got).all() and rel_err(got, ref) <= ATTN_TOL


@pytest.mark.parametrize("impl", IMPLS)
def test_decode_bfp16_query_and_scale(oracle, impl):
    w = W.CONFIGS[2]
    got, ref = run_decode_case(oracle, w, 1, 300, [300], 32, 4, impl, q_mant_bits=8, scale=0.05)
    assert rel_err(got, ref) <= ATTN_TOL
    got, ref = run_decode_case(oracle, w, 1, 300, [300], 64, 4, impl, q_mant_bits=8)
    assert rel_err(got, ref) <= ATTN_TOL
    got, ref = run_decode_case(oracle, w, 1, 300, [300], 32, 8, impl, q_mant_bits=8, scale=0.05)   # 8-bit cache as well
    assert rel_err(got, ref) <= ATTN_TOL
    got, ref = run_decode_case(oracle, w, 1, 300, [300], 64, 6, impl, q_mant_bits=8, scale=0.05)   # and a 6-bit one
    assert rel_err(got, ref) <= ATTN_TOL


@pytest.mark.parametrize("p", [4, 6, 8])
def test_decode_is_deterministic_and_stream_ordered(oracle, p):
    """Two launches on the same inputs give bit-identical outputs (the work split and the merge order are fixed by
    integer arithmetic, no atomics on the data path), also when the calls are enqueued on a stream of their own
    behind the append that fills the cache."""
    w = W.CONFIGS[2]
    S, Bn = 2500, 3
    k, v = W.make_kv(w, n_tokens=S, batch=Bn)
    q = dev(W.make_q(w, batch=Bn))
    lens = dev(torch.tensor([S, 1200, 77], dtype=torch.int32))
    gc = B.Cache(Bn, w.n_kv_heads, 128, 2512, 32, p)
    side = torch.cuda.Stream()
    kd, vd, z = dev(k), dev(v), dev(torch.zeros(Bn, dtype=torch.int32))
    torch.cuda.synchronize()
    with torch.cuda.stream(side):
        B.append(gc, kd, vd, z, stream=side)
        a = B.decode_attn(gc, q, lens, stream=side)
        b = B.decode_attn(gc, q, lens, stream=side)
    side.synchronize()
    c = B.decode_attn(gc, q, lens)
    torch.cuda.synchronize()
    assert B.device_status() == 0
    assert torch.equal(a, b) and torch.equal(a, c)
    oc = oracle_cache(oracle, k, v, w.dtype, 32, p, 2512)
    ref = oracle.decode_attn(oc, W.to_oracle(W.make_q(w, batch=Bn)), w.dtype, w.n_q_heads, [S, 1200, 77])
    assert rel_err(host(a).astype(np.float64), ref) <= ATTN_TOL


@pytest.mark.parametrize("cfg,pinned", [(2, True), (2, False), (4, True)])
def test_decode_step_host_equals_device_path(oracle, cfg, pinned):
    """The step with host buffers (page-locked: read and written in place by the kernels; pageable: copied through
    the staging buffer) gives bit for bit what append + decode_attn give on device tensors, cache planes included."""
    w = W.CONFIGS[cfg]
    Bn, S = 3, 333
    k, v = W.make_kv(w, n_tokens=S, batch=Bn)
    q = W.make_q(w, batch=Bn)
    _, perm, _ = B.calibrate(dev(k.reshape(-1, w.n_kv_heads, 128)), w.n_kv_heads, 128)
    caches = [B.Cache(Bn, w.n_kv_heads, 128, 336, w.block, w.mant_bits, fill=0) for _ in range(2)]
    z = dev(torch.zeros(Bn, dtype=torch.int32))
    sp = dev(torch.full((Bn,), S - 1, dtype=torch.int32))
    lens = dev(torch.full((Bn,), S, dtype=torch.int32))
    for c in caches:
        B.append(c, dev(k[:, :S - 1]), dev(v[:, :S - 1]), z, perm_k=perm)
    kn, vn = k[:, S - 1:].contiguous(), v[:, S - 1:].contiguous()
    B.append(caches[0], dev(kn), dev(vn), sp, perm_k=perm)
    ref = B.decode_attn(caches[0], dev(q), lens, perm_k=perm)
    pin = (lambda t: t.pin_memory()) if pinned else (lambda t: t)
    hk, hv, hq = pin(kn), pin(vn), pin(q.clone())
    hout = pin(torch.zeros(Bn, w.n_q_heads, 128, dtype=torch.float32))
    staging = torch.empty(B.step_staging_bytes(caches[1].fmt, w.n_q_heads, q.dtype), dtype=torch.uint8, device="cuda")
    ws = torch.empty(B.decode_workspace_bytes(caches[1].fmt, w.n_q_heads), dtype=torch.uint8, device="cuda")
    for _ in range(2):                      # twice: the second call rewrites the same row
        B.decode_step_host(caches[1], hk, hv, hq, sp, lens, hout, staging, ws, perm_k=perm)
        assert torch.equal(hout, ref.cpu())
    for name in ("k_mant", "k_exp", "v_mant", "v_exp"):
        assert torch.equal(getattr(caches[0], name), getattr(caches[1], name)), name
    # the same call with its arguments marshalled once, as a decode loop keeps it: the buffers are refilled in place
    step = B.HostStep(caches[1], hk, hv, hq, sp, lens, hout, staging, ws, perm_k=perm)
    hq.copy_(-q)
    hout.zero_()
    assert step() is hout
    ref2 = B.decode_attn(caches[0], dev(-q), lens, perm_k=perm)
    assert torch.equal(hout, ref2.cpu()) and not torch.equal(ref2, ref)
    assert B.device_status() == 0


@pytest.mark.parametrize("cfg,p", [(3, 4), (4, 4), (4, 8), (3, 6)])
def test_back_to_back_steps_equal_synchronised_steps(oracle, cfg, p):
    """The kernels of a step are launched so that each may be set up while the one before it still runs; each waits
    for its predecessor before it touches memory.  Twelve steps issued back to back (append of a new token, decode,
    every step's output kept) must give bit for bit what the same calls give with the device synchronised after every
    single call, cache planes included; the last output is also checked against the oracle."""
    import dataclasses
    w = dataclasses.replace(W.CONFIGS[cfg], mant_bits=p)
    Bn, S0, steps = 3, 700, 12
    k, v = W.make_kv(w, n_tokens=S0 + steps, batch=Bn)
    q0 = W.make_q(w, batch=Bn)
    qs = [torch.roll(q0, 5 * i, dims=-1) * (1.0 + 0.125 * i) for i in range(steps)]      # a different query every step
    _, perm, _ = B.calibrate(dev(k.reshape(-1, w.n_kv_heads, 128)), w.n_kv_heads, 128)
    z = dev(torch.zeros(Bn, dtype=torch.int32))
    runs = []
    for sync in (False, True):
        c = B.Cache(Bn, w.n_kv_heads, 128, 720, w.block, p, fill=0)
        ws = torch.empty(B.decode_workspace_bytes(c.fmt, w.n_q_heads), dtype=torch.uint8, device="cuda")
        B.append(c, dev(k[:, :S0]), dev(v[:, :S0]), z, perm_k=perm)
        kd, vd, qd = dev(k), dev(v), [dev(q) for q in qs]
        sps = [dev(torch.full((Bn,), S0 + i, dtype=torch.int32)) for i in range(steps)]
        lens = [dev(torch.full((Bn,), S0 + i + 1, dtype=torch.int32)) for i in range(steps)]
        outs = [torch.empty(Bn, w.n_q_heads, 128, dtype=torch.float32, device="cuda") for _ in range(steps)]
        torch.cuda.synchronize()
        for i in range(steps):
            B.append(c, kd[:, S0 + i:S0 + i + 1].contiguous(), vd[:, S0 + i:S0 + i + 1].contiguous(), sps[i], perm_k=perm)
            if sync:
                torch.cuda.synchronize()
            B.decode_attn(c, qd[i], lens[i], perm_k=perm, out=outs[i], workspace=ws)
            if sync:
                torch.cuda.synchronize()
        torch.cuda.synchronize()
        runs.append((c, outs))
    assert B.device_status() == 0
    for a, b in zip(runs[0][1], runs[1][1]):
        assert torch.equal(a, b)
    for name in ("k_mant", "k_exp", "v_mant", "v_exp"):
        assert torch.equal(getattr(runs[0][0], name), getattr(runs[1][0], name)), name
    oc = oracle_cache(oracle, k, v, w.dtype, w.block, p, 720, perm_k=host(perm))
    ref = oracle.decode_attn(oc, W.to_oracle(qs[-1]), w.dtype, w.n_q_heads, [S0 + steps] * Bn, perm_k=host(perm))
    assert rel_err(host(runs[0][1][-1]).astype(np.float64), ref) <= ATTN_TOL


def test_two_streams_interleaved_steps(oracle):
    """Steps of two sequences' worth of work issued alternately on two streams (each stream its own cache, workspace
    and outputs; the launches that overlap with their predecessors do so within their stream only) give what the same
    steps give one stream after the other."""
    w = W.CONFIGS[4]
    Bn, S0, steps = 2, 400, 6
    k, v = W.make_kv(w, n_tokens=S0 + steps, batch=Bn)
    q0 = W.make_q(w, batch=Bn)
    _, perm, _ = B.calibrate(dev(k.reshape(-1, w.n_kv_heads, 128)), w.n_kv_heads, 128)
    z = dev(torch.zeros(Bn, dtype=torch.int32))
    kd, vd = dev(k), dev(v)
    results = []
    for concurrent in (False, True):
        streams = [torch.cuda.Stream(), torch.cuda.Stream()]
        rigs = []
        for sidx in range(2):
            c = B.Cache(Bn, w.n_kv_heads, 128, 416, w.block, w.mant_bits, fill=0)
            B.append(c, kd[:, :S0].contiguous(), vd[:, :S0].contiguous(), z, perm_k=perm)
            rigs.append({"cache": c,
                         "ws": torch.empty(B.decode_workspace_bytes(c.fmt, w.n_q_heads), dtype=torch.uint8, device="cuda"),
                         "q": [dev(torch.roll(q0, 3 * i + 7 * sidx, dims=-1)) for i in range(steps)],
                         "outs": [torch.empty(Bn, w.n_q_heads, 128, dtype=torch.float32, device="cuda") for _ in range(steps)],
                         "kn": [kd[:, S0 + i:S0 + i + 1].contiguous() for i in range(steps)],
                         "vn": [vd[:, S0 + i:S0 + i + 1].contiguous() for i in range(steps)],
                         "sp": [dev(torch.full((Bn,), S0 + i, dtype=torch.int32)) for i in range(steps)],
                         "len": [dev(torch.full((Bn,), S0 + i + 1, dtype=torch.int32)) for i in range(steps)]})
        torch.cuda.synchronize()
        order = [(i, sidx) for i in range(steps) for sidx in range(2)] if concurrent else \
                [(i, sidx) for sidx in range(2) for i in range(steps)]
        for i, sidx in order:
            r, st = rigs[sidx], streams[sidx]
            B.append(r["cache"], r["kn"][i], r["vn"][i], r["sp"][i], perm_k=perm, stream=st)
            B.decode_attn(r["cache"], r["q"][i], r["len"][i], perm_k=perm, out=r["outs"][i], workspace=r["ws"], stream=st)
            if not concurrent:
                st.synchronize()
        torch.cuda.synchronize()
        results.append(rigs)
    assert B.device_status() == 0
    for sidx in range(2):
        for a, b in zip(results[0][sidx]["outs"], results[1][sidx]["outs"]):
            assert torch.equal(a, b)
        for name in ("k_mant", "k_exp", "v_mant", "v_exp"):
            assert torch.equal(getattr(results[0][sidx]["cache"], name), getattr(results[1][sidx]["cache"], name)), name


def test_bounded_wait_runs_out_and_context_survives(oracle):
    """The bounded barrier wait of the staged kernels: a barrier whose bytes never arrive makes the wait give up after
    its tries, the kernel returns with KVBFP_FLAG_WAIT_TIMEOUT (and only that flag: the barrier whose bytes do arrive
    was waited for successfully), and the next decode on the same context is correct."""
    assert B.device_status() == 0
    B.selftest_wait_timeout(tries=8, hint_ns=1000)
    assert B.device_status() == B.FLAG_WAIT_TIMEOUT
    assert B.device_status() == 0                                   # reading clears
    with pytest.raises(B.KvbfpError):
        B.selftest_wait_timeout(tries=0)
    w = W.CONFIGS[1]
    got, ref = run_decode_case(oracle, w, 1, 256, [256], 16, 4, B.DECODE_AUTO)
    assert rel_err(got, ref) <= ATTN_TOL


@pytest.mark.parametrize("impl", IMPLS)
@pytest.mark.parametrize("p", P_GRID)
def test_decode_zero_query_is_the_mean_of_values(oracle, impl, p):
    """A query of zeros scores every token alike: the output is the plain mean of the cached values (the fixed-point
    query coefficients of the integer kernels are all zero then, with exponent zero)."""
    w = W.CONFIGS[2]
    Bn, S = 2, 200
    k, v = W.make_kv(w, n_tokens=S, batch=Bn)
    q = torch.zeros(Bn, w.n_q_heads, 128, dtype=W.torch_dtype(w.dtype))
    oc = oracle_cache(oracle, k, v, w.dtype, 32, p, 208)
    ref = oracle.decode_attn(oc, W.to_oracle(q), w.dtype, w.n_q_heads, [S, 77])
    gc = B.Cache(Bn, w.n_kv_heads, 128, 208, 32, p, fill=0xFF)
    B.append(gc, dev(k), dev(v), dev(torch.zeros(Bn, dtype=torch.int32)))
    out = host(B.decode_attn(gc, dev(q), dev(torch.tensor([S, 77], dtype=torch.int32)), impl=impl)).astype(np.float64)
    assert B.device_status() == 0
    assert rel_err(out, ref) <= ATTN_TOL
    vd = np.stack([oracle.dequant(oc, "v", 1, h, 0, 77) for h in range(w.n_kv_heads)])       # [H, 77, d]
    assert rel_err(out[1], vd.mean(axis=1)) <= ATTN_TOL


def test_decode_len_hint_flag(oracle):
    w = W.CONFIGS[2]
    k, v = W.make_kv(w, n_tokens=256)
    gc = B.Cache(1, 32, 128, 256, 32, 4)
    z = dev(torch.zeros(1, dtype=torch.int32))
    B.append(gc, dev(k), dev(v), z)
    q = dev(W.make_q(w))
    lens = dev(torch.tensor([256], dtype=torch.int32))
    a = B.decode_attn(gc, q, lens, max_len_hint=128)
    assert B.device_status() == B.FLAG_LEN_HINT
    b = B.decode_attn(gc, q, dev(torch.tensor([128], dtype=torch.int32)))
    assert B.device_status() == 0
    assert torch.equal(a, b)                               # tokens past the hint were not read
    # a length beyond the capacity is read as the capacity, a negative one as an empty sequence; both are flagged
    full = B.decode_attn(gc, q, lens)
    over = B.decode_attn(gc, q, dev(torch.tensor([300], dtype=torch.int32)))
    assert B.device_status() & B.FLAG_POSITION
    assert torch.equal(over, full)
    neg = B.decode_attn(gc, q, dev(torch.tensor([-5], dtype=torch.int32)))
    assert B.device_status() & B.FLAG_POSITION
    assert not bool(neg.any())


def test_ksort_improves_gpu_cache_quality(oracle):
    """Direction of effect on the GPU path itself: K-sort lowers key MSE and score error."""
    w = W.CONFIGS[2]
    k, v = W.make_kv(w, n_tokens=512)
    kd = dev(k)
    _, perm, _ = B.calibrate(kd.reshape(-1, 32, 128), 32, 128)
    z = dev(torch.zeros(1, dtype=torch.int32))
    plain, sortd = B.Cache(1, 32, 128, 512, 32, 4), B.Cache(1, 32, 128, 512, 32, 4)
    B.append(plain, kd, None, z)
    B.append(sortd, kd, None, z, perm_k=perm)
    mse_p = mse_s = 0.0
    for h in range(32):
        ref = k[0, :, h].float().cuda()
        mse_p += float(((B.dequant(plain, "k", 0, h, 0, 512) - ref) ** 2).mean())
        mse_s += float(((B.dequant(sortd, "k", 0, h, 0, 512, perm=perm) - ref) ** 2).mean())
    assert mse_s < 0.85 * mse_p


@pytest.mark.parametrize("cfg", [2, 4])
def test_quality_report_direction_and_oracle_check(oracle, cfg):
    """The quality report (all heads, GPU path): K-sort lowers key MSE, score error and the error of the attention
    output against UNQUANTISED attention; V-sort lowers value MSE when V has outlier channels.  One sampled head
    of the report is recomputed by the oracle: its key MSE must agree (the planes are bit-exact) and its attention
    output must be the oracle's within the parity tolerance, with an fp64 unquantised attention as yardstick."""
    from paper_2403_20137_b200 import quality as Q
    w = W.CONFIGS[cfg]
    T = 768
    rep = Q.quality_report(w, "cuda", n_tokens=T, per_head=True, draw_on="cpu")
    u, s = rep["unsorted"], rep["ksort"]
    assert s["key_mse"] < 0.85 * u["key_mse"]
    assert s["score_rms_err"] < u["score_rms_err"]
    assert s["attn_out_rel_err_mean"] < u["attn_out_rel_err_mean"]
    assert abs(s["value_mse"] - u["value_mse"]) <= 1e-6 * u["value_mse"]        # K-sort leaves V alone
    repv = Q.quality_report(w, "cuda", n_tokens=T, outliers_in_v=True, sort_v=True)
    assert repv["ksort_vsort"]["value_mse"] < 0.85 * repv["ksort"]["value_mse"]
    # (the output error is dominated by the score errors of the keys, so V-sort need not lower it: not asserted)
    assert B.device_status() == 0
    # ---- one head by the oracle: same seeded tensors, same calibration tokens
    import dataclasses
    h, G = w.n_kv_heads - 3, w.n_q_heads // w.n_kv_heads
    w1 = dataclasses.replace(w, batch=1)
    k, v = W.make_kv(w1, n_tokens=T)
    q = W.make_q(w1)
    calib = W.make_calibration(w, n_tokens=min(w.calib_tokens, 4096))
    _, perm, _ = oracle.calibrate(W.to_oracle(calib), w.dtype, w.n_kv_heads, 128)
    kh, vh = k[:, :, h:h + 1], v[:, :, h:h + 1]
    qh = q[:, h * G:(h + 1) * G]
    for name, pk in (("unsorted", None), ("ksort", perm[h:h + 1])):
        oc = oracle.Cache(1, 1, 128, T, w.block, w.mant_bits)
        oracle.append(oc, W.to_oracle(kh), W.to_oracle(vh), w.dtype, np.zeros(1, np.int32), perm_k=pk)
        kd = oracle.dequant(oc, "k", 0, 0, 0, T, perm=pk)
        mse = float(((kd - kh[0, :, 0].double().numpy()) ** 2).mean())
        assert abs(mse - rep[name]["key_mse_per_head"][h]) <= 1e-5 * mse
        ref = oracle.decode_attn(oc, W.to_oracle(qh), w.dtype, G, [T], perm_k=pk)
        got = host(rep[name]["attn_out"])[:, h * G:(h + 1) * G].astype(np.float64)
        assert rel_err(got, ref) <= ATTN_TOL
    # the yardstick itself: the report's fp32 unquantised attention against fp64 numpy on the same head
    kf, vf, qf = kh[0, :, 0].double().numpy(), vh[0, :, 0].double().numpy(), qh[0].double().numpy()
    sc = qf @ kf.T / math.sqrt(128.0)
    pr = np.exp(sc - sc.max(axis=1, keepdims=True))
    exact = (pr / pr.sum(axis=1, keepdims=True)) @ vf
    assert rel_err(host(rep["unquantised_out"])[0, h * G:(h + 1) * G].astype(np.float64), exact) <= 1e-4


# ------------------------------------------------------------------------------- permuted RoPE
@pytest.mark.parametrize("half_split", [False, True])
def test_rope_tables_and_apply(oracle, half_split):
    """Algorithm 1 step 5 and Eq. (4) on the GPU against the oracle, including the identity
    rotate-then-permute = permute-then-rotate-with-permuted-tables."""
    rng = np.random.default_rng(12)
    H, d, rows = 3, 128, 7
    perm = np.stack([rng.permutation(d) for _ in range(H)]).astype(np.int32)
    inv = np.argsort(perm, axis=1).astype(np.int32)
    th, pa, sg = B.rope_tables(dev(torch.from_numpy(perm)), dev(torch.from_numpy(inv)), H, d, 10000.0, half_split)
    x = rng.standard_normal((rows, H, d)).astype(np.float32)                 # original channel order
    pos = np.array([0, 1, 2, 77, 4095, 32767, 100000], dtype=np.int32)
    xs = np.stack([x[:, h, perm[h]] for h in range(H)], axis=1)             # slot order
    y = host(B.rope_apply(dev(torch.from_numpy(xs)), dev(torch.from_numpy(pos)), th, pa, sg)).astype(np.float64)
    t0, p0, s0 = oracle.rope_tables(d, 10000.0, half_split)
    for h in range(H):
        tp, pp, sp = oracle.rope_permute_tables(perm[h], inv[h], t0, p0, s0)
        assert np.allclose(host(th[h]), tp, rtol=1e-14, atol=0)
        assert np.array_equal(host(pa[h]), pp) and np.array_equal(host(sg[h]).astype(np.float64), sp)
        for r in range(rows):
            ref_slot = oracle.rope_apply(xs[r, h].astype(np.float64), float(pos[r]), tp, pp, sp)
            assert np.allclose(y[r, h], ref_slot, rtol=0, atol=2e-6)
            ref_orig = oracle.rope_apply(x[r, h].astype(np.float64), float(pos[r]), t0, p0, s0)
            assert np.allclose(y[r, h], ref_orig[perm[h]], rtol=0, atol=2e-6)          # commutes with the permutation
    # runs of consecutive positions far out, with a jump backwards and a repeat in the middle; several row chunks
    pos2 = np.concatenate([np.arange(31990, 31990 + 45), np.arange(7, 7 + 30), [7, 7, 123456], np.arange(99990, 99990 + 19)]).astype(np.int32)
    x2 = rng.standard_normal((len(pos2), H, d)).astype(np.float32)
    y2 = host(B.rope_apply(dev(torch.from_numpy(x2)), dev(torch.from_numpy(pos2)), th, pa, sg)).astype(np.float64)
    for h in range(H):
        tp, pp, sp = oracle.rope_permute_tables(perm[h], inv[h], t0, p0, s0)
        for r in range(len(pos2)):
            assert np.allclose(y2[r, h], oracle.rope_apply(x2[r, h].astype(np.float64), float(pos2[r]), tp, pp, sp), rtol=0, atol=2e-6)
    # identity tables and bf16 rows
    th1, pa1, sg1 = B.rope_tables(None, None, H, d, 10000.0, half_split)
    xb = torch.from_numpy(x).to(torch.bfloat16)
    yb = host(B.rope_apply(dev(xb), dev(torch.from_numpy(pos)), th1, pa1, sg1).float()).astype(np.float64)
    for r in (3, 5):
        ref = oracle.rope_apply(xb[r, 1].float().numpy().astype(np.float64), float(pos[r]), t0, p0, s0)
        assert np.allclose(yb[r, 1], ref, rtol=2 ** -8, atol=1e-3)


def test_rope_apply_runs_tiles_and_unpaired_tables(oracle):
    """kvbfp_rope_apply over several row tiles: a run of positions that counts up (the tabulated turn from the
    tile's first angle), with a ragged last tile, in f32 and bf16; and tables that do NOT pair the slots up
    (partner map that is no involution, unrelated frequencies), which take the slot-by-slot form of Eq. (4)."""
    rng = np.random.default_rng(31)
    H, d, rows = 2, 128, 100
    perm = np.stack([rng.permutation(d) for _ in range(H)]).astype(np.int32)
    inv = np.argsort(perm, axis=1).astype(np.int32)
    th, pa, sg = B.rope_tables(dev(torch.from_numpy(perm)), dev(torch.from_numpy(inv)), H, d, 10000.0, False)
    t0, p0, s0 = oracle.rope_tables(d, 10000.0, False)
    tabs = [oracle.rope_permute_tables(perm[h], inv[h], t0, p0, s0) for h in range(H)]
    x = rng.standard_normal((rows, H, d)).astype(np.float32)
    pos = (50000 + np.arange(rows)).astype(np.int32)
    y = host(B.rope_apply(dev(torch.from_numpy(x)), dev(torch.from_numpy(pos)), th, pa, sg)).astype(np.float64)
    xb = torch.from_numpy(x).to(torch.bfloat16)
    yb = host(B.rope_apply(dev(xb), dev(torch.from_numpy(pos)), th, pa, sg).float()).astype(np.float64)
    for h in range(H):
        for r in range(rows):
            ref = oracle.rope_apply(x[r, h].astype(np.float64), float(pos[r]), *tabs[h])
            assert np.allclose(y[r, h], ref, rtol=0, atol=2e-6)
            refb = oracle.rope_apply(xb[r, h].float().numpy().astype(np.float64), float(pos[r]), *tabs[h])
            assert np.allclose(yb[r, h], refb, rtol=2 ** -8, atol=1e-3)
    # free tables
    th_f = rng.uniform(1e-4, 1.0, size=(H, d))
    pa_f = rng.integers(0, d, size=(H, d)).astype(np.int32)
    sg_f = rng.choice([-1.0, 1.0], size=(H, d)).astype(np.float32)
    pos_f = np.concatenate([np.arange(70), rng.integers(0, 90000, size=30)]).astype(np.int32)
    yf = host(B.rope_apply(dev(torch.from_numpy(x)), dev(torch.from_numpy(pos_f)), dev(torch.from_numpy(th_f)),
                           dev(torch.from_numpy(pa_f)), dev(torch.from_numpy(sg_f)))).astype(np.float64)
    for h in range(H):
        for r in range(rows):
            ref = oracle.rope_apply(x[r, h].astype(np.float64), float(pos_f[r]), th_f[h], pa_f[h], sg_f[h].astype(np.float64))
            assert np.allclose(yf[r, h], ref, rtol=0, atol=3e-6)


# ------------------------------------------------------------------------------- full-size workloads
@pytest.mark.parametrize("half_split", [False, True])
@pytest.mark.parametrize("p,n", [(4, 32), (4, 16), (8, 128), (6, 64)])
def test_decode_over_pre_rotation_keys(oracle, half_split, p, n):
    """Keys cached before the rotary embedding and K-sorted; the kernel rotates token t's key to position t after
    the read-back (Sec. III par. 2) with the tables of Algorithm 1 step 5.  GQA, ragged lengths over several
    chunks, positions up to 2999."""
    import dataclasses
    w = dataclasses.replace(W.CONFIGS[4], n_q_heads=8, n_kv_heads=2)
    Bn, S, d, Hkv, Hq = 2, 3000, 128, 2, 8
    lens = [3000, 517]
    k, v = W.make_kv(w, n_tokens=S, batch=Bn)
    q = W.make_q(w, batch=Bn)
    _, pk, ipk = oracle.calibrate(W.to_oracle(k.reshape(-1, Hkv, d)), w.dtype, Hkv, d)
    theta, partner, sign = oracle.rope_tables(d, 10000.0, half_split)
    tabs = [oracle.rope_permute_tables(pk[h], ipk[h], theta, partner, sign) for h in range(Hkv)]
    th, pa, sg = (np.concatenate([t[i] for t in tabs]) for i in range(3))
    oc = oracle_cache(oracle, k, v, w.dtype, n, p, S + 8, perm_k=pk)
    ref = oracle.decode_attn_rope(oc, W.to_oracle(q), w.dtype, Hq, lens, th, pa.astype(np.int32), sg, perm_k=pk)
    plain = oracle.decode_attn(oc, W.to_oracle(q), w.dtype, Hq, lens, perm_k=pk)
    assert rel_err(plain, ref) > 0.05                       # the rotation matters on this input
    t = lambda a: dev(torch.from_numpy(np.ascontiguousarray(a)))
    gth, gpa, gsg = B.rope_tables(t(pk), t(ipk), Hkv, d, 10000.0, half_split)
    assert np.allclose(host(gth).ravel(), th, rtol=1e-14, atol=0) and np.array_equal(host(gpa).ravel(), pa)
    gc = B.Cache(Bn, Hkv, d, S + 8, n, p, fill=0xFF)
    B.append(gc, dev(k), dev(v), dev(torch.zeros(Bn, dtype=torch.int32)), t(pk))
    out = B.decode_attn_rope(gc, dev(q), dev(torch.tensor(lens, dtype=torch.int32)), gth, gpa, gsg, perm_k=t(pk))
    assert B.device_status() == 0
    assert rel_err(host(out).astype(np.float64), ref) <= ATTN_TOL
    with pytest.raises(B.KvbfpError):                       # only the fp32 kernel rotates
        B.decode_attn_rope(gc, dev(q), dev(torch.tensor(lens, dtype=torch.int32)), gth, gpa, gsg, perm_k=t(pk),
                           impl=B.DECODE_MMA)


def _full_size_case(oracle, cfg, sample_pairs, **over):
    """The benchmark's own launch (full batch, full sequence, library-chosen chunking) with inputs drawn on
    the GPU; the oracle recomputes the permutation from the same calibration tokens and sampled (batch, kv head)
    units one by one from the same raw inputs."""
    import dataclasses
    w = dataclasses.replace(W.CONFIGS[cfg], **over)
    S, Bn, Hkv, Hq, d = w.seq, w.batch, w.n_kv_heads, w.n_q_heads, w.head_dim
    G = Hq // Hkv
    dv = torch.device("cuda")
    calib = W.make_calibration(w, device=dv)
    _, perm, _ = B.calibrate(calib, Hkv, d)
    _, perm_o, _ = oracle.calibrate(W.to_oracle(calib), w.dtype, Hkv, d)
    assert np.array_equal(host(perm), perm_o), "permutation differs from the oracle's"
    del calib
    k, v = W.make_kv(w, n_tokens=S, device=dv)
    q = W.make_q(w, device=dv)
    cache = B.Cache(Bn, Hkv, d, S, w.block, w.mant_bits, device=dv)
    zeros = torch.zeros(Bn, dtype=torch.int32, device=dv)
    B.append(cache, k[:, :S - 1].contiguous(), v[:, :S - 1].contiguous(), zeros, perm_k=perm)
    B.append(cache, k[:, S - 1:].contiguous(), v[:, S - 1:].contiguous(),
             torch.full((Bn,), S - 1, dtype=torch.int32, device=dv), perm_k=perm)
    lens = torch.full((Bn,), S, dtype=torch.int32, device=dv)
    out = B.decode_attn(cache, q, lens, perm_k=perm, max_len_hint=S)
    assert B.device_status() == 0
    perm_h = perm_o
    worst = 0.0
    for (b, h) in sample_pairs:
        kk = W.to_oracle(k[b:b + 1, :, h:h + 1])
        vv = W.to_oracle(v[b:b + 1, :, h:h + 1])
        oc = oracle.Cache(1, 1, d, S, w.block, w.mant_bits)
        oracle.append(oc, kk, vv, w.dtype, np.zeros(1, np.int32), perm_k=perm_h[h:h + 1])
        # packed planes of the sampled unit are bit-exact at full size too
        assert np.array_equal(host(cache.k_mant[b, h]), oc.k_mant[0, 0])
        assert np.array_equal(host(cache.v_exp[b, h]), oc.v_exp[0, 0])
        qq = W.to_oracle(q[b:b + 1, h * G:(h + 1) * G])
        ref = oracle.decode_attn(oc, qq, w.dtype, G, [S], perm_k=perm_h[h:h + 1])
        got = host(out[b:b + 1, h * G:(h + 1) * G]).astype(np.float64)
        worst = max(worst, rel_err(got, ref))
    assert worst <= ATTN_TOL
    return worst


def test_full_size_config3_sampled(oracle):
    """B16, H32, S8192 (the benchmark workload): four sampled (batch, head) units."""
    _full_size_case(oracle, 3, [(0, 0), (5, 17), (15, 31), (9, 3)])


def test_full_size_config4_gqa_sampled(oracle):
    """B8, 32 query heads on 8 KV heads, S32768: two sampled (batch, kv head) units, four query heads each."""
    _full_size_case(oracle, 4, [(0, 0), (7, 5)])


def test_full_size_config2_sampled(oracle):
    """B1, H32, S4096 (a launch that does not fill the machine): three sampled heads."""
    _full_size_case(oracle, 2, [(0, 0), (0, 13), (0, 31)])


@pytest.mark.parametrize("p", [6, 8])
def test_full_size_config3_mantissa_sweep_sampled(oracle, p):
    """Config 3's mantissa sweep at full size: the 6-bit and the 8-bit kernels on B16, H32, S8192."""
    _full_size_case(oracle, 3, [(0, 1), (15, 30), (8, 16)], mant_bits=p)


@pytest.mark.parametrize("p", [4, 8])
def test_group_of_8_long_sequences_sampled(oracle, p):
    """Eight query heads per KV head (two 8-column tiles per warp), 64 sequences of 4096 tokens on 4 KV heads:
    256 pairs of 64 items each against about a dozen items per warp, so that many warps' ranges cross from one
    (batch, kv head) pair into the next."""
    _full_size_case(oracle, 4, [(0, 0), (63, 3), (17, 2), (40, 1)], batch=64, seq=4096, n_q_heads=32, n_kv_heads=4,
                    mant_bits=p)


@pytest.mark.parametrize("p,impl", [(4, B.DECODE_AUTO), (8, B.DECODE_AUTO), (6, B.DECODE_AUTO), (4, B.DECODE_SIMT)])
def test_planes_beyond_4_gib(oracle, p, impl):
    """Maximum sizes: a cache whose mantissa planes are larger than 4 GiB (40 sequences x 32 heads x 65536 rows),
    so that row offsets need 64 bits in append, dequant and decode.  300 tokens are written to every sequence;
    the last sequence's units (byte offsets above 2^32) are compared with the oracle run on that sequence alone."""
    w = W.CONFIGS[2]
    Bn, Hkv, d, S_max, T, n = 40, 32, 128, 65536, 300, 32
    dv = torch.device("cuda")
    cache = B.Cache(Bn, Hkv, d, S_max, n, p, device=dv)
    assert cache.k_mant.numel() > (1 << 32)
    k, v = W.make_kv(w, n_tokens=T, device=dv, batch=Bn)
    q = W.make_q(w, device=dv, batch=Bn)
    start = torch.full((Bn,), 1000, dtype=torch.int32, device=dv)
    B.append(cache, k, v, start)
    lens = torch.zeros(Bn, dtype=torch.int32, device=dv)
    lens[Bn - 1] = 1000 + T
    lens[0] = 1000 + T
    # rows [0, 1000) of the two sequences that are read: zeros as keys and values (written, so that they are specified)
    zk = torch.zeros(Bn, 1000, Hkv, d, dtype=k.dtype, device=dv)
    B.append(cache, zk, zk, torch.zeros(Bn, dtype=torch.int32, device=dv))
    del zk
    out = B.decode_attn(cache, q, lens, max_len_hint=1000 + T, impl=impl)
    assert B.device_status() == 0
    assert not host(out[1:Bn - 1]).any()                       # empty sequences
    for b in (0, Bn - 1):
        for h in (0, Hkv - 1):
            kk = np.concatenate([np.zeros((1, 1000, 1, d), np.float32), host(k[b:b + 1, :, h:h + 1].float())], axis=1)
            vv = np.concatenate([np.zeros((1, 1000, 1, d), np.float32), host(v[b:b + 1, :, h:h + 1].float())], axis=1)
            oc = oracle.Cache(1, 1, d, 1312, n, p)
            oracle.append(oc, kk, vv, "f32", np.zeros(1, np.int32))
            assert np.array_equal(host(cache.k_mant[b, h, :1000 + T]), oc.k_mant[0, 0, :1000 + T])
            assert np.array_equal(host(cache.v_exp[b, h, :1000 + T]), oc.v_exp[0, 0, :1000 + T])
            assert np.array_equal(host(B.dequant(cache, "v", b, h, 1000, T)), oracle.dequant(oc, "v", 0, 0, 1000, T).astype(np.float32))
            ref = oracle.decode_attn(oc, W.to_oracle(q[b:b + 1, h:h + 1]), w.dtype, 1, [1000 + T])
            assert rel_err(host(out[b:b + 1, h:h + 1]).astype(np.float64), ref) <= ATTN_TOL
