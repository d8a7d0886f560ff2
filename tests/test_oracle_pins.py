"""Pins for the CPU oracle: closed forms, invariants, special cases and brute force.

Nothing here compares the oracle with itself or with the CUDA path.  Each pin
is chosen so that a plausible mistake (dropped term, wrong sign or index,
transposed operand, wrong tie rule) fails at least one of them.
"""
import itertools
import math
from fractions import Fraction

import numpy as np
import pytest

from paper_2403_20137_b200 import workloads as W

FORMATS_P = [4, 6, 8]
BLOCKS = [16, 32, 64, 128]


def qmax(p):
    return 2 ** (p - 1) - 1


# ---------------------------------------------------------------- I1: powers of two
@pytest.mark.parametrize("p", [3, 4, 6, 8])
def test_powers_of_two_round_trip(oracle, p):
    """Sec. II-B cast + Eq. (1): +-2^k is on the grid of its own block for every binary32 exponent."""
    for k in range(-126, 128):
        for sgn in (1.0, -1.0):
            x = np.zeros(8)
            x[3] = sgn * math.ldexp(1.0, k)
            x[5] = sgn * math.ldexp(1.0, k - 1) if k > -126 else 0.0  # a smaller grid value
            e8, M = oracle.bfp_cast_block(x, p)
            assert e8 == k + 127
            assert M[3] == int(sgn) * 2 ** (p - 2)
            if k > -126:
                assert M[5] == int(sgn) * 2 ** (p - 3)
            for j in range(8):
                assert oracle.bfp_value(M[j], e8, p) == x[j]


@pytest.mark.parametrize("p", [4, 6, 8])
def test_cast_symmetries(oracle, p):
    """What the cast of Sec. II-B must commute with, whatever its internals: a power-of-two scaling moves the shared
    exponent and nothing else, a sign flip negates the mantissas (the range is symmetric and ties go to even), and a
    permutation inside the block permutes the mantissas (the exponent comes from the maximum alone)."""
    rng = np.random.default_rng(31 + p)
    for _ in range(200):
        n = int(rng.choice([16, 32, 64, 128]))
        x = (rng.standard_normal(n) * 2.0 ** rng.integers(-20, 20)).astype(np.float32).astype(np.float64)
        x[rng.integers(0, n)] *= 1.0 + rng.integers(0, 30)                    # sometimes an outlier
        grid = rng.integers(-8, 9, size=n) * 2.0 ** -3                        # plus values that sit on exact ties
        if rng.random() < 0.3:
            x = grid
        e8, M = oracle.bfp_cast_block(x, p)
        k = int(rng.integers(-40, 40))
        e8s, Ms = oracle.bfp_cast_block(np.ldexp(x, k), p)
        if e8 > 0 and 0 < e8 + k < 255:
            assert e8s == e8 + k and np.array_equal(Ms, M)
        e8n, Mn = oracle.bfp_cast_block(-x, p)
        assert e8n == e8 and np.array_equal(Mn, -np.asarray(M))
        perm = rng.permutation(n)
        e8p, Mp = oracle.bfp_cast_block(x[perm], p)
        assert e8p == e8 and np.array_equal(Mp, np.asarray(M)[perm])


def test_zero_and_subnormal_blocks(oracle):
    e8, M = oracle.bfp_cast_block(np.zeros(16), 4)
    assert e8 == 0 and not M.any()
    # below the smallest normal binary32 the exponent byte stays 0 and the grid is 2^(-127-(p-2))
    for p in (4, 8):
        unit = math.ldexp(1.0, -127 - (p - 2))
        x = np.array([3 * unit, -unit, 0.5 * unit, 1.5 * unit, 2.5 * unit])
        e8, M = oracle.bfp_cast_block(x, p)
        assert e8 == 0
        assert list(M) == [3, -1, 0, 2, 2]   # ties go to the even integer


# ---------------------------------------------------------------- I2: grid values / idempotence
@pytest.mark.parametrize("p", FORMATS_P)
@pytest.mark.parametrize("n", [16, 32, 128])
def test_grid_blocks_are_fixed_points(oracle, p, n):
    rng = np.random.default_rng(100 + p * 7 + n)
    for _ in range(200):
        e8 = int(rng.integers(0, 255))
        M = rng.integers(-qmax(p), qmax(p) + 1, size=n)
        top = int(rng.integers(2 ** (p - 2), qmax(p) + 1)) * (1 if rng.random() < 0.5 else -1)
        M[int(rng.integers(0, n))] = top          # forces the exponent to be e8
        x = np.array([math.ldexp(float(m), e8 - 127 - (p - 2)) for m in M])
        e8_o, M_o = oracle.bfp_cast_block(x, p)
        assert e8_o == e8
        assert np.array_equal(M_o, M)


# ---------------------------------------------------------------- I3: error bound
@pytest.mark.parametrize("p", FORMATS_P)
def test_error_bound_and_top_mantissa(oracle, p):
    rng = np.random.default_rng(7 + p)
    for trial in range(300):
        n = int(rng.choice([16, 32, 64]))
        x = rng.standard_normal(n) * math.ldexp(1.0, int(rng.integers(-40, 40)))
        if trial % 3 == 0:
            x[int(rng.integers(0, n))] *= 20.0
        x = x.astype(np.float32).astype(np.float64)
        e8, M = oracle.bfp_cast_block(x, p)
        e = e8 - 127 - (p - 2)
        assert np.max(np.abs(M)) >= 2 ** (p - 2)          # the largest element uses the top bit
        assert np.max(np.abs(M)) <= qmax(p)
        for j in range(n):
            t = Fraction(x[j]) / Fraction(2) ** e
            err = abs(Fraction(x[j]) - Fraction(int(M[j])) * Fraction(2) ** e)
            if abs(t) < qmax(p) + Fraction(1, 2):
                assert err <= Fraction(2) ** e / 2
            else:                                           # clamp zone
                assert abs(M[j]) == qmax(p) and err < Fraction(2) ** e


# ---------------------------------------------------------------- I4: brute force on tiny blocks
@pytest.mark.parametrize("p", [3, 4])
@pytest.mark.parametrize("n", [1, 2, 4])
def test_brute_force_nearest_even(oracle, p, n):
    """Enumerate every allowed mantissa at the prescribed exponent: the cast must pick the closest,
    the even one on exact ties; inputs sit on a 1/8 grid so ties and clamp-zone values all occur."""
    qm = qmax(p)
    cands = list(range(-qm, qm + 1))
    grid = [Fraction(i, 8) for i in range(-8 * 2 ** (p - 1) + 1, 8 * 2 ** (p - 1))]
    rng = np.random.default_rng(11 * p + n)
    for E in (-3, 0, 5):
        unit = Fraction(2) ** (E - (p - 2))
        # the leading element fixes the block exponent: |t0| in [2^(p-2), 2^(p-1))
        lead = [t for t in grid if 2 ** (p - 2) <= abs(t) < 2 ** (p - 1)]
        for t0 in lead:
            others = [grid[int(i)] for i in rng.integers(0, len(grid), size=n - 1)]
            others = [t if abs(t) <= abs(t0) else t0 for t in others]
            ts = [t0] + others
            x = np.array([float(t * unit) for t in ts])
            e8, M = oracle.bfp_cast_block(x, p)
            assert e8 == E + 127
            for t, m in zip(ts, M):
                best = min(abs(t - c) for c in cands)
                winners = [c for c in cands if abs(t - c) == best]
                if len(winners) == 2:
                    winners = [c for c in winners if c % 2 == 0]
                assert int(m) == winners[0]


# ---------------------------------------------------------------- I5: packing
@pytest.mark.parametrize("p", [2, 4, 6, 8])
def test_pack_all_values_all_positions(oracle, p):
    vals = list(range(-(2 ** (p - 1)), 2 ** (p - 1)))
    n = 16
    for pos in range(n):
        for v in vals:
            M = np.zeros(n, dtype=np.int32)
            M[pos] = v
            M[(pos + 5) % n] = -1
            b = oracle.pack_mantissas(M, p)
            # independent writer: one Python integer as the little-endian bit stream
            stream = 0
            for j, m in enumerate(M):
                stream |= ((int(m) + (1 << (p - 1))) % (1 << p)) << (j * p)     # excess code
            ref = np.frombuffer(stream.to_bytes(n * p // 8, "little"), dtype=np.uint8)
            assert np.array_equal(b, ref)
            assert np.array_equal(oracle.unpack_mantissas(b, n, p), M)


def test_pack_nibble_and_six_bit_examples(oracle):
    # p=4, excess-8 code, low nibble = even element.  1 -> 9, -1 -> 7, 7 -> 0xF, -7 -> 1, 0 -> 8
    assert list(oracle.pack_mantissas([1, -1, 7, -7], 4)) == [0x79, 0x1F]
    assert list(oracle.pack_mantissas([0, 0], 4)) == [0x88]
    # p=6, excess-32 code: four elements in three bytes; all zero = fields 32 -> bits 100000 x4
    z = int("100000" * 4, 2)
    assert list(oracle.pack_mantissas([0, 0, 0, 0], 6)) == list(z.to_bytes(3, "little"))
    assert list(oracle.pack_mantissas([1, 0, 0, 0], 6)) == list((z + 1).to_bytes(3, "little"))
    assert list(oracle.pack_mantissas([0, 0, 0, -1], 6)) == list((z - (1 << 18)).to_bytes(3, "little"))
    # p=8, excess-128 code
    assert list(oracle.pack_mantissas([0, 127, -127], 8)) == [128, 255, 1]


# ---------------------------------------------------------------- I9: argsort
def test_argsort_against_rank_count(oracle):
    rng = np.random.default_rng(5)
    for trial in range(50):
        d = 128
        stat = rng.integers(0, 12, size=d).astype(np.float64) if trial % 2 else rng.random(d)
        perm, inv = oracle.argsort_stable(stat)
        assert sorted(perm.tolist()) == list(range(d))
        # brute force: the rank of channel c = #{smaller} + #{equal with lower index}
        for c in range(d):
            rank = sum(1 for o in range(d) if stat[o] < stat[c] or (stat[o] == stat[c] and o < c))
            assert perm[rank] == c and inv[c] == rank
        assert np.all(np.diff(stat[perm]) >= 0)


def test_channel_stat_closed_forms(oracle):
    T, H, d = 37, 3, 8
    x = np.zeros((T, H, d), dtype=np.float32)
    x[5, 1, 2] = -9.0
    x[30, 1, 2] = 4.0
    x[:, 2, 7] = 2.0
    st = oracle.channel_stat(x, "f32", H, d, oracle.STAT_MAXABS)
    assert st[1, 2] == 9.0 and st[2, 7] == 2.0 and st.sum() == 11.0
    l2 = oracle.channel_stat(x, "f32", H, d, oracle.STAT_L2)
    assert l2[1, 2] == math.sqrt(97.0) and abs(l2[2, 7] - 2.0 * math.sqrt(T)) < 1e-12
    # bf16 bit patterns widen exactly: 0x4049 = 3.140625
    xb = np.zeros((2, 1, 4), dtype=np.uint16)
    xb[1, 0, 3] = 0xC049
    assert oracle.channel_stat(xb, "bf16", 1, 4)[0, 3] == 3.140625


def test_calibrate_orders_outlier_channels_last(oracle):
    w = W.CONFIGS[1]
    k, _ = W.make_kv(w)
    st, perm, inv = oracle.calibrate(W.to_oracle(k[0]), "f32", 1, 128)
    assert sorted(perm[0, -4:].tolist()) == sorted(w.fixed_outliers)
    assert np.array_equal(inv[0][perm[0]], np.arange(128))
    assert np.array_equal(st[0], np.abs(k[0, :, 0, :].numpy().astype(np.float64)).max(axis=0))


# ---------------------------------------------------------------- I8: Eq. (2), (3)
def test_joint_permutation_keeps_inner_products(oracle):
    rng = np.random.default_rng(3)
    H, d, d_in = 2, 16, 24
    wq = rng.integers(-5, 6, size=(H, d, d_in)).astype(np.float64)
    wk = rng.integers(-5, 6, size=(H, d, d_in)).astype(np.float64)
    perm = np.stack([rng.permutation(d) for _ in range(H)]).astype(np.int32)
    wq_p, wk_p = oracle.fold_perm(wq, perm), oracle.fold_perm(wk, perm)
    for h in range(H):
        assert np.array_equal(wq_p[h], wq[h][perm[h]])          # row gather
        assert np.array_equal(wq[h].T @ wk[h], wq_p[h].T @ wk_p[h])   # Eq. (2), exact on integers
        x = rng.integers(-3, 4, size=d_in).astype(np.float64)
        assert (wq[h] @ x) @ (wk[h] @ x) == (wq_p[h] @ x) @ (wk_p[h] @ x)   # Eq. (3)


# ---------------------------------------------------------------- cache write / dequant
def _cache_from(oracle, w, k, v, perm_k=None, perm_v=None, block=None, p=None, max_seq=None):
    B, T, H, d = k.shape
    c = oracle.Cache(B, H, d, max_seq or T, block or w.block, p or w.mant_bits)
    oracle.append(c, W.to_oracle(k), W.to_oracle(v), w.dtype, np.zeros(B, dtype=np.int32), perm_k, perm_v)
    return c


def test_append_layout_and_positions(oracle):
    """Rows land at start_pos + t of plane [B, H, S_max, row]; untouched rows stay as they were."""
    B, H, d, S = 2, 3, 32, 10
    c = oracle.Cache(B, H, d, S, 16, 4)
    c.k_mant[:] = 0xAB
    c.k_exp[:] = 0xCD
    k = np.zeros((B, 2, H, d), dtype=np.float32)
    k[1, 1, 2, 0] = 1.0          # batch 1, second new token, head 2, channel 0 -> block 0
    k[1, 1, 2, 17] = -3.0        # block 1
    oracle.append(c, k, None, "f32", np.array([4, 7], dtype=np.int32))
    row = c.k_mant[1, 2, 8]
    assert row[0] == 0x8C and (row[1:8] == 0x88).all()      # M = 2^(p-2) = 4 -> code 12 in the low nibble, zeros -> 8
    assert row[8] == 0x28 and (row[9:] == 0x88).all()       # -3 -> t = -6 -> code 2, odd element
    assert list(c.k_exp[1, 2, 8]) == [127, 128]
    assert (c.k_mant[1, 2, 7] == 0x88).all() and (c.k_exp[1, 2, 7] == 0).all()   # zero row written (code 8 = 0)
    assert (c.k_mant[1, 2, 6] == 0xAB).all() and (c.k_mant[0, 0, 3] == 0xAB).all()
    assert (c.k_mant[0, 0, 4] == 0x88).all() and (c.k_mant[0, 0, 6] == 0xAB).all()
    with pytest.raises(oracle.OracleError) as e:
        oracle.append(c, k, None, "f32", np.array([4, 9], dtype=np.int32))
    assert e.value.status == oracle.CAPACITY


def test_nonfinite_input_is_refused(oracle):
    c = oracle.Cache(1, 1, 16, 4, 16, 4)
    k = np.zeros((1, 1, 1, 16), dtype=np.float32)
    k[0, 0, 0, 3] = np.inf
    with pytest.raises(oracle.OracleError) as e:
        oracle.append(c, k, None, "f32", np.zeros(1, dtype=np.int32))
    assert e.value.status == oracle.NONFINITE


@pytest.mark.parametrize("p", FORMATS_P)
def test_block_equal_head_dim_ignores_permutation(oracle, p):
    """Sanity row of Table I: with one block per head a permutation cannot change anything."""
    w = W.CONFIGS[1]
    k, v = W.make_kv(w, n_tokens=64)
    _, perm, _ = oracle.calibrate(W.to_oracle(k[0]), "f32", 1, 128)
    plain = _cache_from(oracle, w, k, v, block=128, p=p)
    sortd = _cache_from(oracle, w, k, v, perm_k=perm, block=128, p=p)
    a = oracle.dequant(plain, "k", 0, 0, 0, 64)
    b = oracle.dequant(sortd, "k", 0, 0, 0, 64, perm=perm)
    assert np.array_equal(a, b)
    assert np.array_equal(plain.k_exp, sortd.k_exp)


def test_identity_permutation_is_plain_bfp(oracle):
    w = W.CONFIGS[2]
    k, v = W.make_kv(w, n_tokens=16)
    ident = np.tile(np.arange(128, dtype=np.int32), (w.n_kv_heads, 1))
    a = _cache_from(oracle, w, k, v)
    b = _cache_from(oracle, w, k, v, perm_k=ident, perm_v=ident)
    assert np.array_equal(a.k_mant, b.k_mant) and np.array_equal(a.k_exp, b.k_exp)
    assert np.array_equal(a.v_mant, b.v_mant)


def test_dequant_matches_eq1_by_hand(oracle):
    c = oracle.Cache(1, 1, 16, 2, 8, 4)
    c.k_mant[0, 0, 1] = np.frombuffer(bytes([0xA9, 0xCB, 0xED, 0x8F, 0x77, 0x17, 0x88, 0x98]), dtype=np.uint8)
    c.k_exp[0, 0, 1] = [129, 120]
    out = oracle.dequant(c, "k", 0, 0, 1, 1)[0]
    want = [1, 2, 3, 4, 5, 6, 7, 0] + [m * 2.0 ** -9 for m in (-1, -1, -1, -7, 0, 0, 0, 1)]
    assert out.tolist() == want
    perm = np.arange(16, dtype=np.int32)[::-1].copy().reshape(1, 16)
    out_p = oracle.dequant(c, "k", 0, 0, 1, 1, perm=perm)[0]
    assert out_p.tolist() == want[::-1]     # slot j goes back to channel perm[j]


def test_ksort_lowers_key_mse(oracle):
    """Direction of effect (Sec. II-C, Table I): on outlier-structured keys sorted blocks quantise
    better for every block smaller than the head; without outliers sorting changes little."""
    w = W.CONFIGS[1]
    k, v = W.make_kv(w)
    ref = k[0, :, 0, :].numpy().astype(np.float64)
    _, perm, _ = oracle.calibrate(W.to_oracle(k[0]), "f32", 1, 128)
    for n in (16, 32, 64):
        plain = _cache_from(oracle, w, k, v, block=n)
        sortd = _cache_from(oracle, w, k, v, perm_k=perm, block=n)
        mse_plain = np.mean((oracle.dequant(plain, "k", 0, 0, 0, 256) - ref) ** 2)
        mse_sorted = np.mean((oracle.dequant(sortd, "k", 0, 0, 0, 256, perm=perm) - ref) ** 2)
        assert mse_sorted < 0.75 * mse_plain
    # the non-outlier neighbours of an outlier mostly round to zero in the unsorted cache
    plain = _cache_from(oracle, w, k, v, block=16)
    d0 = oracle.dequant(plain, "k", 0, 0, 0, 256)[:, 0:16]
    others = np.delete(d0, 3, axis=1)
    assert np.mean(others == 0.0) > 0.5
    # outlier-free data: sorting by max-abs neither helps nor hurts beyond noise
    rng = np.random.default_rng(1)
    kk = rng.standard_normal((1, 256, 1, 128)).astype(np.float32)
    _, perm2, _ = oracle.calibrate(kk[0], "f32", 1, 128)
    c1, c2 = oracle.Cache(1, 1, 128, 256, 16, 4), oracle.Cache(1, 1, 128, 256, 16, 4)
    z = np.zeros(1, dtype=np.int32)
    oracle.append(c1, kk, None, "f32", z)
    oracle.append(c2, kk, None, "f32", z, perm_k=perm2)
    m1 = np.mean((oracle.dequant(c1, "k", 0, 0, 0, 256) - kk[0, :, 0]) ** 2)
    m2 = np.mean((oracle.dequant(c2, "k", 0, 0, 0, 256, perm=perm2) - kk[0, :, 0]) ** 2)
    assert abs(m1 - m2) < 0.1 * m1


def test_bits_per_element(oracle):
    for n, p in itertools.product(BLOCKS, FORMATS_P):
        c = oracle.Cache(1, 1, 128, 1, n, p)
        bits = 8.0 * (c.k_mant.size + c.k_exp.size) / 128
        assert bits == p + 8.0 / n
        assert c.fmt.row_m == 128 * p // 8 and c.fmt.row_e == 128 // n


# ---------------------------------------------------------------- I10: attention special cases
def _tiny_cache(oracle, K, V, block=16, p=8, max_seq=None):
    """K, V [T, d] float32 values that sit on the BFP grid when small integers are used."""
    T, d = K.shape
    c = oracle.Cache(1, 1, d, max_seq or T, block, p)
    z = np.zeros(1, dtype=np.int32)
    oracle.append(c, K.reshape(1, T, 1, d).astype(np.float32), V.reshape(1, T, 1, d).astype(np.float32), "f32", z)
    return c


def test_attention_special_cases(oracle):
    rng = np.random.default_rng(2)
    d = 32
    V = rng.integers(-100, 101, size=(6, d)).astype(np.float32)
    V[:, 0] = 64.0     # each 16-block carries a power of two >= its other entries/2 so V sits on the grid
    V[:, 16] = 64.0
    V = np.clip(V, -127, 127)
    q = rng.standard_normal((1, 1, d)).astype(np.float32)

    # one token: the output is that token's value row
    c = _tiny_cache(oracle, np.ones((1, d), np.float32), V[:1])
    assert np.array_equal(oracle.decode_attn(c, q, "f32", 1, [1])[0, 0], V[0].astype(np.float64))

    # all keys zero: uniform weights, output = mean of the value rows
    c = _tiny_cache(oracle, np.zeros((6, d), np.float32), V)
    out = oracle.decode_attn(c, q, "f32", 1, [6])[0, 0]
    assert np.allclose(out, V.astype(np.float64).mean(axis=0), rtol=0, atol=1e-12)
    # ...and only over the first seq_len tokens
    out4 = oracle.decode_attn(c, q, "f32", 1, [4])[0, 0]
    assert np.allclose(out4, V[:4].astype(np.float64).mean(axis=0), rtol=0, atol=1e-12)

    # one dominant score: the output is that row
    K = np.zeros((6, d), np.float32)
    K[4, 1] = 64.0
    qq = np.zeros((1, 1, d), np.float32)
    qq[0, 0, 1] = 100.0
    c = _tiny_cache(oracle, K, V)
    out = oracle.decode_attn(c, qq, "f32", 1, [6], softmax_scale=1.0)[0, 0]
    assert np.array_equal(out, V[4].astype(np.float64))

    # two tokens with scores differing by ln 3: weights 1/4 and 3/4
    K = np.zeros((2, d), np.float32)
    K[1, 0] = 1.0
    qq[:] = 0
    qq[0, 0, 0] = 1.0
    c = _tiny_cache(oracle, K, V[:2])
    out = oracle.decode_attn(c, qq, "f32", 1, [2], softmax_scale=math.log(3.0))[0, 0]
    V64 = V.astype(np.float64)
    assert np.allclose(out, 0.25 * V64[0] + 0.75 * V64[1], rtol=1e-14, atol=0)

    # default scale is 1/sqrt(d): same two tokens, score gap = 8/sqrt(32)
    K[1, 0] = 8.0
    c = _tiny_cache(oracle, K, V[:2])
    out = oracle.decode_attn(c, qq, "f32", 1, [2])[0, 0]
    w1 = 1.0 / (1.0 + math.exp(-8.0 / math.sqrt(32.0)))
    assert np.allclose(out, (1 - w1) * V64[0] + w1 * V64[1], rtol=1e-13, atol=0)

    # empty sequence: zeros
    assert not oracle.decode_attn(c, qq, "f32", 1, [0]).any()


def test_attention_matches_numpy_on_dequantised_cache(oracle):
    """The definition itself, with numpy's matmul/softmax as the library routine, GQA included."""
    w = W.CONFIGS[4]
    B, T, Hkv, Hq, d = 2, 40, 2, 8, 128
    rng = np.random.default_rng(9)
    k = (rng.standard_normal((B, T, Hkv, d)) * 3).astype(np.float32)
    v = rng.standard_normal((B, T, Hkv, d)).astype(np.float32)
    q = rng.standard_normal((B, Hq, d)).astype(np.float32)
    perm_k = np.stack([rng.permutation(d) for _ in range(Hkv)]).astype(np.int32)
    perm_v = np.stack([rng.permutation(d) for _ in range(Hkv)]).astype(np.int32)
    inv_v = np.argsort(perm_v, axis=1).astype(np.int32)
    c = oracle.Cache(B, Hkv, d, 48, 32, 4)
    oracle.append(c, k, v, "f32", np.zeros(B, dtype=np.int32), perm_k, perm_v)
    lens = [40, 17]
    out = oracle.decode_attn(c, q, "f32", Hq, lens, perm_k=perm_k, inv_perm_v=inv_v)
    for b in range(B):
        for hq in range(Hq):
            g = hq // (Hq // Hkv)
            Kd = oracle.dequant(c, "k", b, g, 0, lens[b], perm=perm_k)     # original channel order
            Vd = oracle.dequant(c, "v", b, g, 0, lens[b], perm=perm_v)
            s = Kd @ q[b, hq].astype(np.float64) / math.sqrt(d)
            pr = np.exp(s - s.max())
            pr /= pr.sum()
            assert np.allclose(out[b, hq], pr @ Vd, rtol=1e-12, atol=1e-13)


def test_attention_shift_invariance(oracle):
    """Adding a constant to every score (a key direction shared by all tokens) changes nothing."""
    d, T = 32, 12
    rng = np.random.default_rng(4)
    K = rng.integers(-7, 8, size=(T, d)).astype(np.float32)
    K[:, 0] = 4.0
    K[:, 16] = 4.0                   # keeps every block exponent fixed -> K is on the grid
    V = rng.integers(-7, 8, size=(T, d)).astype(np.float32)
    V[:, 0] = 4.0
    V[:, 16] = 4.0
    q = rng.integers(-3, 4, size=(1, 1, d)).astype(np.float32)
    q[0, 0, 16] = 0.0
    c1 = _tiny_cache(oracle, K, V, p=4)
    K2 = K.copy()
    K2[:, 16] = 7.0                  # same constant added to every token's score
    q2 = q.copy()
    q2[0, 0, 16] = 5.0
    c2 = _tiny_cache(oracle, K2, V, p=4)
    o1 = oracle.decode_attn(c1, q, "f32", 1, [T])
    o2 = oracle.decode_attn(c2, q2, "f32", 1, [T])
    assert np.allclose(o1, o2, rtol=1e-12, atol=1e-13)


def test_bfp16_query_cast(oracle):
    """Sec. IV: q in BFP16.  A query already on the 8-bit grid is unchanged; otherwise the result
    equals attention with the query replaced by its own BFP cast."""
    d, T = 32, 5
    rng = np.random.default_rng(6)
    K = rng.standard_normal((T, d)).astype(np.float32)
    V = rng.standard_normal((T, d)).astype(np.float32)
    c = _tiny_cache(oracle, K, V, p=4)
    q = rng.integers(-127, 128, size=(1, 1, d)).astype(np.float32)
    q[0, 0, 0] = 64.0
    q[0, 0, 16] = 127.0
    assert np.array_equal(oracle.decode_attn(c, q, "f32", 1, [T]),
                          oracle.decode_attn(c, q, "f32", 1, [T], q_mant_bits=8))
    q = rng.standard_normal((1, 1, d)).astype(np.float32)
    qc = np.zeros_like(q)
    for blk in range(2):
        e8, M = oracle.bfp_cast_block(q[0, 0, blk * 16:(blk + 1) * 16], 8)
        qc[0, 0, blk * 16:(blk + 1) * 16] = [oracle.bfp_value(m, e8, 8) for m in M]
    assert np.array_equal(oracle.decode_attn(c, qc, "f32", 1, [T]),
                          oracle.decode_attn(c, q, "f32", 1, [T], q_mant_bits=8))
    assert not np.array_equal(qc, q)


# ---------------------------------------------------------------- RoPE (Eq. (4), Algorithm 1 step 5)
@pytest.mark.parametrize("half_split", [False, True])
def test_rope_is_the_block_rotation(oracle, half_split):
    d = 16
    theta, partner, sign = oracle.rope_tables(d, 10000.0, half_split)
    rng = np.random.default_rng(8)
    x = rng.standard_normal(d)
    m = 5.0
    y = oracle.rope_apply(x, m, theta, partner, sign)
    # rotation matrix of Sec. II-D written out pair by pair
    for i in range(d // 2):
        th = 10000.0 ** (-2.0 * i / d)
        a, b = (i, i + d // 2) if half_split else (2 * i, 2 * i + 1)
        assert abs(y[a] - (x[a] * math.cos(m * th) - x[b] * math.sin(m * th))) < 1e-14
        assert abs(y[b] - (x[a] * math.sin(m * th) + x[b] * math.cos(m * th))) < 1e-14
    assert abs(np.linalg.norm(y) - np.linalg.norm(x)) < 1e-13       # orthogonal
    if not half_split:
        assert partner.tolist()[:4] == [1, 0, 3, 2] and sign.tolist()[:4] == [-1, 1, -1, 1]
        assert theta[0] == theta[1] == 1.0


@pytest.mark.parametrize("half_split", [False, True])
def test_permuted_rope_commutes_with_permutation(oracle, half_split):
    d = 32
    rng = np.random.default_rng(10)
    perm = rng.permutation(d).astype(np.int32)
    inv = np.argsort(perm).astype(np.int32)
    theta, partner, sign = oracle.rope_tables(d, 10000.0, half_split)
    tp, pp, sp = oracle.rope_permute_tables(perm, inv, theta, partner, sign)
    x = rng.integers(-9, 10, size=d).astype(np.float64)
    for m in (0.0, 1.0, 77.0):
        y = oracle.rope_apply(x, m, theta, partner, sign)
        yp = oracle.rope_apply(x[perm], m, tp, pp, sp)
        assert np.array_equal(yp, y[perm])       # same products, same order of the two-term sum
    # relative-position property survives: <R_m q, R_n k> depends on m - n only
    qv, kv = rng.standard_normal(d), rng.standard_normal(d)
    a = oracle.rope_apply(qv[perm], 9.0, tp, pp, sp) @ oracle.rope_apply(kv[perm], 4.0, tp, pp, sp)
    b = oracle.rope_apply(qv, 15.0, theta, partner, sign) @ oracle.rope_apply(kv, 10.0, theta, partner, sign)
    assert abs(a - b) < 1e-12


def _tables(oracle, perm, half_split):
    """Per-head tables in stored order, concatenated [H * d]."""
    H, d = perm.shape
    theta, partner, sign = oracle.rope_tables(d, 10000.0, half_split)
    out = [oracle.rope_permute_tables(perm[h], np.argsort(perm[h]).astype(np.int32), theta, partner, sign)
           for h in range(H)]
    return (np.concatenate([o[0] for o in out]), np.concatenate([o[1] for o in out]).astype(np.int32),
            np.concatenate([o[2] for o in out]))


@pytest.mark.parametrize("half_split", [False, True])
def test_attention_over_pre_rotation_keys(oracle, half_split):
    """Attention with the rotary embedding applied after the read-back (Sec. III par. 2), pinned to things other
    than itself: (1) zero frequencies are no rotation at all; (2) the textbook form, complex multiplication of the
    channel pairs by e^{i t theta}, on the dequantised keys with numpy's softmax; (3) with one block per row
    (so that the cast does not depend on the order, Table I's last row) a K-sorted cache with the permuted tables
    of Algorithm 1 step 5 gives what the unsorted cache gives with the plain tables."""
    B, T, Hkv, Hq, d = 2, 37, 2, 4, 128
    rng = np.random.default_rng(21)
    k = (rng.standard_normal((B, T, Hkv, d)) * 2).astype(np.float32)
    v = rng.standard_normal((B, T, Hkv, d)).astype(np.float32)
    q = rng.standard_normal((B, Hq, d)).astype(np.float32)
    lens = [37, 9]
    ident = np.tile(np.arange(d, dtype=np.int32), (Hkv, 1))
    th, pa, sg = _tables(oracle, ident, half_split)
    c = oracle.Cache(B, Hkv, d, 48, 32, 4)
    oracle.append(c, k, v, "f32", np.zeros(B, dtype=np.int32))
    # (1)
    plain = oracle.decode_attn(c, q, "f32", Hq, lens)
    assert np.array_equal(oracle.decode_attn_rope(c, q, "f32", Hq, lens, np.zeros_like(th), pa, sg), plain)
    # (2)
    out = oracle.decode_attn_rope(c, q, "f32", Hq, lens, th, pa, sg)
    assert not np.allclose(out, plain, rtol=1e-3)
    freq = 10000.0 ** (-2.0 * np.arange(d // 2) / d)
    for b in range(B):
        for hq in range(Hq):
            g = hq // (Hq // Hkv)
            Kd = oracle.dequant(c, "k", b, g, 0, lens[b])
            Vd = oracle.dequant(c, "v", b, g, 0, lens[b])
            lo, hi = (Kd[:, :d // 2], Kd[:, d // 2:]) if half_split else (Kd[:, 0::2], Kd[:, 1::2])
            z = (lo + 1j * hi) * np.exp(1j * np.arange(lens[b])[:, None] * freq[None, :])
            Kr = np.empty_like(Kd)
            if half_split:
                Kr[:, :d // 2], Kr[:, d // 2:] = z.real, z.imag
            else:
                Kr[:, 0::2], Kr[:, 1::2] = z.real, z.imag
            s = Kr @ q[b, hq].astype(np.float64) / math.sqrt(d)
            pr = np.exp(s - s.max())
            pr /= pr.sum()
            assert np.allclose(out[b, hq], pr @ Vd, rtol=1e-11, atol=1e-12)
    # (3)
    perm = np.stack([rng.permutation(d) for _ in range(Hkv)]).astype(np.int32)
    tp, pp, sp = _tables(oracle, perm, half_split)
    c1 = oracle.Cache(B, Hkv, d, 48, 128, 4)
    c2 = oracle.Cache(B, Hkv, d, 48, 128, 4)
    oracle.append(c1, k, v, "f32", np.zeros(B, dtype=np.int32))
    oracle.append(c2, k, v, "f32", np.zeros(B, dtype=np.int32), perm)
    a = oracle.decode_attn_rope(c1, q, "f32", Hq, lens, th, pa, sg)
    bb = oracle.decode_attn_rope(c2, q, "f32", Hq, lens, tp, pp, sp, perm_k=perm)
    assert np.allclose(a, bb, rtol=1e-11, atol=1e-12)


# ---------------------------------------------------------------- inputs follow the stated recipe
def test_workload_recipe():
    w = W.CONFIGS[2]
    ch, sc = W.outlier_channels(w)
    assert ch.shape == (32, 6) and all(len(set(r.tolist())) == 6 for r in ch)
    assert 5.0 < float(sc.median()) < 30.0            # LogNormal(2.5, 0.5): median e^2.5 = 12.2
    k, v = W.make_kv(w, n_tokens=64)
    k2, _ = W.make_kv(w, n_tokens=64)
    assert k.dtype.is_floating_point and k.shape == (1, 64, 32, 128) and bool((k == k2).all())
    sd = k.float().std(dim=(0, 1))
    assert float(sd[0, ch[0, 0]]) > 3.0 and abs(float(v.float().std()) - 1.0) < 0.05


# ------------------------------------------------------------------------------- values the paper prints
def _golden(name):
    import os
    out = {}
    with open(os.path.join(os.path.dirname(__file__), "golden", name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            if ":" in line:
                k, v = line.split(":", 1)
                out[k.strip()] = [float(x) for x in v.split()]
            else:
                parts = line.split()
                out[parts[0]] = [float(x) for x in parts[1:]]
    return out


def test_rope_tables_match_the_vectors_the_paper_prints(oracle):
    """Sec. III and its footnote print the frequency, partner-index and sign vectors of the rotary embedding; the
    oracle's tables for a head of 8 channels must be exactly those (tests/golden/rope_order_sec3.txt)."""
    g = _golden("rope_order_sec3.txt")
    d, base = 8, g["base"][0]
    theta, partner, sign = oracle.rope_tables(d, base, False)
    want_theta = np.array([base ** (-2.0 * (i - 1) / d) for i in g["theta_index_interleaved"]])
    assert np.allclose(theta, want_theta, rtol=1e-15, atol=0)
    assert np.array_equal(partner + 1, np.array(g["partner_interleaved"], dtype=np.int32))
    assert np.array_equal(sign, np.array(g["sign_interleaved"]))
    theta_h, partner_h, sign_h = oracle.rope_tables(d, base, True)
    want_h = np.array([base ** (-2.0 * (i - 1) / d) for i in g["theta_index_half_split"]])
    assert np.allclose(theta_h, want_h, rtol=1e-15, atol=0)
    # partners share a frequency and carry opposite signs in both layouts
    for th, pa, sg in ((theta, partner, sign), (theta_h, partner_h, sign_h)):
        assert np.array_equal(th[pa], th) and np.array_equal(sg[pa], -sg) and np.array_equal(pa[pa], np.arange(d))


def test_formats_match_the_ranges_the_paper_prints(oracle):
    """Sec. II-B prints the mantissa range and the two formats in use; the cast must reach both ends of the range and
    never leave it, and a block as large as the head makes K-sort a no-op (Table I, block 128)
    (tests/golden/bfp_formats_sec2b.txt)."""
    g = _golden("bfp_formats_sec2b.txt")
    rng = np.random.default_rng(5)
    for name in ("BFP12", "BFP16"):
        p, b, lo, hi = (int(x) for x in g[name])
        assert b == 8 and lo == -(2 ** (p - 1) - 1) and hi == 2 ** (p - 1) - 1
        scale = np.exp2(float(rng.integers(-20, 20)))
        x = rng.uniform(-0.9, 0.9, 32) * scale
        x[3], x[7] = 1.999 * scale, -1.999 * scale          # both ends round past the range and are clamped to it
        e8, M = oracle.bfp_cast_block(x, p)
        assert M.min() == lo and M.max() == hi and 0 < e8 < 255
        assert np.isclose(p + b / 32.0, {4: 4.25, 8: 8.25}[p])
    assert g["table1_block128_ksort_equals_unsorted"] == [1.0]
    d = 128
    k = (rng.standard_normal((1, 40, 1, d)) * np.where(rng.random(d) < 0.05, 20.0, 1.0)).astype(np.float32)
    _, perm, _ = oracle.calibrate(k.reshape(-1, 1, d), "f32", 1, d)
    plain, sortd = oracle.Cache(1, 1, d, 48, 128, 4), oracle.Cache(1, 1, d, 48, 128, 4)
    z = np.zeros(1, np.int32)
    oracle.append(plain, k, None, "f32", z)
    oracle.append(sortd, k, None, "f32", z, perm_k=perm)
    a = oracle.dequant(plain, "k", 0, 0, 0, 40)
    b_ = oracle.dequant(sortd, "k", 0, 0, 0, 40, perm=perm)
    assert np.array_equal(a, b_)
