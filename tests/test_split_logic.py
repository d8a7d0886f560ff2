"""The integer arithmetic that the persistent decode kernels and the merge kernel share, checked on the host.

Work items (pair-major pieces of a sequence) are cut into one contiguous range per warp; every range writes one
partial result per (batch, kv head) pair it touches, at slot partial_slot(first item of the run in its pair), and the
merge enumerates those runs again from the range boundaries.  The functions under test are the library's own
(range_start, range_of, partial_slot and the host-side plan, exported as kvbfp_split_*): nothing here re-states
them.  Checked over exhaustive small shapes and random large ones: (1) the merge's enumeration finds exactly the
runs the kernel makes, (2) no two runs of a pair share a slot, (3) the ranges tile the items.
"""
import ctypes as C
import random

from paper_2403_20137_b200 import binding as B

CHUNK = 128


def plan(pairs, len_cap, fine_tokens, capacity_blocks, warps_per_block, chunk=CHUNK):
    out = (C.c_int32 * 6)()
    rc = B.lib().kvbfp_split_plan(pairs, len_cap, chunk, fine_tokens, capacity_blocks, warps_per_block, out)
    assert rc == B.OK
    return dict(zip(("grid", "n_warps", "item_tokens", "items_per_pair", "range_items", "range_extra"), out))


def kernel_runs(p, pairs):
    """[(pair, first item in pair, n_items)]: a warp walks its range pair by pair, as the kernels do."""
    L = B.lib()
    ipp, per, extra = p["items_per_pair"], p["range_items"], p["range_extra"]
    runs, prev_end = [], 0
    for w in range(p["n_warps"]):
        i0 = L.kvbfp_split_range_start(w, per, extra)
        i1 = L.kvbfp_split_range_start(w + 1, per, extra)
        assert i0 == prev_end and i1 - i0 == per + (1 if w < extra else 0)
        prev_end = i1
        it = i0
        while it < i1:
            pair, c0 = divmod(it, ipp)
            cnt = min(i1 - it, ipp - c0)
            runs.append((pair, c0, cnt))
            it += cnt
    assert prev_end == pairs * ipp                                   # the ranges tile the items
    return runs


def merge_heads(p, pair, n_live):
    """First items of the runs of `pair` as the merge enumerates them (items < n_live hold tokens)."""
    L = B.lib()
    per, extra = p["range_items"], p["range_extra"]
    first, heads, i = pair * p["items_per_pair"], [], 0
    while i < n_live:
        heads.append(i)
        w = L.kvbfp_split_range_of(first + i, per, extra)
        assert L.kvbfp_split_range_start(w, per, extra) <= first + i < L.kvbfp_split_range_start(w + 1, per, extra)
        i = L.kvbfp_split_range_start(w + 1, per, extra) - first
    return heads


def check_case(pairs, len_cap, fine_tokens, capacity_blocks, warps_per_block, chunk=CHUNK):
    L = B.lib()
    p = plan(pairs, len_cap, fine_tokens, capacity_blocks, warps_per_block, chunk)
    n_chunks = (len_cap + chunk - 1) // chunk
    it, ipp = p["item_tokens"], p["items_per_pair"]
    assert it in (fine_tokens, chunk) and ipp == (len_cap + it - 1) // it
    assert p["n_warps"] == p["grid"] * warps_per_block and 1 <= p["grid"] <= capacity_blocks
    if it != chunk:                       # items of chunk / R tokens: only where the slots of a pair can stay distinct
        R = chunk // it
        assert chunk % it == 0 and it % 16 == 0 and n_chunks >= 2 and p["range_items"] >= 2 * R
    by_pair = {}
    for pr, c0, cnt in kernel_runs(p, pairs):
        by_pair.setdefault(pr, []).append(c0)
    for pr in range(pairs):
        mine = by_pair[pr]
        for n_live in {ipp, max(1, ipp // 3), 1}:                    # full, short and one-item sequences
            assert merge_heads(p, pr, n_live) == [c0 for c0 in mine if c0 < n_live]
        slots = [L.kvbfp_split_partial_slot(c0, it, chunk, n_chunks) for c0 in mine]
        assert len(set(slots)) == len(slots), (pairs, len_cap, capacity_blocks, p, mine, slots)
        assert all(0 <= s < n_chunks for s in slots)
    return p


def test_small_shapes_exhaustively():
    """One to four chunks per pair with ragged and full last chunks, every pair count that matters around the
    points where the plan switches to items of half a chunk and of an eighth of a chunk, and several device sizes."""
    fine_seen = coarse_seen = 0
    pair_counts = [1, 2, 3, 4, 5, 7, 10, 13, 16, 23, 31, 47, 64, 97, 128, 211, 300]
    for n_chunks in (1, 2, 3, 4):
        for len_cap in (128 * n_chunks - 127, 128 * n_chunks - 64, 128 * n_chunks - 63, 128 * n_chunks):
            for blocks in (1, 2, 3, 5, 8, 13):
                for pairs in pair_counts:
                    for fine in (16, 32, 64):
                        p = check_case(pairs, len_cap, fine, blocks, 4)
                        fine_seen += p["item_tokens"] == fine
                        coarse_seen += p["item_tokens"] == 128
    assert fine_seen > 300 and coarse_seen > 300


def test_single_chunk_pairs_are_never_cut_in_half():
    """64 < len_cap <= 128 gives one slot per pair; two finer items of one pair would both map to it, so whatever
    the number of pairs the plan keeps whole chunks there."""
    for pairs in (5, 600, 4440, 5120, 20000):
        for len_cap in (65, 100, 128):
            for fine in (16, 64):
                assert plan(pairs, len_cap, fine, 444, 4)["item_tokens"] == 128
            p = plan(pairs, len_cap, 16, 444, 4)
            assert p["item_tokens"] == 128 and p["items_per_pair"] == 1
    check_case(5120, 128, 16, 444, 4)


def test_large_shapes_randomly():
    rng = random.Random(7)
    cases = [(512, 8192, 16, 296, 4), (64, 32768, 16, 444, 4), (64, 32768, 64, 296, 4), (512, 8192, 32, 444, 4),
             (512, 8192, 64, 444, 4), (3, 7 * 128, 16, 2, 4), (1, 1, 16, 444, 4)]
    for _ in range(60):
        cases.append((rng.randint(1, 400), rng.randint(1, 70 * 128), rng.choice((16, 32, 64)), rng.randint(1, 30),
                      rng.choice((1, 2, 4))))
    for c in cases:
        check_case(*c)
    # caller-chosen chunk sizes are never cut finer
    for chunk in (256, 1024):
        p = check_case(40, 5000, 16, 7, 4, chunk=chunk)
        assert p["item_tokens"] == chunk
