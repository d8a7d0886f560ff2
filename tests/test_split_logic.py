"""The integer arithmetic that the persistent decode kernel and the merge kernel share (host-side check).

Work items (pair-major pieces of a sequence) are cut into one contiguous range per warp; every range writes one
partial per (batch, kv head) it touches, at slot partial_slot(first item).  This re-states that arithmetic in
Python and checks, over many shapes, that (1) the merge's enumeration finds exactly the runs the kernel makes and
(2) no two runs of a pair share a slot.
"""
import random


def partial_slot(item, item_tokens, chunk, n_chunks):
    if item_tokens == chunk:
        return item
    return min((item + 1) >> 1, n_chunks - 1)


def range_start(w, per, extra):
    return w * per + min(w, extra)


def range_of(x, per, extra):
    big = extra * (per + 1)
    return x // (per + 1) if x < big else extra + (x - big) // per


def kernel_runs(pairs, ipp, W):
    """[(pair, first item in pair, n_items)] as the kernel's get_run() walks them."""
    n = pairs * ipp
    per, extra = divmod(n, W)
    runs = []
    for w in range(W):
        i0 = range_start(w, per, extra)
        i1 = i0 + per + (1 if w < extra else 0)
        assert i1 == range_start(w + 1, per, extra)
        it = i0
        while it < i1:
            pair, c0 = divmod(it, ipp)
            cnt = min(i1 - it, ipp - c0)
            runs.append((pair, c0, cnt))
            it += cnt
    return runs


def merge_heads(pair, ipp, W, n, nc):
    """First items of the runs of `pair` as lse_merge enumerates them (items < nc hold tokens)."""
    per, extra = divmod(n, W)
    first, heads, i = pair * ipp, [], 0
    while i < nc:
        heads.append(i)
        w = range_of(first + i, per, extra)
        assert range_start(w, per, extra) <= first + i < range_start(w + 1, per, extra)
        i = range_start(w + 1, per, extra) - first
    return heads


def test_runs_match_merge_and_slots_are_unique():
    rng = random.Random(7)
    cases = [(512, 128, 1776, 64, 128), (64, 512, 1776, 64, 128), (3, 7, 5, 128, 128), (1, 1, 1, 128, 128)]
    for _ in range(300):
        pairs, W = rng.randint(1, 40), rng.randint(1, 97)
        fine = rng.random() < 0.5
        n_chunks = rng.randint(1, 70)
        ipp = 2 * n_chunks - rng.randint(0, 1) if fine else n_chunks
        if fine and pairs * ipp < 4 * W:
            fine, ipp = False, n_chunks             # the library falls back to whole chunks
        cases.append((pairs, ipp, W, 64 if fine else 128, 128))
    for pairs, ipp, W, item_tokens, chunk in cases:
        n = pairs * ipp
        n_chunks = (ipp * item_tokens + chunk - 1) // chunk
        runs = kernel_runs(pairs, ipp, W)
        assert sum(c for _, _, c in runs) == n
        for pair in range(pairs):
            mine = [(c0, cnt) for p, c0, cnt in runs if p == pair]
            for nc in {ipp, max(1, ipp // 3)}:           # full and short sequences
                want = [c0 for c0, _ in mine if c0 < nc]
                assert merge_heads(pair, ipp, W, n, nc) == want
            slots = [partial_slot(c0, item_tokens, chunk, n_chunks) for c0, _ in mine]
            assert len(set(slots)) == len(slots), (pairs, ipp, W, item_tokens, slots)
            assert all(0 <= s < n_chunks for s in slots)
