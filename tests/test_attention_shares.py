"""Host logic of the step kernel's attention shares (no GPU): the cuts of a head's rows into per-CTA shares
are a partition, every share in use holds rows, and the bookkeeping the merge relies on is consistent."""
import numpy as np
import pytest

from paper_2607_11211_b200 import binding, build


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()


def collect(seq_lens, pos, max_seq, step, gm):
    used, shares = binding.attention_shares(seq_lens, pos, max_seq, step, gm)
    return used, shares


CASES = [
    ([1024], 4),                                    # batch 1, the benchmark's first step
    ([0], 4),                                       # empty cache: the new row only
    ([15], 4), ([16], 4), ([63], 4), ([64], 4),
    ([4095], 4),                                    # last free slot of a 4096-row cache
    ([300, 4000, 17, 2300, 1, 900, 2047, 3100], 4), # ragged batch of 8
    ([5, 5, 5, 5, 5, 5, 5, 5], 4),
    ([0, 0, 0], 4),
    ([2300] * 8, 4),
    ([100, 200, 300], 18),                          # few heads: large groups
    ([4000, 3], 32),
    ([7], 1),
]


@pytest.mark.parametrize("lens,gm", CASES)
@pytest.mark.parametrize("step", [0, 3])
def test_shares_partition_the_rows(lens, gm, step):
    max_seq = 4200
    used, shares = collect(lens, lens, max_seq, step, gm)
    rows = [L + step + 1 for L in lens]             # cached rows + the new row
    total = sum(rows)
    assert used == max(1, min(gm, total // 16))
    covered = {b: [] for b in range(len(lens))}
    for g, segs in enumerate(shares):
        if g >= used:
            assert segs == []
            continue
        assert segs, f"share {g} of {used} holds no rows"
        for (b, r0, r1, first, n) in segs:
            assert 0 <= r0 < r1 <= rows[b]
            assert first <= g < first + n           # the share is among the sequence's partials
            covered[b].append((r0, r1, g, first, n))
    for b, pieces in covered.items():
        pieces.sort()
        assert pieces[0][0] == 0 and pieces[-1][1] == rows[b]
        for (a0, a1, *_), (b0, b1, *_) in zip(pieces, pieces[1:]):
            assert a1 == b0                          # no gap, no overlap
        firsts = {p[3] for p in pieces}
        counts = {p[4] for p in pieces}
        assert len(firsts) == 1 and len(counts) == 1
        # the shares of a sequence are consecutive and exactly as many as every one of them says
        assert [p[2] for p in pieces] == list(range(pieces[0][3], pieces[0][3] + pieces[0][4]))


def test_the_share_with_the_new_row_is_the_lightest_at_batch_1():
    used, shares = collect([1024], [1024], 4096, 0, 4)
    sizes = [sum(r1 - r0 for (_, r0, r1, _, _) in s) for s in shares]
    assert used == 4 and sum(sizes) == 1025
    assert sizes[3] < min(sizes[:3])                 # the end of the sequence counts as extra rows
    assert max(sizes[:3]) - min(sizes[:3]) <= 1


def test_invalid_sequences_hold_no_rows():
    # a full cache (seq_len == max_seq) cannot take a new row: the sequence is skipped, the others are served
    used, shares = collect([4096, 100], [4096, 100], 4096, 0, 4)
    seqs = {b for s in shares for (b, *_rest) in s}
    assert seqs == {1}
    used, shares = collect([4096], [4096], 4096, 0, 4)
    assert used == 0 and all(s == [] for s in shares)


def test_bad_arguments_are_refused():
    with pytest.raises(binding.FasttpsError):
        binding.attention_shares([1] * 9, [1] * 9, 64, 0, 4)       # more than 8 sequences
    with pytest.raises(binding.FasttpsError):
        binding.attention_shares([1], [1], 64, 0, 33)              # group larger than the partial table


# ------------------------------------------------- the stand-alone attention kernel's share walk

def _check_walk(lens, heads, max_seq, n_cta):
    from paper_2607_11211_b200 import binding as fb
    lens = np.asarray(lens, np.int32)
    segs = fb.attention_walk(lens, lens, heads, max_seq, n_cta)
    valid = [(0 <= l < max_seq) for l in lens]
    rows = {(b, h): [] for b in range(len(lens)) if valid[b] for h in range(heads)}
    per_cta = {}
    for cta, b, h, r0, r1, first, n in segs:
        assert valid[b] and 0 <= h < heads and 0 <= r0 < r1 <= lens[b] + 1
        assert 1 <= n <= 32 and first <= cta < first + n          # 32 partial records per head, indexed cta - first
        rows[(b, h)].append((r0, r1, cta, first, n))
        per_cta[cta] = per_cta.get(cta, 0) + (r1 - r0)
    for (b, h), parts in rows.items():
        parts.sort()
        assert parts[0][0] == 0 and parts[-1][1] == lens[b] + 1, (b, h)
        assert all(p[1] == q[0] for p, q in zip(parts, parts[1:])), (b, h)       # the shares partition the head's rows
        assert len({(p[3], p[4]) for p in parts}) == 1                          # and agree on the head's CTAs ...
        assert [p[2] for p in parts] == list(range(parts[0][3], parts[0][3] + parts[0][4]))   # ... which all hold rows of it
    total = sum((l + 1) * heads for l, v in zip(lens, valid) if v)
    assert sum(per_cta.values()) == total
    if per_cta:
        assert max(per_cta.values()) - min(per_cta.values()) <= 1              # equal shares
        assert min(per_cta.values()) >= min(16, total)
    return max((p[0][4] for p in rows.values()), default=0), len(per_cta)


def test_attention_walk_partitions_every_head_into_equal_shares_within_the_record_limit():
    rng = np.random.default_rng(11)
    worst = 0
    for _ in range(300):
        batch = int(rng.integers(1, 9))
        heads = int(rng.choice([1, 2, 4, 8, 32]))
        lens = [int(rng.integers(0, 40)) if rng.random() < 0.5 else int(rng.integers(0, 5000)) for _ in range(batch)]
        span, _ = _check_walk(lens, heads, 5008, int(rng.choice([148, 132, 60, 16, 3])))
        worst = max(worst, span)
    assert worst <= 32
    # one long sequence among short ones on few heads: the cut count is held down by the record limit
    span, active = _check_walk([4999, 3, 0, 17], 1, 5008, 148)
    assert span <= 32 and active < 148
    # equal lengths and fewer heads than CTAs: a whole number of CTAs per head
    span, active = _check_walk([4095] * 8, 8, 4096, 148)
    assert active == 128 and span == 2
    # sequences that cannot be served (full cache) contribute no rows
    _check_walk([10, 4096, 7], 4, 4096, 148)
