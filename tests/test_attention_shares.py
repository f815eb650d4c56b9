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
