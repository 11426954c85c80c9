"""Pins for the oracle's pseudo-trajectory functions (Sec. 3.1): the recorded unmask order and the
noisy-sequence equation, against a worked example written out by hand, closed forms for special
trajectories, brute force over all small cases and the one-token-per-step decoder."""
import itertools
import math
from fractions import Fraction

import numpy as np
import pytest

from oracle import d3_oracle as o
from paper_2601_07568_b200 import synth_inputs as si

MASK = 99


def test_worked_example_by_hand():
    """n = 8, tokens 10..17, unmask order (positions from 1): 3, 1, 2, 4, 7, 5, 8, 6.
    Window s = 2, k = 4, t = 1/2: state T_{2 + 2} = T_4 has positions 3, 1, 2, 4 unmasked.
    i <= 2 keep; i in 3..6: position 3 and 4 unmasked in T_4, 5 and 6 masked; i > 6 masked."""
    y = np.arange(10, 18)
    order = [3, 1, 2, 4, 7, 5, 8, 6]
    rank = np.zeros(8, dtype=int)
    for step, pos in enumerate(order, start=1):
        rank[pos - 1] = step
    m = o.ceil_ratio(4, 1, 2)
    assert m == 2
    got = o.noisy_sequence(y, rank, s=2, k=4, m=m, mask_id=MASK)
    assert got.tolist() == [10, 11, 12, 13, MASK, MASK, MASK, MASK]
    # same window, t = 1: T_6 additionally has 7 and 5 unmasked; 7 lies beyond the window and stays masked
    got = o.noisy_sequence(y, rank, s=2, k=4, m=o.ceil_ratio(4, 1, 1), mask_id=MASK)
    assert got.tolist() == [10, 11, 12, 13, 14, MASK, MASK, MASK]
    # window at the start, t = 0: T_0 is all masks, nothing before the window
    assert o.noisy_sequence(y, rank, s=0, k=8, m=0, mask_id=MASK).tolist() == [MASK] * 8
    # s = 1, k = 3, m = 1: T_2 = {3, 1}: position 1 kept (i <= s), 2 masked (rank 3), 3 kept, 4 masked, rest masked
    assert o.noisy_sequence(y, rank, s=1, k=3, m=1, mask_id=MASK).tolist() == [10, MASK, 12, MASK, MASK, MASK, MASK, MASK]
    # the states themselves
    T = o.trajectory_states(y, rank, MASK)
    assert T.shape == (9, 8) and T[0].tolist() == [MASK] * 8 and T[8].tolist() == y.tolist()
    assert T[3].tolist() == [10, 11, 12, MASK, MASK, MASK, MASK, MASK]


@pytest.mark.parametrize("k,num,den", [(0, 1, 2), (5, 0, 1), (5, 1, 1), (32, 4, 5), (7, 1, 3), (32, 1, 32), (9, 2, 3)])
def test_ceil_ratio(k, num, den):
    assert o.ceil_ratio(k, num, den) == math.ceil(Fraction(k * num, den))


def test_left_to_right_trajectory_is_a_prefix():
    """If the teacher decodes strictly left to right, T_j is the first j tokens, so the noisy sequence
    is y up to max(s, min(s + m, s + k)) followed by masks: exactly k - m masks inside the window."""
    n = 12
    y = np.arange(1, n + 1)
    rank = np.arange(1, n + 1)
    for s, k in [(0, 4), (3, 5), (8, 4), (5, 0)]:
        for m in range(k + 1):
            got = o.noisy_sequence(y, rank, s, k, m, MASK)
            keep = s + m
            assert got[:keep].tolist() == y[:keep].tolist() and np.all(got[keep:] == MASK)
            assert int((got[s:s + k] == MASK).sum()) == k - m


def test_all_small_cases_against_rank_comparison():
    """Brute force: every permutation order of n = 5 and every (s, k, m): position i (from 1) keeps its
    token iff i <= s, or i <= s + k and it was unmasked at a step <= s + m."""
    n = 5
    y = np.arange(1, n + 1) * 7
    checked = 0
    for perm in itertools.permutations(range(1, n + 1)):
        rank = np.asarray(perm)
        for s in range(n + 1):
            for k in range(n - s + 1):
                for m in range(k + 1):
                    got = o.noisy_sequence(y, rank, s, k, m, MASK)
                    for i in range(1, n + 1):
                        keep = i <= s or (i <= s + k and rank[i - 1] <= s + m)
                        assert got[i - 1] == (y[i - 1] if keep else MASK)
                    checked += 1
    assert checked > 4000


def test_masks_shrink_as_the_step_grows_and_edges():
    rng = np.random.default_rng(4)
    n = 32
    y = rng.integers(0, 90, size=n)
    rank = rng.permutation(n) + 1
    prev = None
    for m in range(0, 17):
        got = o.noisy_sequence(y, rank, 8, 16, m, MASK)
        masked = got == MASK
        assert not masked[:8].any() and masked[24:].all()
        if prev is not None:
            assert not np.any(masked & ~prev)          # never masks something the smaller step had unmasked
        prev = masked
    assert np.array_equal(o.noisy_sequence(y, rank, n, 0, 0, MASK), y)       # window behind the response: clean
    # a step index beyond the trajectory means its last state
    assert np.array_equal(o.noisy_sequence(y, rank, 20, 12, 12, MASK), y)


def test_rank_of_a_threshold_one_run_is_the_one_token_per_step_order():
    """The extraction run: at threshold 1 every step commits exactly the most confident masked position,
    so the ranks are a permutation of 1..n that replays the separately written sequential decoder."""
    w = si.WORKLOADS["c1"]
    model = o.model_from_shape(w.model, si.gen_weights(w.model), dtype=np.float64)
    ids, lens = si.gen_prompts(w)
    prompt = ids[0, :lens[0]]
    res = model.generate(prompt, w.gen_len, w.block, 1.0)
    rank = o.trajectory_rank(res["commit_step"], w.block)
    assert sorted(rank.tolist()) == list(range(1, w.gen_len + 1))
    tokens, order = model.sequential_decode(prompt, w.gen_len, w.block)
    assert np.array_equal(tokens, res["tokens"])
    assert np.array_equal(rank[order], np.arange(1, w.gen_len + 1))
    # several tokens per step share a rank, blocks keep their order
    res2 = model.generate(prompt, w.gen_len, w.block, 0.05)
    rank2 = o.trajectory_rank(res2["commit_step"], w.block)
    B = w.block
    for j in range(1, w.gen_len // B):
        assert rank2[j * B:(j + 1) * B].min() == rank2[(j - 1) * B:j * B].max() + 1
    assert rank2.max() == res2["n_denoise"]
