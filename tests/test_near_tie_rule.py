"""The near-tie rule used on inputs without planted margins (tests/helpers.py), checked on the CPU with
hand-built cases: a difference inside the band passes, the same difference outside it fails."""
import numpy as np
import pytest
import torch

from helpers import check_merge_unplanted, check_topk_unplanted


def test_topk_band_accepts_a_swap_at_the_cut_only():
    s = np.array([0.9, 0.50004, 0.5, 0.1, 0.8])            # cut between 0.50004 and 0.5 when k = 3
    assert check_topk_unplanted(np.array([0, 1, 4]), s, 3) == 0
    assert check_topk_unplanted(np.array([0, 2, 4]), s, 3) == 2      # 4e-5 apart: either may survive
    with pytest.raises(AssertionError):
        check_topk_unplanted(np.array([0, 3, 4]), s, 3)              # 0.1 is nowhere near the cut
    with pytest.raises(AssertionError):
        check_topk_unplanted(np.array([0, 1]), s, 3)                 # wrong count
    s2 = np.array([0.9, 0.51, 0.5, 0.1, 0.8])
    with pytest.raises(AssertionError):
        check_topk_unplanted(np.array([0, 2, 4]), s2, 3)             # a 1e-2 margin is not a near-tie


def test_merge_band_accepts_the_second_best_slot_only_when_it_is_as_good():
    e = np.eye(4)
    # token 2 is (almost) equally close to kept tokens 0 and 1; token 3 clearly belongs to token 1
    x = np.stack([e[0], e[1], e[0] + (1 - 2e-5) * e[1], 0.1 * e[0] + e[1]])
    kept = np.array([0, 1])

    def run(assign):
        a = np.asarray(assign)
        m = np.stack([x[a == s].mean(axis=0) for s in range(2)])
        c = np.array([(a == s).sum() for s in range(2)], dtype=np.int32)
        return check_merge_unplanted(x, 0, kept, torch.from_numpy(m), torch.from_numpy(a.astype(np.int32)),
                                     torch.from_numpy(c), "f32")
    assert run([0, 1, 0, 1]) == 0          # the oracle's own choice
    assert run([0, 1, 1, 1]) == 1          # the near-tie fell the other way: accepted and counted
    with pytest.raises(AssertionError):
        run([0, 1, 0, 0])                  # token 3 is no near-tie
