"""Pins for the oracle's Topological Reordering (Eq. 5-6) and commit length (Algorithm 1)."""
import itertools

import numpy as np
import pytest

from oracle import wedlm_oracle as orc


def _all_patterns(W):
    return np.array(list(itertools.product([0, 1], repeat=W)), dtype=np.uint8)


@pytest.mark.parametrize("W", [1, 2, 3, 5, 8, 10])
def test_reorder_is_the_stable_partition_of_eq5_eq6(W):
    """Exhaustive over all 2^W fill patterns: perm is a permutation; the observed block comes
    first, each block ascending (Eq. 5); position ids keep the logical index (Eq. 6)."""
    pats = _all_patterns(W)
    P = np.full(len(pats), 37, np.int32)
    r = orc.reorder(pats, P)
    for b, f in enumerate(pats):
        perm = r["perm"][b].tolist()
        assert sorted(perm) == list(range(W))
        No = int(f.sum())
        assert r["n_filled"][b] == No
        obs, msk = perm[:No], perm[No:]
        assert all(f[j] == 1 for j in obs) and all(f[j] == 0 for j in msk)
        assert obs == sorted(obs) and msk == sorted(msk)
        assert (r["pos_ids"][b] - 37).tolist() == perm
        assert all(r["inv_perm"][b][perm[i]] == i for i in range(W))
        # commit length: leading run of filled slots read in logical order
        lead = 0
        while lead < W and f[lead]:
            lead += 1
        assert r["n_commit"][b] == lead
        # in-place commit property: the committed slots are the first physical rows, in order
        assert perm[:lead] == list(range(lead))
        # the (token, position) multiset is preserved
        toks = np.arange(100, 100 + W)
        pairs_logical = {(int(toks[j]), 37 + j) for j in range(W)}
        pairs_phys = {(int(toks[perm[i]]), int(r["pos_ids"][b][i])) for i in range(W)}
        assert pairs_logical == pairs_phys


def test_all_mask_and_all_filled_windows():
    W = 6
    r = orc.reorder(np.zeros((1, W), np.uint8), np.array([10]))
    assert r["perm"][0].tolist() == list(range(W)) and r["n_commit"][0] == 0 and r["n_filled"][0] == 0
    r = orc.reorder(np.ones((1, W), np.uint8), np.array([10]))
    assert r["perm"][0].tolist() == list(range(W)) and r["n_commit"][0] == W and r["n_filled"][0] == W
    assert r["pos_ids"][0].tolist() == list(range(10, 10 + W))


def test_short_window_treats_inactive_slots_as_trailing_masks():
    f = np.array([[1, 0, 1, 1, 1, 1]], np.uint8)
    r = orc.reorder(f, np.array([0]), window_len=np.array([3]))
    # slots 3.. are inactive even though their flag is set
    assert r["perm"][0].tolist() == [0, 2, 1, 3, 4, 5]
    assert r["n_filled"][0] == 2 and r["n_commit"][0] == 1


def test_worked_example_from_the_text():
    """Eq. 5-6 spelled out on a hand example: positions 1..6 (1-based in the paper, 0-based here
    as 0..5), observed set {0, 2, 5}: x~ = [x0, x2, x5, M, M, M], p~ = [0, 2, 5, 1, 3, 4]."""
    f = np.array([[1, 0, 1, 0, 0, 1]], np.uint8)
    r = orc.reorder(f, np.array([0]))
    assert r["pos_ids"][0].tolist() == [0, 2, 5, 1, 3, 4]
    assert r["n_commit"][0] == 1
