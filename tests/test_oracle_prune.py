"""Pins for the one-shot magnitude pruning oracle (paper Sec. 5.2): library sorting on the group norms,
hand-made cases with known winners, invariances and the structure each scheme demands."""
import numpy as np
import pytest

import oracle
from paper_2012_00596_b200 import inputs


def bits(v, n):
    return [i for i in range(n) if (int(v) >> i) & 1]


def test_bp_equals_library_sort_of_group_norms():
    rng = inputs.rng_for(801)
    K, R, S, C, Mb, Nb, keep = 8, 3, 3, 12, 4, 6, 4
    w = rng.standard_normal((K, R, S, C))
    tm = oracle.prune_bp(w, Mb=Mb, Nb=Nb, keep=keep)
    assert tm.shape == (2, 2)
    for fb in range(2):
        for cb in range(2):
            blk = w[fb * Mb:(fb + 1) * Mb, :, :, cb * Nb:(cb + 1) * Nb].reshape(Mb, R * S, Nb)
            score = np.einsum("ftc,ftc->t", blk, blk)
            want = sorted(np.argsort(-score, kind="stable")[:keep].tolist())
            assert bits(tm[fb, cb], 9) == want


def test_bp_hand_made_winners_ties_and_extremes():
    w = np.zeros((2, 1, 4, 2))
    w[:, 0, 1, :] = 3.0            # tap 1: score 4 * 9 = 36
    w[0, 0, 3, 0] = -5.0           # tap 3: score 25
    w[1, 0, 0, 1] = 5.0            # tap 0: score 25 (tie with tap 3: the lower index wins)
    assert bits(oracle.prune_bp(w, Mb=2, Nb=2, keep=1)[0, 0], 4) == [1]
    assert bits(oracle.prune_bp(w, Mb=2, Nb=2, keep=2)[0, 0], 4) == [0, 1]
    assert bits(oracle.prune_bp(w, Mb=2, Nb=2, keep=3)[0, 0], 4) == [0, 1, 3]
    assert bits(oracle.prune_bp(w, Mb=2, Nb=2, keep=4)[0, 0], 4) == [0, 1, 2, 3]
    assert int(oracle.prune_bp(w, Mb=2, Nb=2, keep=0)[0, 0]) == 0
    # 1x1 blocks: every kernel keeps its own largest-magnitude taps (the paper's unstructured-like case)
    tm = oracle.prune_bp(w, Mb=1, Nb=1, keep=1)
    assert bits(tm[0, 0], 4) == [3] and bits(tm[1, 1], 4) == [0]


def test_bp_invariances():
    rng = inputs.rng_for(802)
    w = rng.standard_normal((16, 3, 3, 16))
    tm = oracle.prune_bp(w, Mb=8, Nb=4, keep=3)
    assert all(len(bits(v, 9)) == 3 for v in tm.ravel())
    assert np.array_equal(oracle.prune_bp(-2.5 * w, Mb=8, Nb=4, keep=3), tm)          # sign and scale do not matter
    # pruning by the mask and pruning again is a fixed point
    m = oracle.bp_element_mask(tm, 16, 16, 3, 3, 8, 4)
    assert np.array_equal(oracle.prune_bp(w * m, Mb=8, Nb=4, keep=3), tm)


def test_bb_equals_library_sort_and_structure():
    rng = inputs.rng_for(803)
    O, I, Bo, Bi = 16, 24, 8, 12
    w = rng.standard_normal((O, I))
    rk, ck = oracle.prune_bb(w, Bo=Bo, Bi=Bi, keep_rows=3, keep_cols=5)
    for bo in range(2):
        for bi in range(2):
            blk = w[bo * Bo:(bo + 1) * Bo, bi * Bi:(bi + 1) * Bi]
            assert bits(rk[bo, bi], Bo) == sorted(np.argsort(-(blk ** 2).sum(1), kind="stable")[:3].tolist())
            assert bits(ck[bo, bi], Bi) == sorted(np.argsort(-(blk ** 2).sum(0), kind="stable")[:5].tolist())
    m = oracle.bb_element_mask(rk, ck, O, I, Bo, Bi)
    assert int(m.sum()) == 4 * 3 * 5                                                 # rows x columns product per block


def test_bb_hand_made_and_ties():
    w = np.array([[1.0, 0.0, 2.0], [0.0, 3.0, 0.0], [2.0, 0.0, 1.0]])                 # row scores 5, 9, 5; column scores 5, 9, 5
    rk, ck = oracle.prune_bb(w, Bo=3, Bi=3, keep_rows=2, keep_cols=1)
    assert bits(rk[0, 0], 3) == [0, 1] and bits(ck[0, 0], 3) == [1]
    with pytest.raises(ValueError):
        oracle.prune_bb(w, Bo=3, Bi=3, keep_rows=4, keep_cols=1)


# ---- layer-wide budget (pruning rates such as 2.5x or 7x: per-block counts differ) ---------------

def _group_scores(w, Mb, Nb):
    K, R, S, C = w.shape
    blk = w.reshape(K // Mb, Mb, R * S, C // Nb, Nb)
    return np.einsum("aftbc,aftbc->abt", blk, blk)              # [fb, cb, tap]


def test_bp_global_equals_library_sort_of_all_group_norms():
    """Small integer weights make every score exact, so the order is the same in any summation order."""
    rng = inputs.rng_for(811)
    K, R, S, C, Mb, Nb = 16, 3, 3, 12, 4, 6
    w = rng.integers(-4, 5, size=(K, R, S, C)).astype(np.float64)
    score = _group_scores(w, Mb, Nb).reshape(-1)
    G = score.size
    for n_keep in (0, 1, 7, G * 2 // 5, G // 7, G - 1, G):      # 2.5x and 7x among them
        tm = oracle.prune_bp_global(w, Mb=Mb, Nb=Nb, n_keep=n_keep)
        want = np.zeros(G, dtype=bool)
        want[np.argsort(-score, kind="stable")[:n_keep]] = True
        got = np.array([[(int(v) >> t) & 1 for t in range(9)] for v in tm.ravel()], dtype=bool).reshape(-1)
        assert np.array_equal(got, want), n_keep
        assert int(got.sum()) == n_keep


def test_bp_global_hand_made_ties_and_nesting():
    # every group has the same score: the lowest group indices win, block after block, tap after tap
    w = np.ones((4, 1, 3, 4))
    tm = oracle.prune_bp_global(w, Mb=2, Nb=2, n_keep=7)          # 4 blocks x 3 taps
    assert [int(v) for v in tm.ravel()] == [0b111, 0b111, 0b001, 0]
    # one heavy tap in the last block beats everything; then the ties resume from the front
    w[3, 0, 2, 3] = 10.0
    tm = oracle.prune_bp_global(w, Mb=2, Nb=2, n_keep=2)
    assert [int(v) for v in tm.ravel()] == [0b001, 0, 0, 0b100]
    # nesting: a larger budget keeps a superset; scaling the weights changes nothing
    rng = inputs.rng_for(812)
    w = rng.standard_normal((8, 3, 3, 8))
    prev = np.zeros((4, 4), dtype=np.uint64)
    for n_keep in range(0, 4 * 4 * 9 + 1, 11):
        tm = oracle.prune_bp_global(w, Mb=2, Nb=2, n_keep=n_keep)
        assert np.all((tm & prev) == prev) and sum(bin(int(v)).count("1") for v in tm.ravel()) == n_keep
        assert np.array_equal(tm, oracle.prune_bp_global(4.0 * w, Mb=2, Nb=2, n_keep=n_keep))
        prev = tm
    counts = {bin(int(v)).count("1") for v in oracle.prune_bp_global(w, Mb=2, Nb=2, n_keep=58).ravel()}
    assert len(counts) > 1                                         # 2.5x: the blocks keep different numbers of taps


def test_bp_global_reduces_to_the_per_block_rule_when_blocks_are_alike():
    """If every block holds the same weights, the layer-wide order repeats block by block, and a budget of
    keep * blocks (with scores that differ inside a block) keeps the same `keep` taps in every block."""
    rng = inputs.rng_for(813)
    blk = rng.integers(1, 6, size=(2, 1, 5, 3)).astype(np.float64)
    blk[:, 0, :, :] *= np.arange(1, 6).reshape(1, 5, 1)           # distinct scores per tap
    w = np.tile(blk, (3, 1, 1, 2))                                 # 3 x 2 identical blocks
    per_block = oracle.prune_bp(w, Mb=2, Nb=3, keep=2)
    assert np.array_equal(oracle.prune_bp_global(w, Mb=2, Nb=3, n_keep=2 * 6), per_block)
