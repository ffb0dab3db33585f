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
