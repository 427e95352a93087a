"""Pins of the beam-selection oracle against things other than itself: a hand-worked example, brute force by
Python's own sort on tiny inputs (every candidate compared pairwise), and the properties that define a top-k."""
import itertools

import numpy as np

from oracle import select as osel


def test_hand_worked_example():
    # 2 beams x 3 codes.  Sums: beam 0: [-1.0, -3.0, -2.5]; beam 1 (score -0.5): [-2.5, -0.75, -4.5]
    bs = np.array([0.0, -0.5], np.float32)
    lp = np.array([[-1.0, -3.0, -2.5], [-2.0, -0.25, -4.0]], np.float32)
    par, code, sc = osel.select_beams(bs, lp, 4)
    # best: (1,1) -0.75, (0,0) -1.0, then the tie at -2.5 between flat index 2 = (0,2) and 3 = (1,0): smaller first
    assert par.tolist() == [1, 0, 0, 1]
    assert code.tolist() == [1, 0, 2, 0]
    assert sc.tolist() == [-0.75, -1.0, -2.5, -2.5]


def test_brute_force_on_tiny_inputs():
    rng = np.random.default_rng(7)
    for trial in range(200):
        W, C = int(rng.integers(1, 5)), int(rng.integers(1, 6))
        k = int(rng.integers(1, W * C + 1))
        # coarse values so that ties are frequent
        bs = (rng.integers(-3, 3, W) / 2).astype(np.float32)
        lp = (rng.integers(-4, 1, (W, C)) / 2).astype(np.float32)
        cands = [(float(np.float32(bs[p] + lp[p, c])), p * C + c) for p, c in itertools.product(range(W), range(C))]
        cands.sort(key=lambda t: (-t[0], t[1]))
        par, code, sc = osel.select_beams(bs, lp, k)
        assert [(p * C + c) for p, c in zip(par, code)] == [i for _, i in cands[:k]]
        assert sc.tolist() == [s for s, _ in cands[:k]]


def test_top_k_properties():
    rng = np.random.default_rng(11)
    W, C, k = 37, 64, 50
    bs = rng.normal(size=W).astype(np.float32)
    lp = np.log(rng.dirichlet(np.ones(C), size=W)).astype(np.float32)
    par, code, sc = osel.select_beams(bs, lp, k)
    s = (bs[:, None] + lp).astype(np.float32)
    assert np.all(np.diff(sc) <= 0)                                   # best first
    assert np.array_equal(sc, s[par, code])                           # scores are those of the chosen pairs
    flat = set((par.astype(int) * C + code).tolist())
    assert len(flat) == k                                             # no candidate twice
    rest = np.delete(s.reshape(-1), sorted(flat))
    assert rest.max() <= sc.min()                                     # nothing left out beats anything kept
    assert np.array_equal(np.sort(s.reshape(-1))[::-1][:k], sc)      # the multiset of kept scores is THE top k


def test_k_equal_to_all_candidates_is_a_full_sort_and_k_one_is_argmax():
    rng = np.random.default_rng(3)
    bs = rng.normal(size=5).astype(np.float32)
    lp = rng.normal(size=(5, 7)).astype(np.float32)
    par, code, sc = osel.select_beams(bs, lp, 35)
    assert sorted((par.astype(int) * 7 + code).tolist()) == list(range(35))
    p1, c1, s1 = osel.select_beams(bs, lp, 1)
    s = (bs[:, None] + lp).astype(np.float32)
    assert (int(p1[0]), int(c1[0])) == tuple(int(x) for x in np.unravel_index(np.argmax(s), s.shape))


def test_nan_ranks_last_infinities_and_signed_zero():
    bs = np.zeros(1, np.float32)
    lp = np.array([[np.nan, -np.inf, -0.0, 0.0, np.inf, np.nan, -1.0]], np.float32)
    par, code, sc = osel.select_beams(bs, lp, 7)
    assert code.tolist() == [4, 2, 3, 6, 1, 0, 5]     # +inf; the two zeros by index; -1; -inf; NaNs by index
