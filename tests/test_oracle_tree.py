"""Pins for the oracle's draft-tree construction (Alg. 1 Phase 2; Section 3.2).  The expected trees
below were worked out by hand from the reading stated in the oracle's source; the invariants hold
for any reading in which a child is its parent plus one candidate from the pool."""
import itertools

import numpy as np
import pytest

import oracle
from oracle import theorem1 as T

M = 99


def test_hand_worked_w2d2_with_three_children():
    # pool (row: (token, prob)...): row0 (10,.5) (11,.3); row2 (20,.6) (21,.2); row3 (30,.4) (31,.35)
    root = np.array([M, 5, M, M], np.int32)
    idx = np.array([[10, 11], [0, 0], [20, 21], [30, 31]], np.int32)
    pr = np.array([[.5, .3], [.9, .05], [.6, .2], [.4, .35]], np.float32)
    n, parent, state, prob = oracle.build_draft_tree(root, M, idx, pr, 2, 2, 4)   # W2D2(3): 3 child blocks
    assert n == 4
    # level 1: the two best pool entries (.6 at row 2, .5 at row 0); level 2: node 1 would add (.5),
    # node 2 would add (.6): the more confident child comes first and the budget ends there
    assert parent.tolist() == [-1, 0, 0, 2]
    assert state.tolist() == [[M, 5, M, M], [M, 5, 20, M], [10, 5, M, M], [10, 5, 20, M]]
    assert np.allclose(prob, [1.0, 0.6, 0.5, 0.6])


def test_tree_example_positions_12_18_24():
    # App. B: root with low-confidence positions 12, 18, 24; k = 3 children explore them
    R, k = 32, 3
    root = np.arange(100, 100 + R, dtype=np.int32)
    root[[12, 18, 24]] = M
    idx = np.zeros((R, k), np.int32)
    pr = np.zeros((R, k), np.float32)
    pr[:, 0] = 0.99                                  # filled rows: never in the pool whatever they score
    for row, t, p in ((12, 500, .40), (18, 501, .60), (24, 502, .50)):
        idx[row] = [t, t + 10, t + 20]
        pr[row] = [p, .05, .01]
    n, parent, state, prob = oracle.build_draft_tree(root, M, idx, pr, 3, 1, 4)
    assert n == 4 and parent.tolist() == [-1, 0, 0, 0]
    assert [int(np.flatnonzero(state[b] != root)[0]) for b in (1, 2, 3)] == [18, 24, 12]   # by confidence
    assert [int(state[1][18]), int(state[2][24]), int(state[3][12])] == [501, 502, 500]


def test_size_arithmetic_of_section_3_2():
    rng = np.random.default_rng(0)
    R, k = 32, 3
    root = np.full(R, M, np.int32)
    idx = rng.integers(0, 90, (R, k)).astype(np.int32)
    pr = rng.random((R, k)).astype(np.float32)
    # W = 3, D = 3: at most W*D = 9 drafts (not 3^3 = 27)
    n, parent, _, _ = oracle.build_draft_tree(root, M, idx, pr, 3, 3, 64)
    assert n == 1 + 9
    depth = [0] * n
    for b in range(1, n):
        depth[b] = depth[parent[b]] + 1
    assert [depth.count(d) for d in (1, 2, 3)] == [3, 3, 3]
    # only the root branches (hybrid expansion): deeper nodes have at most one child
    for p in range(1, n):
        assert sum(1 for b in range(1, n) if parent[b] == p) <= 1
    # the budget cuts the tree: W3D3(6) keeps six children
    assert oracle.build_draft_tree(root, M, idx, pr, 3, 3, 7)[0] == 7


def test_invariants_and_brute_force_level_one():
    rng = np.random.default_rng(5)
    for trial in range(200):
        R, k = int(rng.integers(2, 12)), int(rng.integers(1, 5))
        W, D, B = int(rng.integers(1, 5)), int(rng.integers(1, 4)), int(rng.integers(1, 12))
        root = np.where(rng.random(R) < 0.6, M, rng.integers(0, 50, R)).astype(np.int32)
        idx = rng.integers(0, 50, (R, k)).astype(np.int32)
        pr = (rng.integers(1, 40, (R, k)) / 40.0).astype(np.float32)      # coarse: many ties
        pr = -np.sort(-pr, axis=1)                                         # ranks are sorted within a row
        n, parent, state, prob = oracle.build_draft_tree(root, M, idx, pr, W, D, B)
        assert 1 <= n <= min(B, 1 + W * D) and parent[0] == -1 and (state[0] == root).all()
        for b in range(1, n):
            p = parent[b]
            assert 0 <= p < b
            diff = np.flatnonzero(state[b] != state[p])
            assert len(diff) == 1 and state[p][diff[0]] == M                # one fill at a masked row
            r = diff[0]
            assert state[b][r] in idx[r] and prob[b] in pr[r]               # taken from that row's pool
        for b in range(n, B):                                               # unused slots: copies of the root
            assert parent[b] == 0 and (state[b] == root).all()
        # level 1 = the best min(k, W, budget) pool entries in (prob desc, row asc, rank asc) order
        pool = sorted(((-pr[r, j], r, j) for r in range(R) if root[r] == M for j in range(k)))
        lvl1 = [b for b in range(1, n) if parent[b] == 0]
        want = pool[:min(k, W, B - 1)]
        assert len(lvl1) == len(want)
        for b, (negp, r, j) in zip(lvl1, want):
            assert state[b][r] == idx[r, j] and prob[b] == -negp
        # siblings and levels are listed in descending draft confidence
        assert all(prob[lvl1[i]] >= prob[lvl1[i + 1]] for i in range(len(lvl1) - 1))


@pytest.mark.parametrize("tau", [0.9, 1.5])
def test_theorem1_holds_with_this_drafter(tau):
    # exactness does not depend on the drafter (Theorem 1): the Alg. 1 trees only change how many
    # forward passes are needed
    saved = 0
    for seed in range(30):
        model = T.ToyModel(seed)
        s0 = np.full(model.R, model.mask_id, np.int32)
        seq, final = T.sequential_decode(model, s0, tau)
        traj, final2, n_forward, _ = T.speculative_decode(model, s0, tau, "alg1", seed)
        assert traj == seq and np.array_equal(final, final2)
        saved += len(seq) - n_forward
    assert saved > 0
