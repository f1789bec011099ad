"""Pins for the commit oracle: a hand-worked pass, and the exactness theorem (Theorem 1) on the toy
model: the per-row fill steps logged by committing speculative passes must be the sequential
decoder's own step indices, with the same tokens."""
import numpy as np
import pytest

import oracle
from oracle import commit as C
from oracle import theorem1 as T


def test_hand_worked_pass():
    # R = 5, mask = 9.  Path root -> 2 -> 3; node 1 is a rejected sibling.  The pass starts 4
    # sequential steps into the block.  Node 2 filled row 1, node 3 rows 0 and 4; U(node 3) = row 2.
    M = 9
    parent = [-1, 0, 0, 2]
    state = [[M, M, M, 6, M],
             [M, M, 8, 6, M],
             [M, 7, M, 6, M],
             [5, 7, M, 6, 4]]
    o = C.commit_accepted(parent, state, 3, [0, 0, 1, 0, 0], [-1, -1, 3, -1, -1], M, step_base=4)
    assert o["root"].tolist() == [5, 7, 3, 6, 4]
    assert o["fill_step"].tolist() == [5, 4, 6, -1, 5]
    assert o["step_base"] == 7 and o["n_masked"] == 0
    # nothing accepted: only U(root) is filled, one step taken
    o = C.commit_accepted(parent, state, 0, [0, 1, 0, 0, 0], [-1, 7, -1, -1, -1], M, step_base=4)
    assert o["root"].tolist() == [M, 7, M, 6, M] and o["fill_step"].tolist() == [-1, 4, -1, -1, -1]
    assert o["step_base"] == 5 and o["n_masked"] == 3
    # an accepted node that is already full takes no further step
    full = [[M, 1], [2, 1]]
    o = C.commit_accepted([-1, 0], full, 1, [0, 0], [-1, -1], M, step_base=0)
    assert o["root"].tolist() == [2, 1] and o["fill_step"].tolist() == [0, -1] and o["step_base"] == 1


def test_hand_worked_forest_and_kv_hand_over():
    # Two trees in one pass (Section 3.4): nodes 0-2 belong to the current block (root 0), nodes 3-5
    # to the next block (root 3); parents are forest indices.  R = 3, mask = 9.
    M = 9
    parent = [-1, 0, 1, -1, 3, 3]
    state = [[M, M, 1], [2, M, 1], [2, 3, 1],      # chain 0 -> 1 -> 2
             [M, M, M], [4, M, M], [M, 5, M]]      # root 3 with children 4 and 5
    # next block's tree: node 4 accepted (depth 1), U(node 4) = row 2 with token 7
    o = C.commit_accepted(parent, state, 4, [0, 0, 1], [-1, -1, 7], M, step_base=2, tree_root=3)
    assert o["root"].tolist() == [4, M, 7] and o["fill_step"].tolist() == [2, -1, 3]
    assert o["step_base"] == 4 and o["n_masked"] == 1
    # current block's tree: node 2 accepted (depth 2), already full
    o = C.commit_accepted(parent, state, 2, [0, 0, 0], [-1, -1, -1], M, step_base=0, tree_root=0)
    assert o["root"].tolist() == [2, 3, 1] and o["fill_step"].tolist() == [0, 1, -1] and o["step_base"] == 2
    # K/V hand-over: 2 sequences, 3 nodes of R = 2 rows, 1 head, d = 2; value = 100 s + 10 row + c
    draft = np.array([[[[100 * s + 10 * i + c for c in range(2)]] for i in range(6)] for s in range(2)], np.float32)
    got = C.gather_accepted_kv(draft, [2, 0], 2)
    assert got.shape == (2, 2, 1, 2)
    assert got[0].reshape(-1).tolist() == [40, 41, 50, 51]          # node 2 of sequence 0: rows 4, 5
    assert got[1].reshape(-1).tolist() == [100, 101, 110, 111]      # node 0 of sequence 1: rows 0, 1


@pytest.mark.parametrize("tau", [0.9, 1.5])
@pytest.mark.parametrize("mode", ["peek", "alg1", "heuristic"])
def test_committed_steps_are_the_sequential_steps(tau, mode):
    deep = 0
    for seed in range(25):
        model = T.ToyModel(seed)
        s = np.full(model.R, model.mask_id, np.int32)
        seq, final = T.sequential_decode(model, s, tau)
        rng = np.random.Generator(np.random.PCG64(seed))
        fill = np.full(model.R, -1, np.int32)
        base, prev = 0, None
        while (s == model.mask_id).any():
            peek = T.sequential_decode(model, s, tau)[0] if mode == "peek" else None
            if prev is None:
                c0, i0, p0, _ = T._score(model, s[None])
                prev = (c0[0], i0[0], p0[0])
            states, parent = T._draft(model, s, prev[0], prev[1], prev[2], mode, rng, tau, peek)
            conf, idx, prob, _ = T._score(model, states)
            acc = oracle.accept(np.asarray(parent, np.int32)[None], states[None], model.mask_id, conf[None],
                                idx[None, :, :, 0], tau, rule=0, search=seed % 2)
            node = int(acc["accepted_node"][0])
            o = C.commit_accepted(parent, states, node, acc["unmask_flag"][0], acc["unmask_tok"][0],
                                  model.mask_id, base)
            newly = o["fill_step"] >= 0
            assert (fill[newly] == -1).all()             # a row is filled once
            fill[newly] = o["fill_step"][newly]
            open_rows = bool((states[node] == model.mask_id).any())
            assert o["step_base"] == base + int(acc["accepted_len"][0]) + (1 if open_rows else 0)
            deep = max(deep, int(acc["accepted_len"][0]))
            s, base, prev = o["root"], o["step_base"], (conf[node], idx[node], prob[node])
        assert base == len(seq) and np.array_equal(s, final)
        for t, events in enumerate(seq):
            for r, tok in events:
                assert fill[r] == t and s[r] == tok
    if mode == "peek":
        assert deep >= 2
