"""Pins for the oracle's decode rule and acceptance (Alg. 1 Phase 1; Eqs. 6-7;
Section 3.3) and for the exactness theorem on a toy model (Theorem 1)."""
import numpy as np
import pytest

import oracle
from oracle import theorem1 as T
from conftest import load_accept_cases

CASES = load_accept_cases()


@pytest.mark.parametrize("case", CASES, ids=[c["id"] for c in CASES])
def test_hand_worked_trees(case):
    cand = case["top1"] if case["topk"] is None else case["topk"]
    got = oracle.accept(case["parent"], case["state"], case["mask_id"], case["conf"], cand,
                        case["tau"], rule=case["rule"], search=case["search"], topk_m=case["topk_m"],
                        draft_prob=case["draft_prob"])
    e = case["expect"]
    assert got["edge_valid"][0].tolist() == e["edge_valid"]
    assert got["prefix_len"][0].tolist() == e["prefix_len"]
    assert int(got["accepted_node"][0]) == e["accepted_node"]
    assert int(got["accepted_len"][0]) == e["accepted_len"]
    assert int(got["n_new_tokens"][0]) == e["n_new_tokens"]
    assert got["unmask_flag"][0].tolist() == e["unmask_flag"]
    assert got["unmask_tok"][0].tolist() == e["unmask_tok"]


def test_tree_example_positions_12_18_24():
    # App. B: a 32-row root with children exploring positions 12, 18 and 24
    R, M = 32, 999
    root = np.arange(100, 100 + R, dtype=np.int32)
    root[[12, 18, 24]] = M
    kids = []
    for pos, t in ((12, 500), (18, 501), (24, 502)):
        c = root.copy()
        c[pos] = t
        kids.append(c)
    state = np.stack([root] + kids)[None]
    conf = np.full((1, 4, R), 0.99, np.float32)
    conf[0, 0, [12, 18, 24]] = [0.4, 0.6, 0.5]
    conf[0, 2, [12, 24]] = [0.95, 0.93]
    top1 = np.zeros((1, 4, R), np.int32)
    top1[0, 0, [12, 18, 24]] = [500, 501, 502]
    top1[0, 2, [12, 24]] = [600, 601]
    parent = np.array([[-1, 0, 0, 0]], np.int32)
    ex = oracle.accept(parent, state, M, conf, top1, 0.9, rule=0, search=0)
    assert ex["edge_valid"][0].tolist() == [1, 0, 1, 0]       # only position 18 is the next step
    assert int(ex["accepted_node"][0]) == 2 and int(ex["n_new_tokens"][0]) == 1
    assert np.flatnonzero(ex["unmask_flag"][0]).tolist() == [12, 24]
    assert ex["unmask_tok"][0][[12, 24]].tolist() == [600, 601]
    t1 = oracle.accept(parent, state, M, conf, top1, 0.9, rule=1, search=0)
    assert t1["edge_valid"][0].tolist() == [1, 1, 1, 1]       # each matches its row's top prediction
    assert int(t1["accepted_node"][0]) == 1


def _random_tree_case(rng, B=9, R=6, V=12):
    M = V
    parent = np.array([-1] + [int(rng.integers(0, b)) for b in range(1, B)], np.int32)
    conf = rng.random((B, R)).astype(np.float32)
    top1 = rng.integers(0, V, (B, R)).astype(np.int32)
    state = np.full((B, R), M, np.int32)
    fill = rng.random(R) < 0.3
    state[0, fill] = rng.integers(0, V, fill.sum())
    for b in range(1, B):
        p = parent[b]
        c = state[p].copy()
        flag, tok = oracle.decode_rule(state[p], M, conf[p], top1[p], 0.8)
        mode = rng.integers(0, 4)
        if mode <= 1:                       # exact continuation
            c[flag.astype(bool)] = tok[flag.astype(bool)]
        elif mode == 2:                     # top-1 token at an arbitrary masked row
            rows = np.flatnonzero(c == M)
            if len(rows):
                r = rows[rng.integers(len(rows))]
                c[r] = top1[p, r]
        else:                               # arbitrary token
            rows = np.flatnonzero(c == M)
            if len(rows):
                c[rows[0]] = rng.integers(0, V)
        state[b] = c
    return parent[None], state[None], M, conf[None], top1[None]


def test_invariants_on_random_trees():
    rng = np.random.default_rng(11)
    for _ in range(200):
        parent, state, M, conf, top1 = _random_tree_case(rng)
        res = {(r, s): oracle.accept(parent, state, M, conf, top1, 0.8, rule=r, search=s)
               for r in (0, 1) for s in (0, 1)}
        ex, t1 = res[(0, 0)]["edge_valid"][0], res[(1, 0)]["edge_valid"][0]
        assert ((t1 >= ex).all())                      # TOP1-valid is a superset of EXACT-valid
        for r in (0, 1):
            g, l = res[(r, 0)], res[(r, 1)]
            assert np.array_equal(g["edge_valid"], l["edge_valid"])
            assert np.array_equal(g["prefix_len"], l["prefix_len"])
            assert l["accepted_len"][0] >= g["accepted_len"][0]
            # the accepted node's whole path is valid
            for out in (g, l):
                b, n = int(out["accepted_node"][0]), 0
                while b > 0:
                    assert out["edge_valid"][0, b]
                    b, n = int(parent[0, b]), n + 1
                assert n == out["accepted_len"][0]
        # under EXACT all valid children of a node hold the same state; when no node has two
        # of them (no duplicate siblings) the valid path is unique and both searches agree
        B = parent.shape[1]
        dup = any(sum(1 for c in range(1, B) if parent[0, c] == p and ex[c]) > 1 for p in range(B))
        if not dup:
            assert res[(0, 0)]["accepted_node"][0] == res[(0, 1)]["accepted_node"][0]


@pytest.mark.parametrize("tau", [0.9, 1.5])
@pytest.mark.parametrize("mode", ["heuristic", "peek", "random"])
def test_theorem1_speculative_equals_sequential(tau, mode):
    deep = 0
    for seed in range(40):
        model = T.ToyModel(seed)
        s0 = np.full(model.R, model.mask_id, np.int32)
        seq, final = T.sequential_decode(model, s0, tau)
        traj, final2, n_forward, depth = T.speculative_decode(model, s0, tau, mode, seed,
                                                              search=seed % 2)
        assert traj == seq                       # same (position, token) events, same order
        assert np.array_equal(final, final2)     # 100 % token match
        assert n_forward <= len(seq)
        deep = max(deep, depth)
    if mode == "peek":
        assert deep == 3                          # whole draft paths do get accepted
    if mode == "random":
        assert deep <= 1


def test_generator_plan_matches_decode_rule():
    """The workload generator plants which rows a threshold decoder unmasks at
    every node; the oracle must find exactly those rows from the logits."""
    from paper_2608_27514_b200 import workloads as W
    for name in ("cfg1", "cfg2"):
        cfg = W.CONFIGS[name]
        vi = W.verify_inputs(cfg)
        conf, idx, prob, _ = oracle.confidence_topk(vi["logits"], cfg.k)
        S, B, R = cfg.S, cfg.B, cfg.R
        conf32 = conf.astype(np.float32).reshape(S, B, R)
        top1 = idx[:, 0].reshape(S, B, R)
        assert np.abs(conf - cfg.tau).min() > 1e-3
        for s in range(S):
            for b in range(B):
                flag, _ = oracle.decode_rule(vi["state"][s, b], vi["mask_id"], conf32[s, b],
                                             top1[s, b], cfg.tau)
                assert np.array_equal(flag, vi["plan"]["planted_u"][s, b])


# ------------------------------------------------------------------ relaxed tests (Section 3.3)
def _relaxed_case(rng, V=12, k=3):
    """A random tree whose children add tokens drawn from the parent's candidate lists, its
    arg-max or anywhere, over full logits so that every rule can be evaluated."""
    B, R, M = 9, 6, V
    parent = np.array([-1] + [int(rng.integers(0, b)) for b in range(1, B)], np.int32)
    logits = (rng.standard_normal((B, R, V)) * 2).astype(np.float32)
    order = np.argsort(-logits.astype(np.float64), axis=-1, kind="stable")
    topk = order[..., :k].astype(np.int32)
    z = logits.astype(np.float64)
    prob = np.exp(z - z.max(-1, keepdims=True))
    prob /= prob.sum(-1, keepdims=True)
    conf = prob.max(-1).astype(np.float32)
    state = np.full((B, R), M, np.int32)
    state[0, rng.random(R) < 0.3] = 1
    for b in range(1, B):
        c = state[parent[b]].copy()
        rows = np.flatnonzero(c == M)
        for r in rows[: int(rng.integers(1, 3))]:
            mode = rng.integers(0, 3)
            c[r] = topk[parent[b], r, 0] if mode == 0 else (topk[parent[b], r, rng.integers(0, k)] if mode == 1
                                                            else rng.integers(0, V))
        state[b] = c
    return parent[None], state[None], M, conf[None], topk[None], logits[None], prob[None]


def test_draft_token_prob_against_textbook_softmax():
    rng = np.random.default_rng(2)
    for _ in range(30):
        parent, state, M, conf, topk, logits, prob = _relaxed_case(rng)
        got = oracle.draft_token_prob(logits, parent, state, M)[0]
        B, R = state.shape[1:]
        for c in range(B):
            for r in range(R):
                p = parent[0, c]
                added = c > 0 and state[0, p, r] == M and state[0, c, r] != M
                want = prob[0, p, r, state[0, c, r]] if added else 0.0
                assert abs(got[c, r] - want) <= 1e-15


def test_draft_token_prob_closed_forms():
    # uniform logits give 1/V; the probabilities of all V possible drafts of one row sum to 1
    V, M = 7, 7
    parent = np.array([[-1] + [0] * V], np.int32)
    state = np.full((1, V + 1, 2), M, np.int32)
    state[0, 1:, 1] = np.arange(V)              # child t drafts token t at row 1
    rng = np.random.default_rng(0)
    logits = rng.standard_normal((1, V + 1, 2, V)).astype(np.float32)
    got = oracle.draft_token_prob(logits, parent, state, M)[0]
    assert abs(got[1:, 1].sum() - 1.0) < 1e-14 and (got[:, 0] == 0).all() and (got[0] == 0).all()
    got = oracle.draft_token_prob(np.full_like(logits, 3.25), parent, state, M)[0]
    assert np.allclose(got[1:, 1], 1.0 / V, rtol=0, atol=1e-16)
    # a token outside the vocabulary has no probability
    state[0, 3, 1] = V + 5
    assert oracle.draft_token_prob(logits, parent, state, M + 100)[0][3, 1] == 0.0


def test_relaxed_rules_order_and_reductions():
    rng = np.random.default_rng(7)
    seen = set()
    for _ in range(200):
        parent, state, M, conf, topk, logits, prob = _relaxed_case(rng)
        k = topk.shape[-1]
        dp = oracle.draft_token_prob(logits, parent, state, M).astype(np.float32)
        run = lambda rule, m=1, tau=0.8: oracle.accept(parent, state, M, conf, topk, tau, rule=rule, search=1,
                                                       topk_m=m, draft_prob=dp)
        ev = {("top1",): run(1)["edge_valid"][0]}
        for m in range(1, k + 1):
            ev[("topk", m)] = run(2, m)["edge_valid"][0]
        # membership in the first candidate alone is the top-1 test; wider lists only add edges
        assert np.array_equal(ev[("topk", 1)], ev[("top1",)])
        for m in range(1, k):
            assert (ev[("topk", m + 1)] >= ev[("topk", m)]).all()
        # a token more probable than 1/2 is the arg-max, so above tau >= 1/2 PROB implies TOP1;
        # PROB edges shrink as tau grows and vanish at tau = 1
        pr = {tau: run(3, tau=tau)["edge_valid"][0] for tau in (0.5, 0.8, 1.0)}
        assert (ev[("top1",)] >= pr[0.5]).all() and (pr[0.5] >= pr[0.8]).all()
        assert pr[1.0][1:].sum() == 0
        # brute force of the PROB rule from the textbook probabilities
        B, R = state.shape[1:]
        for c in range(1, B):
            p = parent[0, c]
            rows = [r for r in range(R) if state[0, p, r] == M and state[0, c, r] != M]
            want = bool(rows) and all(np.float32(prob[0, p, r, state[0, c, r]]) > np.float32(0.8) for r in rows)
            assert bool(pr[0.8][c]) == want
            seen.add(want)
    assert seen == {True, False}


def test_parent_outside_the_tree_is_an_invalid_edge():
    parent = np.array([[-1, 0, 5, 2, -3]], np.int32)
    state = np.array([[[9, 9], [1, 9], [1, 9], [1, 2], [1, 9]]], np.int32)
    conf = np.full((1, 5, 2), 0.95, np.float32)
    top1 = np.array([[[1, 2]] * 5], np.int32)
    o = oracle.accept(parent, state, 9, conf, top1, 0.9, rule=1, search=1)
    assert o["edge_valid"][0].tolist() == [1, 1, 0, 1, 0]
    assert o["prefix_len"][0].tolist() == [0, 1, 0, 0, 0]      # node 3 hangs off the orphan node 2
    assert o["accepted_node"][0] == 1
