"""GPU parity of the relaxed acceptance tests (Section 3.3: the top-k-membership and probability-above-tau alternatives) against
the oracle: hand-worked trees, random trees scored from full logits through the vocabulary pass,
strictness of the probability test, and the two-tree form."""
import numpy as np
import pytest
import torch

import oracle
from oracle import interblock
from conftest import load_accept_cases
from paper_2608_27514_b200 import binding as B

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
CASES = [c for c in load_accept_cases() if c["topk"] is not None]


def _t(a, dt):
    return None if a is None else torch.as_tensor(np.ascontiguousarray(a), dtype=dt, device=DEV)


def _gpu_relaxed(parent, state, n_cur, M, conf, topk, topk_m, logits, lse, tau, rule, search):
    """parent/state/conf/topk: numpy or device tensors; logits/lse: device tensors or None."""
    dev = lambda a, dt: a if torch.is_tensor(a) else _t(a, dt)
    S, Bn, R = state.shape
    e = lambda shape, dt, v=0: torch.full(shape, v, dtype=dt, device=DEV)
    out = dict(edge_valid=e((S, Bn), torch.uint8), prefix_len=e((S, Bn), torch.int32),
               accepted_node=e((2, S), torch.int32), accepted_len=e((2, S), torch.int32),
               n_new_tokens=e((2, S), torch.int32), unmask_flag=e((2, S, R), torch.uint8),
               unmask_tok=e((2, S, R), torch.int32, -1), draft_prob=e((S, Bn, R), torch.float32, -7.0))
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    B.tsd_accept_relaxed(dev(parent, torch.int32), dev(state, torch.int32), n_cur, M, dev(conf, torch.float32),
                         dev(topk, torch.int32), topk_m, logits, lse, tau, rule, search, status=status, **out)
    torch.cuda.synchronize()
    return {k: v.cpu().numpy() for k, v in out.items()}, status


@pytest.mark.parametrize("case", CASES, ids=[c["id"] for c in CASES])
def test_relaxed_hand_worked_trees(case):
    # the golden cases give the drafted-token probabilities directly; feed them to the kernel as
    # logit = ln(p) with a zero log-sum-exp.  A probability written as exactly tau cannot pass
    # through exp() bit for bit, so it is moved just below (strictness has its own test below).
    state, parent = case["state"], case["parent"]
    S, Bn, R = state.shape
    V = 16
    dp = case["draft_prob"].astype(np.float64).copy()
    dp[dp == np.float32(case["tau"])] -= 1e-3
    logits = np.full((S, Bn, R, V), -30.0, np.float32)
    for c in range(1, Bn):
        p = parent[0, c]
        for r in range(R):
            if state[0, p, r] == case["mask_id"] and state[0, c, r] != case["mask_id"]:
                logits[0, p, r, state[0, c, r]] = np.log(dp[0, c, r]) if dp[0, c, r] > 0 else -30.0
    lse = torch.zeros(S * Bn * R, dtype=torch.float32, device=DEV)
    got, status = _gpu_relaxed(parent, state, Bn, case["mask_id"], case["conf"], case["topk"], case["topk_m"],
                               _t(logits.reshape(-1, V), torch.float32), lse, case["tau"], case["rule"],
                               case["search"])
    ex = case["expect"]
    for key in ("edge_valid", "prefix_len"):
        assert got[key][0].tolist() == ex[key], key
    for key in ("unmask_flag", "unmask_tok"):
        assert got[key][0, 0].tolist() == ex[key], key
    for key in ("accepted_node", "accepted_len", "n_new_tokens"):
        assert int(got[key][0, 0]) == ex[key], key
    added = (state[0, np.maximum(parent[0], 0)] == case["mask_id"]) & (state[0] != case["mask_id"])
    added[0] = False
    assert np.allclose(got["draft_prob"][0][added], dp[0][added], rtol=1e-5, atol=0)
    assert (got["draft_prob"][0][~added] == 0).all()
    assert B.tsd_check_status(status) == B.TSD_OK


def _random_pass(rng, S, Bn, n_cur, R, V, k, dtype):
    """Random forest whose children add candidate tokens of their parents, scored from full logits."""
    M = V
    parent = np.empty((S, Bn), np.int32)
    for b in range(Bn):
        lo = 0 if b < n_cur else n_cur
        parent[:, b] = -1 if b == lo else rng.integers(lo, b, S)
    logits = rng.standard_normal((S, Bn, R, V)).astype(np.float32)
    peak = rng.integers(0, V, (S, Bn, R))
    boost = rng.choice([0.0, 3.0, 6.0, 9.0], (S, Bn, R)).astype(np.float32)
    np.put_along_axis(logits, peak[..., None], (np.take_along_axis(logits, peak[..., None], -1) + boost[..., None]), -1)
    ld = (V + 7) // 8 * 8                                   # rows start on 16-byte boundaries
    lt = torch.zeros((S * Bn * R, ld), dtype=dtype, device=DEV)[:, :V]
    lt.copy_(torch.from_numpy(logits).reshape(-1, V))
    logits = lt.float().cpu().numpy().reshape(S, Bn, R, V)  # what both sides see
    conf, idx, prob, lse = oracle.confidence_topk(logits.reshape(-1, V), k)
    idx = idx.reshape(S, Bn, R, k)
    conf32 = conf.reshape(S, Bn, R).astype(np.float32)
    state = np.full((S, Bn, R), M, np.int32)
    for s in range(S):
        for b in range(Bn):
            p = parent[s, b]
            if p < 0:
                fill = rng.random(R) < 0.3
                state[s, b, fill] = rng.integers(0, V, fill.sum())
                continue
            c = state[s, p].copy()
            rows = np.flatnonzero(c == M)
            mode = rng.integers(0, 4)
            if mode == 0:
                flag, tok = oracle.decode_rule(state[s, p], M, conf32[s, p], idx[s, p, :, 0], 0.8)
                c[flag.astype(bool)] = tok[flag.astype(bool)]
            else:
                for r in rows[rng.permutation(len(rows))[: int(rng.integers(1, 3))]]:
                    c[r] = idx[s, p, r, rng.integers(0, k)] if mode < 3 else rng.integers(0, V)
            state[s, b] = c
    return parent, state, M, lt, logits, conf32, idx


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("Bn,n_cur,R,V,k", [(12, 12, 32, 700, 3), (14, 10, 32, 1500, 4), (20, 7, 64, 333, 2)])
def test_relaxed_rules_from_logits_match_oracle(dtype, Bn, n_cur, R, V, k):
    rng = np.random.default_rng(Bn * 100 + V)
    S = 6
    parent, state, M, lt, logits, conf32, idx = _random_pass(rng, S, Bn, n_cur, R, V, k, dtype)
    # vocabulary pass on the device: confidence, candidates and log-sum-exp stay there
    rows = S * Bn * R
    d_conf = torch.empty(rows, dtype=torch.float32, device=DEV)
    d_idx = torch.empty((rows, k), dtype=torch.int32, device=DEV)
    d_prob = torch.empty((rows, k), dtype=torch.float32, device=DEV)
    d_lse = torch.empty(rows, dtype=torch.float32, device=DEV)
    ws = torch.empty(max(B.tsd_confidence_topk_workspace_bytes(rows, V, k), 16), dtype=torch.uint8, device=DEV)
    B.tsd_confidence_topk(lt, k, d_conf, d_idx, d_prob, d_lse, ws)
    dp = oracle.draft_token_prob(logits, parent, state, M)
    dp32 = dp.astype(np.float32)
    added = dp > 0
    # a threshold that no confidence and no drafted-token probability comes within 1e-4 of:
    # fp32 on the device and fp64 in the oracle then take the same decisions
    tau = next(t for t in (0.8, 0.77, 0.83, 0.71, 0.9) if np.abs(conf32 - t).min() > 1e-4
               and np.abs(dp[added] - t).min() > 1e-4)
    seen = set()
    for rule in (0, 1, 2, 3):
        for search in (0, 1):
            m = k if rule == 2 else 1
            ref = interblock.joint_accept(parent, state, n_cur, M, conf32, idx, tau, rule, search, m, dp32)
            got, status = _gpu_relaxed(parent, state, n_cur, M, d_conf.view(S, Bn, R), d_idx.view(S, Bn, R, k), m,
                                       lt, d_lse, tau, rule, search)
            trees = 2 if n_cur < Bn else 1
            for key, val in ref.items():
                g = got[key] if key in ("edge_valid", "prefix_len") else got[key][:trees]
                v = val if key in ("edge_valid", "prefix_len") else val[:trees]
                assert np.array_equal(g, v), (key, rule, search)
            assert np.abs(got["draft_prob"] - dp).max() <= 1e-5
            assert (got["draft_prob"][~added] == 0).all()
            assert B.tsd_check_status(status) == B.TSD_OK
            seen.add((rule, int(ref["edge_valid"][:, 1:].sum())))
    counts = {r: n for r, n in seen}
    assert counts[0] <= counts[1] <= counts[2] and 0 < counts[3] and counts[0] < counts[2]


def test_prob_rule_is_strict_and_ignores_tokens_outside_the_vocabulary():
    M, V = 50, 8
    parent = np.array([[-1, 0, 0, 0]], np.int32)
    state = np.full((1, 4, 32), M, np.int32)
    state[0, 1, 3] = 2            # drafted with probability exactly 1 (logit - lse = 0)
    state[0, 2, 5] = 4            # probability exp(-1)
    state[0, 3, 7] = V + 3        # not a token
    logits = np.zeros((4 * 32, V), np.float32)
    logits[5, 4] = -1.0
    lse = torch.zeros(4 * 32, dtype=torch.float32, device=DEV)
    conf = np.zeros((1, 4, 32), np.float32)
    topk = np.zeros((1, 4, 32, 1), np.int32)
    run = lambda tau: _gpu_relaxed(parent, state, 4, M, conf, topk, 1, _t(logits, torch.float32), lse, tau,
                                   B.TSD_ACCEPT_PROB, 0)[0]
    got = run(1.0)
    assert got["edge_valid"][0].tolist() == [1, 0, 0, 0]          # 1.0 is not above 1.0
    assert got["draft_prob"][0, 1, 3] == 1.0 and got["draft_prob"][0, 3, 7] == 0.0
    got = run(np.nextafter(np.float32(1.0), np.float32(0.0)))
    assert got["edge_valid"][0].tolist() == [1, 1, 0, 0]
    got = run(0.3)
    assert got["edge_valid"][0].tolist() == [1, 1, 1, 0]
    assert abs(got["draft_prob"][0, 2, 5] - np.exp(-1.0)) < 1e-6


def test_relaxed_argument_checks():
    p = _t(np.zeros(64, np.int32), torch.int32)
    f = torch.zeros(64, dtype=torch.float32, device=DEV)
    outs = dict(edge_valid=p, prefix_len=p, accepted_node=p, accepted_len=p, n_new_tokens=p, unmask_flag=p,
                unmask_tok=p)
    st = p[:32].view(1, 1, 32)
    for kw in (dict(rule=B.TSD_ACCEPT_PROB, logits=None),           # PROB needs the logits
               dict(rule=B.TSD_ACCEPT_TOPK, logits=None, topk_m=2),  # more candidates than the list holds
               dict(rule=7, logits=None)):
        with pytest.raises(B.TsdError) as ei:
            B.tsd_accept_relaxed(p[:1].view(1, 1), st, 1, 9, f[:32].view(1, 1, 32), st, kw.get("topk_m", 1),
                                 kw["logits"], None, 0.9, kw["rule"], 0, **outs)
        assert ei.value.code == B.TSD_ERR_INVALID_ARG
