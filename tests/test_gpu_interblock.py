"""GPU parity of the inter-block variant (Section 3.4, Eq. 3, App. D) against the oracle: joint
visibility bitsets and the dense mask they give, the trigger, attention under the joint mask,
two-tree acceptance, and building both trees of the next pass into one forest on the device."""
import numpy as np
import pytest
import torch

import oracle
from oracle import interblock
from paper_2608_27514_b200 import binding as B
from paper_2608_27514_b200 import workloads as W
from test_gpu_parity import PATHS, _check_attention

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _t(a, dt):
    return None if a is None else torch.as_tensor(np.ascontiguousarray(a), dtype=dt, device=DEV)


def _gpu_vis(S, Bn, n_cur):
    vis = torch.full((S, Bn, (Bn + 63) // 64), -1, dtype=torch.int64, device=DEV)
    B.tsd_build_interblock_vis(n_cur, vis)
    torch.cuda.synchronize()
    return vis


@pytest.mark.parametrize("Bn,n_cur", [(5, 3), (14, 10), (16, 12), (64, 63), (65, 64), (130, 3), (200, 129),
                                      (256, 255), (7, 7), (1, 1)])
def test_vis_matches_oracle(Bn, n_cur):
    got = _gpu_vis(3, Bn, n_cur).cpu().numpy().view(np.uint64)
    ref = interblock.interblock_vis(Bn, n_cur)
    for s in range(3):
        assert np.array_equal(got[s], ref)


def test_trigger_matches_oracle():
    rng = np.random.default_rng(11)
    S, Bn, R, M, tau = 64, 6, 32, 1000, 0.75
    state = np.where(rng.random((S, Bn, R)) < 0.5, M, 3).astype(np.int32)
    conf = (rng.integers(0, 17, (S, Bn, R)) / 16.0).astype(np.float32)     # ties with tau and each other
    node_cur = rng.integers(0, 4, S).astype(np.int32)
    node_next = 4
    state[0, node_cur[0]] = 3          # finished current block
    state[1, node_next] = 3            # finished next block
    state[2, node_cur[2]] = 3
    state[2, node_next] = 3            # both finished
    trig = torch.full((S,), 7, dtype=torch.uint8, device=DEV)
    top = torch.empty((S, 2), dtype=torch.float32, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    B.tsd_interblock_trigger(_t(state, torch.int32), _t(conf, torch.float32), _t(node_cur, torch.int32),
                             node_next, M, tau, trig, top, status)
    torch.cuda.synchronize()
    got, top = trig.cpu().numpy(), top.cpu().numpy()
    seen = set()
    for s in range(S):
        a, b = state[s, node_cur[s]], state[s, node_next]
        want = interblock.interblock_trigger(a, conf[s, node_cur[s]], b, conf[s, node_next], M, tau)
        assert bool(got[s]) == want, s
        assert top[s, 0] == interblock.top_confidence(a, M, conf[s, node_cur[s]])
        assert top[s, 1] == interblock.top_confidence(b, M, conf[s, node_next])
        seen.add(want)
    assert seen == {True, False} and int(status.item()) == 0
    assert list(got[:3]) == [1, 0, 0]
    # node_cur = NULL means node 0; an index outside the forest is reported
    B.tsd_interblock_trigger(_t(state, torch.int32), _t(conf, torch.float32), None, node_next, M, tau, trig)
    torch.cuda.synchronize()
    for s in range(S):
        assert bool(trig[s].item()) == interblock.interblock_trigger(state[s, 0], conf[s, 0], state[s, node_next],
                                                                     conf[s, node_next], M, tau)
    bad = node_cur.copy()
    bad[5] = Bn
    B.tsd_interblock_trigger(_t(state, torch.int32), _t(conf, torch.float32), _t(bad, torch.int32), node_next, M,
                             tau, trig, None, status)
    torch.cuda.synchronize()
    assert B.tsd_check_status(status) == B.TSD_ERR_DEVICE_DATA


@pytest.mark.parametrize("flags", PATHS)
@pytest.mark.parametrize("Bn,n_cur", [(16, 12), (14, 10), (9, 8)])
def test_attention_under_joint_mask(flags, Bn, n_cur):
    # the paper's own form of the inter-block pass: one block per branch, W3D3-sized tree for B_t
    # and a W1D3-sized one for B_{t+1}; the dense mask is compared bit for bit inside the helper
    cfg = W.small(W.CONFIGS["cfg3"], S=2, B=Bn, R=32, Nc=200, Hq=2, Hkv=2)
    vis = _gpu_vis(cfg.S, Bn, n_cur)
    assert np.array_equal(vis[0].cpu().numpy().view(np.uint64), interblock.interblock_vis(Bn, n_cur))
    _check_attention(cfg, W.attention_inputs(cfg, DEV), flags, vis=vis)


def _random_forest(rng, S, Bn, n_cur, R, V, tau):
    """Two random trees per sequence with children that are exact, partial, wrong or malformed."""
    M = V
    parent = np.empty((S, Bn), np.int32)
    for s in range(S):
        for b in range(Bn):
            lo = 0 if b < n_cur else n_cur
            parent[s, b] = -1 if b == lo else int(rng.integers(lo, b))
    conf = rng.random((S, Bn, R)).astype(np.float32)
    conf[rng.random((S, Bn, R)) < 0.2] = tau
    top1 = rng.integers(0, V, (S, Bn, R)).astype(np.int32)
    state = np.full((S, Bn, R), M, np.int32)
    for s in range(S):
        for b in range(Bn):
            p = parent[s, b]
            if p < 0:
                fill = rng.random(R) < 0.3
                state[s, b, fill] = rng.integers(0, V, fill.sum())
                continue
            c = state[s, p].copy()
            flag, tok = oracle.decode_rule(state[s, p], M, conf[s, p], top1[s, p], tau)
            rows = np.flatnonzero(c == M)
            mode = rng.integers(0, 5)
            if mode <= 1:
                c[flag.astype(bool)] = tok[flag.astype(bool)]
            elif mode == 2 and len(rows):
                r = rows[rng.integers(len(rows))]
                c[r] = top1[s, p, r]
            elif mode == 3 and len(rows):
                c[rows[0]] = rng.integers(0, V)
            elif mode == 4 and (c != M).any():
                c[np.flatnonzero(c != M)[0]] = M
            state[s, b] = c
    return parent, state, conf, top1, M


def _gpu_joint_accept(parent, state, n_cur, M, conf, top1, tau, rule, search):
    S, Bn, R = state.shape
    e = lambda shape, dt: torch.full(shape, 0, dtype=dt, device=DEV)
    out = dict(edge_valid=e((S, Bn), torch.uint8), prefix_len=e((S, Bn), torch.int32),
               accepted_node=e((2, S), torch.int32), accepted_len=e((2, S), torch.int32),
               n_new_tokens=e((2, S), torch.int32), unmask_flag=e((2, S, R), torch.uint8),
               unmask_tok=torch.full((2, S, R), -1, dtype=torch.int32, device=DEV))
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    B.tsd_accept_joint_trees(_t(parent, torch.int32), _t(state, torch.int32), n_cur, M, _t(conf, torch.float32),
                             _t(top1, torch.int32), 1, tau, rule, search, status=status, **out)
    torch.cuda.synchronize()
    return {k: v.cpu().numpy() for k, v in out.items()}, status


@pytest.mark.parametrize("Bn,n_cur,R", [(14, 10, 32), (40, 23, 20), (9, 8, 64), (6, 6, 32), (256, 100, 128)])
def test_joint_accept_matches_oracle(Bn, n_cur, R):
    rng = np.random.default_rng(Bn * 7 + R)
    S, V, tau = 12, 50, 0.8
    parent, state, conf, top1, M = _random_forest(rng, S, Bn, n_cur, R, V, tau)
    for rule in (0, 1):
        for search in (0, 1):
            ref = interblock.joint_accept(parent, state, n_cur, M, conf, top1, tau, rule, search)
            got, status = _gpu_joint_accept(parent, state, n_cur, M, conf, top1, tau, rule, search)
            for key, val in ref.items():
                assert np.array_equal(got[key], val), (key, rule, search)
            assert B.tsd_check_status(status) == B.TSD_OK


def test_joint_accept_parent_in_the_other_tree_is_reported():
    rng = np.random.default_rng(3)
    parent, state, conf, top1, M = _random_forest(rng, 2, 8, 5, 32, 50, 0.8)
    parent[1, 6] = 2                      # a node of the second tree hanging off the first
    ref = interblock.joint_accept(parent, state, 5, M, conf, top1, 0.8)
    got, status = _gpu_joint_accept(parent, state, 5, M, conf, top1, 0.8, 0, 0)
    assert B.tsd_check_status(status) == B.TSD_ERR_DEVICE_DATA
    for key, val in ref.items():
        assert np.array_equal(got[key], val), key


def test_next_pass_forest_is_built_on_the_device():
    # after a joint pass: accept both trees, evaluate the trigger, then build the tree of B_t
    # (W3D3) into branches [0, 10) and the compact tree of B_{t+1} (W1D3, only where triggered)
    # into branches [10, 14) of one state array; nothing returns to the host in between
    rng = np.random.default_rng(21)
    S, Bn, n_cur, R, V, k, tau = 24, 14, 10, 32, 300, 3, 0.8
    parent, state, conf, top1, M = _random_forest(rng, S, Bn, n_cur, R, V, tau)
    idx = rng.integers(0, V, (S, Bn, R, k)).astype(np.int32)
    idx[..., 0] = top1
    prob = -np.sort(-(rng.integers(1, 64, (S, Bn, R, k)) / 64.0).astype(np.float32), axis=-1)
    prob[::2, n_cur] *= 0.5            # every other sequence: an unconfident next block, no trigger
    conf = prob[..., 0].copy()

    d = dict(parent=_t(parent, torch.int32), state=_t(state, torch.int32), conf=_t(conf, torch.float32),
             idx=_t(idx, torch.int32), prob=_t(prob, torch.float32))
    e = lambda shape, dt: torch.zeros(shape, dtype=dt, device=DEV)
    acc = dict(edge_valid=e((S, Bn), torch.uint8), prefix_len=e((S, Bn), torch.int32),
               accepted_node=e((2, S), torch.int32), accepted_len=e((2, S), torch.int32),
               n_new_tokens=e((2, S), torch.int32), unmask_flag=e((2, S, R), torch.uint8),
               unmask_tok=e((2, S, R), torch.int32))
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    B.tsd_accept_joint_trees(d["parent"], d["state"], n_cur, M, d["conf"], d["idx"], k, tau, 0, 0,
                             status=status, **acc)
    trig = e((S,), torch.uint8)
    B.tsd_interblock_trigger(d["state"], d["conf"], acc["accepted_node"][0], n_cur, M, tau, trig, None, status)
    new_parent, new_state = e((S, Bn), torch.int32), e((S, Bn, R), torch.int32)
    new_prob, n_nodes = e((S, Bn), torch.float32), e((2, S), torch.int32)
    B.tsd_build_draft_tree(d["state"], acc["accepted_node"][0], acc["unmask_flag"][0], acc["unmask_tok"][0], M,
                           d["idx"], d["prob"], 3, 3, new_parent, new_state, new_prob, n_nodes[0], status,
                           first=0, max_nodes=n_cur)
    B.tsd_build_draft_tree(d["state"], acc["accepted_node"][1], acc["unmask_flag"][1], acc["unmask_tok"][1], M,
                           d["idx"], d["prob"], 1, 3, new_parent, new_state, new_prob, n_nodes[1], status,
                           first=n_cur, max_nodes=Bn - n_cur, enable=trig)
    torch.cuda.synchronize()
    assert int(status.item()) == 0

    ref = interblock.joint_accept(parent, state, n_cur, M, conf, top1, tau)
    got_parent, got_state = new_parent.cpu().numpy(), new_state.cpu().numpy()
    got_n, got_trig = n_nodes.cpu().numpy(), trig.cpu().numpy()
    fired = 0
    for s in range(S):
        a0, a1 = ref["accepted_node"][0, s], ref["accepted_node"][1, s]
        want_trig = interblock.interblock_trigger(state[s, a0], conf[s, a0], state[s, n_cur], conf[s, n_cur], M, tau)
        assert bool(got_trig[s]) == want_trig
        fired += want_trig
        for t, (a, lo, size, Wd, D) in enumerate(((a0, 0, n_cur, 3, 3), (a1, n_cur, Bn - n_cur, 1, 3))):
            root = np.where(ref["unmask_flag"][t, s].astype(bool), ref["unmask_tok"][t, s], state[s, a])
            depth = D if (t == 0 or want_trig) else 0
            n, par, st, _ = oracle.build_draft_tree(root.astype(np.int32), M, idx[s, a], prob[s, a], Wd, depth, size)
            par = np.where(par >= 0, par + lo, par)
            assert got_n[t, s] == n
            assert np.array_equal(got_parent[s, lo:lo + size], par)
            assert np.array_equal(got_state[s, lo:lo + size], st)
    assert 0 < fired < S
