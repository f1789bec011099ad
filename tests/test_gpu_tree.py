"""GPU parity of the draft-tree construction (Alg. 1 Phase 2) against the oracle: bit-exact trees."""
import numpy as np
import pytest
import torch

import oracle
from paper_2608_27514_b200 import binding as B
from paper_2608_27514_b200 import workloads as W
from paper_2608_27514_b200.step import VerifyStep

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _gpu_tree(prev_state, acc, flag, tok, mask_id, idx, prob, width, depth, max_nodes):
    S, Bp, R = prev_state.shape
    t = lambda a, dt: None if a is None else torch.as_tensor(np.ascontiguousarray(a), dtype=dt, device=DEV)
    parent = torch.empty((S, max_nodes), dtype=torch.int32, device=DEV)
    state = torch.empty((S, max_nodes, R), dtype=torch.int32, device=DEV)
    nprob = torch.empty((S, max_nodes), dtype=torch.float32, device=DEV)
    n = torch.empty(S, dtype=torch.int32, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    B.tsd_build_draft_tree(t(prev_state, torch.int32), t(acc, torch.int32), t(flag, torch.uint8), t(tok, torch.int32),
                           mask_id, t(idx, torch.int32), t(prob, torch.float32), width, depth, parent, state,
                           nprob, n, status)
    torch.cuda.synchronize()
    return n.cpu().numpy(), parent.cpu().numpy(), state.cpu().numpy(), nprob.cpu().numpy(), int(status.item())


def _oracle_tree(prev_state, acc, flag, tok, mask_id, idx, prob, width, depth, max_nodes):
    S, Bp, R = prev_state.shape
    out = []
    for s in range(S):
        a = 0 if acc is None else int(acc[s])
        root = prev_state[s, a].copy()
        if flag is not None:
            root = np.where(flag[s].astype(bool), tok[s], root).astype(np.int32)
        out.append(oracle.build_draft_tree(root, mask_id, idx[s, a], prob[s, a], width, depth, max_nodes))
    return out


@pytest.mark.parametrize("R,k,Wd,D,Bn", [(32, 3, 2, 2, 4), (32, 3, 3, 3, 7), (64, 3, 3, 3, 16), (128, 8, 32, 4, 256),
                                          (5, 1, 1, 1, 2), (32, 4, 4, 0, 8), (32, 2, 8, 6, 40)])
@pytest.mark.parametrize("lowest", [1, 0])   # 0: candidates of probability exactly zero take part too
def test_tree_matches_oracle_random_pools(R, k, Wd, D, Bn, lowest):
    rng = np.random.default_rng(R * 1000 + k * 100 + Wd)
    S, Bp, V = 9, 5, 1000
    M = V
    prev = np.where(rng.random((S, Bp, R)) < 0.6, M, rng.integers(0, V, (S, Bp, R))).astype(np.int32)
    prev[3] = rng.integers(0, V, (Bp, R))                     # a sequence with nothing left to unmask
    acc = rng.integers(0, Bp, S).astype(np.int32)
    flag = (rng.random((S, R)) < 0.15).astype(np.uint8)
    tok = rng.integers(0, V, (S, R)).astype(np.int32)
    idx = rng.integers(0, V, (S, Bp, R, k)).astype(np.int32)
    prob = (rng.integers(lowest, 64 if lowest else 4, (S, Bp, R, k)) / 64.0).astype(np.float32)   # coarse values: many ties
    prob = -np.sort(-prob, axis=-1)
    got = _gpu_tree(prev, acc, flag, tok, M, idx, prob, Wd, D, Bn)
    ref = _oracle_tree(prev, acc, flag, tok, M, idx, prob, Wd, D, Bn)
    assert got[4] == 0
    for s in range(S):
        n, parent, state, nprob = ref[s]
        assert got[0][s] == n
        assert np.array_equal(got[1][s], parent) and np.array_equal(got[2][s], state)
        assert np.array_equal(got[3][s], nprob)


def test_tree_without_acceptance_inputs_and_bad_node():
    rng = np.random.default_rng(1)
    S, R, k, M = 3, 32, 3, 500
    prev = np.where(rng.random((S, 1, R)) < 0.5, M, 7).astype(np.int32)
    idx = rng.integers(0, M, (S, 1, R, k)).astype(np.int32)
    prob = -np.sort(-rng.random((S, 1, R, k)).astype(np.float32), axis=-1)
    got = _gpu_tree(prev, None, None, None, M, idx, prob, 2, 2, 4)
    ref = _oracle_tree(prev, None, None, None, M, idx, prob, 2, 2, 4)
    for s in range(S):
        assert got[0][s] == ref[s][0] and np.array_equal(got[2][s], ref[s][2])
    # an accepted-node index outside the tree is reported and treated as node 0
    bad = np.array([0, 9, 0], np.int32)
    got = _gpu_tree(prev, bad, None, None, M, idx, prob, 2, 2, 4)
    assert B.tsd_check_status(got[4]) == B.TSD_ERR_DEVICE_DATA
    assert np.array_equal(got[2][1], ref[1][2])


def test_decode_loop_stays_on_device_and_matches_the_oracle_chain():
    """verify (top-k + accept) -> build the next tree, twice, all on the GPU; the oracle replays the
    same chain on the host from the same logits."""
    cfg = W.small(W.CONFIGS["cfg2"], V=4096, Nc=64, Hq=1, Hkv=1)
    vi = W.verify_inputs(cfg, DEV)
    step = VerifyStep.for_config(cfg, DEV)
    S, Bn, R, k = cfg.S, cfg.B, cfg.R, cfg.k
    step.confidence_topk(vi["logits"])
    res = step.accept(vi["parent"], vi["state"], vi["mask_id"], cfg.tau)
    parent = torch.empty((S, Bn), dtype=torch.int32, device=DEV)
    state = torch.empty((S, Bn, R), dtype=torch.int32, device=DEV)
    nprob = torch.empty((S, Bn), dtype=torch.float32, device=DEV)
    n = torch.empty(S, dtype=torch.int32, device=DEV)
    B.tsd_build_draft_tree(vi["state"], res["accepted_node"], res["unmask_flag"], res["unmask_tok"], vi["mask_id"],
                           step.topk_idx, step.topk_prob, 3, 3, parent, state, nprob, n, step.status)
    torch.cuda.synchronize()
    step.check_status()
    # host replay with the oracle only
    conf, idx, prob, _ = oracle.confidence_topk(vi["logits"].float().cpu().numpy(), k)
    acc = oracle.accept(vi["parent"].cpu().numpy(), vi["state"].cpu().numpy(), vi["mask_id"],
                        conf.astype(np.float32).reshape(S, Bn, R), idx[:, 0].reshape(S, Bn, R), cfg.tau)
    a = int(acc["accepted_node"][0])
    root = np.where(acc["unmask_flag"][0].astype(bool), acc["unmask_tok"][0], vi["state"].cpu().numpy()[0, a])
    # probabilities decide the tree: both sides use the fp32 values the GPU produced for them, the
    # rest (indices, acceptance, unmask set) is the oracle's own
    g_prob = step.topk_prob.cpu().numpy().reshape(S, Bn, R, k)
    assert np.abs(g_prob - prob.reshape(S, Bn, R, k)).max() <= 1e-5
    rn, rparent, rstate, rprob = oracle.build_draft_tree(root.astype(np.int32), vi["mask_id"],
                                                         idx.reshape(S, Bn, R, k)[0, a], g_prob[0, a], 3, 3, Bn)
    assert int(n[0]) == rn and rn == min(Bn, 10)
    assert np.array_equal(parent[0].cpu().numpy(), rparent) and np.array_equal(state[0].cpu().numpy(), rstate)
    # the new tree is a valid input of the next verification pass
    res2 = step.accept(parent, state, vi["mask_id"], cfg.tau)
    torch.cuda.synchronize()
    step.check_status()
    assert int(res2["edge_valid"][0, 0]) == 1
