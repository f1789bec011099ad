"""CPU oracle for inter-block speculation (Section 3.4, Eq. 3, Appendix D).  Test infrastructure,
not the product: plain numpy written from the paper's statements, sharing nothing with the CUDA
library.

Joint layout of one verification pass over two consecutive blocks: the tree of the current block
B_t occupies branches [0, n_cur) with its root at branch 0, the compact tree of the next block
B_{t+1} occupies branches [n_cur, B) with its root at branch n_cur.  Every branch has R rows (one
block).

Reading of the mask (the paper's figure is not available; Section 3.4 and Appendix D in words):
  * the two roots see each other (bidirectional visibility between the roots);
  * a draft of B_t reads the root of B_{t+1}, a draft of B_{t+1} reads the root of B_t;
  * no branch reads any draft other than itself (drafts stay mutually invisible, and a root never
    reads a draft, so the scores of a root do not depend on what was drafted);
  * every branch reads itself and the cached prefix/suffix, as in Section 3.3.
"""
import numpy as np

from . import binding


def interblock_vis(n_branches, n_cur):
    """uint64 [n_branches, ceil(n_branches/64)]: bit j of row b set = branch b reads branch j."""
    assert 1 <= n_cur <= n_branches
    words = (n_branches + 63) // 64
    vis = np.zeros((n_branches, words), dtype=np.uint64)

    def put(b, j):
        vis[b, j // 64] |= np.uint64(1) << np.uint64(j % 64)

    for b in range(n_branches):
        put(b, b)
        if n_cur < n_branches:          # a next-block tree exists
            if b < n_cur:
                put(b, n_cur)           # B_t's root and drafts read the root of B_{t+1}
            else:
                put(b, 0)               # B_{t+1}'s root and drafts read the root of B_t
    return vis


def top_confidence(state, mask_id, conf):
    """c^(1) of one block: the largest confidence among its still-masked rows (-inf if none)."""
    state = np.asarray(state)
    conf = np.asarray(conf, dtype=np.float32)
    masked = state == mask_id
    return np.float32(conf[masked].max()) if masked.any() else np.float32(-np.inf)


def interblock_trigger(state_cur, conf_cur, state_next, conf_next, mask_id, tau):
    """Eq. 3: speculate over B_{t+1} as well iff c_{t+1}^(1) > c_t^(1) or c_{t+1}^(1) > tau.
    A next block with no masked row has nothing to draft: no trigger."""
    c_cur = top_confidence(state_cur, mask_id, conf_cur)
    c_next = top_confidence(state_next, mask_id, conf_next)
    if c_next == -np.inf:
        return False
    return bool(c_next > c_cur or c_next > np.float32(tau))


def joint_accept(parent, state, n_cur, mask_id, conf, top1, tau, rule=0, search=0, topk_m=1, draft_prob=None):
    """Acceptance of the two trees of a joint pass, each by the single-tree procedure of
    Section 3.3 on its own branches.  parent [S,B] holds forest indices (parent[:, n_cur] = -1).
    Returns per-branch arrays over the forest and per-tree arrays with a leading axis of 2
    (tree 0 = B_t, tree 1 = B_{t+1}); accepted_node is a forest index."""
    parent = np.asarray(parent, dtype=np.int32)
    state = np.asarray(state, dtype=np.int32)
    conf = np.asarray(conf, dtype=np.float32)
    top1 = np.asarray(top1, dtype=np.int32)
    S, B, R = state.shape
    out = dict(edge_valid=np.zeros((S, B), np.uint8), prefix_len=np.zeros((S, B), np.int32),
               accepted_node=np.zeros((2, S), np.int32), accepted_len=np.zeros((2, S), np.int32),
               n_new_tokens=np.zeros((2, S), np.int32), unmask_flag=np.zeros((2, S, R), np.uint8),
               unmask_tok=np.full((2, S, R), -1, np.int32))
    for t, (lo, hi) in enumerate(((0, n_cur), (n_cur, B))):
        if hi == lo:
            continue
        par = parent[:, lo:hi].copy()
        par[:, 1:] -= lo                 # indices local to the tree
        par[:, 0] = -1
        o = binding.accept(par, state[:, lo:hi], mask_id, conf[:, lo:hi], top1[:, lo:hi], tau, rule, search,
                           topk_m, None if draft_prob is None else np.asarray(draft_prob)[:, lo:hi])
        out["edge_valid"][:, lo:hi] = o["edge_valid"]
        out["prefix_len"][:, lo:hi] = o["prefix_len"]
        out["accepted_node"][t] = o["accepted_node"] + lo
        for key in ("accepted_len", "n_new_tokens", "unmask_flag", "unmask_tok"):
            out[key][t] = o[key]
    return out
