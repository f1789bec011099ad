"""CPU oracle for the step after the path: committing what a verification pass accepted (test
infrastructure, not the product; plain numpy, shares nothing with the CUDA library).

Section 3.3 ends a pass with the longest verified trajectory; Section 3.1 makes its last node the
start of the next pass.  Every edge of the accepted path is one step of the sequential decoder
(Theorem 1: its delta is exactly what threshold decoding would have unmasked there), and the unmask
set U(accepted node) is one more.  So a pass that starts `step_base` sequential steps into the block
and accepts a node of depth n fills
    the delta of the path node at depth j   at sequential step step_base + j - 1   (j = 1..n)
    U(accepted node)                         at sequential step step_base + n
and leaves the block step_base + n + 1 steps in (step_base + n if the accepted node was already
full, in which case U is empty and no step is taken).
"""
import numpy as np


def gather_accepted_kv(draft, accepted_node, R):
    """draft [S, B*R, H, d], accepted_node [S] -> [S, R, H, d]: the draft rows of the accepted node
    (Appendix A / Section 3.1: the block's K/V under the tokens that were kept)."""
    draft = np.asarray(draft)
    return np.stack([draft[s, int(a) * R:(int(a) + 1) * R] for s, a in enumerate(np.asarray(accepted_node))])


def commit_accepted(parent, state, accepted_node, unmask_flag, unmask_tok, mask_id, step_base=0, tree_root=0):
    """One sequence.  parent [B], state [B,R] -> dict(root [R] = the next root, fill_step [R] = the
    sequential step at which a row was filled by this pass (-1 for rows it did not fill),
    step_base = the new step count, n_masked = rows still masked in the next root).  tree_root is
    the index of the tree's root when the arrays hold a forest (Section 3.4: two trees per pass)."""
    parent = np.asarray(parent, dtype=np.int64)
    state = np.asarray(state, dtype=np.int32)
    flag = np.asarray(unmask_flag).astype(bool)
    tok = np.asarray(unmask_tok, dtype=np.int32)
    R = state.shape[1]
    path = [int(accepted_node)]
    while path[-1] != tree_root:
        path.append(int(parent[path[-1]]))
    path.reverse()                                   # root .. accepted node
    fill_step = np.full(R, -1, dtype=np.int32)
    for j in range(1, len(path)):
        p, c = path[j - 1], path[j]
        for r in range(R):
            if state[p, r] == mask_id and state[c, r] != mask_id:
                fill_step[r] = step_base + j - 1
    n = len(path) - 1
    acc_state = state[path[-1]]
    root = acc_state.copy()
    took_step = bool((acc_state == mask_id).any())
    for r in range(R):
        if flag[r] and acc_state[r] == mask_id:
            root[r] = tok[r]
            fill_step[r] = step_base + n
    return dict(root=root, fill_step=fill_step, step_base=step_base + n + (1 if took_step else 0),
                n_masked=int((root == mask_id).sum()))
