"""Speculative decoding of one block as a sequence of libtsd calls (Alg. 1, Sections 3.1-3.3).

``BlockDecoder`` strings the library's kernels into the paper's loop.  One pass =

    caller's model forward over every node of the tree   (its attention layers call
                                                          ``VerifyStep.attention``)
    -> tsd_confidence_topk      scores of this pass = candidate pool of the next (Section 3.1)
    -> tsd_accept_trajectories  longest verified trajectory (Section 3.3)
    -> tsd_commit_accepted      next root into the token buffer, sequential step indices
    -> tsd_build_draft_tree     tree of the next pass (Alg. 1 Phase 2)

All of it is enqueued on the current stream; the only thing read back per pass is the count of
rows still masked (4 bytes per sequence), which ends the loop.  The class allocates and marshals;
every step of the arithmetic runs in the library's kernels.
"""
import torch

from . import binding as B


class BlockDecoder:
    def __init__(self, step, width, depth, tau, mask_id, rule=B.TSD_ACCEPT_EXACT, search=B.TSD_SEARCH_GREEDY):
        """step: a VerifyStep whose layout (batch, branches, rows) fixes the tree size: every pass
        verifies step.B nodes per sequence (unused slots are copies of the root)."""
        self.step, self.width, self.depth, self.tau, self.mask_id = step, int(width), int(depth), float(tau), int(mask_id)
        self.rule, self.search = rule, search
        S, Bn, R, dev = step.S, step.B, step.R, step.device
        i32 = lambda *shape: torch.zeros(shape, dtype=torch.int32, device=dev)
        # two copies of the tree: the builder reads the verified tree while it writes the next one
        self.trees = [dict(parent=i32(S, Bn), state=i32(S, Bn, R), prob=torch.zeros((S, Bn), device=dev),
                           n=i32(S)) for _ in range(2)]
        self.cur = 0
        self.root = i32(S, R)
        self.fill_step = i32(S, R)
        self.step_base = i32(S)
        self.n_masked = i32(S)
        self.n_forward = 0

    @property
    def tree(self):
        return self.trees[self.cur]

    def start(self, root_state):
        """Begin a block from root_state int32 [S, R]; the first pass has no candidate pool yet, so
        its tree is the root alone (copies in the unused slots)."""
        t = self.tree
        t["state"].copy_(root_state.to(torch.int32)[:, None, :].expand_as(t["state"]))
        t["parent"].zero_()
        t["parent"][:, 0] = -1
        t["n"].fill_(1)
        self.fill_step.fill_(-1)
        self.step_base.zero_()
        # the root alone, nothing accepted, nothing to unmask: the commit kernel copies it to
        # self.root and counts its masked rows
        B.tsd_commit_accepted(t["parent"], t["state"], None, None, None, self.mask_id, root_out=self.root,
                              n_masked=self.n_masked, status=self.step.status)
        self.n_forward = 0

    def advance(self, logits, tokens=None, block_start=None):
        """One pass after the caller's forward: logits [S*B*R, V] of the current tree's nodes."""
        st, t, nxt = self.step, self.tree, self.trees[1 - self.cur]
        st.confidence_topk(logits)
        if self.rule in (B.TSD_ACCEPT_EXACT, B.TSD_ACCEPT_TOP1):
            st.accept(t["parent"], t["state"], self.mask_id, self.tau, self.rule, self.search)
        else:
            st.accept_relaxed(t["parent"], t["state"], self.mask_id, self.tau, self.rule, self.search,
                              logits if self.rule == B.TSD_ACCEPT_PROB else None)
        B.tsd_commit_accepted(t["parent"], t["state"], st.accepted_node, st.unmask_flag, st.unmask_tok,
                              self.mask_id, tokens, block_start, self.root, self.fill_step, self.step_base,
                              self.n_masked, st.status)
        B.tsd_build_draft_tree(t["state"], st.accepted_node, st.unmask_flag, st.unmask_tok, self.mask_id,
                               st.topk_idx, st.topk_prob, self.width, self.depth, nxt["parent"], nxt["state"],
                               nxt["prob"], nxt["n"], st.status)
        self.cur = 1 - self.cur
        self.n_forward += 1

    def decode(self, forward, tokens=None, block_start=None, max_passes=None):
        """Run passes until no sequence has a masked row left.  forward(state int32 [S,B,R]) must
        return the logits [S*B*R, V] of every node (a device tensor the vocabulary pass accepts)."""
        limit = self.step.R + 1 if max_passes is None else max_passes
        while self.n_forward < limit and int(self.n_masked.max().item()) > 0:
            self.advance(forward(self.tree["state"]), tokens, block_start)
        self.step.check_status()
        return self.root
