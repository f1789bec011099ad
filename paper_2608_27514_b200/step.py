"""One blockwise verification step as a sequence of libtsd calls.

``VerifyStep`` owns the device buffers (outputs, mask blob, workspaces) for a
fixed layout and enqueues the stages on the current stream: mask once per tree
shape, then attention -> confidence/top-k -> acceptance per step.  It only
allocates and marshals; all arithmetic runs in the library's kernels.
"""
import torch

from . import binding as B


class VerifyStep:
    def __init__(self, S, n_branches, R, Nc, Hq, Hkv, d, V, k, dtype, device="cuda:0"):
        self.S, self.B, self.R, self.Nc, self.Hq, self.Hkv, self.d, self.V, self.k = (
            S, n_branches, R, Nc, Hq, Hkv, d, V, k)
        self.dtype = dtype
        self.device = torch.device(device)
        self.layout = B.make_layout(S, n_branches, R, Nc, Hq, Hkv, d, dtype)
        dev = self.device
        N, rows = n_branches * R, S * n_branches * R
        self.N, self.rows = N, rows
        u8 = lambda n: torch.empty(max(int(n), 16), dtype=torch.uint8, device=dev)
        self.mask = u8(B.tsd_branch_mask_bytes(self.layout))
        self.attn_ws = u8(B.tsd_verify_attention_workspace_bytes(self.layout))
        # zeroed once, as the header asks: the calls keep its ticket words at 0 from then on
        self.topk_ws = torch.zeros(max(int(B.tsd_confidence_topk_workspace_bytes(rows, V, k)), 16),
                                   dtype=torch.uint8, device=dev)
        self.out = torch.empty((S, N, Hq, d), dtype=dtype, device=dev)
        self.attn_lse = torch.empty((S, Hq, N), dtype=torch.float32, device=dev)
        self.conf = torch.empty(rows, dtype=torch.float32, device=dev)
        self.topk_idx = torch.empty((rows, k), dtype=torch.int32, device=dev)
        self.topk_prob = torch.empty((rows, k), dtype=torch.float32, device=dev)
        self.lse = torch.empty(rows, dtype=torch.float32, device=dev)
        self.edge_valid = torch.empty((S, n_branches), dtype=torch.uint8, device=dev)
        self.prefix_len = torch.empty((S, n_branches), dtype=torch.int32, device=dev)
        self.accepted_node = torch.empty(S, dtype=torch.int32, device=dev)
        self.accepted_len = torch.empty(S, dtype=torch.int32, device=dev)
        self.n_new_tokens = torch.empty(S, dtype=torch.int32, device=dev)
        self.unmask_flag = torch.empty((S, R), dtype=torch.uint8, device=dev)
        self.unmask_tok = torch.empty((S, R), dtype=torch.int32, device=dev)
        self.status = torch.zeros(1, dtype=torch.int32, device=dev)
        self.mask_built = False

    @classmethod
    def for_config(cls, cfg, device="cuda:0"):
        return cls(cfg.S, cfg.B, cfg.R, cfg.Nc, cfg.Hq, cfg.Hkv, cfg.d, cfg.V, cfg.k, cfg.torch_dtype, device)

    def build_mask(self, vis=None, cache_lens=None, dense_out=None):
        B.tsd_build_branch_mask(self.layout, vis, cache_lens, self.mask, dense_out)
        self.mask_built = True

    def attention(self, q, k_cache, v_cache, k_draft, v_draft, sm_scale, flags=0, out=None, lse=None):
        if not self.mask_built:
            self.build_mask()
        B.tsd_verify_attention(self.layout, self.mask, q, k_cache, v_cache, k_draft, v_draft,
                               self.out if out is None else out,
                               self.attn_lse if lse is None else lse, sm_scale, self.attn_ws, flags,
                               self.status)
        return self.out if out is None else out

    def confidence_topk(self, logits):
        B.tsd_confidence_topk(logits, self.k, self.conf, self.topk_idx, self.topk_prob, self.lse,
                              self.topk_ws, self.status)
        return self.conf, self.topk_idx, self.topk_prob

    def accept(self, parent, state, mask_id, tau, rule=B.TSD_ACCEPT_EXACT, search=B.TSD_SEARCH_GREEDY,
               conf=None, top1=None, top1_stride=None):
        B.tsd_accept_trajectories(
            parent, state, mask_id, self.conf if conf is None else conf,
            self.topk_idx if top1 is None else top1, self.k if top1_stride is None else top1_stride,
            tau, rule, search, self.edge_valid, self.prefix_len, self.accepted_node, self.accepted_len,
            self.n_new_tokens, self.unmask_flag, self.unmask_tok, self.status)
        return self.accept_outputs()

    def accept_relaxed(self, parent, state, mask_id, tau, rule, search=B.TSD_SEARCH_LONGEST, logits=None,
                       topk_m=None):
        """Acceptance under any rule, on the candidates and log-sum-exp of the last vocabulary pass;
        the probability rule gathers from `logits` (the tensor that pass read)."""
        if logits is not None and not hasattr(self, "draft_prob"):
            self.draft_prob = torch.empty((self.S, self.B, self.R), dtype=torch.float32, device=self.device)
        B.tsd_accept_relaxed(
            parent, state, self.B, mask_id, self.conf, self.topk_idx.view(self.S, self.B, self.R, self.k),
            self.k if topk_m is None else topk_m, logits, self.lse if logits is not None else None, tau, rule,
            search, self.edge_valid, self.prefix_len, self.accepted_node, self.accepted_len, self.n_new_tokens,
            self.unmask_flag, self.unmask_tok, getattr(self, "draft_prob", None) if logits is not None else None,
            self.status)
        return self.accept_outputs()

    def accept_outputs(self):
        return dict(edge_valid=self.edge_valid, prefix_len=self.prefix_len,
                    accepted_node=self.accepted_node, accepted_len=self.accepted_len,
                    n_new_tokens=self.n_new_tokens, unmask_flag=self.unmask_flag,
                    unmask_tok=self.unmask_tok)

    def run(self, attn, logits, parent, state, mask_id, tau, rule=B.TSD_ACCEPT_EXACT,
            search=B.TSD_SEARCH_GREEDY, flags=0):
        """The whole hot path: attention -> confidence/top-k -> acceptance."""
        self.attention(attn["q"], attn["k_cache"], attn["v_cache"], attn["k_draft"], attn["v_draft"],
                       attn["sm_scale"], flags)
        self.confidence_topk(logits)
        return self.accept(parent, state, mask_id, tau, rule, search)

    def check_status(self):
        rc = B.tsd_check_status(self.status)
        if rc != B.TSD_OK:
            raise B.TsdError(rc, "device status")
