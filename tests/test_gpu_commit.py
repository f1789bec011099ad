"""GPU parity of tsd_commit_accepted against the commit oracle, and the exactness theorem
(Theorem 1) end to end on the device: a toy model decoded block by block through the library's
loop gives the same (row, token, step) trajectory with and without speculation."""
import numpy as np
import pytest
import torch

import oracle
from oracle import commit as C
from paper_2608_27514_b200 import binding as B
from paper_2608_27514_b200.decode import BlockDecoder
from paper_2608_27514_b200.step import VerifyStep

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _t(a, dt):
    return None if a is None else torch.as_tensor(np.ascontiguousarray(a), dtype=dt, device=DEV)


def _valid_trees(rng, S, Bn, R, V):
    """Random trees whose children extend their parents by one to three rows (so every path is a
    possible accepted path), plus an unmask set for a chosen node."""
    M = V
    parent = np.stack([[-1] + [int(rng.integers(0, b)) for b in range(1, Bn)] for _ in range(S)]).astype(np.int32)
    state = np.full((S, Bn, R), M, np.int32)
    for s in range(S):
        fill = rng.random(R) < 0.25
        state[s, 0, fill] = rng.integers(0, V, fill.sum())
        for b in range(1, Bn):
            c = state[s, parent[s, b]].copy()
            rows = np.flatnonzero(c == M)
            for r in rows[rng.permutation(len(rows))[: int(rng.integers(1, 4))]]:
                c[r] = rng.integers(0, V)
            state[s, b] = c
    acc = rng.integers(0, Bn, S).astype(np.int32)
    flag = np.zeros((S, R), np.uint8)
    tok = np.full((S, R), -1, np.int32)
    for s in range(S):
        rows = np.flatnonzero(state[s, acc[s]] == M)
        pick = rows[rng.permutation(len(rows))[: int(rng.integers(0, 4))]]
        flag[s, pick] = 1
        tok[s, pick] = rng.integers(0, V, len(pick))
        extra = np.flatnonzero(state[s, acc[s]] != M)[:1]     # a flag on a filled row must be ignored
        flag[s, extra] = 1
        tok[s, extra] = 12345
    return parent, state, acc, flag, tok, M


@pytest.mark.parametrize("Bn,R", [(8, 32), (40, 64), (256, 128), (1, 5), (13, 100)])
def test_commit_matches_oracle(Bn, R):
    rng = np.random.default_rng(Bn + R)
    S, V, L = 17, 1000, 300
    parent, state, acc, flag, tok, M = _valid_trees(rng, S, Bn, R, V)
    base = rng.integers(0, 20, S).astype(np.int32)
    start = rng.integers(0, L - R + 1, S).astype(np.int32)
    tokens = torch.full((S, L), -5, dtype=torch.int32, device=DEV)
    root = torch.empty((S, R), dtype=torch.int32, device=DEV)
    fill = torch.full((S, R), -1, dtype=torch.int32, device=DEV)
    d_base, n_masked = _t(base, torch.int32), torch.empty(S, dtype=torch.int32, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    B.tsd_commit_accepted(_t(parent, torch.int32), _t(state, torch.int32), _t(acc, torch.int32),
                          _t(flag, torch.uint8), _t(tok, torch.int32), M, tokens, _t(start, torch.int32), root, fill,
                          d_base, n_masked, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    tokens = tokens.cpu().numpy()
    for s in range(S):
        o = C.commit_accepted(parent[s], state[s], acc[s], flag[s], tok[s], M, int(base[s]))
        assert np.array_equal(root[s].cpu().numpy(), o["root"])
        assert np.array_equal(fill[s].cpu().numpy(), o["fill_step"])
        assert int(d_base[s]) == o["step_base"] and int(n_masked[s]) == o["n_masked"]
        want = np.full(L, -5, np.int32)
        want[start[s]:start[s] + R] = o["root"]
        assert np.array_equal(tokens[s], want)


def test_commit_defaults_and_bad_inputs():
    rng = np.random.default_rng(0)
    parent, state, acc, flag, tok, M = _valid_trees(rng, 3, 6, 32, 50)
    root = torch.empty((3, 32), dtype=torch.int32, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    # no accepted node, no unmask set, no token buffer: the next root is node 0 itself
    B.tsd_commit_accepted(_t(parent, torch.int32), _t(state, torch.int32), None, None, None, M, root_out=root,
                          status=status)
    torch.cuda.synchronize()
    assert np.array_equal(root.cpu().numpy(), state[:, 0]) and int(status.item()) == 0
    # a block that does not fit the token buffer is reported and not written
    tokens = torch.full((3, 40), -5, dtype=torch.int32, device=DEV)
    start = _t(np.array([0, 9, 8], np.int32), torch.int32)
    B.tsd_commit_accepted(_t(parent, torch.int32), _t(state, torch.int32), None, None, None, M, tokens, start,
                          status=status)
    torch.cuda.synchronize()
    assert B.tsd_check_status(status) == B.TSD_ERR_DEVICE_DATA
    assert (tokens[1] == -5).all() and (tokens[2, 8:] == _t(state[2, 0], torch.int32)).all()
    # a parent chain that leaves the tree: reported, U(root) only
    status.zero_()
    bad = parent.copy()
    bad[0, 3] = 4
    B.tsd_commit_accepted(_t(bad, torch.int32), _t(state, torch.int32), _t(np.array([3, 0, 0], np.int32), torch.int32),
                          None, None, M, root_out=root, status=status)
    torch.cuda.synchronize()
    assert B.tsd_check_status(status) == B.TSD_ERR_DEVICE_DATA
    assert np.array_equal(root[0].cpu().numpy(), state[0, 0])


class ToyModel:
    """Embedding + one attention layer over a fixed cache (the library's verify attention) +
    un-embedding; bf16 activations.  The matmuls are torch's: with the same tree size in both runs
    they give every row the same result whatever the other rows hold."""

    def __init__(self, step, seed, V=512, gain=5.0):
        g = torch.Generator(device="cpu").manual_seed(seed)
        H, d, R = step.Hq, step.d, step.R
        D = H * d
        rn = lambda *shape: torch.randn(shape, generator=g)
        self.step, self.V, self.mask_id, self.D = step, V, V, D
        self.E = rn(V + 1, D).to(DEV).bfloat16()
        self.P = rn(R, D).to(DEV).bfloat16()
        self.Wq, self.Wk, self.Wv = ((rn(D, D) / D ** 0.5).to(DEV).bfloat16() for _ in range(3))
        self.Wo = (rn(D, V) * gain / D ** 0.5).to(DEV).bfloat16()
        self.kc = rn(step.S, step.Nc, H, d).to(DEV).bfloat16()
        self.vc = rn(step.S, step.Nc, H, d).to(DEV).bfloat16()

    def forward(self, state):
        st = self.step
        S, Bn, R = state.shape
        x = self.E[state.long()] + self.P[None, None]
        x = x.reshape(S * Bn * R, self.D)
        shape = (S, Bn * R, st.Hq, st.d)
        q, k, v = ((x @ w).reshape(shape) for w in (self.Wq, self.Wk, self.Wv))
        att = st.attention(q, self.kc, self.vc, k, v, 1.0 / st.d ** 0.5)
        h = x + att.reshape(S * Bn * R, self.D)
        return (h @ self.Wo).contiguous()


@pytest.mark.parametrize("tau", [0.9, 1.5])
@pytest.mark.parametrize("search", [B.TSD_SEARCH_GREEDY, B.TSD_SEARCH_LONGEST])
def test_theorem1_on_the_device(tau, search):
    S, Bn, R, Nc, H, d, k = 6, 8, 32, 96, 2, 128, 3
    step = VerifyStep(S, Bn, R, Nc, H, H, d, 512, k, torch.bfloat16, DEV)
    model = ToyModel(step, seed=int(tau * 10) + search)
    root = torch.full((S, R), model.mask_id, dtype=torch.int32, device=DEV)
    root[1, :20] = 7                                   # a block that starts partly decoded
    runs = {}
    for name, depth in (("sequential", 0), ("speculative", 3)):
        dec = BlockDecoder(step, 3, depth, tau, model.mask_id, B.TSD_ACCEPT_EXACT, search)
        dec.start(root)
        tokens = torch.zeros((S, R + 8), dtype=torch.int32, device=DEV)
        final = dec.decode(model.forward, tokens, torch.full((S,), 4, dtype=torch.int32, device=DEV))
        torch.cuda.synchronize()
        assert int(dec.n_masked.max()) == 0 and (final != model.mask_id).all()
        assert torch.equal(tokens[:, 4:4 + R], final)
        runs[name] = (final.cpu().numpy(), dec.fill_step.cpu().numpy(), dec.step_base.cpu().numpy(), dec.n_forward)
    seq, spec = runs["sequential"], runs["speculative"]
    assert np.array_equal(seq[0], spec[0])             # same tokens
    assert np.array_equal(seq[1], spec[1])             # filled at the same sequential step
    assert np.array_equal(seq[2], spec[2])             # same number of sequential steps
    assert seq[3] == seq[2].max()                      # without drafts: one forward per step
    assert spec[3] < seq[3]                            # speculation saved forwards


def test_commit_both_trees_of_a_joint_pass():
    # Section 3.4: one pass carries the tree of the current block (root 0) and a tree of the next
    # block (root n_cur); parents and accepted nodes are forest indices.  Each tree commits on its own.
    rng = np.random.default_rng(21)
    S, R, V, n_cur, n_nxt = 9, 32, 500, 7, 5
    Bn, M = n_cur + n_nxt, 500
    pa, sa, acc_a, fa, ta, _ = _valid_trees(rng, S, n_cur, R, V)
    pb, sb, acc_b, fb, tb, _ = _valid_trees(rng, S, n_nxt, R, V)
    parent = np.concatenate([pa, np.where(pb < 0, -1, pb + n_cur)], axis=1).astype(np.int32)
    state = np.concatenate([sa, sb], axis=1)
    for root_idx, acc, flag, tok in ((0, acc_a, fa, ta), (n_cur, acc_b + n_cur, fb, tb)):
        root = torch.empty((S, R), dtype=torch.int32, device=DEV)
        fill = torch.full((S, R), -1, dtype=torch.int32, device=DEV)
        base, n_masked = torch.full((S,), 3, dtype=torch.int32, device=DEV), torch.empty(S, dtype=torch.int32, device=DEV)
        status = torch.zeros(1, dtype=torch.int32, device=DEV)
        B.tsd_commit_accepted(_t(parent, torch.int32), _t(state, torch.int32), _t(acc, torch.int32),
                              _t(flag, torch.uint8), _t(tok, torch.int32), M, root_out=root, fill_step=fill,
                              step_base=base, n_masked=n_masked, status=status, tree_root=root_idx)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        for s in range(S):
            o = C.commit_accepted(parent[s], state[s], acc[s], flag[s], tok[s], M, 3, tree_root=root_idx)
            assert np.array_equal(root[s].cpu().numpy(), o["root"])
            assert np.array_equal(fill[s].cpu().numpy(), o["fill_step"])
            assert int(base[s]) == o["step_base"] and int(n_masked[s]) == o["n_masked"]
    # an accepted node of the other tree is outside this one: reported, U(root) only
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    root = torch.empty((S, R), dtype=torch.int32, device=DEV)
    B.tsd_commit_accepted(_t(parent, torch.int32), _t(state, torch.int32), _t(acc_a, torch.int32), None, None, M,
                          root_out=root, status=status, tree_root=n_cur)
    torch.cuda.synchronize()
    assert B.tsd_check_status(status) == B.TSD_ERR_DEVICE_DATA
    assert np.array_equal(root.cpu().numpy(), state[:, n_cur])


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_gather_accepted_kv_matches_oracle(dtype):
    # the accepted node's draft K/V rows -> a slot of the caller's cache, from strided views of a
    # fused projection output into a strided view of a wider cache tensor
    g = torch.Generator(device=DEV).manual_seed(3)
    S, Bn, R, H, d, rows = 5, 6, 32, 3, 128, 200
    qkv = torch.randn((S, Bn * R, 2 * H + 1, d), generator=g, device=DEV).to(dtype)
    k_draft, v_draft = qkv[:, :, 1:1 + H], qkv[:, :, 1 + H:]
    cache = torch.full((S, rows, 2 * H, d), 7.0, dtype=dtype, device=DEV)
    k_out, v_out = cache[:, :, :H], cache[:, :, H:]
    acc = torch.tensor([3, 0, 5, 1, 2], dtype=torch.int32, device=DEV)
    row0 = torch.tensor([0, 168, 10, 64, 96], dtype=torch.int32, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    B.tsd_gather_accepted_kv(acc, R, k_draft, v_draft, k_out, v_out, row0, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    wk = C.gather_accepted_kv(k_draft.float().cpu().numpy(), acc.cpu().numpy(), R)
    wv = C.gather_accepted_kv(v_draft.float().cpu().numpy(), acc.cpu().numpy(), R)
    want = np.full((S, rows, 2 * H, d), 7.0, np.float32)
    for s in range(S):
        r0 = int(row0[s])
        want[s, r0:r0 + R, :H] = wk[s]
        want[s, r0:r0 + R, H:] = wv[s]
    assert np.array_equal(cache.float().cpu().numpy(), want)       # a copy: bit-exact, nothing else touched
    # K only, default node (0) and default destination row (0)
    cache.fill_(7.0)
    B.tsd_gather_accepted_kv(None, R, k_draft, None, k_out, None)
    torch.cuda.synchronize()
    assert torch.equal(k_out[:, :R], k_draft[:, :R]) and (cache[:, R:] == 7.0).all() and (v_out == 7.0).all()
    # a node outside the tree, a destination past the end: reported, those sequences untouched
    cache.fill_(7.0)
    bad_acc = torch.tensor([3, 6, 5, -1, 2], dtype=torch.int32, device=DEV)
    bad_row0 = torch.tensor([0, 0, 169, 0, 96], dtype=torch.int32, device=DEV)
    B.tsd_gather_accepted_kv(bad_acc, R, k_draft, v_draft, k_out, v_out, bad_row0, status)
    torch.cuda.synchronize()
    assert B.tsd_check_status(status) == B.TSD_ERR_DEVICE_DATA
    assert (cache[1] == 7.0).all() and (cache[2] == 7.0).all() and (cache[3] == 7.0).all()
    assert torch.equal(k_out[0, :R], k_draft[0, 3 * R:4 * R]) and torch.equal(v_out[4, 96:96 + R], v_draft[4, 2 * R:3 * R])


def test_a_bounded_wait_that_runs_out_is_reported_and_the_context_stays_usable():
    # the library's bounded barrier wait on a barrier nothing completes: the kernel gives up after
    # the poll limit, returns by itself and raises the time-out bit; the device keeps working
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    B.tsd_selftest_bounded_wait(status, poll_limit=32)
    torch.cuda.synchronize()
    assert int(status.item()) == 1
    assert B.tsd_check_status(status) == B.TSD_ERR_TIMEOUT
    x = torch.arange(1000, device=DEV).sum().item()                # the context still answers
    assert x == 499500
    # the attention stage reports through the same word: a clean run leaves it at 0
    from paper_2608_27514_b200 import workloads as W
    cfg = W.small(W.CONFIGS["cfg2"], B=4, Nc=64, Hq=2, Hkv=2)
    step = VerifyStep.for_config(cfg, DEV)
    attn = W.attention_inputs(cfg, DEV)
    step.attention(attn["q"], attn["k_cache"], attn["v_cache"], attn["k_draft"], attn["v_draft"], attn["sm_scale"])
    torch.cuda.synchronize()
    assert B.tsd_check_status(step.status) == B.TSD_OK
