"""GPU parity: every stage of the verification step, called through the C ABI, against the CPU
oracle on the same seeded inputs.  Integer results (indices, validity, lengths) must be bit-exact;
attention within 2e-2 abs + 1e-2 rel for bf16 (1e-5 for fp32); probabilities within 1e-5."""
import numpy as np
import pytest
import torch

import oracle
from conftest import load_accept_cases
from paper_2608_27514_b200 import binding as B
from paper_2608_27514_b200 import workloads as W
from paper_2608_27514_b200.step import VerifyStep

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
PATHS = [pytest.param(0, id="default"), pytest.param(B.TSD_ATTN_FORCE_SIMT, id="simt")]


def _np(t):
    return t.detach().float().cpu().numpy() if t.dtype == torch.bfloat16 else t.detach().cpu().numpy()


def _attn_tol(cfg, ref):
    if cfg.dtype == "bf16":
        return 2e-2 + 1e-2 * np.abs(ref)
    return 1e-5 + 1e-5 * np.abs(ref)


def _run_attention(cfg, attn, flags, vis=None, cache_lens=None, want_dense=False):
    step = VerifyStep.for_config(cfg, DEV)
    dense = None
    if want_dense:
        dense = torch.empty((cfg.S, cfg.N, cfg.Nc + cfg.N), dtype=torch.uint8, device=DEV)
    step.build_mask(vis, cache_lens, dense)
    step.attention(attn["q"], attn["k_cache"], attn["v_cache"], attn["k_draft"], attn["v_draft"],
                   attn["sm_scale"], flags)
    torch.cuda.synchronize()
    step.check_status()
    return step, dense


def _compare_attention(step, cfg, attn, mask, heads=None, seqs=None):
    """`step.out` / `step.attn_lse` against the oracle; `heads`/`seqs` restrict the oracle to a sample."""
    seqs = list(range(cfg.S)) if seqs is None else seqs
    group = cfg.Hq // cfg.Hkv
    kv_heads = list(range(cfg.Hkv)) if heads is None else heads
    worst = 0.0
    for s in seqs:
        for g in kv_heads:
            hs = slice(g * group, (g + 1) * group)
            sl = lambda t, h: _np(t[s:s + 1][:, :, h])
            ref, ref_lse = oracle.masked_attention(
                sl(attn["q"], hs), sl(attn["k_cache"], slice(g, g + 1)), sl(attn["v_cache"], slice(g, g + 1)),
                sl(attn["k_draft"], slice(g, g + 1)), sl(attn["v_draft"], slice(g, g + 1)),
                mask[s:s + 1], attn["sm_scale"])
            got = _np(step.out[s:s + 1][:, :, hs]).astype(np.float64)
            err = np.abs(got - ref)
            assert (err <= _attn_tol(cfg, ref)).all(), "attention off by %g (seq %d kv head %d)" % (err.max(), s, g)
            got_lse = step.attn_lse[s:s + 1, hs].cpu().numpy()
            assert np.abs(got_lse - ref_lse).max() <= (2e-2 if cfg.dtype == "bf16" else 1e-4)
            worst = max(worst, err.max())
    return worst


def _check_attention(cfg, attn, flags, vis=None, cache_lens=None, heads=None, seqs=None):
    """Run the attention stage and compare with the oracle (dense mask bit for bit as well)."""
    step, dense = _run_attention(cfg, attn, flags, vis, cache_lens, want_dense=True)
    mask = oracle.dense_mask(cfg.S, cfg.B, cfg.R, cfg.Nc,
                             None if vis is None else vis.cpu().numpy(),
                             None if cache_lens is None else cache_lens.cpu().numpy())
    assert np.array_equal(dense.cpu().numpy(), mask)
    return _compare_attention(step, cfg, attn, mask, heads, seqs)


# ----------------------------------------------------------------------------- mask
@pytest.mark.parametrize("flags", PATHS)
def test_attention_reports_a_mask_built_for_another_layout(flags):
    cfg = W.small(W.CONFIGS["cfg2"], S=1, B=4, R=32, Nc=64, Hq=2, Hkv=2)
    other = VerifyStep.for_config(W.small(cfg, B=8), DEV)
    other.build_mask()                                  # a (larger) blob for 8 branches
    step = VerifyStep.for_config(cfg, DEV)
    step.mask, step.mask_built = other.mask, True
    step.out.fill_(7.0)
    attn = W.attention_inputs(cfg, DEV)
    step.attention(attn["q"], attn["k_cache"], attn["v_cache"], attn["k_draft"], attn["v_draft"], attn["sm_scale"],
                   flags)
    torch.cuda.synchronize()
    assert B.tsd_check_status(step.status) == B.TSD_ERR_DEVICE_DATA
    assert (step.out == 7.0).all()                      # nothing was written


def test_mask_dense_matches_oracle_with_vis_and_ragged_cache():
    cfg = W.small(W.CONFIGS["cfg2"], S=3, B=9, Nc=100, Hq=1, Hkv=1)
    rng = np.random.default_rng(0)
    vis = torch.from_numpy(rng.integers(0, 1 << 9, (cfg.S, cfg.B, 1)).astype(np.int64)).to(DEV)
    lens = torch.tensor([100, 0, 37], dtype=torch.int32, device=DEV)
    step = VerifyStep.for_config(cfg, DEV)
    dense = torch.empty((cfg.S, cfg.N, cfg.Nc + cfg.N), dtype=torch.uint8, device=DEV)
    step.build_mask(vis, lens, dense)
    torch.cuda.synchronize()
    ref = oracle.dense_mask(cfg.S, cfg.B, cfg.R, cfg.Nc, vis.cpu().numpy().astype(np.uint64), lens.cpu().numpy())
    assert np.array_equal(dense.cpu().numpy(), ref)


# ------------------------------------------------------------------------ attention
@pytest.mark.parametrize("flags", PATHS)
def test_attention_cfg1_fp32(flags):
    cfg = W.CONFIGS["cfg1"]
    worst = _check_attention(cfg, W.attention_inputs(cfg, DEV), flags)
    assert worst < 1e-5


@pytest.mark.parametrize("flags", PATHS)
@pytest.mark.parametrize("R", [32, 64, 128])
def test_attention_small_bf16_ragged_gqa(flags, R):
    # 5 branches: the last query tile is ragged; 4 query heads share 2 kv heads; ragged caches
    cfg = W.small(W.CONFIGS["cfg2"], S=2, B=5, R=R, Nc=300, Hq=4, Hkv=2)
    attn = W.attention_inputs(cfg, DEV)
    lens = torch.tensor([300, 173], dtype=torch.int32, device=DEV)
    _check_attention(cfg, attn, flags, cache_lens=lens)


@pytest.mark.parametrize("seed", range(12))
def test_attention_random_shapes_masks_and_cache_lengths(seed):
    # shapes, visibility bitsets and cache lengths drawn at random: partial query tiles, empty and
    # ragged caches, grouped heads, branches that read several others
    rng = np.random.default_rng(100 + seed)
    R = int(rng.choice([32, 64, 128]))
    Bn = int(rng.integers(1, 21 if R == 32 else 9))
    Hkv = int(rng.choice([1, 2]))
    Hq = Hkv * int(rng.choice([1, 2, 3]))
    cfg = W.small(W.CONFIGS["cfg2"], S=int(rng.integers(1, 4)), B=Bn, R=R, Nc=int(rng.choice([0, 1, 63, 64, 65, 200, 333])),
                  Hq=Hq, Hkv=Hkv)
    vis = np.zeros((cfg.S, Bn, 1), dtype=np.int64)
    for s_ in range(cfg.S):
        for b in range(Bn):
            if rng.random() < 0.4:
                vis[s_, b, 0] = int(rng.integers(0, 1 << Bn))
    cache_lens = None
    if cfg.Nc:
        cache_lens = torch.from_numpy(rng.integers(0, cfg.Nc + 1, cfg.S).astype(np.int32)).to(DEV)
    flags = B.TSD_ATTN_FORCE_SIMT if seed % 4 == 3 else 0
    _check_attention(cfg, W.attention_inputs(cfg, DEV), flags, vis=torch.from_numpy(vis).to(DEV), cache_lens=cache_lens)


@pytest.mark.parametrize("flags", PATHS)
def test_attention_strided_views_of_packed_tensors(flags):
    # Q / draft K / draft V as slices of one fused projection output, cached K / V as slices of one
    # cache tensor, the output as a view into a wider buffer: same bits as the contiguous call
    cfg = W.small(W.CONFIGS["cfg2"], S=2, B=5, R=32, Nc=200, Hq=4, Hkv=2)
    attn = W.attention_inputs(cfg, DEV)
    step, _ = _run_attention(cfg, attn, flags)
    ref_out, ref_lse = step.out.clone(), step.attn_lse.clone()
    qkv = torch.empty((cfg.S, cfg.N, cfg.Hq + 2 * cfg.Hkv, cfg.d), dtype=attn["q"].dtype, device=DEV)
    qkv[:, :, :cfg.Hq] = attn["q"]
    qkv[:, :, cfg.Hq:cfg.Hq + cfg.Hkv] = attn["k_draft"]
    qkv[:, :, cfg.Hq + cfg.Hkv:] = attn["v_draft"]
    cache = torch.empty((cfg.S, cfg.Nc, 2 * cfg.Hkv, cfg.d), dtype=attn["q"].dtype, device=DEV)
    cache[:, :, :cfg.Hkv] = attn["k_cache"]
    cache[:, :, cfg.Hkv:] = attn["v_cache"]
    wide = torch.full((cfg.S, cfg.N + 3, cfg.Hq + 1, cfg.d), 9.0, dtype=attn["q"].dtype, device=DEV)
    out = wide[:, 1:cfg.N + 1, :cfg.Hq]
    step2 = VerifyStep.for_config(cfg, DEV)
    step2.build_mask()
    step2.attention(qkv[:, :, :cfg.Hq], cache[:, :, :cfg.Hkv], cache[:, :, cfg.Hkv:],
                    qkv[:, :, cfg.Hq:cfg.Hq + cfg.Hkv], qkv[:, :, cfg.Hq + cfg.Hkv:], attn["sm_scale"], flags, out=out)
    torch.cuda.synchronize()
    step2.check_status()
    assert torch.equal(out, ref_out) and torch.equal(step2.attn_lse, ref_lse)
    # nothing outside the view was touched
    assert (wide[:, 0] == 9.0).all() and (wide[:, cfg.N + 1:] == 9.0).all() and (wide[:, :, cfg.Hq] == 9.0).all()


@pytest.mark.parametrize("flags", PATHS)
def test_attention_custom_visibility(flags):
    # asymmetric visibility as in the inter-block variant (Section 3.4): drafts read the root
    cfg = W.small(W.CONFIGS["cfg2"], S=2, B=7, R=32, Nc=128, Hq=2, Hkv=2)
    vis = np.zeros((cfg.S, cfg.B, 1), dtype=np.int64)
    vis[0, 1:, 0] = 1            # every draft of sequence 0 also reads branch 0
    vis[1, 0, 0] = 0b1111111     # the root of sequence 1 reads everything
    vis[1, 5, 0] = 0b0000110
    _check_attention(cfg, W.attention_inputs(cfg, DEV), flags, vis=torch.from_numpy(vis).to(DEV))


@pytest.mark.parametrize("flags", PATHS)
def test_attention_no_cache_and_tiny_cache(flags):
    for nc in (0, 16):
        cfg = W.small(W.CONFIGS["cfg2"], B=4, Nc=nc, Hq=2, Hkv=2)
        _check_attention(cfg, W.attention_inputs(cfg, DEV), flags)


@pytest.mark.parametrize("flags", PATHS)
def test_attention_poisoned_branches_do_not_leak(flags):
    cfg = W.small(W.CONFIGS["cfg2"], B=8, Nc=256, Hq=2, Hkv=2)
    clean = W.attention_inputs(cfg, DEV)
    keep = 5
    rows = slice(keep * cfg.R, (keep + 1) * cfg.R)
    base, _ = _run_attention(cfg, clean, flags)
    dirty, _ = _run_attention(cfg, W.poison_other_branches(cfg, clean, keep), flags)
    # the kept branch cannot see the poisoned ones: bit-identical output
    assert torch.equal(base.out[:, rows], dirty.out[:, rows])
    assert dirty.out[:, rows].float().abs().max() < 10.0


@pytest.mark.parametrize("flags", PATHS)
def test_attention_unreadable_rows_may_hold_anything(flags):
    # Inf / NaN in rows that no query row of a tile may read must not reach its output (a weight of
    # 0 times NaN is NaN): cached rows past cache_lens, whatever the unused capacity holds, and
    # the rows of the branches of a listed draft tile that the query tile cannot see.
    cfg = W.small(W.CONFIGS["cfg2"], S=2, B=8, R=32, Nc=200, Hq=2, Hkv=1)
    attn = W.attention_inputs(cfg, DEV)
    lens = torch.tensor([137, 64], dtype=torch.int32, device=DEV)
    for s_, n in enumerate(lens.tolist()):
        attn["k_cache"][s_, n:] = float("nan")
        attn["v_cache"][s_, n:] = float("inf")
        attn["v_cache"][s_, n::2] = float("nan")
    # query tile 0 (branches 0-3) lists draft tile 1 only because branch 0 reads branch 4: the
    # rows of branches 5-7 are loaded with it and are unreadable for every row of the tile
    vis = np.zeros((cfg.S, cfg.B, 1), dtype=np.int64)
    vis[:, 0, 0] = 1 << 4
    bad = slice(5 * cfg.R, 8 * cfg.R)
    attn["k_draft"][:, bad] = float("nan")
    attn["v_draft"][:, bad] = float("-inf")
    vis_t = torch.from_numpy(vis).to(DEV)
    step, _ = _run_attention(cfg, attn, flags, vis_t, lens)
    mask = oracle.dense_mask(cfg.S, cfg.B, cfg.R, cfg.Nc, vis.astype(np.uint64), lens.cpu().numpy())
    # branches 5-7 read their own NaN, and branch 4 shares its query tile with them (draft rows
    # that some row of a query tile may read have to be finite): unspecified
    good = slice(0, 4 * cfg.R)
    ref, ref_lse = oracle.masked_attention(_np(attn["q"]), _np(attn["k_cache"]), _np(attn["v_cache"]),
                                           _np(attn["k_draft"]), _np(attn["v_draft"]), mask, attn["sm_scale"])
    got = _np(step.out).astype(np.float64)[:, good]
    assert np.isfinite(got).all()
    assert (np.abs(got - ref[:, good]) <= _attn_tol(cfg, ref[:, good])).all()
    assert np.abs(step.attn_lse.cpu().numpy()[:, :, good] - ref_lse[:, :, good]).max() <= 2e-2


@pytest.mark.parametrize("flags", PATHS)
def test_attention_sharp_scores(flags):
    # queries scaled x4: near one-hot softmax rows, where a leaked or dropped key would show
    cfg = W.small(W.CONFIGS["cfg2"], B=8, Nc=512, Hq=2, Hkv=2)
    _check_attention(cfg, W.attention_inputs(cfg, DEV, q_gain=4.0), flags)


@pytest.mark.parametrize("flags", PATHS)
@pytest.mark.parametrize("name", ["cfg2", "cfg3"])
def test_attention_full_config(flags, name):
    cfg = W.CONFIGS[name]
    worst = _check_attention(cfg, W.attention_inputs(cfg, DEV), flags, heads=[0, 13, 31] if name == "cfg3" else None)
    assert worst < 1e-2


@pytest.mark.parametrize("name,seqs,heads", [("cfg4", [0, 15], [0, 31]), ("cfg5", [3], [0, 3])])
def test_attention_full_size_sampled(name, seqs, heads):
    # full-size launch as the benchmark times it; the oracle checks sampled (sequence, kv head) pairs
    cfg = W.CONFIGS[name]
    _check_attention(cfg, W.attention_inputs(cfg, DEV), 0, seqs=seqs, heads=heads)


def test_attention_is_deterministic():
    cfg = W.small(W.CONFIGS["cfg3"], Hq=4, Hkv=4)
    attn = W.attention_inputs(cfg, DEV)
    a, _ = _run_attention(cfg, attn, 0)
    b, _ = _run_attention(cfg, attn, 0)
    assert torch.equal(a.out, b.out) and torch.equal(a.attn_lse, b.attn_lse)


# ----------------------------------------------------------------- confidence / top-k
def _check_topk(logits, k, rows=None):
    n, V = logits.shape
    conf = torch.empty(n, dtype=torch.float32, device=DEV)
    idx = torch.empty((n, k), dtype=torch.int32, device=DEV)
    prob = torch.empty((n, k), dtype=torch.float32, device=DEV)
    lse = torch.empty(n, dtype=torch.float32, device=DEV)
    ws = torch.empty(max(16, B.tsd_confidence_topk_workspace_bytes(n, V, k)), dtype=torch.uint8, device=DEV)
    B.tsd_confidence_topk(logits, k, conf, idx, prob, lse, ws)
    torch.cuda.synchronize()
    sel = slice(None) if rows is None else torch.as_tensor(rows, device=DEV)
    host = _np(logits[sel])
    r_conf, r_idx, r_prob, r_lse = oracle.confidence_topk(host, k)
    assert np.array_equal(idx[sel].cpu().numpy(), r_idx)
    assert np.abs(conf[sel].cpu().numpy() - r_conf).max() <= 1e-5
    assert np.abs(prob[sel].cpu().numpy() - r_prob).max() <= 1e-5
    finite = np.isfinite(r_lse)
    assert np.abs(lse[sel].cpu().numpy()[finite] - r_lse[finite]).max() <= 1e-4
    return conf, idx, prob


@pytest.mark.parametrize("name", ["cfg1", "cfg2", "cfg3"])
def test_topk_full_config(name):
    cfg = W.CONFIGS[name]
    vi = W.verify_inputs(cfg, DEV)
    _check_topk(vi["logits"], cfg.k)


@pytest.mark.parametrize("name", ["cfg4", "cfg5"])
def test_topk_full_size_sampled(name):
    cfg = W.CONFIGS[name]
    vi = W.verify_inputs(cfg, DEV)
    rows = np.random.default_rng(1).choice(cfg.rows, 96, replace=False)
    rows.sort()
    _check_topk(vi["logits"], cfg.k, rows)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("k", [1, 2, 3, 4, 5, 8])
def test_topk_ragged_vocab_and_heavy_ties(dtype, k):
    g = torch.Generator(device=DEV).manual_seed(k)
    for n, V in ((7, 1000), (3, 40), (300, 2056), (5000, 520)):
        # rounding to halves makes most of the top entries tie: index order decides
        pitch = (V + 7) // 8 * 8 + 8          # rows padded: row pitch != vocabulary
        buf = (torch.randn((n, pitch), generator=g, device=DEV) * 2).mul(2).round().div(2).to(dtype)
        _check_topk(buf[:, :V], min(k, V))


@pytest.mark.parametrize("seed", range(10))
def test_topk_random_rows_vocab_k_and_dtype(seed):
    # sizes drawn at random: one value per row up to a wide vocabulary, one row up to several waves of
    # blocks, segmented and whole rows, ragged tails, a sharp peak in some rows, -inf in others
    rng = np.random.default_rng(500 + seed)
    V = int(rng.choice([1, 2, 7, 8, 9, 31, 257, 1000, 4099, 20000, 70001]))
    n = int(rng.choice([1, 2, 5, 40, 147, 149, 300, 700]))
    if n * V > 30_000_000:
        n = max(1, 30_000_000 // V)
    k = int(min(rng.integers(1, 9), V))
    dtype = torch.float32 if seed % 2 else torch.bfloat16
    pitch = (V + 7) // 8 * 8
    g = torch.Generator(device=DEV).manual_seed(seed)
    buf = (torch.randn((n, pitch), generator=g, device=DEV) * float(rng.choice([0.5, 3.0, 10.0]))).to(dtype)
    x = buf[:, :V]
    rows = torch.arange(n, device=DEV)
    x[rows[::3], torch.randint(0, V, (len(rows[::3]),), generator=g, device=DEV)] += 12.0      # sharp peaks
    if V > 4:
        x[rows[1::4], :2] = float("-inf")
    _check_topk(x, k)


def test_topk_minus_inf_and_split_rows():
    V = 126464
    g = torch.Generator(device=DEV).manual_seed(5)
    x = (torch.randn((6, V), generator=g, device=DEV) * 3).bfloat16()
    x[0, :] = float("-inf")
    x[0, 77] = 1.0                       # one finite entry: the rest tie at -inf, lowest indices first
    x[1, 5:] = float("-inf")
    x[2, V - 1] = 40.0                    # maximum in the last position of the last segment
    x[3, 0] = 40.0
    conf, idx, prob = _check_topk(x, 4)
    assert idx[0].tolist() == [77, 0, 1, 2] and prob[0, 1] == 0


@pytest.mark.parametrize("fill", ["ones", "random", "last_call"])
def test_topk_workspace_needs_no_clearing(fill):
    # few rows: each row is split over several blocks that meet through ticket words in the
    # workspace; whatever the workspace held before (all bits set, noise, the previous call's
    # leftovers), the results are the oracle's
    V, k = 50000, 3
    g = torch.Generator(device=DEV).manual_seed(11)
    x = (torch.randn((5, V), generator=g, device=DEV) * 3).bfloat16()
    nbytes = B.tsd_confidence_topk_workspace_bytes(5, V, k)
    assert nbytes > 0
    if fill == "ones":
        ws = torch.full((nbytes,), 0xFF, dtype=torch.uint8, device=DEV)
    else:
        ws = torch.randint(0, 256, (nbytes,), generator=g, device=DEV, dtype=torch.uint8)
    r_conf, r_idx, r_prob, _ = oracle.confidence_topk(_np(x), k)
    for call in range(3 if fill == "last_call" else 1):
        conf = torch.zeros(5, dtype=torch.float32, device=DEV)
        idx = torch.zeros((5, k), dtype=torch.int32, device=DEV)
        prob = torch.zeros((5, k), dtype=torch.float32, device=DEV)
        B.tsd_confidence_topk(x, k, conf, idx, prob, None, ws)
        torch.cuda.synchronize()
        assert np.array_equal(idx.cpu().numpy(), r_idx)
        assert np.abs(conf.cpu().numpy() - r_conf).max() <= 1e-5
        assert np.abs(prob.cpu().numpy() - r_prob).max() <= 1e-5


def test_topk_all_equal_rows_whole_and_split():
    # every value ties with the bound: far more candidates than the block's candidate pool holds,
    # so the lowest indices must come out of the slower merge path, for whole and for split rows
    for n, V in ((3, 126464), (200, 30000), (2, 777)):
        x = torch.full((n, (V + 7) // 8 * 8), 1.5, dtype=torch.bfloat16, device=DEV)[:, :V]
        x[0, V // 2:] = 2.0          # the upper half of row 0 ties at a higher value
        conf, idx, prob = _check_topk(x, 4)
        assert idx[0].tolist() == [V // 2 + j for j in range(4)]
        assert idx[1].tolist() == [0, 1, 2, 3]


def test_topk_is_deterministic():
    cfg = W.CONFIGS["cfg2"]
    vi = W.verify_inputs(cfg, DEV)
    outs = []
    for _ in range(3):
        s = VerifyStep.for_config(cfg, DEV)
        s.confidence_topk(vi["logits"])
        torch.cuda.synchronize()
        outs.append((s.conf.clone(), s.topk_idx.clone(), s.topk_prob.clone(), s.lse.clone()))
    for o in outs[1:]:
        assert all(torch.equal(a, b) for a, b in zip(outs[0], o))


# ------------------------------------------------------------------------ acceptance
def _gpu_accept(parent, state, mask_id, conf, top1, tau, rule, search, stride=1):
    S, Bn, R = state.shape
    t = lambda a, dt: torch.as_tensor(np.ascontiguousarray(a), dtype=dt, device=DEV)
    e = lambda shape, dt: torch.empty(shape, dtype=dt, device=DEV)
    out = dict(edge_valid=e((S, Bn), torch.uint8), prefix_len=e((S, Bn), torch.int32),
               accepted_node=e(S, torch.int32), accepted_len=e(S, torch.int32),
               n_new_tokens=e(S, torch.int32), unmask_flag=e((S, R), torch.uint8),
               unmask_tok=e((S, R), torch.int32))
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    B.tsd_accept_trajectories(t(parent, torch.int32), t(state, torch.int32), mask_id, t(conf, torch.float32),
                              t(top1, torch.int32), stride, tau, rule, search, status=status, **out)
    torch.cuda.synchronize()
    return {k: v.cpu().numpy() for k, v in out.items()}, status


CASES = [c for c in load_accept_cases() if c["rule"] <= 1]   # the relaxed rules: test_gpu_relaxed.py


@pytest.mark.parametrize("case", CASES, ids=[c["id"] for c in CASES])
def test_accept_hand_worked_trees(case):
    got, _ = _gpu_accept(case["parent"], case["state"], case["mask_id"], case["conf"], case["top1"],
                         case["tau"], case["rule"], case["search"])
    e = case["expect"]
    for key in ("edge_valid", "prefix_len", "unmask_flag", "unmask_tok"):
        assert got[key][0].tolist() == e[key], key
    for key in ("accepted_node", "accepted_len", "n_new_tokens"):
        assert int(got[key][0]) == e[key], key


@pytest.mark.parametrize("R", [4, 32, 64, 100])
def test_accept_random_trees_match_oracle(R):
    rng = np.random.default_rng(R)
    S, Bn, V = 33, 40, 50
    M = V
    parent = np.stack([[-1] + [int(rng.integers(0, b)) for b in range(1, Bn)] for _ in range(S)]).astype(np.int32)
    conf = rng.random((S, Bn, R)).astype(np.float32)
    conf[rng.random((S, Bn, R)) < 0.2] = 0.8           # exact ties with tau and among rows
    top1 = rng.integers(0, V, (S, Bn, R)).astype(np.int32)
    state = np.full((S, Bn, R), M, np.int32)
    for s in range(S):
        fill = rng.random(R) < 0.3
        state[s, 0, fill] = rng.integers(0, V, fill.sum())
        for b in range(1, Bn):
            p = parent[s, b]
            c = state[s, p].copy()
            flag, tok = oracle.decode_rule(state[s, p], M, conf[s, p], top1[s, p], 0.8)
            mode = rng.integers(0, 5)
            rows = np.flatnonzero(c == M)
            if mode <= 1:
                c[flag.astype(bool)] = tok[flag.astype(bool)]
            elif mode == 2 and len(rows):
                r = rows[rng.integers(len(rows))]
                c[r] = top1[s, p, r]
            elif mode == 3 and len(rows):
                c[rows[0]] = rng.integers(0, V)
            elif mode == 4:
                filled = np.flatnonzero(c != M)
                if len(filled):
                    c[filled[0]] = M if rng.random() < 0.5 else (c[filled[0]] + 1) % V   # malformed
            state[s, b] = c
    for rule in (0, 1):
        for search in (0, 1):
            ref = oracle.accept(parent, state, M, conf, top1, 0.8, rule, search)
            got, status = _gpu_accept(parent, state, M, conf, top1, 0.8, rule, search)
            for key, val in ref.items():
                assert np.array_equal(got[key], val), (key, rule, search)
            assert B.tsd_check_status(status) == B.TSD_OK


@pytest.mark.parametrize("seed", range(10))
def test_accept_random_shapes_chains_and_broken_parents(seed):
    # tree sizes and block lengths drawn at random, up to the limits (256 nodes, 128 rows); some
    # trees are long chains (the walk climbs many levels), some have parents that point nowhere
    # (an invalid edge hanging off nothing, whose descendants inherit a prefix of 0)
    rng = np.random.default_rng(9000 + seed)
    R = int(rng.choice([1, 4, 31, 32, 33, 64, 100, 128]))
    Bn = int(rng.choice([1, 2, 5, 8, 33, 64, 130, 256]))
    S, V = int(rng.integers(1, 6)), 50
    M = V
    deep = seed % 3 == 0
    parent = np.stack([[-1] + [int(b - 1 if deep and rng.random() < 0.8 else rng.integers(0, b))
                               for b in range(1, Bn)] for _ in range(S)]).astype(np.int32)
    broken = seed % 2 == 1 and Bn > 2
    if broken:
        for s in range(S):
            for b in rng.integers(1, Bn, 2):
                parent[s, b] = int(rng.choice([-1, b, b + 3, -5]))
    conf = rng.random((S, Bn, R)).astype(np.float32)
    conf[rng.random((S, Bn, R)) < 0.2] = 0.8
    top1 = rng.integers(0, V, (S, Bn, R)).astype(np.int32)
    state = np.full((S, Bn, R), M, np.int32)
    for s in range(S):
        fill = rng.random(R) < 0.3
        state[s, 0, fill] = rng.integers(0, V, fill.sum())
        for b in range(1, Bn):
            p = parent[s, b] if 0 <= parent[s, b] < b else 0
            c = state[s, p].copy()
            flag, tok = oracle.decode_rule(state[s, p], M, conf[s, p], top1[s, p], 0.8)
            mode = rng.integers(0, 5)
            rows = np.flatnonzero(c == M)
            if mode <= 2:
                c[flag.astype(bool)] = tok[flag.astype(bool)]
            elif mode == 3 and len(rows):
                r = rows[rng.integers(len(rows))]
                c[r] = top1[s, p, r]
            elif len(rows):
                c[rows[0]] = rng.integers(0, V)
            state[s, b] = c
    for rule in (0, 1):
        for search in (0, 1):
            ref = oracle.accept(parent, state, M, conf, top1, 0.8, rule, search)
            got, status = _gpu_accept(parent, state, M, conf, top1, 0.8, rule, search)
            for key, val in ref.items():
                assert np.array_equal(got[key], val), (key, rule, search)
            want = B.TSD_ERR_DEVICE_DATA if broken else B.TSD_OK
            assert B.tsd_check_status(status) == want


def test_accept_reports_bad_parent_without_faulting():
    parent = np.array([[-1, 0, 7, 1]], np.int32)       # node 2 points past itself
    state = np.full((1, 4, 32), 9, np.int32)
    conf = np.zeros((1, 4, 32), np.float32)
    top1 = np.zeros((1, 4, 32), np.int32)
    got, status = _gpu_accept(parent, state, 9, conf, top1, 0.9, 0, 0)
    assert B.tsd_check_status(status) == B.TSD_ERR_DEVICE_DATA
    assert got["edge_valid"][0, 2] == 0


# ---------------------------------------------------------------- the whole hot path
@pytest.mark.parametrize("name", ["cfg1", "cfg2", "cfg3"])
def test_whole_step_matches_oracle(name):
    cfg = W.CONFIGS[name]
    attn = W.attention_inputs(cfg, DEV)
    vi = W.verify_inputs(cfg, DEV)
    step = VerifyStep.for_config(cfg, DEV)
    res = step.run(attn, vi["logits"], vi["parent"], vi["state"], vi["mask_id"], cfg.tau)
    torch.cuda.synchronize()
    step.check_status()
    S, Bn, R = cfg.S, cfg.B, cfg.R
    conf, idx, prob, _ = oracle.confidence_topk(_np(vi["logits"]), cfg.k)
    assert np.array_equal(step.topk_idx.cpu().numpy(), idx)
    g_conf = step.conf.cpu().numpy()
    assert np.abs(g_conf - conf).max() <= 1e-5
    # (a) same fp32 confidences on both sides: every decision bit-exact
    same = oracle.accept(_np(vi["parent"]), _np(vi["state"]), vi["mask_id"], g_conf.reshape(S, Bn, R),
                         idx[:, 0].reshape(S, Bn, R), cfg.tau)
    # (b) the oracle's own chain (fp64 softmax rounded to fp32): the generator keeps confidences
    # clear of tau and of each other, so the decisions agree as well
    own = oracle.accept(_np(vi["parent"]), _np(vi["state"]), vi["mask_id"],
                        conf.astype(np.float32).reshape(S, Bn, R), idx[:, 0].reshape(S, Bn, R), cfg.tau)
    for key in same:
        assert np.array_equal(res[key].cpu().numpy(), same[key]), key
        assert np.array_equal(res[key].cpu().numpy(), own[key]), key
    # the plan the generator planted is what the decoder found
    assert int(res["edge_valid"].sum()) >= S


@pytest.mark.parametrize("name,seqs,heads", [("cfg4", [0, 9], [5, 31]), ("cfg5", [2], [1, 3])])
def test_whole_step_full_size_matches_oracle(name, seqs, heads):
    # the two large workloads through VerifyStep.run, as the benchmark launches them: the oracle
    # scores EVERY row of the vocabulary pass (logits streamed to the host in slabs), the
    # acceptance runs on the full planted trees, attention is compared on sampled (sequence, kv
    # head) pairs (its fp64 oracle needs minutes for the whole batch)
    cfg = W.CONFIGS[name]
    attn = W.attention_inputs(cfg, DEV)
    vi = W.verify_inputs(cfg, DEV)
    step = VerifyStep.for_config(cfg, DEV)
    res = step.run(attn, vi["logits"], vi["parent"], vi["state"], vi["mask_id"], cfg.tau)
    torch.cuda.synchronize()
    step.check_status()
    S, Bn, R = cfg.S, cfg.B, cfg.R
    g_idx, g_conf, g_prob = step.topk_idx.cpu().numpy(), step.conf.cpu().numpy(), step.topk_prob.cpu().numpy()
    conf = np.empty(cfg.rows, np.float64)
    top1 = np.empty(cfg.rows, np.int32)
    slab = 1024
    for r0 in range(0, cfg.rows, slab):
        r1 = min(cfg.rows, r0 + slab)
        o_conf, o_idx, o_prob, _ = oracle.confidence_topk(_np(vi["logits"][r0:r1]), cfg.k)
        assert np.array_equal(g_idx[r0:r1], o_idx), "top-k indices, rows %d..%d" % (r0, r1)
        assert np.abs(g_conf[r0:r1] - o_conf).max() <= 1e-5
        assert np.abs(g_prob[r0:r1] - o_prob).max() <= 1e-5
        conf[r0:r1], top1[r0:r1] = o_conf, o_idx[:, 0]
    parent, state = _np(vi["parent"]), _np(vi["state"])
    same = oracle.accept(parent, state, vi["mask_id"], g_conf.reshape(S, Bn, R), top1.reshape(S, Bn, R), cfg.tau)
    own = oracle.accept(parent, state, vi["mask_id"], conf.astype(np.float32).reshape(S, Bn, R),
                        top1.reshape(S, Bn, R), cfg.tau)
    for key in same:
        assert np.array_equal(res[key].cpu().numpy(), same[key]), key
        assert np.array_equal(res[key].cpu().numpy(), own[key]), key
    assert int(res["accepted_len"].sum()) > 0            # planted continuations really are accepted
    mask = oracle.dense_mask(cfg.S, cfg.B, cfg.R, cfg.Nc)
    _compare_attention(step, cfg, attn, mask, heads=heads, seqs=seqs)


def test_topk_subnormal_and_signed_zero_logits():
    # thresholds that sit at +-0 or at subnormal bf16 values must still order exactly
    V = 4096
    x = torch.full((4, V), -1.0, dtype=torch.bfloat16, device=DEV)
    tiny = torch.tensor([1e-40], dtype=torch.float32).bfloat16().item()   # a subnormal bf16
    x[0, 100], x[0, 2000], x[0, 3000], x[0, 50] = 0.0, -0.0, tiny, 2 * tiny
    x[1, :] = -0.0
    x[1, 3000] = 0.0
    x[2, :] = tiny
    x[2, 7] = 2 * tiny
    x[2, 4000] = 3 * tiny
    x[3, :] = -tiny
    x[3, 9], x[3, 10] = -0.0, 0.0
    _check_topk(x, 4)


# ------------------------------------------------------------------------ extremes
@pytest.mark.parametrize("flags", PATHS)
def test_attention_many_branches_all_visible(flags):
    # 256 branches (the maximum) that all see each other: every query tile lists all 64 draft tiles
    cfg = W.small(W.CONFIGS["cfg2"], B=256, R=32, Nc=64, Hq=1, Hkv=1)
    vis = torch.full((cfg.S, cfg.B, 4), -1, dtype=torch.int64, device=DEV)
    _check_attention(cfg, W.attention_inputs(cfg, DEV), flags, vis=vis)


@pytest.mark.parametrize("flags", PATHS)
def test_attention_batch_with_an_empty_cache(flags):
    # one sequence of the batch has no valid cached token at all: only its own branch is visible
    cfg = W.small(W.CONFIGS["cfg2"], S=3, B=4, R=64, Nc=200, Hq=2, Hkv=1)
    lens = torch.tensor([200, 0, 1], dtype=torch.int32, device=DEV)
    _check_attention(cfg, W.attention_inputs(cfg, DEV), flags, cache_lens=lens)


def test_topk_k_equals_vocab_and_single_row():
    g = torch.Generator(device=DEV).manual_seed(9)
    x = torch.randn((5, 8), generator=g, device=DEV).bfloat16()
    _check_topk(x, 8)                                  # every entry is a candidate
    y = torch.randn((1, 300000), generator=g, device=DEV)
    _check_topk(y, 8)                                  # one long fp32 row: segments + ticket merge
    z = torch.randn((3, 16), generator=g, device=DEV)
    _check_topk(z[:, :1], 1)                           # vocabulary of one


def test_accept_largest_tree():
    rng = np.random.default_rng(3)
    S, Bn, R, V = 2, 256, 128, 1000
    M = V
    parent = np.stack([[-1] + [int(rng.integers(max(0, b - 3), b)) for b in range(1, Bn)] for _ in range(S)]).astype(np.int32)
    conf = rng.random((S, Bn, R)).astype(np.float32)
    top1 = rng.integers(0, V, (S, Bn, R)).astype(np.int32)
    state = np.full((S, Bn, R), M, np.int32)
    for s in range(S):
        for b in range(1, Bn):
            p = parent[s, b]
            c = state[s, p].copy()
            flag, tok = oracle.decode_rule(state[s, p], M, conf[s, p], top1[s, p], 0.97)
            if rng.random() < 0.8:
                c[flag.astype(bool)] = tok[flag.astype(bool)]
            else:
                rows = np.flatnonzero(c == M)
                if len(rows):
                    c[rows[-1]] = rng.integers(0, V)
            state[s, b] = c
    for rule in (0, 1):
        for search in (0, 1):
            ref = oracle.accept(parent, state, M, conf, top1, 0.97, rule, search)
            got, status = _gpu_accept(parent, state, M, conf, top1, 0.97, rule, search)
            for key, val in ref.items():
                assert np.array_equal(got[key], val), (key, rule, search)
            assert ref["accepted_len"].max() > 3          # deep chains really are accepted
