"""Pins for the oracle's mask and masked attention (Section 3.3).  Each check
compares the C oracle with something that is not the oracle: a textbook
formula written here with numpy, a closed form, or an invariant."""
import numpy as np
import pytest

import oracle


def _rand(rng, *shape):
    return rng.standard_normal(shape).astype(np.float32)


def _inputs(rng, S, B, R, Nc, Hq, Hkv, d):
    N = B * R
    return (_rand(rng, S, N, Hq, d), _rand(rng, S, Nc, Hkv, d), _rand(rng, S, Nc, Hkv, d),
            _rand(rng, S, N, Hkv, d), _rand(rng, S, N, Hkv, d))


def _textbook(q, k, v, scale):
    """softmax(q k^T * scale) v for one head, all keys visible."""
    a = (q.astype(np.float64) @ k.astype(np.float64).T) * scale
    a = a - a.max(axis=1, keepdims=True)
    p = np.exp(a)
    p /= p.sum(axis=1, keepdims=True)
    return p @ v.astype(np.float64)


def test_mask_rules_small():
    # two branches of two rows over three cached tokens, written out by hand
    m = oracle.dense_mask(1, 2, 2, 3)[0]
    expect = np.array([[1, 1, 1, 1, 1, 0, 0],
                       [1, 1, 1, 1, 1, 0, 0],
                       [1, 1, 1, 0, 0, 1, 1],
                       [1, 1, 1, 0, 0, 1, 1]], dtype=np.uint8)
    assert np.array_equal(m, expect)


def test_mask_cache_lens_and_vis():
    vis = np.zeros((2, 3, 1), dtype=np.uint64)
    vis[0, 2, 0] = 0b001          # seq 0: branch 2 also reads branch 0 (not symmetric)
    vis[1, 0, 0] = 0b110          # seq 1: branch 0 reads branches 1 and 2
    m = oracle.dense_mask(2, 3, 2, 4, vis=vis, cache_lens=np.array([4, 2], np.int32))
    # cached part
    assert m[0, :, :4].all() and m[1, :, :2].all() and not m[1, :, 2:4].any()
    d0 = m[0, :, 4:].reshape(3, 2, 3, 2)[:, 0, :, 0]
    d1 = m[1, :, 4:].reshape(3, 2, 3, 2)[:, 0, :, 0]
    assert np.array_equal(d0, [[1, 0, 0], [0, 1, 0], [1, 0, 1]])
    assert np.array_equal(d1, [[1, 1, 1], [0, 1, 0], [0, 0, 1]])


def test_single_branch_is_ordinary_attention():
    # a one-node tree is non-speculative blockwise decoding: R rows over Nc + R keys
    rng = np.random.default_rng(1)
    S, B, R, Nc, Hq, Hkv, d = 2, 1, 8, 11, 3, 3, 16
    q, kc, vc, kd, vd = _inputs(rng, S, B, R, Nc, Hq, Hkv, d)
    out, lse = oracle.masked_attention(q, kc, vc, kd, vd, oracle.dense_mask(S, B, R, Nc), 0.25)
    for s in range(S):
        for h in range(Hq):
            k = np.concatenate([kc[s, :, h], kd[s, :, h]])
            v = np.concatenate([vc[s, :, h], vd[s, :, h]])
            ref = _textbook(q[s, :, h], k, v, 0.25)
            assert np.abs(out[s, :, h] - ref).max() < 1e-12


def test_full_visibility_is_plain_bidirectional_attention():
    rng = np.random.default_rng(2)
    S, B, R, Nc, Hq, Hkv, d = 1, 3, 4, 5, 2, 2, 8
    q, kc, vc, kd, vd = _inputs(rng, S, B, R, Nc, Hq, Hkv, d)
    vis = np.full((S, B, 1), 0b111, dtype=np.uint64)
    mask = oracle.dense_mask(S, B, R, Nc, vis=vis)
    assert mask.all()
    out, _ = oracle.masked_attention(q, kc, vc, kd, vd, mask, 0.3)
    for h in range(Hq):
        k = np.concatenate([kc[0, :, h], kd[0, :, h]])
        v = np.concatenate([vc[0, :, h], vd[0, :, h]])
        assert np.abs(out[0, :, h] - _textbook(q[0, :, h], k, v, 0.3)).max() < 1e-12


def test_brute_force_gathered_keys_gqa_ragged():
    # per row: gather exactly the keys the two rules allow, then textbook attention
    rng = np.random.default_rng(3)
    S, B, R, Nc, Hq, Hkv, d = 2, 4, 3, 7, 4, 2, 8
    N = B * R
    q, kc, vc, kd, vd = _inputs(rng, S, B, R, Nc, Hq, Hkv, d)
    lens = np.array([7, 4], np.int32)
    out, lse = oracle.masked_attention(q, kc, vc, kd, vd,
                                       oracle.dense_mask(S, B, R, Nc, cache_lens=lens), 0.5)
    for s in range(S):
        for h in range(Hq):
            g = h // (Hq // Hkv)
            for i in range(N):
                b = i // R
                keys = [kc[s, j, g] for j in range(lens[s])] + [kd[s, b * R + r, g] for r in range(R)]
                vals = [vc[s, j, g] for j in range(lens[s])] + [vd[s, b * R + r, g] for r in range(R)]
                a = np.array([0.5 * float(np.dot(q[s, i, h].astype(np.float64), kk.astype(np.float64)))
                              for kk in keys])
                w = np.exp(a - a.max())
                ref = (w[:, None] * np.array(vals, dtype=np.float64)).sum(0) / w.sum()
                assert np.abs(out[s, i, h] - ref).max() < 1e-12
                assert abs(lse[s, h, i] - (a.max() + np.log(w.sum()))) < 1e-12


def test_branch_independence_is_bit_exact():
    rng = np.random.default_rng(4)
    S, B, R, Nc, Hq, Hkv, d = 1, 4, 4, 6, 2, 1, 8
    q, kc, vc, kd, vd = _inputs(rng, S, B, R, Nc, Hq, Hkv, d)
    mask = oracle.dense_mask(S, B, R, Nc)
    out1, _ = oracle.masked_attention(q, kc, vc, kd, vd, mask, 0.35)
    keep = slice(2 * R, 3 * R)
    q2, kd2, vd2 = (100 * _rand(rng, *a.shape) for a in (q, kd, vd))
    for a, a2 in ((q, q2), (kd, kd2), (vd, vd2)):
        a2[:, keep] = a[:, keep]
    out2, _ = oracle.masked_attention(q2, kc, vc, kd2, vd2, mask, 0.35)
    assert np.array_equal(out1[:, keep], out2[:, keep])


def test_closed_forms():
    rng = np.random.default_rng(5)
    S, B, R, Nc, Hq, Hkv, d = 1, 2, 4, 5, 1, 1, 8
    q, kc, vc, kd, vd = _inputs(rng, S, B, R, Nc, Hq, Hkv, d)
    mask = oracle.dense_mask(S, B, R, Nc)
    # q = 0: uniform weights, output = mean of the visible value rows, lse = log(#visible)
    out, lse = oracle.masked_attention(np.zeros_like(q), kc, vc, kd, vd, mask, 1.0)
    for b in range(B):
        mean = np.concatenate([vc[0, :, 0], vd[0, b * R:(b + 1) * R, 0]]).astype(np.float64).mean(0)
        assert np.abs(out[0, b * R:(b + 1) * R, 0] - mean).max() < 1e-14
    assert np.abs(lse - np.log(Nc + R)).max() < 1e-14
    # constant V: output is that constant
    out, _ = oracle.masked_attention(q, kc, np.full_like(vc, 0.75), kd, np.full_like(vd, 0.75), mask, 1.0)
    assert np.abs(out - 0.75).max() < 1e-14
    # one cached key 40 above every other score: output is its value row
    kc2 = np.zeros_like(kc)
    q2 = np.zeros_like(q)
    q2[..., 0] = 1.0
    kc2[0, 3, 0, 0] = 40.0
    out, _ = oracle.masked_attention(q2, kc2, vc, np.zeros_like(kd), vd, mask, 1.0)
    assert np.abs(out[0, :, 0] - vc[0, 3, 0].astype(np.float64)).max() < 1e-15


def test_permuting_cached_keys_changes_nothing_and_output_is_convex():
    rng = np.random.default_rng(6)
    S, B, R, Nc, Hq, Hkv, d = 1, 3, 4, 9, 2, 2, 8
    q, kc, vc, kd, vd = _inputs(rng, S, B, R, Nc, Hq, Hkv, d)
    mask = oracle.dense_mask(S, B, R, Nc)
    out1, lse1 = oracle.masked_attention(q, kc, vc, kd, vd, mask, 0.4)
    perm = rng.permutation(Nc)
    out2, lse2 = oracle.masked_attention(q, kc[:, perm], vc[:, perm], kd, vd, mask, 0.4)
    assert np.abs(out1 - out2).max() < 1e-13 and np.abs(lse1 - lse2).max() < 1e-13
    vmax = max(np.abs(vc).max(), np.abs(vd).max())
    assert np.abs(out1).max() <= vmax + 1e-12


def test_lse_merge_identity():
    # attention over cache-only and over own-branch-only, merged by their lse
    # weights, equals the one-shot result (the basis of split-KV evaluation)
    rng = np.random.default_rng(7)
    S, B, R, Nc, Hq, Hkv, d = 1, 2, 4, 6, 2, 2, 8
    N = B * R
    q, kc, vc, kd, vd = _inputs(rng, S, B, R, Nc, Hq, Hkv, d)
    full = oracle.dense_mask(S, B, R, Nc)
    out, lse = oracle.masked_attention(q, kc, vc, kd, vd, full, 0.4)
    m_cache = full.copy()
    m_cache[:, :, Nc:] = 0
    m_own = full.copy()
    m_own[:, :, :Nc] = 0
    o1, l1 = oracle.masked_attention(q, kc, vc, kd, vd, m_cache, 0.4)
    o2, l2 = oracle.masked_attention(q, kc, vc, kd, vd, m_own, 0.4)
    l1t, l2t = l1.transpose(0, 2, 1)[..., None], l2.transpose(0, 2, 1)[..., None]
    lm = np.logaddexp(l1t, l2t)
    merged = np.exp(l1t - lm) * o1 + np.exp(l2t - lm) * o2
    assert np.abs(merged - out).max() < 1e-12
    assert np.abs(lm[..., 0].transpose(0, 2, 1) - lse).max() < 1e-12


def test_generated_workload_shapes():
    from paper_2608_27514_b200 import workloads as W
    cfg = W.CONFIGS["cfg1"]
    a = W.attention_inputs(cfg)
    assert a["q"].shape == (1, 128, 4, 64) and a["k_cache"].shape == (1, 256, 4, 64)
    assert W.tree_parents(cfg) == [-1, 0, 0, 1]            # W2D2(3), Section 3.2
    for name, rows, keys in (("cfg2", 256, 768), ("cfg3", 1024, 1536), ("cfg4", 16384, 1536),
                             ("cfg5", 16384, 5120)):
        c = W.CONFIGS[name]
        assert c.rows == rows and c.Nc + c.R == keys
        par = W.tree_parents(c)
        assert par[0] == -1 and all(0 <= par[b] < b for b in range(1, c.B))
    # Prop. 1's worked number (printed as "about 45.6"): 0.85*32 + 0.85*0.68*32
    assert abs(0.85 * 32 + 0.85 * 0.68 * 32 - 45.7) < 0.05
