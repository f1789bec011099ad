"""Pins for the inter-block oracle (Section 3.4, Eq. 3, Appendix D): a hand-written mask and truth
table, closed forms for the visible-key counts, the reduction to a two-block bidirectional window
(textbook attention written here with numpy), and isolation from other drafts."""
import os

import numpy as np
import pytest

import oracle
from oracle import interblock

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "interblock_mask.txt")


def _golden():
    head, rows, trig = None, [], []
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        f = line.split()
        if f[0] == "n_cache":
            head = dict(zip(f[0::2], map(int, f[1::2])))
        elif f[0] == "trigger":
            trig.append((float(f[1]), float(f[2]), float(f[3]), bool(int(f[4]))))
        else:
            rows.append([int(ch) for ch in "".join(f)])
    return head, np.array(rows, dtype=np.uint8), trig


def _dense(B, R, Nc, n_cur):
    return oracle.dense_mask(1, B, R, Nc, vis=interblock.interblock_vis(B, n_cur)[None])[0]


def test_mask_matches_hand_written_case():
    head, expect, _ = _golden()
    m = _dense(head["n_branches"], head["rows_per_branch"], head["n_cache"], head["n_cur"])
    assert np.array_equal(m, expect)


def test_trigger_truth_table():
    _, _, trig = _golden()
    M = 7
    for c_cur, c_next, tau, want in trig:
        # the block maxima sit among lower confidences; filled rows carry a high confidence that
        # must be ignored
        state_cur = np.array([3, M, M, M], np.int32)
        conf_cur = np.array([0.99, c_cur, c_cur - 0.1, 0.0], np.float32)
        state_next = np.array([M, M, 5, M], np.int32)
        conf_next = np.array([c_next - 0.2, c_next, 0.999, 0.1], np.float32)
        assert interblock.interblock_trigger(state_cur, conf_cur, state_next, conf_next, M, tau) is want


def test_trigger_degenerate_blocks():
    M = 7
    full = np.array([1, 2], np.int32)
    open_ = np.array([M, M], np.int32)
    c = np.array([0.3, 0.2], np.float32)
    # a finished current block has no top confidence: any open next block triggers
    assert interblock.interblock_trigger(full, c, open_, c, M, 0.9) is True
    # a finished next block has nothing to draft
    assert interblock.interblock_trigger(open_, c, full, c, M, 0.9) is False


@pytest.mark.parametrize("B,n_cur,R,Nc", [(5, 3, 2, 1), (14, 10, 4, 3), (70, 66, 1, 0), (130, 3, 1, 2)])
def test_mask_closed_forms(B, n_cur, R, Nc):
    m = _dense(B, R, Nc, n_cur)
    # every row reads the cache, its own branch and exactly one other branch (a root)
    assert (m.sum(axis=1) == Nc + 2 * R).all()
    blk = m[:, Nc:].reshape(B, R, B, R)
    assert (blk == blk[:, :1, :, :1]).all()          # visibility is per branch pair
    v = blk[:, 0, :, 0].astype(bool)
    assert v.diagonal().all()
    off = v & ~np.eye(B, dtype=bool)
    # the only mutual pair is the two roots; nobody reads a draft
    assert np.array_equal(np.argwhere(off & off.T), [[0, n_cur], [n_cur, 0]])
    drafts = [b for b in range(B) if b not in (0, n_cur)]
    assert not off[:, drafts].any()
    assert off[:n_cur, n_cur].all() and off[n_cur:, 0].all()


def test_no_next_tree_is_the_isolated_mask():
    assert np.array_equal(_dense(6, 3, 4, 6), oracle.dense_mask(1, 6, 3, 4)[0])


def _textbook(q, k, v, scale):
    a = (q.astype(np.float64) @ k.astype(np.float64).T) * scale
    a -= a.max(axis=1, keepdims=True)
    p = np.exp(a)
    return (p / p.sum(axis=1, keepdims=True)) @ v.astype(np.float64)


def test_joint_pass_reduces_to_two_block_windows():
    # each branch of a joint pass is ordinary attention over cache + itself + the root it reads;
    # for the roots that is the bidirectional two-block window of Section 3.4
    rng = np.random.default_rng(5)
    B, n_cur, R, Nc, H, d = 6, 4, 5, 7, 2, 8
    N = B * R
    q = rng.standard_normal((1, N, H, d)).astype(np.float32)
    kc, vc = (rng.standard_normal((1, Nc, H, d)).astype(np.float32) for _ in range(2))
    kd, vd = (rng.standard_normal((1, N, H, d)).astype(np.float32) for _ in range(2))
    mask = _dense(B, R, Nc, n_cur)[None]
    out, _ = oracle.masked_attention(q, kc, vc, kd, vd, mask, 0.3)
    rows = lambda b: slice(b * R, (b + 1) * R)
    for b in range(B):
        other = n_cur if b < n_cur else 0
        for h in range(H):
            k = np.concatenate([kc[0, :, h], kd[0, rows(b), h], kd[0, rows(other), h]])
            v = np.concatenate([vc[0, :, h], vd[0, rows(b), h], vd[0, rows(other), h]])
            np.testing.assert_allclose(out[0, rows(b), h], _textbook(q[0, rows(b), h], k, v, 0.3),
                                       rtol=1e-12, atol=1e-12)
    # what was drafted never reaches a root or another draft
    kd2, vd2 = kd.copy(), vd.copy()
    kd2[0, rows(1)] += 100.0
    vd2[0, rows(5)] -= 50.0
    out2, _ = oracle.masked_attention(q, kc, vc, kd2, vd2, mask, 0.3)
    keep = [b for b in range(B) if b not in (1, 5)]
    for b in keep:
        assert np.array_equal(out[0, rows(b)], out2[0, rows(b)])


def test_joint_accept_is_two_single_tree_acceptances(accept_cases):
    # glue two hand-worked single-tree cases into one forest: every per-tree result must equal the
    # hand-worked expectation of that case
    M = 99
    by_shape = {}
    for c in accept_cases:
        if c["rule"] > 1:          # the relaxed rules need more inputs than this glue passes on
            continue
        by_shape.setdefault((c["state"].shape[2], c["rule"], c["search"], c["tau"]), []).append(c)
    pairs = [(v[0], v[-1]) for v in by_shape.values() if len(v) >= 2]
    assert pairs
    for a, b in pairs:
        n_cur = a["state"].shape[1]
        parent_b = b["parent"].copy()
        parent_b[:, 1:] += n_cur
        parent_b[:, 0] = -1
        parent = np.concatenate([a["parent"], parent_b], axis=1)
        cat = lambda key: np.concatenate([a[key], b[key]], axis=1)
        o = interblock.joint_accept(parent, cat("state"), n_cur, M, cat("conf"), cat("top1"), a["tau"],
                                    a["rule"], a["search"])
        assert o["accepted_node"][0, 0] == a["expect"]["accepted_node"]
        assert o["accepted_node"][1, 0] == b["expect"]["accepted_node"] + n_cur
        assert o["accepted_len"][0, 0] == a["expect"]["accepted_len"]
        assert o["accepted_len"][1, 0] == b["expect"]["accepted_len"]
