"""Toy-model harness for the exactness theorem (Theorem 1; test infrastructure).

Theorem 1: with cached prefix/suffix K/V, no inter-block speculation and
deterministic decoding, the speculative decoder emits the same sequence of
(position, token) unmask events as the sequential dual-cache decoder.  The
paper checks it on real models (App. "Exactness Proof and Empirical
Verification": 100 % token match, 0.00 logit error); here the "model" is a
small deterministic fp64 network whose only mixing layer is the oracle's
masked attention over a fixed random cache plus the node's own rows.

  sequential:   s <- s + U(f(s))                                    until full
  speculative:  score root s and its draft children in ONE masked call,
                accept by the oracle's rule, s <- state[acc] + U(acc)

Both use oracle.decode_rule for U and oracle.accept for the tree walk; the
batched forward uses oracle.dense_mask + oracle.masked_attention.
"""
import numpy as np

from . import binding as _o


class ToyModel:
    def __init__(self, seed, V=64, d=16, R=8, Nc=16, gain=6.0):
        rng = np.random.Generator(np.random.PCG64(seed))
        self.V, self.d, self.R, self.Nc = V, d, R, Nc
        self.mask_id = V  # one extra embedding row for [MASK]
        self.E = rng.standard_normal((V + 1, d))
        self.P = rng.standard_normal((R, d))
        self.Wq, self.Wk, self.Wv = (rng.standard_normal((d, d)) / np.sqrt(d) for _ in range(3))
        self.Wo = rng.standard_normal((d, V)) * gain / np.sqrt(d)
        # fp32-representable cache (the oracle takes fp32 carriers)
        self.kc = rng.standard_normal((1, Nc, 1, d)).astype(np.float32)
        self.vc = rng.standard_normal((1, Nc, 1, d)).astype(np.float32)

    def _qkv(self, states):
        """states [B,R] -> x, q, k, v with B*R rows (fp32-representable)."""
        B, R = states.shape
        x = self.E[states.reshape(-1)] + np.tile(self.P, (B, 1))
        f32 = lambda a: a.astype(np.float32).reshape(1, B * R, 1, self.d)
        return x, f32(x @ self.Wq), f32(x @ self.Wk), f32(x @ self.Wv)

    def logits(self, states):
        """One masked call over all nodes: logits [B,R,V], branches isolated
        (Section 3.3)."""
        states = np.asarray(states)
        B, R = states.shape
        x, q, k, v = self._qkv(states)
        mask = _o.dense_mask(1, B, R, self.Nc)
        att, _ = _o.masked_attention(q, self.kc, self.vc, k, v, mask, 1.0 / np.sqrt(self.d))
        h = x + att.reshape(B * R, self.d)
        return (h @ self.Wo).reshape(B, R, self.V)


def _score(model, states):
    """conf (fp32), top-1 and top-3 per row through the oracle's Eq. 2."""
    B, R = np.asarray(states).shape
    full = model.logits(states)
    lg = full.astype(np.float32).reshape(B * R, model.V)
    conf, idx, prob, _ = _o.confidence_topk(lg, 3)
    return (conf.astype(np.float32).reshape(B, R), idx.reshape(B, R, 3), prob.reshape(B, R, 3), full)


def sequential_decode(model, s0, tau):
    """Threshold decoding one step at a time; returns the list of unmask
    events, one frozenset of (row, token) per step."""
    s = np.array(s0, dtype=np.int32)
    traj = []
    while (s == model.mask_id).any():
        conf, idx, _, _ = _score(model, s[None])
        flag, tok = _o.decode_rule(s, model.mask_id, conf[0], idx[0, :, 0], tau)
        traj.append(frozenset((int(r), int(tok[r])) for r in np.flatnonzero(flag)))
        s = np.where(flag.astype(bool), tok, s).astype(np.int32)
    return traj, s


def _draft(model, root, conf, idx, prob, mode, rng, tau, peek):
    """Children of the root and one grandchild under the first child.

    heuristic: guess from the previous forward's scores that the next step
    unmasks the best remaining rows (level 1: three alternatives; deeper: the
    parent's best unused candidate).  peek: the true next steps (so deep
    acceptance is exercised), with one deliberately wrong sibling.  random:
    arbitrary fills (always rejected unless lucky).
    """
    R = root.shape[0]
    masked = [int(r) for r in np.flatnonzero(root == model.mask_id)]
    nodes, parent = [root.copy()], [-1]

    def add(par, fills):
        c = nodes[par].copy()
        for r, t in fills:
            c[r] = t
        nodes.append(c)
        parent.append(par)
        return len(nodes) - 1

    if not masked:
        return np.stack(nodes), parent
    if mode == "alg1":
        # the library's reading of Alg. 1 Phase 2 on the previous pass's candidate pool (W2D2(3))
        n, par, st, _ = _o.build_draft_tree(root, model.mask_id, idx, prob.astype(np.float32), 2, 2, 4)
        return st[:n].astype(np.int32), [int(x) for x in par[:n]]
    if mode == "peek":
        steps = peek[:3]
        wrong_r = masked[int(rng.integers(len(masked)))]
        add(0, [(wrong_r, int(rng.integers(model.V)))])       # wrong sibling first
        if steps:
            c1 = add(0, sorted(steps[0]))
            if len(steps) > 1:
                c2 = add(c1, sorted(steps[1]))
                add(c1, [(r, (t + 1) % model.V) for r, t in sorted(steps[1])])  # wrong token
                if len(steps) > 2:
                    add(c2, sorted(steps[2]))
    elif mode == "random":
        for _ in range(3):
            r = masked[int(rng.integers(len(masked)))]
            add(0, [(r, int(rng.integers(model.V)))])
        if nodes[1][masked[-1]] == model.mask_id:
            add(1, [(masked[-1], int(rng.integers(model.V)))])
    else:
        order = sorted(masked, key=lambda r: -conf[r])
        hi = [r for r in masked if conf[r] > tau]
        first = [(r, int(idx[r, 0])) for r in hi] if hi else [(order[0], int(idx[order[0], 0]))]
        c1 = add(0, first)
        if len(order) > 1:
            add(0, [(order[1], int(idx[order[1], 0]))])
        add(0, [(order[0], int(idx[order[0], 1]))])
        rest = [r for r in order if nodes[c1][r] == model.mask_id]
        if rest:
            c2 = add(c1, [(rest[0], int(idx[rest[0], 0]))])
            if len(rest) > 1:
                add(c2, [(rest[1], int(idx[rest[1], 0]))])
    return np.stack(nodes), parent


def speculative_decode(model, s0, tau, mode="heuristic", seed=0, search=0, check_isolation=True):
    """Returns (trajectory, final state, forwards used, max accepted depth)."""
    rng = np.random.Generator(np.random.PCG64(seed))
    s = np.array(s0, dtype=np.int32)
    traj, n_forward, max_depth = [], 0, 0
    prev = None  # scores of the node the current root came from
    while (s == model.mask_id).any():
        peek = sequential_decode(model, s, tau)[0] if mode == "peek" else None
        if prev is None:
            conf0, idx0, prob0, _ = _score(model, s[None])
            prev = (conf0[0], idx0[0], prob0[0])
        states, parent = _draft(model, s, prev[0], prev[1], prev[2], mode, rng, tau, peek)
        B = states.shape[0]
        conf, idx, prob, lg = _score(model, states)
        n_forward += 1
        if check_isolation:
            for b in range(B):
                alone = model.logits(states[b:b + 1])[0]
                assert np.array_equal(alone, lg[b]), "branch leaked"
        acc = _o.accept(np.asarray(parent, np.int32)[None], states[None], model.mask_id,
                        conf[None], idx[None, :, :, 0], tau, rule=0, search=search)
        node = int(acc["accepted_node"][0])
        path = []
        b = node
        while b > 0:
            path.append(b)
            b = parent[b]
        for b in reversed(path):
            p = parent[b]
            traj.append(frozenset((int(r), int(states[b][r]))
                                  for r in np.flatnonzero(states[b] != states[p])))
        max_depth = max(max_depth, len(path))
        flag, tok = acc["unmask_flag"][0].astype(bool), acc["unmask_tok"][0]
        if (states[node] == model.mask_id).any():
            traj.append(frozenset((int(r), int(tok[r])) for r in np.flatnonzero(flag)))
        s = np.where(flag, tok, states[node]).astype(np.int32)
        prev = (conf[node], idx[node], prob[node])
    return traj, s, n_forward, max_depth
