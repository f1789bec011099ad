"""Seeded synthetic inputs for the blockwise verification step.

This module only *makes inputs*: tensors shaped and distributed like the
paper's workloads (Section 5.1: generation length 512, block size 32; trees
named WxDy(n) in Section 3.2), plus draft trees whose children are planted to
be right or nearly right.  It holds none of the verification arithmetic and is
the only code that the CUDA path's tests/benchmark and the CPU oracle's tests
both use.  The one normaliser it evaluates (a log-sum-exp of a noise row) is
there to place planted peaks at a chosen probability, i.e. to shape the input
distribution; no decision of the method is taken here.

Everything is a function of (config, seed): numpy PCG64 for the discrete
plan, torch's seeded generator for the dense tensors.
"""
from dataclasses import dataclass, replace
import math

import numpy as np
import torch


@dataclass(frozen=True)
class Config:
    name: str
    S: int          # independent sequences
    Hq: int         # query heads
    Hkv: int        # key/value heads
    d: int          # head dim
    Nc: int         # cached prefix+suffix tokens
    B: int          # tree nodes ("branches") per sequence, node 0 = root
    R: int          # query rows per branch: 32 (one block) or 64 (current + next)
    V: int          # vocabulary
    k: int          # candidates per row
    tau: float
    dtype: str      # "f32" | "bf16"
    sigma: float    # std of the noise logits
    arity: int      # breadth-first fill arity of the tree (0 = explicit shape)
    seed: int
    f_high: float = 0.2       # fraction of rows planted above tau
    literal_peaks: bool = False  # cfg 1: "+4 at a random token on 50 % of positions"

    @property
    def N(self):
        return self.B * self.R

    @property
    def rows(self):
        return self.S * self.B * self.R

    @property
    def torch_dtype(self):
        return torch.float32 if self.dtype == "f32" else torch.bfloat16


# The five workloads.  Cache length = prompt + generation - rows of one branch.
CONFIGS = {
    "cfg1": Config("cfg1", 1, 4, 4, 64, 256, 4, 32, 4096, 3, 0.9, "f32", 2.0, 0, 0, literal_peaks=True),
    "cfg2": Config("cfg2", 1, 32, 32, 128, 736, 8, 32, 126464, 3, 0.9, "bf16", 3.0, 0, 1),
    "cfg3": Config("cfg3", 1, 32, 32, 128, 1472, 16, 64, 126464, 3, 0.9, "bf16", 3.0, 3, 2),
    "cfg4": Config("cfg4", 16, 32, 32, 128, 1504, 32, 32, 126464, 3, 0.9, "bf16", 3.0, 3, 3),
    "cfg5": Config("cfg5", 4, 28, 4, 128, 5056, 64, 64, 152064, 4, 0.9, "bf16", 3.0, 4, 4),
}


def small(cfg, **kw):
    """A reduced copy of a config (tests use it to keep the oracle fast)."""
    return replace(cfg, **kw)


def tree_parents(cfg):
    """parent[b] for one sequence; node 0 is the root, parent[b] < b.

    cfg1 is W2D2(3): root, two children, one grandchild.  cfg2 is the hybrid
    shape for k=3, D=3: root + 3 children + one grandchild each + one
    great-grandchild.  The others fill breadth-first with the given arity.
    """
    if cfg.name == "cfg1" and cfg.B == 4:
        return [-1, 0, 0, 1]
    if cfg.name == "cfg2" and cfg.B == 8:
        return [-1, 0, 0, 0, 1, 2, 3, 4]
    a = max(cfg.arity, 1)
    return [-1] + [(b - 1) // a for b in range(1, cfg.B)]


def _randn(shape, gen, device, dtype, scale=1.0):
    x = torch.randn(shape, generator=gen, device=device, dtype=torch.float32)
    if scale != 1.0:
        x.mul_(scale)
    return x.to(dtype)


def attention_inputs(cfg, device="cpu", q_gain=1.0, seed_offset=0):
    """Q, cached K/V and draft K/V ~ N(0,1) in the config's dtype.

    Layouts: q [S,N,Hq,d]; k_cache/v_cache [S,Nc,Hkv,d]; k_draft/v_draft
    [S,N,Hkv,d]; draft row index = branch*R + r.  ``q_gain`` > 1 sharpens the
    softmax so that a leaked key would move the output visibly.
    """
    dev = torch.device(device)
    gen = torch.Generator(device=dev)
    gen.manual_seed(1000 + 17 * cfg.seed + seed_offset)
    dt = cfg.torch_dtype
    q = _randn((cfg.S, cfg.N, cfg.Hq, cfg.d), gen, dev, dt, q_gain)
    kc = _randn((cfg.S, cfg.Nc, cfg.Hkv, cfg.d), gen, dev, dt)
    vc = _randn((cfg.S, cfg.Nc, cfg.Hkv, cfg.d), gen, dev, dt)
    kd = _randn((cfg.S, cfg.N, cfg.Hkv, cfg.d), gen, dev, dt)
    vd = _randn((cfg.S, cfg.N, cfg.Hkv, cfg.d), gen, dev, dt)
    return dict(q=q, k_cache=kc, v_cache=vc, k_draft=kd, v_draft=vd,
                sm_scale=1.0 / math.sqrt(cfg.d))


def _logit(p):
    return math.log(p / (1.0 - p))


def plan_tree(cfg, alpha=(0.85, 0.68)):
    """Discrete plan: tree, block states and which (row, token) peaks to plant.

    Per node every row gets a planted top token and a target probability
    p*: "high" rows (p* in [0.93, 0.995], above tau) or "low" rows (p* in
    [0.30, 0.80] before the two runner-up tokens are added, which leaves the
    top-1 probability below 0.6).  The set a threshold decoder would unmask at
    a node is then known by construction: its masked high rows, or, when it
    has none, the masked low row with the largest p* (kept 0.08 clear of the
    runner-up row).  A child is the parent plus that set ("correct draft",
    probability alpha[0] at depth 1 and alpha[1] deeper, Section 4.2) or a near
    miss of it; at most one child of a node is correct.
    """
    rng = np.random.Generator(np.random.PCG64(5000 + cfg.seed))
    S, B, R, V = cfg.S, cfg.B, cfg.R, cfg.V
    mask_id = V - 1
    par = tree_parents(cfg)
    children = [[c for c in range(B) if par[c] == b] for b in range(B)]
    depth = [0] * B
    for b in range(1, B):
        depth[b] = depth[par[b]] + 1
    state = np.full((S, B, R), mask_id, dtype=np.int32)
    kind = np.zeros((S, B, R), dtype=np.int8)      # 1 high, 2 low (top-3 structure), 3 literal +4
    tok = np.zeros((S, B, R, 3), dtype=np.int64)   # planted top-1 and two runner-ups
    pstar = np.zeros((S, B, R), dtype=np.float64)
    planted_u = np.zeros((S, B, R), dtype=np.uint8)
    n_correct = 0
    for s in range(S):
        masked = rng.random(R) < 0.6
        while masked.sum() < 4:
            masked[rng.integers(R)] = True
        state[s, 0] = np.where(masked, mask_id, rng.integers(0, V - 1, size=R))
        for b in range(B):
            st = state[s, b]
            m_rows = np.flatnonzero(st == mask_id)
            # three distinct planted tokens per row
            t = rng.integers(0, V - 1, size=(R, 3))
            while True:
                dup = (t[:, 0] == t[:, 1]) | (t[:, 0] == t[:, 2]) | (t[:, 1] == t[:, 2])
                if not dup.any():
                    break
                t[dup] = rng.integers(0, V - 1, size=(int(dup.sum()), 3))
            tok[s, b] = t
            no_high = rng.random() < 0.25
            hi = rng.random(R) < cfg.f_high
            if no_high:
                hi[m_rows] = False
            kind[s, b] = np.where(hi, 1, 2)
            pstar[s, b] = np.where(hi, rng.uniform(0.93, 0.995, R), rng.uniform(0.30, 0.80, R))
            if cfg.literal_peaks:
                # literal recipe on the rows that steer nothing; steering rows stay calibrated
                lit = rng.random(R) < 0.5
                lit[m_rows] = False
                kind[s, b][lit] = 3
                kind[s, b][~lit & ~np.isin(np.arange(R), m_rows)] = 0
            u_rows = [r for r in m_rows if hi[r]]
            second = None
            if not u_rows and len(m_rows) > 0:
                order = sorted(m_rows, key=lambda r: -pstar[s, b, r])
                top = order[0]
                if len(order) > 1:
                    second = order[1]
                    pstar[s, b, top] = min(0.88, max(pstar[s, b, top], pstar[s, b, second] + 0.08))
                    for r in order[1:]:
                        pstar[s, b, r] = min(pstar[s, b, r], pstar[s, b, top] - 0.08)
                u_rows = [top]
            planted_u[s, b, u_rows] = 1
            kids = children[b]
            if not kids or not u_rows:
                for c in kids:
                    state[s, c] = st
                continue
            a = alpha[0] if depth[b] == 0 else alpha[1]
            correct = -1
            if rng.random() < a:
                correct = 0 if rng.random() < 0.7 else int(rng.integers(len(kids)))
                n_correct += 1
            for ci, c in enumerate(kids):
                child = st.copy()
                for r in u_rows:
                    child[r] = t[r, 0]
                if ci != correct:
                    variant = (ci + b) % 4
                    r0 = u_rows[int(rng.integers(len(u_rows)))]
                    if variant == 0:        # right row, runner-up token
                        child[r0] = t[r0, 1]
                    elif variant == 1 and second is not None:   # wrong row, its own top token
                        child[r0] = mask_id
                        child[second] = t[second, 0]
                    elif variant == 2 and len(u_rows) > 1:      # strict subset
                        child[r0] = mask_id
                    else:                   # superset: one extra low row, or a wrong token
                        extra = [r for r in m_rows if r not in u_rows]
                        if extra:
                            e = extra[int(rng.integers(len(extra)))]
                            child[e] = t[e, 0]
                        else:
                            child[r0] = t[r0, 2]
                state[s, c] = child
    parent = np.tile(np.asarray(par, dtype=np.int32), (S, 1))
    return dict(parent=parent, state=state, mask_id=mask_id, kind=kind, tok=tok,
                pstar=pstar, planted_u=planted_u, n_correct=n_correct, depth=depth)


def logits_from_plan(cfg, plan, device="cpu", chunk_rows=512):
    """[rows, V] logits: N(0, sigma^2) noise with the planned peaks written in.

    A planted top token sits at lnZ0 + logit(p*), lnZ0 being the noise row's
    log-normaliser; "low" rows also get two runner-ups 0.7 and 1.6 below it.
    """
    dev = torch.device(device)
    gen = torch.Generator(device=dev)
    gen.manual_seed(9000 + 31 * cfg.seed)
    rows, V = cfg.rows, cfg.V
    dt = cfg.torch_dtype
    out = torch.empty((rows, V), device=dev, dtype=dt)
    kind = torch.from_numpy(plan["kind"].reshape(rows)).to(dev)
    tok = torch.from_numpy(plan["tok"].reshape(rows, 3)).to(dev)
    lg = torch.from_numpy(np.log(plan["pstar"] / (1.0 - plan["pstar"])).reshape(rows)).to(dev)
    for r0 in range(0, rows, chunk_rows):
        r1 = min(rows, r0 + chunk_rows)
        x = torch.randn((r1 - r0, V), generator=gen, device=dev, dtype=torch.float32)
        x.mul_(cfg.sigma)
        x = x.to(dt).float()
        lnz0 = torch.logsumexp(x.double(), dim=1)
        kd, tk, l0 = kind[r0:r1], tok[r0:r1], lg[r0:r1]
        ar = torch.arange(r1 - r0, device=dev)
        top = (lnz0 + l0).float()
        cal = (kd == 1) | (kd == 2)
        x[ar[cal], tk[cal, 0]] = top[cal]
        low = kd == 2
        x[ar[low], tk[low, 1]] = top[low] - 0.7
        x[ar[low], tk[low, 2]] = top[low] - 1.6
        lit = kd == 3
        x[ar[lit], tk[lit, 0]] += 4.0
        out[r0:r1] = x.to(dt)
    return out


def verify_inputs(cfg, device="cpu"):
    """Tree, block states and logits for one verification step."""
    plan = plan_tree(cfg)
    logits = logits_from_plan(cfg, plan, device)
    dev = torch.device(device)
    return dict(
        parent=torch.from_numpy(plan["parent"]).to(dev),
        state=torch.from_numpy(plan["state"]).to(dev),
        mask_id=int(plan["mask_id"]),
        logits=logits,
        tau=cfg.tau,
        k=cfg.k,
        plan=plan,
    )


def poison_other_branches(cfg, inp, keep_branch):
    """Copy of attention inputs in which every draft branch except
    ``keep_branch`` has K aligned with the kept branch's queries and V = +-1e4:
    any leak across branches (Section 3.3, rule 2) then swamps the output."""
    out = dict(inp)
    kd = inp["k_draft"].clone()
    vd = inp["v_draft"].clone()
    R = cfg.R
    group = cfg.Hq // cfg.Hkv
    qk = inp["q"][:, keep_branch * R:(keep_branch + 1) * R, ::group, :]
    for b in range(cfg.B):
        if b == keep_branch:
            continue
        kd[:, b * R:(b + 1) * R] = (8.0 * qk).to(kd.dtype)
        sign = 1.0 if b % 2 == 0 else -1.0
        vd[:, b * R:(b + 1) * R] = sign * 1.0e4
    out["k_draft"], out["v_draft"] = kd, vd
    return out
