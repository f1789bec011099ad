"""ctypes binding of the C oracle: argument marshalling only (numpy arrays in,
numpy arrays out).  The arithmetic lives in ``tsd_oracle.c``."""
import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "tsd_oracle.c")
_LIB = os.path.join(_HERE, "libtsd_oracle.so")
_lib = None


# -ffp-contract=off keeps every product and sum a separate IEEE operation (no fused multiply-add
# slipped in by -march=native), so the oracle's bits do not depend on the host's instruction set;
# nothing is reassociated without -ffast-math.
BUILD_FLAGS = "-O3 -march=native -ffp-contract=off -fopenmp"
_FLAGS_FILE = os.path.join(_HERE, "libtsd_oracle.flags")


def build(force=False):
    """Compile the oracle with gcc (OpenMP over rows); rebuilt when the source or the flags change."""
    stale = force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
    if not stale:
        try:
            with open(_FLAGS_FILE) as f:
                stale = f.read().strip() != BUILD_FLAGS
        except OSError:
            stale = True
    if stale:
        tmp = _LIB + ".%d.tmp" % os.getpid()
        subprocess.check_call(["gcc"] + BUILD_FLAGS.split() + ["-std=c11", "-fPIC", "-shared", _SRC, "-o", tmp, "-lm"])
        os.replace(tmp, _LIB)
        with open(_FLAGS_FILE, "w") as f:
            f.write(BUILD_FLAGS + "\n")
    return _LIB


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.oracle_num_threads.restype = ctypes.c_int
        _lib.oracle_decode_rule.restype = ctypes.c_int
    return _lib


def num_threads():
    return int(_load().oracle_num_threads())


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _arr(x, dtype):
    if x is None:
        return None
    if hasattr(x, "detach"):  # torch tensor
        x = x.detach().cpu()
        if str(x.dtype) == "torch.bfloat16":
            x = x.float()
        x = x.numpy()
    return np.ascontiguousarray(x, dtype=dtype)


def dense_mask(S, B, R, Nc, vis=None, cache_lens=None):
    """uint8 [S, B*R, Nc+B*R], 1 = visible (Section 3.3)."""
    vis = _arr(vis, np.uint64)
    cache_lens = _arr(cache_lens, np.int32)
    out = np.empty((S, B * R, Nc + B * R), dtype=np.uint8)
    _load().oracle_dense_mask(S, B, R, Nc, _ptr(vis), _ptr(cache_lens), _ptr(out))
    return out


def masked_attention(q, k_cache, v_cache, k_draft, v_draft, mask, sm_scale):
    """q [S,N,Hq,d], k/v_cache [S,Nc,Hkv,d], k/v_draft [S,N,Hkv,d], mask
    [S,N,Nc+N] -> (out fp64 [S,N,Hq,d], lse fp64 [S,Hq,N])."""
    q = _arr(q, np.float32)
    kc, vc = _arr(k_cache, np.float32), _arr(v_cache, np.float32)
    kd, vd = _arr(k_draft, np.float32), _arr(v_draft, np.float32)
    mask = _arr(mask, np.uint8)
    S, N, Hq, d = q.shape
    Nc, Hkv = kc.shape[1], kc.shape[2]
    assert kc.shape == (S, Nc, Hkv, d) and vc.shape == kc.shape
    assert kd.shape == (S, N, Hkv, d) and vd.shape == kd.shape
    assert mask.shape == (S, N, Nc + N) and Hq % Hkv == 0
    out = np.empty((S, N, Hq, d), dtype=np.float64)
    lse = np.empty((S, Hq, N), dtype=np.float64)
    _load().oracle_masked_attention(
        S, N, Nc, Hq, Hkv, d, _ptr(q), _ptr(kc), _ptr(vc), _ptr(kd), _ptr(vd),
        _ptr(mask), ctypes.c_double(float(sm_scale)), _ptr(out), _ptr(lse))
    return out, lse


def confidence_topk(logits, k):
    """logits [rows, V] -> conf fp64 [rows], idx int32 [rows,k], prob fp64
    [rows,k], lse fp64 [rows] (Eq. 2; order: logit desc, index asc)."""
    logits = _arr(logits, np.float32)
    rows, V = logits.shape
    assert 1 <= k <= V
    conf = np.empty(rows, dtype=np.float64)
    idx = np.empty((rows, k), dtype=np.int32)
    prob = np.empty((rows, k), dtype=np.float64)
    lse = np.empty(rows, dtype=np.float64)
    _load().oracle_confidence_topk(
        _ptr(logits), ctypes.c_int64(rows), V, ctypes.c_int64(V), k,
        _ptr(conf), _ptr(idx), _ptr(prob), _ptr(lse))
    return conf, idx, prob, lse


def decode_rule(state, mask_id, conf, top1, tau):
    """One node: (flag uint8 [R], tok int32 [R]) = U(node)."""
    state = _arr(state, np.int32)
    conf = _arr(conf, np.float32)
    top1 = _arr(top1, np.int32)
    R = state.shape[0]
    flag = np.empty(R, dtype=np.uint8)
    tok = np.empty(R, dtype=np.int32)
    _load().oracle_decode_rule(R, _ptr(state), ctypes.c_int32(mask_id), _ptr(conf),
                               _ptr(top1), ctypes.c_float(tau), _ptr(flag), _ptr(tok))
    return flag, tok


def accept(parent, state, mask_id, conf, top1, tau, rule=0, search=0, topk_m=1, draft_prob=None):
    """parent [S,B], state [S,B,R], conf [S,B,R] fp32, top1 [S,B,R] or the
    candidate lists [S,B,R,k] (entry 0 = arg-max; rule 2 tests the first
    topk_m), draft_prob fp32 [S,B,R] (rule 3) -> dict of edge_valid,
    prefix_len, accepted_node, accepted_len, n_new_tokens, unmask_flag,
    unmask_tok."""
    parent = _arr(parent, np.int32)
    state = _arr(state, np.int32)
    conf = _arr(conf, np.float32)
    top1 = _arr(top1, np.int32)
    draft_prob = _arr(draft_prob, np.float32)
    S, B, R = state.shape
    stride = 1 if top1.ndim == 3 else top1.shape[3]
    assert parent.shape == (S, B) and conf.shape == (S, B, R) and top1.shape[:3] == (S, B, R)
    assert 1 <= topk_m <= stride and (rule != 3 or draft_prob.shape == (S, B, R))
    o = dict(
        edge_valid=np.empty((S, B), np.uint8),
        prefix_len=np.empty((S, B), np.int32),
        accepted_node=np.empty(S, np.int32),
        accepted_len=np.empty(S, np.int32),
        n_new_tokens=np.empty(S, np.int32),
        unmask_flag=np.empty((S, R), np.uint8),
        unmask_tok=np.empty((S, R), np.int32),
    )
    _load().oracle_accept(
        S, B, R, _ptr(parent), _ptr(state), ctypes.c_int32(mask_id), _ptr(conf),
        _ptr(top1), ctypes.c_int64(stride), int(topk_m), _ptr(draft_prob), ctypes.c_float(tau),
        int(rule), int(search),
        _ptr(o["edge_valid"]), _ptr(o["prefix_len"]), _ptr(o["accepted_node"]),
        _ptr(o["accepted_len"]), _ptr(o["n_new_tokens"]), _ptr(o["unmask_flag"]),
        _ptr(o["unmask_tok"]))
    return o


def draft_token_prob(logits, parent, state, mask_id):
    """logits [S,B,R,V], parent [S,B], state [S,B,R] -> fp64 [S,B,R]: probability of each drafted
    token under its parent's distribution at that row (0 where the child adds nothing)."""
    logits = _arr(logits, np.float32)
    parent = _arr(parent, np.int32)
    state = _arr(state, np.int32)
    S, B, R, V = logits.shape
    assert parent.shape == (S, B) and state.shape == (S, B, R)
    out = np.empty((S, B, R), dtype=np.float64)
    _load().oracle_draft_token_prob(S, B, R, V, _ptr(logits), _ptr(parent), _ptr(state),
                                    ctypes.c_int32(mask_id), _ptr(out))
    return out


def build_draft_tree(root_state, mask_id, topk_idx, topk_prob, W, D, max_nodes):
    """One sequence: root_state [R], topk_idx/topk_prob [R,k] -> (n_nodes, parent [B], state [B,R],
    node_prob [B]) by Alg. 1 Phase 2 (see the C source for the reading of its three helpers)."""
    root_state = _arr(root_state, np.int32)
    topk_idx = _arr(topk_idx, np.int32)
    topk_prob = _arr(topk_prob, np.float32)
    R, k = topk_idx.shape
    parent = np.empty(max_nodes, np.int32)
    state = np.empty((max_nodes, R), np.int32)
    prob = np.empty(max_nodes, np.float32)
    lib = _load()
    lib.oracle_build_draft_tree.restype = ctypes.c_int
    n = lib.oracle_build_draft_tree(R, k, _ptr(root_state), ctypes.c_int32(mask_id), _ptr(topk_idx),
                                    _ptr(topk_prob), int(W), int(D), int(max_nodes), _ptr(parent),
                                    _ptr(state), _ptr(prob))
    return int(n), parent, state, prob
