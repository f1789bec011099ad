"""Thin ctypes binding over the libtsd C ABI: same names, argument marshalling only.

Tensors are torch CUDA tensors used purely as device memory; each call extracts
raw pointers and strides and enqueues the library's kernels on torch's current
stream (or the one given).  There is no fallback: if the library is missing or
an argument is rejected, the call raises.
"""
import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libtsd.so")

TSD_F32, TSD_BF16 = 0, 1
TSD_ACCEPT_EXACT, TSD_ACCEPT_TOP1, TSD_ACCEPT_TOPK, TSD_ACCEPT_PROB = 0, 1, 2, 3
TSD_SEARCH_GREEDY, TSD_SEARCH_LONGEST = 0, 1
TSD_ATTN_FORCE_SIMT = 0x1
TSD_OK, TSD_ERR_INVALID_ARG, TSD_ERR_UNSUPPORTED, TSD_ERR_WORKSPACE = 0, -1, -2, -3
TSD_ERR_CUDA, TSD_ERR_TIMEOUT, TSD_ERR_DEVICE_DATA = -4, -5, -6

EXPORTS = (
    "tsd_strerror", "tsd_last_cuda_error", "tsd_check_status",
    "tsd_branch_mask_bytes", "tsd_build_branch_mask",
    "tsd_verify_attention_workspace_bytes", "tsd_verify_attention",
    "tsd_confidence_topk_workspace_bytes", "tsd_confidence_topk",
    "tsd_confidence_topk_static_capacity", "tsd_confidence_topk_static",
    "tsd_accept_trajectories", "tsd_build_draft_tree",
    "tsd_build_interblock_vis", "tsd_interblock_trigger", "tsd_accept_joint_trees", "tsd_accept_relaxed",
    "tsd_commit_accepted", "tsd_verify_attention_fp8_cache_workspace_bytes", "tsd_verify_attention_fp8_cache",
    "tsd_gather_accepted_kv", "tsd_selftest_bounded_wait",
)


class TsdError(RuntimeError):
    def __init__(self, code, where):
        self.code = code
        msg = "%s failed: %s (%d)" % (where, strerror(code), code)
        if code == TSD_ERR_CUDA:
            msg += ": " + last_cuda_error()
        super().__init__(msg)


class tsd_layout(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in (
        "batch", "n_branches", "rows_per_branch", "n_cache", "n_q_heads", "n_kv_heads",
        "head_dim", "dtype")]


_lib = None
_vp, _i32, _i64, _u32, _f32, _sz = (ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64,
                                     ctypes.c_uint32, ctypes.c_float, ctypes.c_size_t)


def lib():
    """The loaded library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError("libtsd.so is missing (%s): build it with "
                               "`python -m paper_2608_27514_b200.build`; there is no fallback" % LIB_PATH)
        L = ctypes.CDLL(LIB_PATH)
        L.tsd_strerror.restype = ctypes.c_char_p
        L.tsd_strerror.argtypes = [ctypes.c_int]
        L.tsd_last_cuda_error.restype = ctypes.c_char_p
        L.tsd_check_status.argtypes = [_u32]
        L.tsd_branch_mask_bytes.restype = _sz
        L.tsd_branch_mask_bytes.argtypes = [ctypes.POINTER(tsd_layout)]
        L.tsd_build_branch_mask.argtypes = [ctypes.POINTER(tsd_layout), _vp, _vp, _vp, _sz, _vp, _vp]
        L.tsd_verify_attention_workspace_bytes.restype = _sz
        L.tsd_verify_attention_workspace_bytes.argtypes = [ctypes.POINTER(tsd_layout)]
        L.tsd_verify_attention.argtypes = (
            [ctypes.POINTER(tsd_layout), _vp] + [_vp, _i64, _i64, _i64] + [_vp, _vp, _i64, _i64, _i64]
            + [_vp, _vp, _i64, _i64, _i64] + [_vp, _i64, _i64, _i64] + [_vp, _f32, _vp, _sz, _u32, _vp, _vp])
        L.tsd_confidence_topk_workspace_bytes.restype = _sz
        L.tsd_confidence_topk_workspace_bytes.argtypes = [_i64, _i32, _i32]
        L.tsd_confidence_topk.argtypes = [_vp, _i32, _i64, _i32, _i64, _i32, _vp, _vp, _vp, _vp, _vp,
                                          _sz, _vp, _vp]
        L.tsd_confidence_topk_static_capacity.restype = _sz
        L.tsd_confidence_topk_static_capacity.argtypes = []
        L.tsd_confidence_topk_static.argtypes = [_vp, _i32, _i64, _i32, _i64, _i32, _vp, _vp, _vp, _vp, _vp, _vp]
        L.tsd_accept_trajectories.argtypes = [_i32, _i32, _i32, _vp, _vp, _i32, _vp, _vp, _i32, _f32,
                                              _i32, _i32] + [_vp] * 9
        L.tsd_build_draft_tree.argtypes = [_i32, _i32, _i32, _i32, _vp, _vp, _vp, _vp, _i32, _vp, _vp, _i32,
                                           _i32, _i32, _i32, _i32, _vp, _vp, _vp, _vp, _vp, _vp, _vp]
        L.tsd_build_interblock_vis.argtypes = [_i32, _i32, _i32, _vp, _vp]
        L.tsd_interblock_trigger.argtypes = [_i32, _i32, _i32, _vp, _vp, _vp, _i32, _i32, _f32, _vp, _vp, _vp,
                                             _vp]
        L.tsd_accept_joint_trees.argtypes = [_i32, _i32, _i32, _i32, _vp, _vp, _i32, _vp, _vp, _i32, _f32,
                                             _i32, _i32] + [_vp] * 9
        L.tsd_accept_relaxed.argtypes = ([_i32, _i32, _i32, _i32, _vp, _vp, _i32, _vp, _vp, _i32, _i32, _vp, _i32,
                                          _i64, _i64, _vp, _f32, _i32, _i32] + [_vp] * 10)
        L.tsd_commit_accepted.argtypes = [_i32, _i32, _i32, _i32, _vp, _vp, _vp, _vp, _vp, _i32, _vp, _i64, _vp, _vp,
                                          _vp, _vp, _vp, _vp, _vp]
        L.tsd_gather_accepted_kv.argtypes = [_i32, _i32, _i32, _i32, _i32, _i32, _vp, _vp, _vp, _i64, _i64, _i64,
                                             _vp, _vp, _i64, _i64, _i64, _vp, _i32, _vp, _vp]
        L.tsd_selftest_bounded_wait.argtypes = [_vp, _u32, _vp]
        L.tsd_verify_attention_fp8_cache_workspace_bytes.restype = _sz
        L.tsd_verify_attention_fp8_cache_workspace_bytes.argtypes = [ctypes.POINTER(tsd_layout)]
        L.tsd_verify_attention_fp8_cache.argtypes = (
            [ctypes.POINTER(tsd_layout), _vp] + [_vp, _i64, _i64, _i64] + [_vp, _vp, _i64, _i64, _i64, _vp, _vp]
            + [_vp, _vp, _i64, _i64, _i64] + [_vp, _i64, _i64, _i64] + [_vp, _f32, _vp, _sz, _u32, _vp, _vp])
        _lib = L
    return _lib


def strerror(code):
    return lib().tsd_strerror(int(code)).decode()


def last_cuda_error():
    return lib().tsd_last_cuda_error().decode()


def tsd_check_status(status):
    """status: int word or a 1-element uint32/int32 tensor (copied back here)."""
    word = int(status.item()) & 0xFFFFFFFF if hasattr(status, "item") else int(status)
    return lib().tsd_check_status(word)


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream))


def _check(rc, where):
    if rc != TSD_OK:
        raise TsdError(rc, where)


def dtype_code(dt):
    if dt == torch.float32:
        return TSD_F32
    if dt == torch.bfloat16:
        return TSD_BF16
    raise TsdError(TSD_ERR_UNSUPPORTED, "dtype %s" % dt)


def make_layout(batch, n_branches, rows_per_branch, n_cache, n_q_heads, n_kv_heads, head_dim, dtype):
    code = dtype if isinstance(dtype, int) else dtype_code(dtype)
    return tsd_layout(batch, n_branches, rows_per_branch, n_cache, n_q_heads, n_kv_heads, head_dim, code)


def tsd_branch_mask_bytes(layout):
    return int(lib().tsd_branch_mask_bytes(ctypes.byref(layout)))


def tsd_build_branch_mask(layout, vis, cache_lens, mask_out, dense_out=None, stream=None):
    rc = lib().tsd_build_branch_mask(ctypes.byref(layout), _ptr(vis), _ptr(cache_lens), _ptr(mask_out),
                                     mask_out.numel() * mask_out.element_size(), _ptr(dense_out),
                                     _stream(stream))
    _check(rc, "tsd_build_branch_mask")


def tsd_verify_attention_workspace_bytes(layout):
    return int(lib().tsd_verify_attention_workspace_bytes(ctypes.byref(layout)))


def _strides3(t):
    # [batch, rows, heads, dim] -> (batch, row, head) strides in elements
    assert t.dim() == 4 and t.stride(3) == 1, "head_dim must be contiguous"
    return t.stride(0), t.stride(1), t.stride(2)


def tsd_verify_attention(layout, mask, q, k_cache, v_cache, k_draft, v_draft, out, lse=None,
                         sm_scale=1.0, workspace=None, flags=0, status=None, stream=None):
    assert v_cache is None or v_cache.stride() == k_cache.stride()
    assert v_draft.stride() == k_draft.stride()
    cs = _strides3(k_cache) if k_cache is not None else (0, 0, layout.head_dim)
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    rc = lib().tsd_verify_attention(
        ctypes.byref(layout), _ptr(mask), _ptr(q), *_strides3(q), _ptr(k_cache), _ptr(v_cache), *cs,
        _ptr(k_draft), _ptr(v_draft), *_strides3(k_draft), _ptr(out), *_strides3(out), _ptr(lse),
        float(sm_scale), _ptr(workspace), ws_bytes, int(flags), _ptr(status), _stream(stream))
    _check(rc, "tsd_verify_attention")


def tsd_confidence_topk_workspace_bytes(n_rows, vocab, k):
    return int(lib().tsd_confidence_topk_workspace_bytes(int(n_rows), int(vocab), int(k)))


def tsd_confidence_topk(logits, k, conf, topk_idx, topk_prob, lse=None, workspace=None, status=None,
                        stream=None):
    assert logits.dim() == 2 and logits.stride(1) == 1
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    rc = lib().tsd_confidence_topk(
        _ptr(logits), dtype_code(logits.dtype), logits.shape[0], logits.shape[1], logits.stride(0),
        int(k), _ptr(conf), _ptr(topk_idx), _ptr(topk_prob), _ptr(lse), _ptr(workspace), ws_bytes,
        _ptr(status), _stream(stream))
    _check(rc, "tsd_confidence_topk")


def tsd_confidence_topk_static_capacity():
    return int(lib().tsd_confidence_topk_static_capacity())


def tsd_confidence_topk_static(logits, k, conf, topk_idx, topk_prob, lse=None, status=None, stream=None):
    """tsd_confidence_topk for callers that cannot provide a workspace: the scratch is the fixed
    array inside the library (see the header for its limit and sharing rules)."""
    assert logits.dim() == 2 and logits.stride(1) == 1
    rc = lib().tsd_confidence_topk_static(
        _ptr(logits), dtype_code(logits.dtype), logits.shape[0], logits.shape[1], logits.stride(0),
        int(k), _ptr(conf), _ptr(topk_idx), _ptr(topk_prob), _ptr(lse), _ptr(status), _stream(stream))
    _check(rc, "tsd_confidence_topk_static")


def tsd_accept_trajectories(parent, state, mask_id, conf, top1_idx, top1_stride, tau, rule, search,
                            edge_valid, prefix_len, accepted_node, accepted_len, n_new_tokens,
                            unmask_flag, unmask_tok, status=None, stream=None):
    S, B, R = state.shape
    rc = lib().tsd_accept_trajectories(
        S, B, R, _ptr(parent), _ptr(state), int(mask_id), _ptr(conf), _ptr(top1_idx), int(top1_stride),
        float(tau), int(rule), int(search), _ptr(edge_valid), _ptr(prefix_len), _ptr(accepted_node),
        _ptr(accepted_len), _ptr(n_new_tokens), _ptr(unmask_flag), _ptr(unmask_tok), _ptr(status),
        _stream(stream))
    _check(rc, "tsd_accept_trajectories")


def _slice_ptr(t, first):
    """Address of branch `first` of sequence 0 in a contiguous [S, B, ...] tensor."""
    return ctypes.c_void_p(t.data_ptr() + first * t.stride(1) * t.element_size())


def tsd_build_draft_tree(prev_state, accepted_node, unmask_flag, unmask_tok, mask_id, topk_idx, topk_prob,
                         width, depth, parent, state, node_prob, n_nodes, status=None, stream=None,
                         first=0, max_nodes=None, enable=None):
    """prev_state [S,Bp,R]; topk_idx/topk_prob [S*Bp*R, k] (or any shape with that many entries);
    outputs parent [S,B], state [S,B,R], node_prob [S,B], n_nodes [S].  With `first`/`max_nodes`
    the tree fills branches [first, first + max_nodes) of the (larger) output arrays and its
    parent indices count from `first`; `enable` uint8 [S] keeps a sequence's tree at its root."""
    S, Bp, R = prev_state.shape
    k = topk_idx.shape[-1]
    B = state.shape[1]
    max_nodes = B - first if max_nodes is None else int(max_nodes)
    assert state.is_contiguous() and parent.is_contiguous() and node_prob.is_contiguous()
    assert 0 <= first and first + max_nodes <= B
    rc = lib().tsd_build_draft_tree(
        S, Bp, R, k, _ptr(prev_state), _ptr(accepted_node), _ptr(unmask_flag), _ptr(unmask_tok), int(mask_id),
        _ptr(topk_idx), _ptr(topk_prob), int(width), int(depth), max_nodes, B, int(first), _ptr(enable),
        _slice_ptr(parent, first), _slice_ptr(state, first), _slice_ptr(node_prob, first), _ptr(n_nodes),
        _ptr(status), _stream(stream))
    _check(rc, "tsd_build_draft_tree")


def tsd_build_interblock_vis(n_cur, vis, stream=None):
    """vis uint64/int64 [S, B, ceil(B/64)] (written)."""
    S, B, W = vis.shape
    assert W == (B + 63) // 64 and vis.is_contiguous() and vis.element_size() == 8
    _check(lib().tsd_build_interblock_vis(S, B, int(n_cur), _ptr(vis), _stream(stream)),
           "tsd_build_interblock_vis")


def tsd_interblock_trigger(state, conf, node_cur, node_next, mask_id, tau, trigger, top_conf=None,
                           status=None, stream=None):
    S, B, R = state.shape
    rc = lib().tsd_interblock_trigger(S, B, R, _ptr(state), _ptr(conf), _ptr(node_cur), int(node_next),
                                      int(mask_id), float(tau), _ptr(trigger), _ptr(top_conf), _ptr(status),
                                      _stream(stream))
    _check(rc, "tsd_interblock_trigger")


def tsd_accept_joint_trees(parent, state, n_cur, mask_id, conf, top1_idx, top1_stride, tau, rule, search,
                           edge_valid, prefix_len, accepted_node, accepted_len, n_new_tokens,
                           unmask_flag, unmask_tok, status=None, stream=None):
    """Forest layout: parent/edge_valid/prefix_len [S,B]; accepted_* and n_new_tokens [2,S];
    unmask_* [2,S,R]."""
    S, B, R = state.shape
    rc = lib().tsd_accept_joint_trees(
        S, B, int(n_cur), R, _ptr(parent), _ptr(state), int(mask_id), _ptr(conf), _ptr(top1_idx),
        int(top1_stride), float(tau), int(rule), int(search), _ptr(edge_valid), _ptr(prefix_len),
        _ptr(accepted_node), _ptr(accepted_len), _ptr(n_new_tokens), _ptr(unmask_flag), _ptr(unmask_tok),
        _ptr(status), _stream(stream))
    _check(rc, "tsd_accept_joint_trees")


def tsd_accept_relaxed(parent, state, n_cur, mask_id, conf, topk_idx, topk_m, logits, lse, tau, rule, search,
                       edge_valid, prefix_len, accepted_node, accepted_len, n_new_tokens, unmask_flag,
                       unmask_tok, draft_prob=None, status=None, stream=None):
    """Any of the four rules on one tree (n_cur = B) or two; topk_idx [S,B,R,k]; logits
    [S*B*R, V] (or None) with lse [S*B*R]; per-tree outputs [2,S,...] (row 0 only for one tree)."""
    S, B, R = state.shape
    if logits is not None:
        assert logits.dim() == 2 and logits.stride(1) == 1 and logits.shape[0] == S * B * R
    rc = lib().tsd_accept_relaxed(
        S, B, int(n_cur), R, _ptr(parent), _ptr(state), int(mask_id), _ptr(conf), _ptr(topk_idx),
        int(topk_idx.shape[-1]) if topk_idx.dim() == 4 else 1, int(topk_m), _ptr(logits),
        0 if logits is None else dtype_code(logits.dtype), 0 if logits is None else logits.shape[1],
        0 if logits is None else logits.stride(0), _ptr(lse), float(tau), int(rule), int(search),
        _ptr(edge_valid), _ptr(prefix_len), _ptr(accepted_node), _ptr(accepted_len), _ptr(n_new_tokens),
        _ptr(unmask_flag), _ptr(unmask_tok), _ptr(draft_prob), _ptr(status), _stream(stream))
    _check(rc, "tsd_accept_relaxed")


def tsd_commit_accepted(parent, state, accepted_node, unmask_flag, unmask_tok, mask_id, tokens=None,
                        block_start=None, root_out=None, fill_step=None, step_base=None, n_masked=None,
                        status=None, stream=None, tree_root=0):
    """parent [S,B], state [S,B,R]; tokens [S,L] (row stride = tokens.stride(0)); the rest [S] / [S,R];
    tree_root = forest index of the tree's root (the next block's tree of a joint pass)."""
    S, B, R = state.shape
    if tokens is not None:
        assert tokens.dim() == 2 and tokens.stride(1) == 1
    rc = lib().tsd_commit_accepted(
        S, B, R, int(tree_root), _ptr(parent), _ptr(state), _ptr(accepted_node), _ptr(unmask_flag), _ptr(unmask_tok),
        int(mask_id), _ptr(tokens), 0 if tokens is None else tokens.stride(0), _ptr(block_start), _ptr(root_out),
        _ptr(fill_step), _ptr(step_base), _ptr(n_masked), _ptr(status), _stream(stream))
    _check(rc, "tsd_commit_accepted")


def tsd_gather_accepted_kv(accepted_node, rows_per_branch, k_draft, v_draft, k_out, v_out, out_row0=None,
                           status=None, stream=None):
    """k/v_draft [S, B*R, Hkv, d] -> k/v_out [S, rows, Hkv, d] at row out_row0[s] (views allowed; the
    last dimension contiguous); v_draft / v_out may both be None."""
    S, N, H, d = k_draft.shape
    assert k_draft.stride(3) == 1 and k_out.stride(3) == 1 and k_out.shape[0] == S and k_out.shape[2:] == (H, d)
    if v_draft is not None:
        assert v_draft.stride() == k_draft.stride() and v_out.stride() == k_out.stride()
    rc = lib().tsd_gather_accepted_kv(
        S, N // rows_per_branch, int(rows_per_branch), H, d, dtype_code(k_draft.dtype), _ptr(accepted_node),
        _ptr(k_draft), _ptr(v_draft), k_draft.stride(0), k_draft.stride(1), k_draft.stride(2),
        _ptr(k_out), _ptr(v_out), k_out.stride(0), k_out.stride(1), k_out.stride(2), _ptr(out_row0),
        k_out.shape[1], _ptr(status), _stream(stream))
    _check(rc, "tsd_gather_accepted_kv")


def tsd_selftest_bounded_wait(status, poll_limit=64, stream=None):
    """Runs the library's bounded barrier wait on a barrier nothing completes; sets TSD_STATUS_TIMEOUT."""
    _check(lib().tsd_selftest_bounded_wait(_ptr(status), int(poll_limit), _stream(stream)),
           "tsd_selftest_bounded_wait")


def tsd_verify_attention_fp8_cache_workspace_bytes(layout):
    return int(lib().tsd_verify_attention_fp8_cache_workspace_bytes(ctypes.byref(layout)))


def tsd_verify_attention_fp8_cache(layout, mask, q, k_cache_e4m3, v_cache_e4m3, k_scale, v_scale, k_draft, v_draft,
                                   out, workspace, lse=None, sm_scale=1.0, flags=0, status=None, stream=None):
    """k/v_cache_e4m3: uint8 (or float8_e4m3fn) tensors [S, Nc, Hkv, d]; k/v_scale fp32 [S, Hkv] or None."""
    assert v_cache_e4m3 is None or v_cache_e4m3.stride() == k_cache_e4m3.stride()
    assert v_draft.stride() == k_draft.stride()
    cs = _strides3(k_cache_e4m3) if k_cache_e4m3 is not None else (0, 0, layout.head_dim)
    rc = lib().tsd_verify_attention_fp8_cache(
        ctypes.byref(layout), _ptr(mask), _ptr(q), *_strides3(q), _ptr(k_cache_e4m3), _ptr(v_cache_e4m3), *cs,
        _ptr(k_scale), _ptr(v_scale), _ptr(k_draft), _ptr(v_draft), *_strides3(k_draft), _ptr(out), *_strides3(out),
        _ptr(lse), float(sm_scale), _ptr(workspace), workspace.numel() * workspace.element_size(), int(flags),
        _ptr(status), _stream(stream))
    _check(rc, "tsd_verify_attention_fp8_cache")
