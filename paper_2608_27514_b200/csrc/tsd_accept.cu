// Stage 3: acceptance of draft trajectories (paper Section 3.3 "Verification procedure";
// Alg. 1 Phase 1 for the high/low confidence split; Eqs. 6-7 for the top-1 fallback).
//
// One thread block per sequence.  Warps take tree nodes in turn: first the decode rule U(p) of
// every node (what threshold decoding would unmask next), then the validity of every edge, both
// as warp ballots over the block's rows; one warp then walks the tree, a lane per node.
// Integer and float compares only: the result is exact.
//
// Besides the exact and top-1 tests, the two relaxed readings of the verification test
// (the top-k-membership and probability-above-tau alternatives of that passage): membership of the drafted token in the parent's first
// topk_m candidates, and the probability of the drafted token under the parent's distribution,
// gathered here from the logits and the row's log-sum-exp (one scattered load per drafted token;
// the vocabulary pass has already produced the log-sum-exp).
//
// The joint pass of inter-block speculation (Section 3.4) verifies two trees at once: branches
// [0, n_cur) and [n_cur, B) of the same arrays.  blockIdx.y picks the tree; per-branch outputs
// keep their position in the forest, per-tree outputs are tree-major ([2, batch, ...]).
#include <limits.h>
#include <math_constants.h>
#include "tsd_common.cuh"

namespace tsd {

constexpr int kMaxBranches = 256;
constexpr int kMaxRows = 128;
constexpr int kRowWords = kMaxRows / 32;
constexpr int kAcceptThreads = 256;      // a warp per node up to 8 nodes ...
constexpr int kAcceptMaxThreads = 1024;  // ... and up to 32 warps for larger trees (nodes are taken in turn)
constexpr int kStageCells = 4096;        // trees of up to this many (node, row) cells are staged in shared memory

struct RelaxedArgs {
  int topk_m;           // candidates per row that count for TSD_ACCEPT_TOPK
  const void* logits;   // [batch, B, R, vocab] rows `ld` elements apart, nullable
  int dtype;
  int64_t vocab, ld;
  const float* lse;     // [batch, B, R] natural-log sum-exp of each logits row
  float* draft_prob;    // [batch, B, R] out, nullable
};

// WORDS = 32-row words per node that the unrolled loops cover (R <= 32 * WORDS).
template <int WORDS>
__global__ void __launch_bounds__(kAcceptMaxThreads)
accept_kernel(int B_all, int n_cur, int R, const int32_t* __restrict__ parent, const int32_t* __restrict__ state,
              int mask_id, const float* __restrict__ conf, const int32_t* __restrict__ top1,
              int top1_stride, float tau, int rule, int search, uint8_t* __restrict__ edge_valid,
              int32_t* __restrict__ prefix_len, int32_t* __restrict__ accepted_node,
              int32_t* __restrict__ accepted_len, int32_t* __restrict__ n_new_tokens,
              uint8_t* __restrict__ unmask_flag, int32_t* __restrict__ unmask_tok,
              uint32_t* __restrict__ status, RelaxedArgs x) {
  __shared__ uint32_t s_u[kMaxBranches][kRowWords];  // U(p) as a row bitset
  __shared__ uint8_t s_valid[kMaxBranches];
  __shared__ int s_par[kMaxBranches];
  __shared__ int s_pl[kMaxBranches];  // prefix_len, kept on chip for the walk (global reads of values
                                      // just written would cost one L2 round trip per node)
  __shared__ int s_acc;
  // Small trees: every warp loads its node's tokens and top-1 candidates once, together with the
  // confidences, and the later phases (the parent's rows for the edge test, the accepted node's
  // candidates for the unmask set) read them from here instead of making two more dependent round
  // trips to global memory.
  __shared__ int32_t s_st[kStageCells], s_t1[kStageCells];
  const int s = blockIdx.x, tree = blockIdx.y, batch = gridDim.x;
  const int lo = tree ? n_cur : 0;          // first branch of this tree = its root
  const int B = tree ? B_all - n_cur : n_cur;  // its size (0: nothing to verify)
  const size_t ts = (size_t)tree * batch + s;  // slot in the tree-major outputs
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
  const unsigned full = 0xffffffffu;
  if (B <= 0) return;
  const int32_t* st = state + ((size_t)s * B_all + lo) * R;
  const float* cf = conf + ((size_t)s * B_all + lo) * R;
  const int32_t* t1 = top1 + ((size_t)s * B_all + lo) * R * top1_stride;
  const int words = min((R + 31) / 32, WORDS);
  const bool staged = B * R <= kStageCells;

  // decode rule U(p) for every node
  for (int p = warp; p < B; p += n_warps) {
    // the node's parent is requested together with its rows (one address for the whole warp)
    const int raw_parent = p > 0 ? parent[(size_t)s * B_all + lo + p] : -1;  // forest index
    uint32_t hi[WORDS], any_hi = 0, any_masked = 0;
    float best = -CUDART_INF_F;
    int best_r = INT_MAX;
#pragma unroll
    for (int w = 0; w < WORDS; ++w) {
      hi[w] = 0;
      if (w < words) {
        const int r = w * 32 + lane;
        bool masked = false, high = false;
        if (r < R) {
          const int32_t tok = st[p * R + r];
          if (staged) {
            s_st[p * R + r] = tok;
            s_t1[p * R + r] = t1[(size_t)(p * R + r) * top1_stride];
          }
          masked = tok == mask_id;
          const float c = cf[p * R + r];

          high = masked && c > tau;  // strictly above the threshold
          if (masked && (best_r == INT_MAX || c > best)) { best = c; best_r = r; }  // rows ascend
        }
        hi[w] = __ballot_sync(full, high);
        any_hi |= hi[w];
        any_masked |= __ballot_sync(full, masked);
      }
    }
    if (!any_hi && any_masked) {  // no row above tau: the single most confident masked row
#pragma unroll
      for (int off = 16; off; off >>= 1) {
        const float ov = __shfl_xor_sync(full, best, off);
        const int orow = __shfl_xor_sync(full, best_r, off);
        const bool take = orow != INT_MAX &&
                          (best_r == INT_MAX || ov > best || (ov == best && orow < best_r));
        if (take) { best = ov; best_r = orow; }
      }
#pragma unroll
      for (int w = 0; w < WORDS; ++w) hi[w] = (best_r >> 5) == w ? (1u << (best_r & 31)) : 0u;
    }
    if (lane == 0) {
#pragma unroll
      for (int w = 0; w < WORDS; ++w) s_u[p][w] = hi[w];
      int par = -1;
      if (p > 0) par = raw_parent >= lo ? raw_parent - lo : -1;  // local to the tree
      if (p > 0 && (par < 0 || par >= p)) {
        if (status) atomicOr(status, TSD_STATUS_BAD_PARENT);
        par = -1;  // treated as an invalid edge hanging off nothing
      }
      s_par[p] = par;
    }
  }
  __syncthreads();

  // validity of every edge parent -> c
  for (int c = warp; c < B; c += n_warps) {
    const int p = s_par[c];
    bool ok = true, malformed = false, delta = false;
    for (int w = 0; w < words; ++w) {
      const int r = w * 32 + lane;
      if (r < R) {
        float pr = 0.f;  // probability of the token this child adds at r, under its parent
        if (c > 0 && p >= 0) {
          const int sp = staged ? s_st[p * R + r] : st[p * R + r];
          const int sc = staged ? s_st[c * R + r] : st[c * R + r];
          const bool p_masked = sp == mask_id, c_masked = sc == mask_id;
          const bool in_u = (s_u[p][w] >> lane) & 1u;
          if (!p_masked) {
            malformed |= sc != sp;
          } else if (c_masked) {
            if (rule == TSD_ACCEPT_EXACT && in_u) ok = false;  // U has a row the child lacks
          } else {
            delta = true;
            const int32_t* cand = t1 + (size_t)(p * R + r) * top1_stride;
            bool tok_ok = (staged ? s_t1[p * R + r] : cand[0]) == sc;
            if (rule == TSD_ACCEPT_TOPK)
              for (int j = 1; j < x.topk_m; ++j) tok_ok |= cand[j] == sc;
            if (x.logits && sc >= 0 && sc < x.vocab) {
              const size_t row = ((size_t)s * B_all + lo + p) * R + r;
              const float z = x.dtype == TSD_BF16
                                  ? __bfloat162float(static_cast<const __nv_bfloat16*>(x.logits)[row * x.ld + sc])
                                  : static_cast<const float*>(x.logits)[row * x.ld + sc];
              pr = expf(z - x.lse[row]);
            }
            if (rule == TSD_ACCEPT_EXACT) ok &= in_u && tok_ok;
            else if (rule == TSD_ACCEPT_PROB) ok &= pr > tau;  // strictly above, as in Alg. 1
            else ok &= tok_ok;
          }
        }
        if (x.draft_prob) x.draft_prob[((size_t)s * B_all + lo + c) * R + r] = pr;
      }
    }
    const bool all_ok = __all_sync(full, ok), any_bad = __any_sync(full, malformed),
               any_delta = __any_sync(full, delta);
    if (lane == 0) s_valid[c] = c == 0 ? 1 : (p >= 0 && all_ok && !any_bad && any_delta);
  }
  __syncthreads();

  // tree walk by warp 0, a lane per node: the lane climbs from its node to the root (trees are a few
  // levels deep), counting the steps (= depth) and remembering the invalid edge nearest the root;
  // the leading valid edges on the path root -> node are the ones above that edge.
  if (warp == 0) {
    int32_t* pl = prefix_len + (size_t)s * B_all + lo;
    uint8_t* ev = edge_valid + (size_t)s * B_all + lo;
    int best_depth = 0, best_node = 0;  // longest fully valid path seen by this lane (root: depth 0)
    for (int b = lane; b < B; b += 32) {
      int depth = 0, bad_at = -1;  // bad_at: steps from b up to the child end of that invalid edge
      for (int a = b; a > 0; a = s_par[a]) {
        if (!s_valid[a]) bad_at = depth;
        ++depth;
      }
      const int plb = bad_at < 0 ? depth : depth - bad_at - 1;
      s_pl[b] = plb;
      pl[b] = plb;
      ev[b] = b == 0 ? 1 : s_valid[b];
      if (bad_at < 0 && depth > best_depth) { best_depth = depth; best_node = b; }  // nodes ascend per lane
    }
    int acc = 0, acc_depth = 0;
    if (search == TSD_SEARCH_LONGEST) {
      // deepest fully valid node, lowest index among equals
#pragma unroll
      for (int off = 16; off; off >>= 1) {
        const int od = __shfl_xor_sync(full, best_depth, off), on = __shfl_xor_sync(full, best_node, off);
        if (od > best_depth || (od == best_depth && on < best_node)) { best_depth = od; best_node = on; }
      }
      acc = best_node;
      acc_depth = best_depth;
    } else {
      // greedy: from the root, keep moving to the lowest-index valid child
      for (;;) {
        int next = -1;
        for (int b0 = 0; b0 < B && next < 0; b0 += 32) {
          const int b = b0 + lane;
          const unsigned m = __ballot_sync(full, b < B && b > acc && s_par[b] == acc && s_valid[b]);
          if (m) next = b0 + __ffs(m) - 1;
        }
        if (next < 0) break;
        acc = next;
        ++acc_depth;
      }
    }
    if (lane == 0) {
      accepted_node[ts] = lo + acc;  // index in the forest
      accepted_len[ts] = acc_depth;
      s_acc = acc;
    }
  }
  __syncthreads();

  // tokens gained and the next unmask set U(accepted node)
  const int acc = s_acc;
  if (warp == 0) {
    int gained = 0;
    for (int w = 0; w < words; ++w) {
      const int r = w * 32 + lane;
      bool f0 = false, fa = false;
      if (r < R) {
        f0 = (staged ? s_st[r] : st[r]) != mask_id;
        fa = (staged ? s_st[acc * R + r] : st[acc * R + r]) != mask_id;
      }
      gained += __popc(__ballot_sync(full, fa)) - __popc(__ballot_sync(full, f0));
      if (r < R) {
        const bool in_u = (s_u[acc][w] >> lane) & 1u;
        unmask_flag[ts * R + r] = in_u ? 1 : 0;
        unmask_tok[ts * R + r] =
            in_u ? (staged ? s_t1[acc * R + r] : t1[(size_t)(acc * R + r) * top1_stride]) : -1;
      }
    }
    if (lane == 0) n_new_tokens[ts] = gained;
  }
}

}  // namespace tsd

static int accept_launch(int32_t batch, int32_t n_branches, int32_t n_cur, int32_t rows_per_branch,
                         const int32_t* parent, const int32_t* state, int32_t mask_id, const float* conf,
                         const int32_t* top1_idx, int32_t top1_stride, float tau, int32_t rule,
                         int32_t search, uint8_t* edge_valid, int32_t* prefix_len, int32_t* accepted_node,
                         int32_t* accepted_len, int32_t* n_new_tokens, uint8_t* unmask_flag,
                         int32_t* unmask_tok, uint32_t* status, tsd_stream_t stream,
                         const tsd::RelaxedArgs& x) {
  if (batch < 0 || n_cur < 1 || n_cur > n_branches || n_branches < 1 || n_branches > tsd::kMaxBranches || rows_per_branch < 1 ||
      rows_per_branch > tsd::kMaxRows || top1_stride < 1)
    return TSD_ERR_INVALID_ARG;
  if (rule < TSD_ACCEPT_EXACT || rule > TSD_ACCEPT_PROB) return TSD_ERR_INVALID_ARG;
  if (rule == TSD_ACCEPT_TOPK && (x.topk_m < 1 || x.topk_m > top1_stride)) return TSD_ERR_INVALID_ARG;
  if (rule == TSD_ACCEPT_PROB && !x.logits) return TSD_ERR_INVALID_ARG;
  if (x.logits) {
    if (x.dtype != TSD_F32 && x.dtype != TSD_BF16) return TSD_ERR_UNSUPPORTED;
    if (!x.lse || x.vocab < 1 || x.ld < x.vocab) return TSD_ERR_INVALID_ARG;
  }
  if (search != TSD_SEARCH_GREEDY && search != TSD_SEARCH_LONGEST) return TSD_ERR_INVALID_ARG;
  if (!(tau == tau)) return TSD_ERR_INVALID_ARG;  // NaN threshold
  if (batch == 0) return TSD_OK;
  if (!parent || !state || !conf || !top1_idx || !edge_valid || !prefix_len || !accepted_node ||
      !accepted_len || !n_new_tokens || !unmask_flag || !unmask_tok)
    return TSD_ERR_INVALID_ARG;
  const dim3 grid(batch, n_cur < n_branches ? 2 : 1);
  const int tree_max = n_cur > n_branches - n_cur ? n_cur : n_branches - n_cur;
  const int threads = tree_max * 32 < tsd::kAcceptThreads ? tsd::kAcceptThreads
                      : (tree_max * 32 > tsd::kAcceptMaxThreads ? tsd::kAcceptMaxThreads : tree_max * 32);
  auto kernel = rows_per_branch <= 32 ? tsd::accept_kernel<1>
                : rows_per_branch <= 64 ? tsd::accept_kernel<2> : tsd::accept_kernel<tsd::kRowWords>;
  kernel<<<grid, threads, 0, stream>>>(
      n_branches, n_cur, rows_per_branch, parent, state, mask_id, conf, top1_idx, top1_stride, tau, rule,
      search, edge_valid, prefix_len, accepted_node, accepted_len, n_new_tokens, unmask_flag,
      unmask_tok, status, x);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return tsd::cuda_fail(e, "accept_kernel");
  return TSD_OK;
}

extern "C" int tsd_accept_trajectories(int32_t batch, int32_t n_branches, int32_t rows_per_branch,
                                       const int32_t* parent, const int32_t* state, int32_t mask_id,
                                       const float* conf, const int32_t* top1_idx, int32_t top1_stride,
                                       float tau, int32_t rule, int32_t search, uint8_t* edge_valid,
                                       int32_t* prefix_len, int32_t* accepted_node,
                                       int32_t* accepted_len, int32_t* n_new_tokens,
                                       uint8_t* unmask_flag, int32_t* unmask_tok, uint32_t* status,
                                       tsd_stream_t stream) {
  if (rule != TSD_ACCEPT_EXACT && rule != TSD_ACCEPT_TOP1) return TSD_ERR_INVALID_ARG;
  return accept_launch(batch, n_branches, n_branches, rows_per_branch, parent, state, mask_id, conf, top1_idx,
                       top1_stride, tau, rule, search, edge_valid, prefix_len, accepted_node, accepted_len,
                       n_new_tokens, unmask_flag, unmask_tok, status, stream, tsd::RelaxedArgs{});
}

extern "C" int tsd_accept_joint_trees(int32_t batch, int32_t n_branches, int32_t n_cur,
                                      int32_t rows_per_branch, const int32_t* parent, const int32_t* state,
                                      int32_t mask_id, const float* conf, const int32_t* top1_idx,
                                      int32_t top1_stride, float tau, int32_t rule, int32_t search,
                                      uint8_t* edge_valid, int32_t* prefix_len, int32_t* accepted_node,
                                      int32_t* accepted_len, int32_t* n_new_tokens, uint8_t* unmask_flag,
                                      int32_t* unmask_tok, uint32_t* status, tsd_stream_t stream) {
  if (rule != TSD_ACCEPT_EXACT && rule != TSD_ACCEPT_TOP1) return TSD_ERR_INVALID_ARG;
  return accept_launch(batch, n_branches, n_cur, rows_per_branch, parent, state, mask_id, conf, top1_idx,
                       top1_stride, tau, rule, search, edge_valid, prefix_len, accepted_node, accepted_len,
                       n_new_tokens, unmask_flag, unmask_tok, status, stream, tsd::RelaxedArgs{});
}

extern "C" int tsd_accept_relaxed(int32_t batch, int32_t n_branches, int32_t n_cur, int32_t rows_per_branch,
                                  const int32_t* parent, const int32_t* state, int32_t mask_id,
                                  const float* conf, const int32_t* topk_idx, int32_t topk_stride,
                                  int32_t topk_m, const void* logits, int32_t dtype, int64_t vocab,
                                  int64_t row_stride, const float* lse, float tau, int32_t rule,
                                  int32_t search, uint8_t* edge_valid, int32_t* prefix_len,
                                  int32_t* accepted_node, int32_t* accepted_len, int32_t* n_new_tokens,
                                  uint8_t* unmask_flag, int32_t* unmask_tok, float* draft_prob,
                                  uint32_t* status, tsd_stream_t stream) {
  tsd::RelaxedArgs x{};
  x.topk_m = topk_m;
  x.logits = logits;
  x.dtype = dtype;
  x.vocab = vocab;
  x.ld = row_stride;
  x.lse = lse;
  x.draft_prob = logits ? draft_prob : nullptr;
  return accept_launch(batch, n_branches, n_cur, rows_per_branch, parent, state, mask_id, conf, topk_idx,
                       topk_stride, tau, rule, search, edge_valid, prefix_len, accepted_node, accepted_len,
                       n_new_tokens, unmask_flag, unmask_tok, status, stream, x);
}
