// Draft-tree construction (paper Alg. 1, Phase 2 "speculative expansion"; Section 3.2), the step
// right before the verification pass, fused with the root update that follows acceptance.
//
// One warp per sequence.  The next root is the accepted node's block state plus its unmask set
// (what tsd_accept_trajectories returned); the candidate pool is the top-k (token, probability) of
// every row still masked in that root, read from the scores of the pass that has just been verified
// (Section 3.1: the verification of step t provides the logits for drafting step t+1).
//   level 1  : the k most probable pool entries, one child each (root + one (row, token));
//   level > 1: every frontier node gets one child = the node + the most probable pool entry whose
//              row is still masked in it;
//   pruning  : the W most probable children of a level survive, in that order, and form the next
//              frontier; the tree stops at max_nodes nodes.
// Ties go to the lower row, then the lower rank, then the earlier child.  Lanes own rows
// (row = lane + 32 i); every selection is a warp arg-best reduction, so the result is exact and
// deterministic.  Unused node slots are copies of the root hanging off the root (an empty delta is
// never accepted).
//
// For the joint pass of inter-block speculation (Section 3.4) the tree can be written into a slice
// of a larger forest: `out_stride` branches per sequence in the output arrays, `node_base` added
// to every parent index, and a per-sequence `enable` byte (the trigger of Eq. 3) that, when 0,
// leaves the tree at its root.
#include <limits.h>
#include <math_constants.h>
#include "tsd_common.cuh"

namespace tsd {

constexpr int kTreeMaxRows = 128;   // rows per branch
constexpr int kTreeRowsPerLane = kTreeMaxRows / 32;
constexpr int kTreeMaxK = 8;
constexpr int kTreeMaxWidth = 32;   // one lane per child when a level is pruned

struct Cand {
  float p;
  int row, rank;
};
__device__ __forceinline__ bool cand_before(const Cand& a, const Cand& b) {  // a beats b
  if (b.row < 0) return a.row >= 0;
  if (a.row < 0) return false;
  if (a.p != b.p) return a.p > b.p;
  if (a.row != b.row) return a.row < b.row;
  return a.rank < b.rank;
}
// The best candidate of the warp in two warp-wide reductions (redux.sync): probabilities are
// non-negative, so their bit patterns order like unsigned integers; among the lanes that hold the
// largest one, the smallest (row, rank) wins.  Every lane returns with the winner.
__device__ __forceinline__ Cand warp_best(Cand c) {
  const unsigned full = 0xffffffffu;
  const bool valid = c.row >= 0 && c.p >= 0.f;
  const unsigned pk = valid ? (c.p > 0.f ? __float_as_uint(c.p) + 1u : 1u) : 0u;  // 0 = no candidate in this lane
  const unsigned pmax = __reduce_max_sync(full, pk);
  Cand w = {0.f, -1, 0};
  if (pmax == 0u) return w;
  const unsigned rr = (valid && pk == pmax) ? ((unsigned)c.row << 8) | (unsigned)c.rank : 0xffffffffu;
  const unsigned rmin = __reduce_min_sync(full, rr);
  w.p = __uint_as_float(pmax - 1u);  // a zero of either sign comes back as +0
  w.row = (int)(rmin >> 8);
  w.rank = (int)(rmin & 0xffu);
  return w;
}

// RPL = rows per lane (R <= 32 * RPL), KK = candidates per row held in registers (k <= KK): the
// selection loops are unrolled over RPL x KK, so the common block of 32 rows with k <= 4 runs a
// tenth of the instructions of the largest case (a single warp is bound by instruction latency).
template <int RPL, int KK>
__global__ void __launch_bounds__(32)
build_draft_tree_kernel(int prev_branches, int R, int k, const int32_t* __restrict__ prev_state,
                        const int32_t* __restrict__ accepted_node, const uint8_t* __restrict__ unmask_flag,
                        const int32_t* __restrict__ unmask_tok, int mask_id,
                        const int32_t* __restrict__ topk_idx, const float* __restrict__ topk_prob, int W,
                        int D, int max_nodes, int out_stride, int node_base,
                        const uint8_t* __restrict__ enable, int32_t* __restrict__ parent, int32_t* __restrict__ state,
                        float* __restrict__ node_prob, int32_t* __restrict__ n_nodes,
                        uint32_t* __restrict__ status) {
  __shared__ int s_front[kTreeMaxWidth];
  __shared__ int s_cpar[kTreeMaxWidth], s_crow[kTreeMaxWidth], s_crank[kTreeMaxWidth];
  __shared__ float s_cp[kTreeMaxWidth];
  __shared__ uint32_t s_mask[256][RPL];  // per node: which rows are still masked
  const int s = blockIdx.x, lane = threadIdx.x;
  int acc = accepted_node ? accepted_node[s] : 0;
  if (acc < 0 || acc >= prev_branches) {  // inconsistent device data: report, fall back to node 0
    if (lane == 0 && status) atomicOr(status, TSD_STATUS_BAD_PARENT);
    acc = 0;
  }
  const size_t src = ((size_t)s * prev_branches + acc) * R;  // rows of the accepted node
  const int32_t* idx = topk_idx + src * k;
  const float* prb = topk_prob + src * k;
  int32_t* st = state + (size_t)s * out_stride * R;
  int32_t* par = parent + (size_t)s * out_stride;
  float* np_ = node_prob + (size_t)s * out_stride;
  if (enable && !enable[s]) D = 0;

  // next root = accepted state + its unmask set; every node slot starts as a copy of it
  bool root_masked[RPL];
#pragma unroll
  for (int i = 0; i < RPL; ++i) {
    const int r = lane + 32 * i;
    root_masked[i] = false;
    if (r < R) {
      int v = prev_state[src + r];
      if (unmask_flag && unmask_flag[(size_t)s * R + r]) v = unmask_tok[(size_t)s * R + r];
      root_masked[i] = v == mask_id;
      for (int b = 0; b < max_nodes; ++b) st[(size_t)b * R + r] = v;
    }
  }
  for (int b = lane; b < max_nodes; b += 32) {
    par[b] = b == 0 ? -1 : node_base;
    np_[b] = b == 0 ? 1.f : 0.f;
  }
  // the pool lives in registers (this lane's rows x k) and the nodes' masked-row sets in shared
  // memory, so the selection rounds below touch no global memory
  float pool[RPL][KK];
#pragma unroll
  for (int i = 0; i < RPL; ++i) {
    const int r = lane + 32 * i;
#pragma unroll
    for (int j = 0; j < KK; ++j) pool[i][j] = (r < R && j < k) ? prb[(size_t)r * k + j] : -1.f;
    const uint32_t word = __ballot_sync(0xffffffffu, root_masked[i]);
    if (lane == 0) s_mask[0][i] = word;
  }
  __syncwarp();

  int n = 1, n_front = 1;
  if (lane == 0) s_front[0] = 0;
  for (int level = 1; level <= D && n < max_nodes && n_front > 0; ++level) {
    int n_child = 0;
    if (level == 1) {
      // the k best pool entries: k rounds, the winner's entry is marked used in its lane
      uint32_t used = 0;
      for (int t = 0; t < k; ++t) {
        Cand best = {0.f, -1, 0};
#pragma unroll
        for (int i = 0; i < RPL; ++i) {
          const int r = lane + 32 * i;
          if (r < R && root_masked[i]) {
#pragma unroll
            for (int j = 0; j < KK; ++j) {
              if (j >= k || ((used >> (i * KK + j)) & 1u)) continue;
              const Cand c = {pool[i][j], r, j};
              if (cand_before(c, best)) best = c;
            }
          }
        }
        const Cand win = warp_best(best);
        if (win.row < 0) break;  // pool exhausted (uniform: every lane sees the same winner)
        if ((win.row & 31) == lane) used |= 1u << ((win.row >> 5) * KK + win.rank);
        if (lane == 0) { s_cpar[n_child] = 0; s_crow[n_child] = win.row; s_crank[n_child] = win.rank; s_cp[n_child] = win.p; }
        ++n_child;
      }
    } else {
      for (int f = 0; f < n_front; ++f) {
        const int node = s_front[f];
        Cand best = {0.f, -1, 0};
#pragma unroll
        for (int i = 0; i < RPL; ++i) {
          const int r = lane + 32 * i;
          if (r < R && ((s_mask[node][i] >> lane) & 1u)) {
#pragma unroll
            for (int j = 0; j < KK; ++j) {
              if (j >= k) continue;
              const Cand c = {pool[i][j], r, j};
              if (cand_before(c, best)) best = c;
            }
          }
        }
        const Cand win = warp_best(best);
        if (win.row < 0) continue;  // the node is full
        if (lane == 0) { s_cpar[n_child] = node; s_crow[n_child] = win.row; s_crank[n_child] = win.rank; s_cp[n_child] = win.p; }
        ++n_child;
      }
    }
    __syncwarp();
    // prune: lane c ranks child c by (probability descending, generation order); the first
    // min(W, budget) become nodes n, n+1, ... and the next frontier
    const int keep = min(min(W, max_nodes - n), n_child);
    int pos = INT_MAX;
    if (lane < n_child) {
      pos = 0;
      for (int c = 0; c < n_child; ++c)
        pos += (s_cp[c] > s_cp[lane] || (s_cp[c] == s_cp[lane] && c < lane)) ? 1 : 0;
    }
    __syncwarp();
    int my_par = -1, my_row = 0, my_tok = 0;
    float my_p = 0.f;
    if (pos < keep) {
      my_par = s_cpar[lane]; my_row = s_crow[lane]; my_p = s_cp[lane];
      my_tok = idx[(size_t)my_row * k + s_crank[lane]];
    }
    __syncwarp();
    if (pos < keep) {
      s_front[pos] = n + pos;
      par[n + pos] = node_base + my_par;
      np_[n + pos] = my_p;
    }
    // materialise the kept children: node = copy of its parent + one filled row
    for (int q = 0; q < keep; ++q) {
      // lane that owns position q broadcasts its child
      const unsigned owner_mask = __ballot_sync(0xffffffffu, pos == q);
      const int owner = __ffs(owner_mask) - 1;
      const int cpar = __shfl_sync(0xffffffffu, my_par, owner);
      const int crow = __shfl_sync(0xffffffffu, my_row, owner);
      const int ctok = __shfl_sync(0xffffffffu, my_tok, owner);
#pragma unroll
      for (int i = 0; i < RPL; ++i) {
        const int r = lane + 32 * i;
        if (r < R) st[(size_t)(n + q) * R + r] = r == crow ? ctok : st[(size_t)cpar * R + r];
        if (lane == 0) s_mask[n + q][i] = s_mask[cpar][i] & ~((crow >> 5) == i ? (1u << (crow & 31)) : 0u);
      }
    }
    __syncwarp();
    n += keep;
    n_front = keep;
  }
  if (lane == 0) n_nodes[s] = n;
}

}  // namespace tsd

extern "C" int tsd_build_draft_tree(int32_t batch, int32_t prev_branches, int32_t rows_per_branch, int32_t k,
                                    const int32_t* prev_state, const int32_t* accepted_node,
                                    const uint8_t* unmask_flag, const int32_t* unmask_tok, int32_t mask_id,
                                    const int32_t* topk_idx, const float* topk_prob, int32_t width,
                                    int32_t depth, int32_t max_nodes, int32_t out_stride,
                                    int32_t node_base, const uint8_t* enable, int32_t* parent,
                                    int32_t* state, float* node_prob, int32_t* n_nodes, uint32_t* status,
                                    tsd_stream_t stream) {
  if (batch < 0 || prev_branches < 1 || rows_per_branch < 1 || rows_per_branch > tsd::kTreeMaxRows || k < 1 ||
      k > tsd::kTreeMaxK || width < 1 || width > tsd::kTreeMaxWidth || depth < 0 || max_nodes < 1 ||
      max_nodes > 256 || out_stride < max_nodes || node_base < 0)
    return TSD_ERR_INVALID_ARG;
  if ((unmask_flag == nullptr) != (unmask_tok == nullptr)) return TSD_ERR_INVALID_ARG;
  if (batch == 0) return TSD_OK;
  if (!prev_state || !topk_idx || !topk_prob || !parent || !state || !node_prob || !n_nodes)
    return TSD_ERR_INVALID_ARG;
  auto launch = [&](auto kernel) {
    kernel<<<batch, 32, 0, stream>>>(prev_branches, rows_per_branch, k, prev_state, accepted_node, unmask_flag,
                                     unmask_tok, mask_id, topk_idx, topk_prob, width, depth, max_nodes, out_stride,
                                     node_base, enable, parent, state, node_prob, n_nodes, status);
  };
  const int rpl = (rows_per_branch + 31) / 32;
  if (rpl == 1 && k <= 4) launch(tsd::build_draft_tree_kernel<1, 4>);
  else if (rpl <= 2 && k <= 4) launch(tsd::build_draft_tree_kernel<2, 4>);
  else launch(tsd::build_draft_tree_kernel<tsd::kTreeRowsPerLane, tsd::kTreeMaxK>);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return tsd::cuda_fail(e, "build_draft_tree_kernel");
  return TSD_OK;
}
