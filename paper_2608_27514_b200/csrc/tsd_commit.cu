// The step after the path: commit what a verification pass accepted (paper Section 3.3, last
// paragraph of "Verification procedure"; Section 3.1: the accepted node is where the next pass
// starts; Theorem 1: every edge of the accepted path is one step of the sequential decoder).
//
// One warp per sequence, lanes own rows.  The accepted path is walked from the accepted node up to
// the root (bounded by the number of branches); a row filled by the path node at depth j is logged
// at sequential step step_base + j - 1, the rows of U(accepted node) at step_base + depth.  The
// next root is written into the sequence's token buffer at the block's position, and the block's
// step counter moves on by depth + 1 (depth, if the accepted node had nothing left to unmask).
#include <algorithm>
#include "tsd_common.cuh"

namespace tsd {

constexpr int kCommitMaxRows = 128;
constexpr int kCommitRowsPerLane = kCommitMaxRows / 32;
constexpr int kCommitMaxBranches = 256;

__global__ void __launch_bounds__(32)
commit_kernel(int B, int R, int root, const int32_t* __restrict__ parent, const int32_t* __restrict__ state,
              const int32_t* __restrict__ accepted_node, const uint8_t* __restrict__ unmask_flag,
              const int32_t* __restrict__ unmask_tok, int mask_id, int32_t* __restrict__ tokens,
              int64_t seq_stride, const int32_t* __restrict__ block_start, int32_t* __restrict__ root_out,
              int32_t* __restrict__ fill_step, int32_t* __restrict__ step_base,
              int32_t* __restrict__ n_masked, uint32_t* __restrict__ status) {
  __shared__ int s_path[kCommitMaxBranches];  // accepted node first, root last
  __shared__ int s_depth;
  const int s = blockIdx.x, lane = threadIdx.x;
  const int32_t* par = parent + (size_t)s * B;
  const int32_t* st = state + (size_t)s * B * R;
  if (lane == 0) {
    // `root` is the forest index of this tree's root (0 for a tree of its own); node and parent
    // indices are forest indices, and a tree's nodes follow its root
    int b = accepted_node ? accepted_node[s] : root, n = 0;
    bool bad = b < root || b >= B;
    if (bad) b = root;
    s_path[0] = b;
    while (b > root && n < B) {  // parents precede their children, so this ends within B steps
      const int p = par[b];
      if (p < root || p >= b) { bad = true; break; }
      b = p;
      s_path[++n] = b;
    }
    if (bad) {  // inconsistent tree: commit nothing but U(root)
      if (status) atomicOr(status, TSD_STATUS_BAD_PARENT);
      s_path[0] = root;
      n = 0;
    }
    s_depth = n;
  }
  __syncwarp();
  const int depth = s_depth, acc = s_path[0];
  const int base = step_base ? step_base[s] : 0;
  const int64_t start = block_start ? block_start[s] : 0;
  const bool in_range = start >= 0 && start + R <= seq_stride;
  if (tokens && !in_range && lane == 0 && status) atomicOr(status, TSD_STATUS_BAD_INDEX);
  int still = 0, open_rows = 0;
#pragma unroll
  for (int i = 0; i < kCommitRowsPerLane; ++i) {
    const int r = lane + 32 * i;
    if (r >= R) continue;
    int v = st[(size_t)acc * R + r];
    int step = -1;
    if (v == mask_id) {
      ++open_rows;
      if (unmask_flag && unmask_flag[(size_t)s * R + r]) {
        v = unmask_tok[(size_t)s * R + r];
        step = base + depth;
      }
    } else if (st[(size_t)root * R + r] == mask_id) {
      // filled somewhere on the path: by the shallowest node that holds it
      int j = depth;  // s_path[depth - j] is the path node at depth j
      while (j > 1 && st[(size_t)s_path[depth - j + 1] * R + r] != mask_id) --j;
      step = base + j - 1;
    }
    if (v == mask_id) ++still;
    if (root_out) root_out[(size_t)s * R + r] = v;
    if (tokens && in_range) tokens[(size_t)s * seq_stride + start + r] = v;
    if (fill_step && step >= 0) fill_step[(size_t)s * R + r] = step;
  }
#pragma unroll
  for (int off = 16; off; off >>= 1) {
    still += __shfl_xor_sync(0xffffffffu, still, off);
    open_rows += __shfl_xor_sync(0xffffffffu, open_rows, off);
  }
  if (lane == 0) {
    if (n_masked) n_masked[s] = still;
    if (step_base) step_base[s] = base + depth + (open_rows > 0 ? 1 : 0);
  }
}

// The accepted node's draft K/V rows -> a destination of the caller's (one layer per call): 16-byte
// vectors, one thread each; grid.y = sequence.  The accepted node comes from device memory, so a
// decode loop can chain this after the acceptance without a read-back.
__global__ void __launch_bounds__(256)
gather_accepted_kv_kernel(int B, int R, int H, int vec_per_head, const int32_t* __restrict__ accepted_node,
                          const uint4* __restrict__ k_src, const uint4* __restrict__ v_src, int64_t ss_b,
                          int64_t ss_r, int64_t ss_h, uint4* __restrict__ k_dst, uint4* __restrict__ v_dst,
                          int64_t ds_b, int64_t ds_r, int64_t ds_h, const int32_t* __restrict__ dst_row0,
                          int dst_rows, uint32_t* __restrict__ status) {
  const int s = blockIdx.y;
  const int node = accepted_node ? accepted_node[s] : 0;
  const int64_t row0 = dst_row0 ? dst_row0[s] : 0;
  if (node < 0 || node >= B || row0 < 0 || row0 + R > dst_rows) {  // nothing of this sequence is written
    if (threadIdx.x == 0 && blockIdx.x == 0 && status) atomicOr(status, TSD_STATUS_BAD_INDEX);
    return;
  }
  const int total = R * H * vec_per_head;
  for (int t = blockIdx.x * blockDim.x + threadIdx.x; t < total; t += gridDim.x * blockDim.x) {
    const int c = t % vec_per_head, h = (t / vec_per_head) % H, r = t / (vec_per_head * H);
    const int64_t src = s * ss_b + ((int64_t)node * R + r) * ss_r + h * ss_h + c;   // in 16-byte units
    const int64_t dst = s * ds_b + (row0 + r) * ds_r + h * ds_h + c;
    k_dst[dst] = k_src[src];
    if (v_src) v_dst[dst] = v_src[src];
  }
}

}  // namespace tsd

extern "C" int tsd_gather_accepted_kv(int32_t batch, int32_t n_branches, int32_t rows_per_branch, int32_t n_kv_heads,
                                      int32_t head_dim, int32_t dtype, const int32_t* accepted_node,
                                      const void* k_draft, const void* v_draft, int64_t d_stride_b,
                                      int64_t d_stride_row, int64_t d_stride_head, void* k_out, void* v_out,
                                      int64_t o_stride_b, int64_t o_stride_row, int64_t o_stride_head,
                                      const int32_t* out_row0, int32_t out_rows, uint32_t* status,
                                      tsd_stream_t stream) {
  if (batch < 0 || n_branches < 1 || n_branches > tsd::kCommitMaxBranches || rows_per_branch < 1 ||
      rows_per_branch > tsd::kCommitMaxRows || n_kv_heads < 1 || head_dim < 1 || out_rows < rows_per_branch)
    return TSD_ERR_INVALID_ARG;
  if (dtype != TSD_F32 && dtype != TSD_BF16) return TSD_ERR_UNSUPPORTED;
  const int esize = dtype == TSD_F32 ? 4 : 2;
  if ((head_dim * esize) % 16 != 0) return TSD_ERR_UNSUPPORTED;
  if (batch == 0) return TSD_OK;
  if (!k_draft || !k_out || (v_draft == nullptr) != (v_out == nullptr)) return TSD_ERR_INVALID_ARG;
  const void* ptrs[] = {k_draft, v_draft, k_out, v_out};
  for (const void* p : ptrs)
    if (p && !tsd::aligned16(p)) return TSD_ERR_INVALID_ARG;
  const int64_t strides[] = {d_stride_b, d_stride_row, d_stride_head, o_stride_b, o_stride_row, o_stride_head};
  for (int64_t st : strides)
    if (st < 0 || (st * esize) % 16 != 0) return TSD_ERR_INVALID_ARG;
  if (d_stride_head < head_dim || o_stride_head < head_dim) return TSD_ERR_INVALID_ARG;
  const int per16 = 16 / esize, vec_per_head = head_dim / per16;
  const int total = rows_per_branch * n_kv_heads * vec_per_head;
  dim3 grid((unsigned)std::min((total + 255) / 256, 64), (unsigned)batch);
  tsd::gather_accepted_kv_kernel<<<grid, 256, 0, stream>>>(
      n_branches, rows_per_branch, n_kv_heads, vec_per_head, accepted_node, static_cast<const uint4*>(k_draft),
      static_cast<const uint4*>(v_draft), d_stride_b / per16, d_stride_row / per16, d_stride_head / per16,
      static_cast<uint4*>(k_out), static_cast<uint4*>(v_out), o_stride_b / per16, o_stride_row / per16,
      o_stride_head / per16, out_row0, out_rows, status);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return tsd::cuda_fail(e, "gather_accepted_kv_kernel");
  return TSD_OK;
}

extern "C" int tsd_commit_accepted(int32_t batch, int32_t n_branches, int32_t rows_per_branch, int32_t tree_root,
                                   const int32_t* parent, const int32_t* state, const int32_t* accepted_node,
                                   const uint8_t* unmask_flag, const int32_t* unmask_tok, int32_t mask_id,
                                   int32_t* tokens, int64_t seq_stride, const int32_t* block_start,
                                   int32_t* root_out, int32_t* fill_step, int32_t* step_base,
                                   int32_t* n_masked, uint32_t* status, tsd_stream_t stream) {
  if (batch < 0 || n_branches < 1 || n_branches > tsd::kCommitMaxBranches || rows_per_branch < 1 ||
      rows_per_branch > tsd::kCommitMaxRows)
    return TSD_ERR_INVALID_ARG;
  if (tree_root < 0 || tree_root >= n_branches) return TSD_ERR_INVALID_ARG;
  if ((unmask_flag == nullptr) != (unmask_tok == nullptr)) return TSD_ERR_INVALID_ARG;
  if (tokens && seq_stride < rows_per_branch) return TSD_ERR_INVALID_ARG;
  if (batch == 0) return TSD_OK;
  if (!parent || !state) return TSD_ERR_INVALID_ARG;
  tsd::commit_kernel<<<batch, 32, 0, stream>>>(n_branches, rows_per_branch, tree_root, parent, state, accepted_node,
                                               unmask_flag, unmask_tok, mask_id, tokens, seq_stride, block_start,
                                               root_out, fill_step, step_base, n_masked, status);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return tsd::cuda_fail(e, "commit_kernel");
  return TSD_OK;
}
