// Inter-block speculation helpers (paper Section 3.4, Eq. 3, Appendix D): the branch-visibility
// bitsets of a joint pass over the trees of two consecutive blocks, and the trigger that decides
// whether the next block gets drafts at all.
//
// Joint layout: branches [0, n_cur) = tree of the current block (root 0), branches [n_cur, B) =
// compact tree of the next block (root n_cur).  The roots read each other, a draft reads the other
// block's root, nobody reads a draft but the draft itself.  tsd_build_branch_mask turns the
// bitsets into the tile lists the attention kernel walks.
#include <math_constants.h>
#include "tsd_common.cuh"

namespace tsd {

__global__ void interblock_vis_kernel(int B, int n_cur, int words, uint64_t* __restrict__ vis, size_t total) {
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;  // one (sequence, branch, word)
  if (i >= total) return;
  const int w = (int)(i % words);
  const int b = (int)((i / words) % B);
  uint64_t bits = 0;
  if ((b >> 6) == w) bits |= 1ull << (b & 63);
  if (n_cur < B) {
    const int other = b < n_cur ? n_cur : 0;  // the root this branch reads besides itself
    if ((other >> 6) == w) bits |= 1ull << (other & 63);
  }
  vis[i] = bits;
}

// One warp per sequence: c^(1) of a block = the largest confidence among its masked rows.
__global__ void __launch_bounds__(32)
interblock_trigger_kernel(int B, int R, const int32_t* __restrict__ state, const float* __restrict__ conf,
                          const int32_t* __restrict__ node_cur, int node_next, int mask_id, float tau,
                          uint8_t* __restrict__ trigger, float* __restrict__ top_conf,
                          uint32_t* __restrict__ status) {
  const int s = blockIdx.x, lane = threadIdx.x;
  int cur = node_cur ? node_cur[s] : 0;
  if (cur < 0 || cur >= B) {
    if (lane == 0 && status) atomicOr(status, TSD_STATUS_BAD_PARENT);
    cur = 0;
  }
  float c[2] = {-CUDART_INF_F, -CUDART_INF_F};
  const int node[2] = {cur, node_next};
#pragma unroll
  for (int t = 0; t < 2; ++t) {
    const size_t base = ((size_t)s * B + node[t]) * R;
    for (int r = lane; r < R; r += 32)
      if (state[base + r] == mask_id) c[t] = fmaxf(c[t], conf[base + r]);
#pragma unroll
    for (int off = 16; off; off >>= 1) c[t] = fmaxf(c[t], __shfl_xor_sync(0xffffffffu, c[t], off));
  }
  if (lane == 0) {
    trigger[s] = (c[1] != -CUDART_INF_F && (c[1] > c[0] || c[1] > tau)) ? 1 : 0;
    if (top_conf) { top_conf[2 * s] = c[0]; top_conf[2 * s + 1] = c[1]; }
  }
}

}  // namespace tsd

extern "C" int tsd_build_interblock_vis(int32_t batch, int32_t n_branches, int32_t n_cur, uint64_t* vis,
                                        tsd_stream_t stream) {
  if (batch < 0 || n_branches < 1 || n_branches > 256 || n_cur < 1 || n_cur > n_branches)
    return TSD_ERR_INVALID_ARG;
  if (batch == 0) return TSD_OK;
  if (!vis) return TSD_ERR_INVALID_ARG;
  const int words = (n_branches + 63) / 64;
  const size_t total = (size_t)batch * n_branches * words;
  tsd::interblock_vis_kernel<<<(unsigned)((total + 255) / 256), 256, 0, stream>>>(n_branches, n_cur, words, vis,
                                                                               total);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return tsd::cuda_fail(e, "interblock_vis_kernel");
  return TSD_OK;
}

extern "C" int tsd_interblock_trigger(int32_t batch, int32_t n_branches, int32_t rows_per_branch,
                                      const int32_t* state, const float* conf, const int32_t* node_cur,
                                      int32_t node_next, int32_t mask_id, float tau, uint8_t* trigger,
                                      float* top_conf, uint32_t* status, tsd_stream_t stream) {
  if (batch < 0 || n_branches < 1 || rows_per_branch < 1 || node_next < 0 || node_next >= n_branches ||
      !(tau == tau))
    return TSD_ERR_INVALID_ARG;
  if (batch == 0) return TSD_OK;
  if (!state || !conf || !trigger) return TSD_ERR_INVALID_ARG;
  tsd::interblock_trigger_kernel<<<batch, 32, 0, stream>>>(n_branches, rows_per_branch, state, conf, node_cur,
                                                           node_next, mask_id, tau, trigger, top_conf, status);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return tsd::cuda_fail(e, "interblock_trigger_kernel");
  return TSD_OK;
}
