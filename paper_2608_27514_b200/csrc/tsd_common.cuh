// Internal helpers shared by the tsd kernels (not part of the C ABI).
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include "../../include/tsd.h"

namespace tsd {

// Records a failed CUDA runtime call for tsd_last_cuda_error(); returns TSD_ERR_CUDA.
int cuda_fail(cudaError_t e, const char* where);

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// ---- branch-mask blob (written by tsd_build_branch_mask, read by the attention kernels) ----
// int32 words: header[8] | cache_len[round4(S)] | records[S * n_qt], each record =
// { count, 0, (draft_tile, bits) * n_qt }.  A query tile is 128 consecutive draft rows of one
// sequence = 128/R branch slots; bit (qs*4 + ks) of `bits` = slot qs of the query tile may read
// slot ks of draft tile `draft_tile`.
constexpr int kMaskMagic = 0x54534431;
constexpr int kTile = 128;
constexpr int kHdrWords = 8;
enum { H_MAGIC = 0, H_S, H_B, H_R, H_NC, H_NQT, H_REC_WORDS, H_RECS_OFF };

struct MaskDims {
  int n_qt;        // query tiles per sequence
  int rec_words;   // words per (sequence, query tile) record
  int lens_off;    // word offset of cache_len[]
  int recs_off;    // word offset of the records
  size_t bytes;
};

inline MaskDims mask_dims(const tsd_layout& L) {
  MaskDims m;
  const int N = L.n_branches * L.rows_per_branch;
  m.n_qt = (N + kTile - 1) / kTile;
  m.rec_words = 2 + 2 * m.n_qt;
  m.lens_off = kHdrWords;
  m.recs_off = kHdrWords + ((L.batch + 3) / 4) * 4;
  m.bytes = (size_t)(m.recs_off + (size_t)L.batch * m.n_qt * m.rec_words) * 4;
  m.bytes = (m.bytes + 15) / 16 * 16;
  return m;
}

int validate_layout(const tsd_layout* L);
int check_attention_args(const tsd_layout* L, const void* mask, const void* q, int64_t q_stride_b,
                         int64_t q_stride_row, int64_t q_stride_head, const void* k_cache, const void* v_cache,
                         int64_t c_stride_b, int64_t c_stride_row, int64_t c_stride_head, const void* k_draft,
                         const void* v_draft, int64_t d_stride_b, int64_t d_stride_row, int64_t d_stride_head,
                         const void* out, int64_t o_stride_b, int64_t o_stride_row, int64_t o_stride_head,
                         float sm_scale, const void* workspace);

// attention launchers (defined in their own translation units)
struct AttnArgs {
  tsd_layout L;
  const int32_t* mask;
  const void *q, *kc, *vc, *kd, *vd;
  void* out;
  float* lse;
  int64_t qs_b, qs_r, qs_h, cs_b, cs_r, cs_h, ds_b, ds_r, ds_h, os_b, os_r, os_h;
  float sm_scale;
  void* workspace;
  size_t workspace_bytes;
  uint32_t* status;
  cudaStream_t stream;
};
int launch_attention_simt(const AttnArgs& a);
bool attention_tc_supported(const AttnArgs& a);
size_t attention_tc_workspace_bytes(const tsd_layout& L);
int launch_attention_tc(const AttnArgs& a);

// ---- ticket words: blocks that share a result meet without waiting for each other ----
// Each block publishes its part, then arrives on the ticket word; the last arrival reads the
// others' parts and finishes the result.  A word in use carries kTicketTag in its upper 24 bits
// and the number of arrivals so far in the lower 8; any other content counts as idle and the last
// arrival writes 0, so the memory that holds the words needs no clearing between calls.
constexpr unsigned kTicketTag = 0x7FC3A9u;

#ifdef __CUDACC__
// One arrival; true for the last of n arrivals (n <= 255).
__device__ __forceinline__ bool ticket_arrive(unsigned* t, int n) {
  unsigned old = *reinterpret_cast<volatile unsigned*>(t), assumed, cnt;
  do {
    assumed = old;
    cnt = (assumed >> 8) == kTicketTag ? (assumed & 0xffu) : 0u;
    const unsigned next = (cnt + 1 == (unsigned)n) ? 0u : ((kTicketTag << 8) | (cnt + 1));
    old = atomicCAS(t, assumed, next);
  } while (old != assumed);
  return cnt + 1 == (unsigned)n;
}
// Arrivals so far (a snapshot: more may follow at any time).
__device__ __forceinline__ unsigned ticket_count(const unsigned* t) {
  const unsigned v = *reinterpret_cast<const volatile unsigned*>(t);
  return (v >> 8) == kTicketTag ? (v & 0xffu) : 0u;
}
#endif

__device__ __forceinline__ float to_float(float x) { return x; }
__device__ __forceinline__ float to_float(__nv_bfloat16 x) { return __bfloat162float(x); }
__device__ __forceinline__ void from_float(float& d, float x) { d = x; }
__device__ __forceinline__ void from_float(__nv_bfloat16& d, float x) { d = __float2bfloat16_rn(x); }

}  // namespace tsd
