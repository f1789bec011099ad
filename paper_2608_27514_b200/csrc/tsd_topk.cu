// Stage 2: confidence and top-k candidates in one streaming pass over the logits
// (paper Eq. 2: c = max softmax(logits); Section 3.2: top-k candidates per position).
//
// HBM-bound: every logit is read exactly once with 128-bit coalesced loads.  Each thread keeps a
// running (max, sum of exp) pair and a sorted k-entry candidate list in registers; the hot loop
// spends one compare against the list's last entry per element, so the insert path is rare.
// Lists are merged by warp shuffles (k rounds of an arg-best reduction), then across the warps of
// the block through shared memory.  With few rows a row is split into segments handled by
// different blocks; the last block to finish a row (a ticket counter in the workspace, no
// spinning) merges the segment partials in segment order, so the result does not depend on
// arrival order.
//
// Ordering is (logit descending, index ascending) on the raw input values (bf16 and fp32 both
// widen to fp32 exactly), so indices are uniquely defined.
#include <limits.h>
#include <math_constants.h>
#include <algorithm>
#include "tsd_common.cuh"

namespace tsd {

constexpr int kTopkThreads = 256;
constexpr int kTopkWarps = kTopkThreads / 32;
constexpr int kTopkUnroll = 4;
constexpr int kMaxSegments = 32;
constexpr float kLog2e = 1.4426950408889634f;

__device__ __forceinline__ bool key_before(float va, int ia, float vb, int ib) {
  return va > vb || (va == vb && ia < ib);
}

__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__device__ __forceinline__ uint4 ld_stream(const uint4* p) {
  uint4 r;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "l"(p));
  return r;
}

template <int K>
struct Acc {
  float v[K];  // candidate logits, sorted by key order
  int i[K];    // their vocabulary indices
  float m;     // v[0], or 0 while nothing finite has been seen (keeps x - m free of inf - inf)
  float s;     // sum of exp(x - m) over the elements seen

  __device__ __forceinline__ void init() {
#pragma unroll
    for (int j = 0; j < K; ++j) { v[j] = -CUDART_INF_F; i[j] = INT_MAX; }
    m = 0.f;
    s = 0.f;
  }

  // (x, xi) is known to come before the last entry: insert it, dropping the last.
  __device__ __forceinline__ void insert(float x, int xi) {
    bool placed = false;
#pragma unroll
    for (int j = K - 1; j >= 1; --j) {
      if (!placed) {
        if (key_before(x, xi, v[j - 1], i[j - 1])) { v[j] = v[j - 1]; i[j] = i[j - 1]; }
        else { v[j] = x; i[j] = xi; placed = true; }
      }
    }
    if (!placed) { v[0] = x; i[0] = xi; }
  }

  __device__ __forceinline__ void push(float x, int xi) {
    if (x >= v[K - 1]) {  // rare once the list holds k large entries
      if (key_before(x, xi, v[K - 1], i[K - 1])) {
        if (x > v[0]) {  // new running maximum: rebase the sum
          s *= ex2_approx((m - x) * kLog2e);
          if (v[0] == -CUDART_INF_F) s = 0.f;
          m = x;
        }
        insert(x, xi);
      }
    }
    s += ex2_approx((x - m) * kLog2e);
  }

  __device__ __forceinline__ void pop_front() {
#pragma unroll
    for (int j = 0; j < K - 1; ++j) { v[j] = v[j + 1]; i[j] = i[j + 1]; }
    v[K - 1] = -CUDART_INF_F;
    i[K - 1] = INT_MAX;
  }
};

// Combines the 32 lanes' accumulators; every lane returns with the merged result.
template <int K>
__device__ __forceinline__ void warp_merge(Acc<K>& a) {
  const unsigned full = 0xffffffffu;
  float M = a.v[0];
#pragma unroll
  for (int off = 16; off; off >>= 1) M = fmaxf(M, __shfl_xor_sync(full, M, off));
  float s = (a.v[0] == -CUDART_INF_F) ? 0.f : a.s * ex2_approx((a.v[0] - M) * kLog2e);
#pragma unroll
  for (int off = 16; off; off >>= 1) s += __shfl_xor_sync(full, s, off);
  float ov[K];
  int oi[K];
#pragma unroll
  for (int r = 0; r < K; ++r) {
    float bv = a.v[0];
    int bi = a.i[0];
#pragma unroll
    for (int off = 16; off; off >>= 1) {
      const float pv = __shfl_xor_sync(full, bv, off);
      const int pi = __shfl_xor_sync(full, bi, off);
      if (key_before(pv, pi, bv, bi)) { bv = pv; bi = pi; }
    }
    ov[r] = bv;
    oi[r] = bi;
    if (a.v[0] == bv && a.i[0] == bi) a.pop_front();
  }
#pragma unroll
  for (int r = 0; r < K; ++r) { a.v[r] = ov[r]; a.i[r] = oi[r]; }
  a.s = s;
  a.m = (M == -CUDART_INF_F) ? 0.f : M;
}

template <int K>
struct Partial {  // one segment's result, as stored in the workspace
  float m, s;
  float v[K];
  int i[K];
};

template <int K>
__device__ __forceinline__ void finalize(const Acc<K>& a, int k, int64_t row, float* conf,
                                         int32_t* topk_idx, float* topk_prob, float* lse) {
  const float M = a.v[0], Z = a.s;
  const float inv = 1.f / Z;
#pragma unroll
  for (int j = 0; j < K; ++j) {
    if (j < k) {
      const float p = expf(a.v[j] - M) * inv;
      topk_idx[row * k + j] = a.i[j];
      topk_prob[row * k + j] = p;
      if (j == 0) conf[row] = p;
    }
  }
  if (lse) lse[row] = M + logf(Z);
}

template <typename T>
struct Unpack;
template <>
struct Unpack<float> {
  static constexpr int kElems = 4;
  template <int K>
  static __device__ __forceinline__ void push(Acc<K>& a, const uint4& w, int base) {
    a.push(__uint_as_float(w.x), base);
    a.push(__uint_as_float(w.y), base + 1);
    a.push(__uint_as_float(w.z), base + 2);
    a.push(__uint_as_float(w.w), base + 3);
  }
};
template <>
struct Unpack<__nv_bfloat16> {
  static constexpr int kElems = 8;
  template <int K>
  static __device__ __forceinline__ void push(Acc<K>& a, const uint4& w, int base) {
    a.push(__uint_as_float(w.x << 16), base);
    a.push(__uint_as_float(w.x & 0xffff0000u), base + 1);
    a.push(__uint_as_float(w.y << 16), base + 2);
    a.push(__uint_as_float(w.y & 0xffff0000u), base + 3);
    a.push(__uint_as_float(w.z << 16), base + 4);
    a.push(__uint_as_float(w.z & 0xffff0000u), base + 5);
    a.push(__uint_as_float(w.w << 16), base + 6);
    a.push(__uint_as_float(w.w & 0xffff0000u), base + 7);
  }
};

// grid.x = n_rows * n_seg; block = kTopkThreads.
template <typename T, int K>
__global__ void __launch_bounds__(kTopkThreads)
confidence_topk_kernel(const T* __restrict__ logits, int vocab, int64_t row_stride, int k, int n_seg,
                       int chunks_per_seg, float* __restrict__ conf, int32_t* __restrict__ topk_idx,
                       float* __restrict__ topk_prob, float* __restrict__ lse,
                       Partial<K>* __restrict__ partials, unsigned* __restrict__ tickets) {
  constexpr int E = Unpack<T>::kElems;
  const int64_t row = blockIdx.x / n_seg;
  const int seg = blockIdx.x % n_seg;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const T* rowp = logits + row * row_stride;
  const uint4* rowv = reinterpret_cast<const uint4*>(rowp);
  const int chunks_total = vocab / E;
  const int c0 = seg * chunks_per_seg;
  const int c1 = min(c0 + chunks_per_seg, chunks_total);

  Acc<K> a;
  a.init();
  for (int base = c0 + tid; base < c1; base += kTopkThreads * kTopkUnroll) {
    uint4 buf[kTopkUnroll];
#pragma unroll
    for (int u = 0; u < kTopkUnroll; ++u) {
      const int c = base + u * kTopkThreads;
      if (c < c1) buf[u] = ld_stream(rowv + c);
    }
#pragma unroll
    for (int u = 0; u < kTopkUnroll; ++u) {
      const int c = base + u * kTopkThreads;
      if (c < c1) Unpack<T>::push(a, buf[u], c * E);
    }
  }
  if (seg == n_seg - 1 && tid == 0) {  // ragged tail of a vocabulary that is not a multiple of E
    for (int x = chunks_total * E; x < vocab; ++x) a.push(to_float(rowp[x]), x);
  }

  warp_merge(a);
  __shared__ Partial<K> sm[kTopkWarps];
  if (lane == 0) {
    sm[warp].m = a.v[0];
    sm[warp].s = a.s;
#pragma unroll
    for (int j = 0; j < K; ++j) { sm[warp].v[j] = a.v[j]; sm[warp].i[j] = a.i[j]; }
  }
  __syncthreads();
  if (warp != 0) return;
  a.init();
  if (lane < kTopkWarps) {
    a.s = sm[lane].s;
#pragma unroll
    for (int j = 0; j < K; ++j) { a.v[j] = sm[lane].v[j]; a.i[j] = sm[lane].i[j]; }
  }
  warp_merge(a);
  if (n_seg == 1) {
    if (lane == 0) finalize(a, k, row, conf, topk_idx, topk_prob, lse);
    return;
  }
  // several segments per row: publish this one, the last to arrive merges all of them
  unsigned ticket = 0;
  if (lane == 0) {
    Partial<K>* p = partials + row * n_seg + seg;
    p->m = a.v[0];
    p->s = a.s;
#pragma unroll
    for (int j = 0; j < K; ++j) { p->v[j] = a.v[j]; p->i[j] = a.i[j]; }
    __threadfence();
    ticket = atomicInc(tickets + row, (unsigned)(n_seg - 1));  // wraps back to 0 after n_seg arrivals
    __threadfence();
  }
  ticket = __shfl_sync(0xffffffffu, ticket, 0);
  if (ticket != (unsigned)(n_seg - 1)) return;
  a.init();
  if (lane < n_seg) {
    const Partial<K>* p = partials + row * n_seg + lane;
    a.s = __ldcg(&p->s);
#pragma unroll
    for (int j = 0; j < K; ++j) { a.v[j] = __ldcg(&p->v[j]); a.i[j] = __ldcg(&p->i[j]); }
  }
  warp_merge(a);
  if (lane == 0) finalize(a, k, row, conf, topk_idx, topk_prob, lse);
}

struct TopkPlan {
  int n_seg, chunks_per_seg, K;
  size_t partial_bytes, ticket_off, total_bytes;
};

static int round_k(int k) { return k <= 4 ? k : (k <= 6 ? 6 : 8); }

static TopkPlan topk_plan(int64_t n_rows, int vocab, int k, int elems_per_chunk) {
  TopkPlan p;
  p.K = round_k(k);
  const int chunks = vocab / elems_per_chunk;
  const int64_t target_units = 148 * 16;
  int64_t n_seg = n_rows >= target_units ? 1 : (target_units + n_rows - 1) / n_rows;
  n_seg = std::min<int64_t>(n_seg, kMaxSegments);
  n_seg = std::min<int64_t>(n_seg, std::max(1, chunks / 1024));
  p.n_seg = (int)std::max<int64_t>(n_seg, 1);
  p.chunks_per_seg = (chunks + p.n_seg - 1) / p.n_seg;
  if (p.chunks_per_seg == 0) p.chunks_per_seg = 1;
  const size_t rec = 8 + 8 * (size_t)p.K;
  p.partial_bytes = p.n_seg > 1 ? (size_t)n_rows * p.n_seg * rec : 0;
  p.ticket_off = (p.partial_bytes + 15) / 16 * 16;
  p.total_bytes = p.n_seg > 1 ? p.ticket_off + ((size_t)n_rows * 4 + 15) / 16 * 16 : 0;
  return p;
}

template <typename T, int K>
static cudaError_t launch_topk(const void* logits, int64_t n_rows, int vocab, int64_t row_stride, int k,
                               const TopkPlan& p, float* conf, int32_t* idx, float* prob, float* lse,
                               void* ws, cudaStream_t st) {
  Partial<K>* partials = reinterpret_cast<Partial<K>*>(ws);
  unsigned* tickets = reinterpret_cast<unsigned*>(static_cast<char*>(ws) + p.ticket_off);
  if (p.n_seg > 1) {
    cudaError_t e = cudaMemsetAsync(tickets, 0, (size_t)n_rows * 4, st);
    if (e != cudaSuccess) return e;
  }
  confidence_topk_kernel<T, K><<<(unsigned)(n_rows * p.n_seg), kTopkThreads, 0, st>>>(
      static_cast<const T*>(logits), vocab, row_stride, k, p.n_seg, p.chunks_per_seg, conf, idx, prob,
      lse, partials, tickets);
  return cudaGetLastError();
}

template <typename T>
static cudaError_t dispatch_k(int K, const void* logits, int64_t n_rows, int vocab, int64_t row_stride,
                              int k, const TopkPlan& p, float* conf, int32_t* idx, float* prob,
                              float* lse, void* ws, cudaStream_t st) {
  switch (K) {
    case 1: return launch_topk<T, 1>(logits, n_rows, vocab, row_stride, k, p, conf, idx, prob, lse, ws, st);
    case 2: return launch_topk<T, 2>(logits, n_rows, vocab, row_stride, k, p, conf, idx, prob, lse, ws, st);
    case 3: return launch_topk<T, 3>(logits, n_rows, vocab, row_stride, k, p, conf, idx, prob, lse, ws, st);
    case 4: return launch_topk<T, 4>(logits, n_rows, vocab, row_stride, k, p, conf, idx, prob, lse, ws, st);
    case 6: return launch_topk<T, 6>(logits, n_rows, vocab, row_stride, k, p, conf, idx, prob, lse, ws, st);
    default: return launch_topk<T, 8>(logits, n_rows, vocab, row_stride, k, p, conf, idx, prob, lse, ws, st);
  }
}

}  // namespace tsd

extern "C" {

static int topk_check(int64_t n_rows, int32_t vocab, int32_t k) {
  if (n_rows < 0 || vocab < 1 || k < 1 || k > 8 || k > vocab) return TSD_ERR_INVALID_ARG;
  if (n_rows * (int64_t)tsd::kMaxSegments > 0x7fffffffLL) return TSD_ERR_INVALID_ARG;
  return TSD_OK;
}

size_t tsd_confidence_topk_workspace_bytes(int64_t n_rows, int32_t vocab, int32_t k) {
  if (topk_check(n_rows, vocab, k) != TSD_OK || n_rows == 0) return 0;
  // sized for the narrower element type (more chunks per row can only mean more segments)
  const size_t a = tsd::topk_plan(n_rows, vocab, k, 8).total_bytes;
  const size_t b = tsd::topk_plan(n_rows, vocab, k, 4).total_bytes;
  return a > b ? a : b;
}

int tsd_confidence_topk(const void* logits, int32_t dtype, int64_t n_rows, int32_t vocab,
                        int64_t row_stride, int32_t k, float* conf, int32_t* topk_idx,
                        float* topk_prob, float* lse, void* workspace, size_t workspace_bytes,
                        uint32_t* status, tsd_stream_t stream) {
  (void)status;
  int rc = topk_check(n_rows, vocab, k);
  if (rc != TSD_OK) return rc;
  if (dtype != TSD_F32 && dtype != TSD_BF16) return TSD_ERR_UNSUPPORTED;
  if (n_rows == 0) return TSD_OK;
  const int esize = dtype == TSD_F32 ? 4 : 2;
  if (!logits || !conf || !topk_idx || !topk_prob) return TSD_ERR_INVALID_ARG;
  if (row_stride < vocab || !tsd::aligned16(logits) || (row_stride * esize) % 16 != 0)
    return TSD_ERR_INVALID_ARG;
  const tsd::TopkPlan p = tsd::topk_plan(n_rows, vocab, k, 16 / esize);
  const size_t need = tsd_confidence_topk_workspace_bytes(n_rows, vocab, k);
  if (need > 0) {  // the documented size is required whichever dtype is passed
    if (!workspace || !tsd::aligned16(workspace)) return TSD_ERR_INVALID_ARG;
    if (workspace_bytes < need) return TSD_ERR_WORKSPACE;
  }
  cudaError_t e = dtype == TSD_F32
      ? tsd::dispatch_k<float>(p.K, logits, n_rows, vocab, row_stride, k, p, conf, topk_idx, topk_prob,
                               lse, workspace, stream)
      : tsd::dispatch_k<__nv_bfloat16>(p.K, logits, n_rows, vocab, row_stride, k, p, conf, topk_idx,
                                       topk_prob, lse, workspace, stream);
  if (e != cudaSuccess) return tsd::cuda_fail(e, "confidence_topk_kernel");
  return TSD_OK;
}

}  // extern "C"
