// Stage 2: confidence and top-k candidates in one streaming pass over the logits
// (paper Eq. 2: c = max softmax(logits); Section 3.2: top-k candidates per position).
//
// HBM-bound, so the streaming loop is branch-free.  A block handles one row (or one segment of a
// row when there are few rows) in three phases:
//   1. stream: 128-bit coalesced loads, four chunks per thread in flight.  Per batch the thread
//      takes the packed maximum of its 32 values, rebases its running sum to the new maximum with
//      one multiply, adds 2^(x*log2e - e) for every value (one FFMA + one ex2 each), and stores the
//      batch maximum in shared memory.
//   2. bound: the k-th largest of the warps' maxima (one shuffle reduction per warp, then every
//      warp ranks the 8 or 16 values, one per lane).  At least k values of the row are
//      >= it, so it is a valid lower bound of the k-th best.
//   3. collect: each warp re-reads only those of its batches whose maximum reaches the bound
//      (a handful per row, served by L2); the values >= bound go into a small pool in shared
//      memory, from which one warp picks the k best by counting ranks (no sort, no shuffles).
//      A pool that would overflow (heavy ties) falls back to merging per-lane lists by shuffles.
// With few rows a row is split into segments handled by different blocks; the last block to finish
// a row (a ticket word in the workspace, no spinning, no clearing between calls) merges the
// segment partials in segment order, so the result does not depend on arrival order.
//
// Ordering is (logit descending, index ascending) on the raw input values (bf16 and fp32 both
// widen to fp32 exactly), so indices are uniquely defined.
#include <limits.h>
#include <math_constants.h>
#include <algorithm>
#include "tsd_common.cuh"

namespace tsd {

constexpr int kTopkUnroll = 4;            // chunks per thread per batch
constexpr int kTopkSegChunks = 32768;     // chunks per segment at most (batch maxima: 32 KB of smem)
constexpr int kMaxSegments = 32;
constexpr int kPoolCap = 64;              // candidate pool of a block (entries)
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

__device__ __forceinline__ void prefetch_l2(const void* p) {
  asm volatile("prefetch.global.L2 [%0];" ::"l"(p));
}

// packed pairs of fp32 (one instruction for two lanes of arithmetic)
__device__ __forceinline__ uint64_t pack2(uint32_t lo, uint32_t hi) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "r"(lo), "r"(hi));
  return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float& lo, float& hi) {
  uint32_t a, b;
  asm("mov.b64 {%0, %1}, %2;" : "=r"(a), "=r"(b) : "l"(v));
  lo = __uint_as_float(a);
  hi = __uint_as_float(b);
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}

__device__ __forceinline__ uint32_t bmax2(uint32_t a, uint32_t b) {
  uint32_t r;
  asm("max.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
  return r;
}

// Sorted candidate list (key order) plus the row statistics that travel with it through merges:
// the sum is kept as s * 2^e with e = fl(M * log2e) for the maximum M, so that one FFMA feeds
// the exponential; the rounding of e is undone exactly in finalize().
template <int K>
struct Acc {
  float v[K];
  int i[K];
  float e;  // exponent base; meaningful only when `seen`
  float s;
  bool seen;  // a finite value contributed

  __device__ __forceinline__ void init() {
#pragma unroll
    for (int j = 0; j < K; ++j) { v[j] = -CUDART_INF_F; i[j] = INT_MAX; }
    e = 0.f;
    s = 0.f;
    seen = false;
  }
  // insert (x, xi) if it comes before the last entry
  __device__ __forceinline__ void offer(float x, int xi) {
    if (!key_before(x, xi, v[K - 1], i[K - 1])) return;
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
  float E = a.seen ? a.e : -CUDART_INF_F;
#pragma unroll
  for (int off = 16; off; off >>= 1) E = fmaxf(E, __shfl_xor_sync(full, E, off));
  float s = a.seen ? a.s * ex2_approx(a.e - E) : 0.f;
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
  a.seen = E != -CUDART_INF_F;
  a.e = a.seen ? E : 0.f;
}

template <int K>
struct Partial {  // one segment's result, as stored in the workspace
  float e, s;     // e = -inf when nothing finite was seen
  float v[K];
  int i[K];
};

// Every lane of the warp holds the merged result; lane j writes candidate j.
template <int K>
__device__ __forceinline__ void finalize(const Acc<K>& a, int k, int64_t row, int lane, float* conf,
                                         int32_t* topk_idx, float* topk_prob, float* lse) {
  // a.s = sum 2^(x*log2e - e) with e = fl(M*log2e): the FMA residual d = M*log2e - e is exact
  const float M = a.v[0];
  const float d = fmaf(M, kLog2e, -a.e);
  const float Z = a.s * exp2f(-d);  // sum exp(x - M)
  const float inv = 1.f / Z;
#pragma unroll
  for (int j = 0; j < K; ++j) {
    if (j == lane && j < k) {
      const float p = expf(a.v[j] - M) * inv;
      topk_idx[row * k + j] = a.i[j];
      topk_prob[row * k + j] = p;
      if (j == 0) conf[row] = p;
    }
  }
  if (lse && lane == 0) lse[row] = M + logf(Z);
}

template <typename T>
struct Unpack;
template <>
struct Unpack<float> {
  static constexpr int kElems = 4;
  static constexpr uint32_t kNegInfWord = 0xff800000u;
  static __device__ __forceinline__ float chunk_max(const uint4& w) {
    return fmaxf(fmaxf(__uint_as_float(w.x), __uint_as_float(w.y)),
                 fmaxf(__uint_as_float(w.z), __uint_as_float(w.w)));
  }
  static __device__ __forceinline__ float batch_max(const uint4 (&b)[kTopkUnroll]) {
    return fmaxf(fmaxf(chunk_max(b[0]), chunk_max(b[1])), fmaxf(chunk_max(b[2]), chunk_max(b[3])));
  }
  static __device__ __forceinline__ float elem(const uint4& w, int j) {
    return __uint_as_float(j == 0 ? w.x : (j == 1 ? w.y : (j == 2 ? w.z : w.w)));
  }
  static __device__ __forceinline__ float sum_exp(const uint4& w, float ne, float s) {
    s += ex2_approx(fmaf(__uint_as_float(w.x), kLog2e, ne));
    s += ex2_approx(fmaf(__uint_as_float(w.y), kLog2e, ne));
    s += ex2_approx(fmaf(__uint_as_float(w.z), kLog2e, ne));
    s += ex2_approx(fmaf(__uint_as_float(w.w), kLog2e, ne));
    return s;
  }
};
template <>
struct Unpack<__nv_bfloat16> {
  static constexpr int kElems = 8;
  static constexpr uint32_t kNegInfWord = 0xff80ff80u;
  static __device__ __forceinline__ float batch_max(const uint4 (&b)[kTopkUnroll]) {
    uint32_t m = bmax2(bmax2(bmax2(b[0].x, b[0].y), bmax2(b[0].z, b[0].w)),
                       bmax2(bmax2(b[1].x, b[1].y), bmax2(b[1].z, b[1].w)));
    m = bmax2(m, bmax2(bmax2(bmax2(b[2].x, b[2].y), bmax2(b[2].z, b[2].w)),
                       bmax2(bmax2(b[3].x, b[3].y), bmax2(b[3].z, b[3].w))));
    return fmaxf(__uint_as_float(m << 16), __uint_as_float(m & 0xffff0000u));
  }
  static __device__ __forceinline__ float elem(const uint4& w, int j) {
    const uint32_t word = j < 2 ? w.x : (j < 4 ? w.y : (j < 6 ? w.z : w.w));
    return __uint_as_float((j & 1) ? (word & 0xffff0000u) : (word << 16));
  }
  static __device__ __forceinline__ float sum_exp(const uint4& w, float ne, float s) {
    // a bf16 pair widens to an fp32 pair with one shift and one mask; the scale-and-shift and the
    // accumulation run as packed fp32 pairs, only the exponentials are per value
    const uint64_t l2 = pack2(__float_as_uint(kLog2e), __float_as_uint(kLog2e));
    const uint64_t ne2 = pack2(__float_as_uint(ne), __float_as_uint(ne));
    uint64_t acc = pack2(0u, 0u);
    const uint32_t words[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      float t0, t1;
      unpack2(fma2(pack2(words[q] << 16, words[q] & 0xffff0000u), l2, ne2), t0, t1);
      acc = add2(acc, pack2(__float_as_uint(ex2_approx(t0)), __float_as_uint(ex2_approx(t1))));
    }
    float a0, a1;
    unpack2(acc, a0, a1);
    return s + (a0 + a1);
  }
};

// grid.x = n_rows * n_seg; block = THREADS (256 when many blocks share an SM; 512 when there are so
// few rows that a block has to keep the SM busy on its own: twice the warps per row).
template <typename T, int K, int THREADS>
__global__ void __launch_bounds__(THREADS)
confidence_topk_kernel(const T* __restrict__ logits, int vocab, int64_t row_stride, int k, int n_seg,
                       int chunks_per_seg, float* __restrict__ conf, int32_t* __restrict__ topk_idx,
                       float* __restrict__ topk_prob, float* __restrict__ lse,
                       Partial<K>* __restrict__ partials, unsigned* __restrict__ tickets, int prefetch) {
  constexpr int E_ = Unpack<T>::kElems;
  constexpr int kTopkThreads = THREADS, kTopkWarps = THREADS / 32;
  constexpr int kTopkBatch = THREADS * kTopkUnroll;        // chunks per block per batch
  constexpr int kTopkMaxIter = kTopkSegChunks / kTopkBatch;  // batches per segment
  __shared__ float s_bmax[kTopkMaxIter][kTopkThreads];  // per-thread batch maxima
  __shared__ __align__(16) float s_wmax[kTopkWarps];  // per-warp maxima
  __shared__ float s_wsum[kTopkWarps];                // per-warp sums on the block's exponent base
  __shared__ float s_pool_v[kPoolCap];                // candidates found by the collect phase
  __shared__ int s_pool_i[kPoolCap];
  __shared__ int s_cnt;
  __shared__ float s_res_v[K];
  __shared__ int s_res_i[K];
  __shared__ Partial<K> s_part[kTopkWarps];           // shuffle-merge path only
  const int64_t row = blockIdx.x / n_seg;
  const int seg = blockIdx.x % n_seg;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const T* rowp = logits + row * row_stride;
  const uint4* rowv = reinterpret_cast<const uint4*>(rowp);
  const int chunks_total = vocab / E_;
  const int c0 = seg * chunks_per_seg;
  const int c1 = min(c0 + chunks_per_seg, chunks_total);
  const int n_iter = (c1 - c0 + kTopkBatch - 1) / kTopkBatch;  // <= kTopkMaxIter (host-enforced)
  const bool has_tail = seg == n_seg - 1 && tid == 0 && chunks_total * E_ < vocab;

  // ---- phase 1: stream.  Two register buffers: the loads of batch it+1 are in flight while
  // batch it is processed, so a block overlaps memory latency with its own arithmetic.
  float m = -CUDART_INF_F, e = 0.f, s = 0.f;
  auto load_batch = [&](uint4 (&buf)[kTopkUnroll], int it) {
    const int base = c0 + it * kTopkBatch + tid;
#pragma unroll
    for (int u = 0; u < kTopkUnroll; ++u) {
      const int c = base + u * kTopkThreads;
      if (c < c1) buf[u] = ld_stream(rowv + c);
      else  // past the segment: -inf adds nothing and is never a candidate
        buf[u] = make_uint4(Unpack<T>::kNegInfWord, Unpack<T>::kNegInfWord, Unpack<T>::kNegInfWord,
                            Unpack<T>::kNegInfWord);
    }
  };
  auto process_batch = [&](const uint4 (&buf)[kTopkUnroll], int it) {
    const float bm = Unpack<T>::batch_max(buf);
    s_bmax[it][tid] = bm;
    const float m_new = fmaxf(m, bm);
    const float e_new = (m_new == -CUDART_INF_F) ? 0.f : m_new * kLog2e;
    s *= (m == -CUDART_INF_F) ? 0.f : ex2_approx(e - e_new);  // rebase: 1 when the maximum stays
    m = m_new;
    e = e_new;
    float part[kTopkUnroll];  // independent partial sums keep the dependent add chains short
    if ((it + 1) * kTopkBatch <= c1 - c0) {
#pragma unroll
      for (int u = 0; u < kTopkUnroll; ++u) part[u] = Unpack<T>::sum_exp(buf[u], -e, 0.f);
    } else {  // the segment's last, partly filled batch: no exponentials for the padding
      const int base = c0 + it * kTopkBatch + tid;
#pragma unroll
      for (int u = 0; u < kTopkUnroll; ++u)
        part[u] = base + u * kTopkThreads < c1 ? Unpack<T>::sum_exp(buf[u], -e, 0.f) : 0.f;
    }
    s += (part[0] + part[1]) + (part[2] + part[3]);
  };
  // Optional L2 prefetch `prefetch` batches ahead of the register loads, one 128-byte line per
  // thread (the launcher turns it on for large grids only).
  auto prefetch_batch = [&](int it) {
    constexpr int kLines = kTopkBatch * 16 / 128;  // lines per batch (<= THREADS)
    const int c = c0 + it * kTopkBatch + tid * 8;  // first chunk of this thread's line
    if (tid < kLines && it < n_iter && c < c1) prefetch_l2(rowv + c);
  };
  {
    uint4 buf_a[kTopkUnroll], buf_b[kTopkUnroll];
    if (n_iter > 0) load_batch(buf_a, 0);
    for (int p = 1; p <= prefetch; ++p) prefetch_batch(p);
    for (int it = 0; it < n_iter; it += 2) {
      if (it + 1 < n_iter) load_batch(buf_b, it + 1);
      if (prefetch) { prefetch_batch(it + prefetch + 1); prefetch_batch(it + prefetch + 2); }
      process_batch(buf_a, it);
      if (it + 1 < n_iter) {
        if (it + 2 < n_iter) load_batch(buf_a, it + 2);
        process_batch(buf_b, it + 1);
      }
    }
  }
  float tail_max = -CUDART_INF_F;
  if (has_tail) {  // ragged tail of a vocabulary that is not a multiple of the chunk size
    for (int x = chunks_total * E_; x < vocab; ++x) tail_max = fmaxf(tail_max, to_float(rowp[x]));
    const float m_new = fmaxf(m, tail_max);
    const float e_new = (m_new == -CUDART_INF_F) ? 0.f : m_new * kLog2e;
    s *= (m == -CUDART_INF_F) ? 0.f : ex2_approx(e - e_new);
    m = m_new;
    e = e_new;
    for (int x = chunks_total * E_; x < vocab; ++x) s += ex2_approx(fmaf(to_float(rowp[x]), kLog2e, -e));
  }

  // ---- phase 2: bound = k-th largest of the warps' maxima.  Each of the k best warps holds a
  // value equal to its maximum, so at least k values of the segment reach the bound.  One shuffle
  // reduction per warp, one block-wide barrier, then a rank count per warp.
  if (tid == 0) s_cnt = 0;
  {
    float wm = m;
#pragma unroll
    for (int off = 16; off; off >>= 1) wm = fmaxf(wm, __shfl_xor_sync(0xffffffffu, wm, off));
    if (lane == 0) s_wmax[warp] = wm;
  }
  __syncthreads();
  // lane l < WARPS takes warp maximum l and counts the maxima that come before it (larger, or
  // equal from a lower warp): ranks are unique, rank 0 is the block maximum, rank K-1 the bound
  float M, bound;
  {
    const float mine = lane < kTopkWarps ? s_wmax[lane] : -CUDART_INF_F;
    int rank = 0;
#pragma unroll
    for (int q = 0; q < kTopkWarps; ++q) {
      const float o = s_wmax[q];
      rank += (o > mine || (o == mine && q < lane)) ? 1 : 0;
    }
    const bool in = lane < kTopkWarps;
    const unsigned b0 = __ballot_sync(0xffffffffu, in && rank == 0);
    const unsigned bk = __ballot_sync(0xffffffffu, in && rank == K - 1);
    M = __shfl_sync(0xffffffffu, mine, __ffs(b0) - 1);
    bound = __shfl_sync(0xffffffffu, mine, __ffs(bk) - 1);
  }
  // the block's sum on the block's exponent base; the per-warp sums meet after the next barrier
  const float E = (M == -CUDART_INF_F) ? 0.f : M * kLog2e;
  {
    float sr = (m == -CUDART_INF_F) ? 0.f : s * ex2_approx(e - E);
#pragma unroll
    for (int off = 16; off; off >>= 1) sr += __shfl_xor_sync(0xffffffffu, sr, off);
    if (lane == 0) s_wsum[warp] = sr;
  }

  // ---- phase 3: collect the values >= bound from the few batches that hold one
  Acc<K> a;
  a.init();
  // The whole block waits for its slowest warp here, so a hit batch (32 values for bf16, 16 for
  // fp32) is examined by the warp together: lane l re-reads value l of the batch (an L2 hit) and
  // offers it to its own list.
  for (int it = 0; it < n_iter; ++it) {
    unsigned hits = __ballot_sync(0xffffffffu, s_bmax[it][tid] >= bound);
    while (hits) {
      const int src = __ffs(hits) - 1;
      hits &= hits - 1;
      if (lane < kTopkUnroll * E_) {
        const int c = c0 + it * kTopkBatch + (warp * 32 + src) + (lane / E_) * kTopkThreads;
        if (c < c1) {
          const int xi = c * E_ + lane % E_;
          const float x = to_float(rowp[xi]);
          if (x >= bound) a.offer(x, xi);
        }
      }
    }
  }
  if (has_tail && tail_max >= bound) {
    for (int x = chunks_total * E_; x < vocab; ++x) {
      const float v = to_float(rowp[x]);
      if (v >= bound) a.offer(v, x);
    }
  }
  // The lanes that found something (a handful per block) put their entries into a small pool in
  // shared memory.  If the pool would overflow (heavy ties: many values equal to the bound), the
  // lists are merged by shuffles instead, which is slower but has no capacity.
  {
    int n_mine = 0;
#pragma unroll
    for (int j = 0; j < K; ++j) n_mine += a.i[j] != INT_MAX;
    if (n_mine > 0) {
      const int at = atomicAdd(&s_cnt, n_mine);
      if (at + n_mine <= kPoolCap) {
#pragma unroll
        for (int j = 0; j < K; ++j)
          if (j < n_mine) { s_pool_v[at + j] = a.v[j]; s_pool_i[at + j] = a.i[j]; }
      }
    }
  }
  __syncthreads();
  const int n_pool = s_cnt;
  if (n_pool > kPoolCap) {
    a.seen = m != -CUDART_INF_F;
    a.e = e;
    a.s = s;
    warp_merge(a);
    if (lane == 0) {
      s_part[warp].e = a.seen ? a.e : -CUDART_INF_F;
      s_part[warp].s = a.s;
#pragma unroll
      for (int j = 0; j < K; ++j) { s_part[warp].v[j] = a.v[j]; s_part[warp].i[j] = a.i[j]; }
    }
    __syncthreads();
    if (warp != 0) return;
    a.init();
    if (lane < kTopkWarps) {
      a.seen = s_part[lane].e != -CUDART_INF_F;
      a.e = a.seen ? s_part[lane].e : 0.f;
      a.s = s_part[lane].s;
#pragma unroll
      for (int j = 0; j < K; ++j) { a.v[j] = s_part[lane].v[j]; a.i[j] = s_part[lane].i[j]; }
    }
    warp_merge(a);
  } else {
    if (warp != 0) return;
    // sum of the warps' sums (fixed tree), and the pool's best K by rank: every lane counts the
    // entries that come before its own (keys are unique), so rank r goes to slot r without a sort
    float st = lane < kTopkWarps ? s_wsum[lane] : 0.f;
#pragma unroll
    for (int off = 16; off; off >>= 1) st += __shfl_xor_sync(0xffffffffu, st, off);
    if (lane < K) { s_res_v[lane] = -CUDART_INF_F; s_res_i[lane] = INT_MAX; }
    __syncwarp();
#pragma unroll
    for (int h = 0; h < kPoolCap / 32; ++h) {
      const int q = lane + 32 * h;
      if (q < n_pool) {
        const float v = s_pool_v[q];
        const int i = s_pool_i[q];
        int rank = 0;
        for (int o = 0; o < n_pool; ++o) rank += key_before(s_pool_v[o], s_pool_i[o], v, i);
        if (rank < K) { s_res_v[rank] = v; s_res_i[rank] = i; }
      }
    }
    __syncwarp();
#pragma unroll
    for (int j = 0; j < K; ++j) { a.v[j] = s_res_v[j]; a.i[j] = s_res_i[j]; }
    a.seen = M != -CUDART_INF_F;
    a.e = E;
    a.s = st;
  }
  if (n_seg == 1) {
    finalize(a, k, row, lane, conf, topk_idx, topk_prob, lse);
    return;
  }
  // several segments per row: publish this one, the last to arrive merges all of them
  bool last = false;
  if (lane == 0) {
    Partial<K>* p = partials + row * n_seg + seg;
    p->e = a.seen ? a.e : -CUDART_INF_F;
    p->s = a.s;
#pragma unroll
    for (int j = 0; j < K; ++j) { p->v[j] = a.v[j]; p->i[j] = a.i[j]; }
    __threadfence();
    last = ticket_arrive(tickets + row, n_seg);
    __threadfence();
  }
  if (!__shfl_sync(0xffffffffu, last, 0)) return;
  a.init();
  if (lane < n_seg) {
    const Partial<K>* p = partials + row * n_seg + lane;
    const float pe = __ldcg(&p->e);
    a.seen = pe != -CUDART_INF_F;
    a.e = a.seen ? pe : 0.f;
    a.s = __ldcg(&p->s);
#pragma unroll
    for (int j = 0; j < K; ++j) { a.v[j] = __ldcg(&p->v[j]); a.i[j] = __ldcg(&p->i[j]); }
  }
  warp_merge(a);
  finalize(a, k, row, lane, conf, topk_idx, topk_prob, lse);
}

struct TopkPlan {
  int n_seg, chunks_per_seg, K, threads, prefetch;
  size_t partial_bytes, ticket_off, total_bytes;
};

static int round_k(int k) { return k <= 4 ? k : (k <= 6 ? 6 : 8); }

static TopkPlan topk_plan(int64_t n_rows, int vocab, int k, int elems_per_chunk) {
  TopkPlan p;
  p.K = round_k(k);
  const int chunks = vocab / elems_per_chunk;
  // Few rows: split rows only until every SM has a block (more segments add per-block latency
  // and merge work faster than they add parallelism; measured on cfg2- and cfg3-sized inputs).
  const int64_t target_units = 148;
  int64_t n_seg = n_rows >= target_units ? 1 : (target_units + n_rows - 1) / n_rows;
  n_seg = std::min<int64_t>(n_seg, kMaxSegments);
  n_seg = std::min<int64_t>(n_seg, std::max(1, chunks / 2048));
  // a segment may span at most kTopkSegChunks chunks (its batch maxima live in shared memory)
  n_seg = std::max<int64_t>(n_seg, (chunks + kTopkSegChunks - 1) / kTopkSegChunks);
  p.n_seg = (int)std::max<int64_t>(n_seg, 1);
  // up to two 512-thread blocks fit an SM: use them while that still gives every block a slot at once
  p.threads = (n_rows * p.n_seg <= 2 * 148) ? 512 : 256;
  // L2 prefetch distance in batches (measured): with several waves of blocks, requesting lines
  // three batches ahead adds 3 % of bandwidth; with few blocks it only delays the demand loads
  p.prefetch = (n_rows * p.n_seg >= 2048) ? 3 : 0;
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
  if (p.threads == 512)
    confidence_topk_kernel<T, K, 512><<<(unsigned)(n_rows * p.n_seg), 512, 0, st>>>(
        static_cast<const T*>(logits), vocab, row_stride, k, p.n_seg, p.chunks_per_seg, conf, idx, prob,
        lse, partials, tickets, p.prefetch);
  else
    confidence_topk_kernel<T, K, 256><<<(unsigned)(n_rows * p.n_seg), 256, 0, st>>>(
        static_cast<const T*>(logits), vocab, row_stride, k, p.n_seg, p.chunks_per_seg, conf, idx, prob,
        lse, partials, tickets, p.prefetch);
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
  // rows longer than kMaxSegments segments of kTopkMaxIter batches (4 Mi fp32 / 8 Mi bf16 logits)
  if ((int64_t)vocab / 4 > (int64_t)tsd::kTopkSegChunks * tsd::kMaxSegments)
    return TSD_ERR_INVALID_ARG;
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

// ---------------------------------------------------------------------------------------------
// Allocation-free variant.  Some hosts can hand this library nothing but their inputs and outputs:
// an inference-server plug-in whose device memory pool is sized once at start-up and then frozen,
// or a decode loop in which calling cudaMalloc is ruled out because it would stall the whole
// device in the middle of a step.  For them the per-segment partial results and the per-row
// tickets live in a fixed array that is part of the library image: every GPU that loads the
// library carries these bytes until the process exits, which is why the size is kept modest.
namespace tsd {

constexpr size_t kStaticScratchBytes = 1u << 20;  // 1 MiB per device
static __device__ __align__(256) unsigned char g_topk_scratch[kStaticScratchBytes];

// In host code `g_topk_scratch` is only a handle for the runtime, not an address a kernel can use:
// the device address has to be asked for, with the device current.  The lookup is a host-side
// query that allocates nothing; it is repeated on every call rather than remembered, so that the
// address is never one from before a device reset (the first lookup on a device loads the
// library's module there, which is why that first call belongs before any stream capture).
static cudaError_t static_scratch_address(void** out) {
  void* ptr = nullptr;
  cudaError_t e = cudaGetSymbolAddress(&ptr, g_topk_scratch);
  if (e != cudaSuccess) return e;
  *out = ptr;
  return cudaSuccess;
}

}  // namespace tsd

extern "C" size_t tsd_confidence_topk_static_capacity(void) { return tsd::kStaticScratchBytes; }

extern "C" int tsd_confidence_topk_static(const void* logits, int32_t dtype, int64_t n_rows, int32_t vocab,
                                          int64_t row_stride, int32_t k, float* conf, int32_t* topk_idx,
                                          float* topk_prob, float* lse, uint32_t* status,
                                          tsd_stream_t stream) {
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
  // this shape would need more scratch than the library carries: the caller has to use
  // tsd_confidence_topk with a workspace of its own.  The test is on the documented size
  // (tsd_confidence_topk_workspace_bytes, the larger of the two dtypes' needs), so that the check a
  // caller makes beforehand and this one agree.
  if (tsd_confidence_topk_workspace_bytes(n_rows, vocab, k) > tsd::kStaticScratchBytes) return TSD_ERR_WORKSPACE;
  void* scratch = nullptr;
  if (p.total_bytes > 0) {
    cudaError_t e = tsd::static_scratch_address(&scratch);
    if (e != cudaSuccess) return tsd::cuda_fail(e, "cudaGetSymbolAddress(g_topk_scratch)");
  }
  // ticket words need no clearing (a word that does not carry the in-use tag counts as idle, and
  // the last arrival of a row returns it to idle); the partial-result slots are fully rewritten by
  // every call that reads them
  cudaError_t e = dtype == TSD_F32
      ? tsd::dispatch_k<float>(p.K, logits, n_rows, vocab, row_stride, k, p, conf, topk_idx, topk_prob,
                               lse, scratch, stream)
      : tsd::dispatch_k<__nv_bfloat16>(p.K, logits, n_rows, vocab, row_stride, k, p, conf, topk_idx,
                                       topk_prob, lse, scratch, stream);
  if (e != cudaSuccess) return tsd::cuda_fail(e, "confidence_topk_kernel (static scratch)");
  return TSD_OK;
}
