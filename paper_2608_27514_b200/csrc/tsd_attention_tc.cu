// Stage 1b on tensor cores: masked verify attention (paper Section 3.3) for bf16, head_dim 128.
//
// One thread block per (sequence, query head, tile of 128 draft rows = 128/R branches).  The key
// tiles of a block are the cached prefix/suffix tiles, shared by every branch (a dense GEMM), then
// the draft tiles listed for this query tile in the mask blob; inside a draft tile only the
// (query branch, key branch) pairs whose bit is set are visible, everything else gets weight 0.
// Tiles of branches a query tile cannot see are never loaded.
//
// Warp roles: warps 0-3 = softmax (one query row per thread, TMEM lane = row), warp 4 = TMA
// producer, warp 5 = tcgen05 MMA issuer (also owns the TMEM allocation).
//   S = Q K^T : tcgen05.mma, A and B K-major from 128B-swizzled shared memory, fp32 in TMEM
//   softmax  : tcgen05.ld S -> registers, running max / sum in the exp2 domain, P -> bf16 -> TMEM
//              (tcgen05.st over the first 32 columns of that S buffer: two bf16 per 32-bit column)
//   O += P V : tcgen05.mma, A = P from TMEM, B = V (MN-major: head_dim contiguous), fp32 in TMEM
// Key tiles are 64 keys wide.  S is double-buffered in TMEM (2 x 64 columns) so that Q K^T of tile
// j+1 runs while the softmax of tile j is on the CUDA cores, and two blocks share an SM (each 256 of
// the 512 TMEM columns and ~97 KB of shared memory) so that one block's P V fills the gaps of the
// other.  MMAs issued by one thread execute in order, so an S/P buffer may be overwritten by a later
// Q K^T as soon as the P V that reads it has been issued.
// The running maximum used as exponent offset only moves when the row maximum grows by more than
// 2^8, so rescaling O in TMEM is rare; the final division by the row sum makes the result exact.
// Every mbarrier wait is bounded: on expiry the block raises TSD_STATUS_TIMEOUT, stops issuing
// work, frees its TMEM and returns.
#include <cuda.h>
#include <math_constants.h>
#include <mutex>
#include "tsd_common.cuh"

namespace tsd {

constexpr int kTcThreads = 192;
constexpr uint32_t kSub = 16384;          // bytes of one [128 rows x 64 elements] bf16 sub-tile
constexpr uint32_t kTileBytes = 2 * kSub;  // a [128 x 128] bf16 tile
constexpr int kKeys = 64;                       // keys per tile
constexpr uint32_t kSubKV = 8192;              // bytes of one [64 keys x 64 elements] bf16 sub-tile
constexpr uint32_t kKVBytes = 2 * kSubKV;      // a [64 x 128] bf16 K or V tile
constexpr uint32_t kOffQ = 0, kOffK = kTileBytes, kOffV = kTileBytes + 2 * kKVBytes;  // 2 stages each
constexpr uint32_t kOffBar = kTileBytes + 4 * kKVBytes;
constexpr uint32_t kColS = 0, kColO = 128;     // S buffers at columns 0 and 64; P aliases 32 columns of each
constexpr uint32_t kSmemBytes = kOffBar + 256 + 1024;  // + barriers + slack to align the base to 1 KB
constexpr uint32_t kSpinLimit = 1u << 21;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

// S_FULL[b] (Q K^T of a tile complete) also frees that tile's K stage; PV_DONE[b] (P V complete)
// also frees its V stage: a tcgen05.commit costs ~100 clocks of the issuing thread, so each event
// gets exactly one.
enum Bar { Q_FULL = 0, K_FULL = 1, V_FULL = 3, S_FULL = 5, P_FULL = 7, PV_DONE = 9, N_BARS = 11 };

// ------------------------------------------------------------------ PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile("{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}"
               : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
__device__ __forceinline__ bool mbar_test_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile("{\n.reg .pred p;\nmbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}"
               : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait.  Returns false when the block is aborting (this wait or another one ran out).
// The non-blocking test comes first: a phase that has already completed costs one shared-memory
// round trip instead of a suspend / wake-up.
// `sleep_ns` > 0 backs off between polls: used by the roles that run far ahead (the TMA producer),
// whose spinning would otherwise take issue slots from the softmax warps on the same scheduler.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag,
                                          uint32_t sleep_ns = 0) {
  if (mbar_test_wait(bar, parity)) return true;
  for (uint32_t it = 0; it < kSpinLimit; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if (sleep_ns) __nanosleep(sleep_ns);
    if ((it & 255u) == 255u && *abort_flag) return false;
  }
  *abort_flag = 1u;
  return false;
}

__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1,
                                            int c2, int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}

__device__ __forceinline__ void tma_store_4d(const CUtensorMap* map, uint32_t src, int c0, int c1, int c2, int c3) {
  asm volatile("cp.async.bulk.tensor.4d.global.shared::cta.bulk_group [%0, {%2, %3, %4, %5}], [%1];"
               ::"l"(map), "r"(src), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}

// True in exactly one lane of a converged warp; the compiler recognises the pattern and keeps the
// warp's address arithmetic on the uniform datapath, which the tcgen05 instructions read.
__device__ __forceinline__ bool elect_one() {
  uint32_t pred = 0;
  asm volatile("{\n.reg .pred p;\nelect.sync _|p, 0xffffffff;\n@p mov.u32 %0, 1;\n}" : "+r"(pred));
  return pred != 0;
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// ACC is a compile-time constant so that the accumulate predicate costs nothing at issue time; the
// issue rate of the elected thread is what keeps the tensor pipe fed (64 clocks per 128x128x16 MMA).
template <bool ACC>
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc) {
  if (ACC)
    asm volatile("{\n.reg .pred p;\nsetp.eq.b32 p, 0, 0;\n"
                 "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
                 ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc) : "memory");
  else
    asm volatile("{\n.reg .pred p;\nsetp.ne.b32 p, 0, 0;\n"
                 "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
                 ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc) : "memory");
}

template <bool ACC>
__device__ __forceinline__ void tc_mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc) {
  if (ACC)
    asm volatile("{\n.reg .pred p;\nsetp.eq.b32 p, 0, 0;\n"
                 "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n}"
                 ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc) : "memory");
  else
    asm volatile("{\n.reg .pred p;\nsetp.ne.b32 p, 0, 0;\n"
                 "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n}"
                 ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc) : "memory");
}

#define TSD_R32(a, o) "=r"(a[o+0]), "=r"(a[o+1]), "=r"(a[o+2]), "=r"(a[o+3]), "=r"(a[o+4]), "=r"(a[o+5]), "=r"(a[o+6]), "=r"(a[o+7]), \
  "=r"(a[o+8]), "=r"(a[o+9]), "=r"(a[o+10]), "=r"(a[o+11]), "=r"(a[o+12]), "=r"(a[o+13]), "=r"(a[o+14]), "=r"(a[o+15]), \
  "=r"(a[o+16]), "=r"(a[o+17]), "=r"(a[o+18]), "=r"(a[o+19]), "=r"(a[o+20]), "=r"(a[o+21]), "=r"(a[o+22]), "=r"(a[o+23]), \
  "=r"(a[o+24]), "=r"(a[o+25]), "=r"(a[o+26]), "=r"(a[o+27]), "=r"(a[o+28]), "=r"(a[o+29]), "=r"(a[o+30]), "=r"(a[o+31])
#define TSD_W32(a, o) "r"(a[o+0]), "r"(a[o+1]), "r"(a[o+2]), "r"(a[o+3]), "r"(a[o+4]), "r"(a[o+5]), "r"(a[o+6]), "r"(a[o+7]), \
  "r"(a[o+8]), "r"(a[o+9]), "r"(a[o+10]), "r"(a[o+11]), "r"(a[o+12]), "r"(a[o+13]), "r"(a[o+14]), "r"(a[o+15]), \
  "r"(a[o+16]), "r"(a[o+17]), "r"(a[o+18]), "r"(a[o+19]), "r"(a[o+20]), "r"(a[o+21]), "r"(a[o+22]), "r"(a[o+23]), \
  "r"(a[o+24]), "r"(a[o+25]), "r"(a[o+26]), "r"(a[o+27]), "r"(a[o+28]), "r"(a[o+29]), "r"(a[o+30]), "r"(a[o+31])

// 32 consecutive fp32 columns of this thread's TMEM lane -> registers a[o .. o+31]
#define TSD_TMEM_LD32(a, o, taddr)                                                                         \
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "                                                   \
               "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"                                   \
               "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"                  \
               : TSD_R32(a, o) : "r"(taddr) : "memory")
#define TSD_TMEM_ST32(a, o, taddr)                                                                         \
  asm volatile("tcgen05.st.sync.aligned.32x32b.x32.b32 [%32], "                                            \
               "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"                                   \
               "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31};"                         \
               ::TSD_W32(a, o), "r"(taddr) : "memory")
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ float ex2f(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}

// Packed fp32 pairs (two lanes per instruction on this architecture) and the 3-input maximum.
__device__ __forceinline__ uint64_t pack2(uint32_t lo, uint32_t hi) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "r"(lo), "r"(hi));
  return r;
}
__device__ __forceinline__ uint64_t pack2f(float lo, float hi) { return pack2(__float_as_uint(lo), __float_as_uint(hi)); }
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
__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
// 2^t for a pair, t in [-126, 16], on the FMA pipe: t = n + f with n = round(t), f in [-0.5, 0.5];
// 2^f by a degree-3 polynomial (relative error 7.5e-5, well below the bf16 rounding of P), and n
// added into the exponent field.  Takes load off the 16-per-clock special-function unit.
__device__ __forceinline__ void exp2_poly2(uint64_t t2, float& p0, float& p1) {
  float t0, t1;
  unpack2(t2, t0, t1);
  t2 = pack2f(fmaxf(t0, -126.f), fmaxf(t1, -126.f));
  const uint64_t magic = pack2f(12582912.f, 12582912.f);          // 1.5 * 2^23: rounds to an integer
  const uint64_t y = add2(t2, magic);
  const uint64_t n = add2(y, pack2f(-12582912.f, -12582912.f));
  const uint64_t f = fma2(n, pack2f(-1.f, -1.f), t2);
  uint64_t r = fma2(f, pack2f(0.05517165f, 0.05517165f), pack2f(0.24261113f, 0.24261113f));
  r = fma2(r, f, pack2f(0.69326097f, 0.69326097f));
  r = fma2(r, f, pack2f(0.99992806f, 0.99992806f));
  float y0, y1, r0, r1;
  unpack2(y, y0, y1);
  unpack2(r, r0, r1);
  p0 = __uint_as_float(__float_as_uint(r0) + (__float_as_uint(y0) << 23));
  p1 = __uint_as_float(__float_as_uint(r1) + (__float_as_uint(y1) << 23));
}
constexpr int kPolyOf8 = 2;  // of every 8 score pairs, this many take the polynomial exp2 (unmasked tiles)

// Shared-memory matrix descriptor, 128-byte swizzle (descriptor version 1 = this architecture).
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  return (uint64_t)((addr >> 4) & 0x3FFFu) | ((uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16) |
         ((uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32) | (1ull << 46) | (2ull << 61);
}
// Instruction descriptor: fp32 accumulate, bf16 x bf16, M = 128, N = n; b_mn = 1 when B is MN-major.
__host__ __device__ constexpr uint32_t instr_desc(uint32_t n, uint32_t b_mn) {
  return (1u << 4) | (1u << 7) | (1u << 10) | (b_mn << 16) | ((n >> 3) << 17) | ((128u >> 4) << 24);
}

struct TcParams {
  const int32_t* mask;
  __nv_bfloat16* out;
  float* lse;
  uint32_t* status;
  int64_t os_b, os_r, os_h;
  int S, B, R, Nc, N, Hq, group;
  int recs_off, n_qt, rec_words;  // layout of the mask blob, computed on the host from the same tsd_layout
  float scale_log2e;  // sm_scale * log2(e), > 0
};

__global__ void __launch_bounds__(kTcThreads, 2)
attention_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_kc,
                    const __grid_constant__ CUtensorMap map_vc, const __grid_constant__ CUtensorMap map_kd,
                    const __grid_constant__ CUtensorMap map_vd, const __grid_constant__ CUtensorMap map_o,
                    const TcParams p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* base_ptr = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t bars = base + kOffBar;
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(base_ptr + kOffBar + 128);
  volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(base_ptr + kOffBar + 132);
  auto bar = [&](int i) { return bars + 8u * (uint32_t)i; };

  const int qt = blockIdx.x, h = blockIdx.y, s = blockIdx.z;
  const int g = h / p.group;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  // Everything the block needs from the mask blob is requested at once (the blob's layout follows
  // from the tsd_layout, so no address depends on a loaded value); the producer thread meanwhile
  // sets up the barriers and starts the Q load, so the two latencies overlap.
  const int32_t* mask = p.mask;
  const int32_t* rec = mask + p.recs_off + (size_t)(s * p.n_qt + qt) * p.rec_words;
  const int h_magic = mask[H_MAGIC], h_s = mask[H_S], h_b = mask[H_B], h_r = mask[H_R], h_nc = mask[H_NC];
  const int clen = mask[kHdrWords + s];
  const int n_dt_raw = rec[0];  // visible 128-row draft tiles = 2 key tiles each

  if (warp == 4 && lane == 0) {
    abort_flag[0] = 0;
    abort_flag[1] = 0;  // scratch flag for the producer's drain waits
    mbar_init(bar(Q_FULL), 1);
    for (int i = 0; i < 2; ++i) {
      mbar_init(bar(K_FULL + i), 1);
      mbar_init(bar(V_FULL + i), 1);
      mbar_init(bar(S_FULL + i), 1);
      mbar_init(bar(P_FULL + i), 4);
      mbar_init(bar(PV_DONE + i), 1);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_async_smem();
    mbar_expect_tx(bar(Q_FULL), kTileBytes);
    tma_load_4d(base + kOffQ, &map_q, bar(Q_FULL), 0, h, qt * kTile, s);
    tma_load_4d(base + kOffQ + kSub, &map_q, bar(Q_FULL), 64, h, qt * kTile, s);
  }
  if (warp == 5) {  // TMEM: 2 x S/P (64 columns each) + O (128 columns); two blocks share the SM's 512
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 256;" ::"r"(bars + 128u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  // A blob that was built for another layout: report it and run the block with no key tiles and
  // no output (the Q load in flight is still waited for before the block leaves).
  const bool hdr_ok = h_magic == kMaskMagic && h_s == p.S && h_b == p.B && h_r == p.R && h_nc == p.Nc;
  if (!hdr_ok && tid == 0 && p.status) atomicOr(p.status, TSD_STATUS_BAD_MASK);
  const int n_ct = hdr_ok ? (clen + kKeys - 1) / kKeys : 0;  // cached tiles of 64 keys
  const int n_dt = hdr_ok ? n_dt_raw : 0;
  const int T = n_ct + 2 * n_dt;

  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  if (warp == 4) {
    // ------------------------------------------------------------ TMA producer (one lane)
    if (lane == 0) {
      auto load_tile = [&](uint32_t dst, uint32_t full_bar, const CUtensorMap* mc, const CUtensorMap* md, int j) {
        mbar_expect_tx(full_bar, kKVBytes);
        const bool cached = j < n_ct;
        const CUtensorMap* m = cached ? mc : md;
        const int e = j - n_ct;  // draft key tile e = half (e & 1) of the listed 128-row tile e >> 1
        const int row = cached ? j * kKeys : rec[2 + 2 * (e >> 1)] * kTile + (e & 1) * kKeys;
        tma_load_4d(dst, m, full_bar, 0, g, row, s);
        tma_load_4d(dst + kSubKV, m, full_bar, 64, g, row, s);
      };
      bool ok = true;
      int k_issued = 0, v_issued = 0;
      auto load_k = [&](int j) {
        if (j >= 2) ok = ok && mbar_wait(bar(S_FULL + (j & 1)), ((j >> 1) - 1) & 1, abort_flag, 100);
        if (ok) { load_tile(base + kOffK + (j & 1) * kKVBytes, bar(K_FULL + (j & 1)), &map_kc, &map_kd, j); k_issued = j + 1; }
      };
      auto load_v = [&](int j) {
        if (j >= 2) ok = ok && mbar_wait(bar(PV_DONE + (j & 1)), ((j >> 1) - 1) & 1, abort_flag, 100);
        if (ok) { load_tile(base + kOffV + (j & 1) * kKVBytes, bar(V_FULL + (j & 1)), &map_vc, &map_vd, j); v_issued = j + 1; }
      };
      if (T > 0) load_k(0);
      for (int j = 0; j < T && ok; ++j) {
        if (j + 1 < T) load_k(j + 1);
        if (ok) load_v(j);
      }
      if (*abort_flag) {
        // aborting: give the copies already issued a bounded time to land before the block exits
        mbar_wait(bar(Q_FULL), 0, abort_flag + 1);
        for (int j = max(0, k_issued - 2); j < k_issued; ++j) mbar_wait(bar(K_FULL + (j & 1)), (j >> 1) & 1, abort_flag + 1);
        for (int j = max(0, v_issued - 2); j < v_issued; ++j) mbar_wait(bar(V_FULL + (j & 1)), (j >> 1) & 1, abort_flag + 1);
      }
    }
  } else if (warp == 5) {
    // ------------------------------------------------------------ MMA issuer
    // The whole warp walks the loop (uniform control flow, all lanes wait on the barriers); one
    // elected lane issues the MMAs and commits.
    {
      constexpr uint32_t idesc_qk = instr_desc(kKeys, 0), idesc_pv = instr_desc(128, 1);
      bool ok = mbar_wait(bar(Q_FULL), 0, abort_flag);
      // Every operand is built once, from values the compiler can see are warp-uniform (a lane-0
      // broadcast), and kept in registers: descriptors differ only in their 14-bit address field.
      const uint32_t ubase = __shfl_sync(0xffffffffu, base, 0);
      const uint32_t utmem = __shfl_sync(0xffffffffu, tmem, 0);
      uint64_t qd[8], kd[2][8], vd[2][kKeys / 16];
#pragma unroll
      for (int kk = 0; kk < 8; ++kk) {
        qd[kk] = smem_desc(ubase + kOffQ + (kk >> 2) * kSub + (kk & 3) * 32, 16, 1024);
#pragma unroll
        for (int b = 0; b < 2; ++b)
          kd[b][kk] = smem_desc(ubase + kOffK + b * kKVBytes + (kk >> 2) * kSubKV + (kk & 3) * 32, 16, 1024);
      }
#pragma unroll
      for (int b = 0; b < 2; ++b)
#pragma unroll
        for (int kk = 0; kk < kKeys / 16; ++kk)
          vd[b][kk] = smem_desc(ubase + kOffV + b * kKVBytes + kk * 2048, kSubKV, 1024);
      // S[j&1] = Q K_j^T (8 MMAs of K = 16 over head_dim).  The buffer was last read by P V of tile
      // j-2, which was issued earlier, so in-order execution makes it safe to overwrite.
      auto issue_qk = [&](int j) {
        const int b = j & 1;
        ok = ok && mbar_wait(bar(K_FULL + b), (j >> 1) & 1, abort_flag);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) return;
        tc_fence_after();
        if (elect_one()) {
          if (b == 0) {
            tc_mma<false>(utmem + kColS, qd[0], kd[0][0], idesc_qk);
#pragma unroll
            for (int kk = 1; kk < 8; ++kk) tc_mma<true>(utmem + kColS, qd[kk], kd[0][kk], idesc_qk);
          } else {
            tc_mma<false>(utmem + kColS + kKeys, qd[0], kd[1][0], idesc_qk);
#pragma unroll
            for (int kk = 1; kk < 8; ++kk) tc_mma<true>(utmem + kColS + kKeys, qd[kk], kd[1][kk], idesc_qk);
          }
          tc_commit(bar(S_FULL + b));
        }
        __syncwarp();
      };
      if (ok && T > 0) issue_qk(0);
      for (int j = 0; j < T && ok; ++j) {
        if (j + 1 < T) issue_qk(j + 1);  // runs while the softmax of tile j is on the CUDA cores
        // O += P_j V_j: P from TMEM (16 keys = 8 packed columns per MMA), V MN-major from shared memory
        const int b = j & 1;
        ok = ok && mbar_wait(bar(V_FULL + b), (j >> 1) & 1, abort_flag);
        ok = ok && mbar_wait(bar(P_FULL + b), (j >> 1) & 1, abort_flag);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        tc_fence_after();
        if (elect_one()) {
          if (j == 0) {
            tc_mma_ts<false>(utmem + kColO, utmem + kColS, vd[0][0], idesc_pv);
#pragma unroll
            for (int kk = 1; kk < kKeys / 16; ++kk) tc_mma_ts<true>(utmem + kColO, utmem + kColS + kk * 8, vd[0][kk], idesc_pv);
          } else if (b == 0) {
#pragma unroll
            for (int kk = 0; kk < kKeys / 16; ++kk) tc_mma_ts<true>(utmem + kColO, utmem + kColS + kk * 8, vd[0][kk], idesc_pv);
          } else {
#pragma unroll
            for (int kk = 0; kk < kKeys / 16; ++kk)
              tc_mma_ts<true>(utmem + kColO, utmem + kColS + kKeys + kk * 8, vd[1][kk], idesc_pv);
          }
          tc_commit(bar(PV_DONE + b));
        }
        __syncwarp();
      }
    }
  } else {
    // ------------------------------------------------------------ softmax, one query row per thread
    const int r = tid;
    const uint32_t t_lane = tmem + ((uint32_t)(warp * 32) << 16);
    const int qs = r / p.R;
    const float c = p.scale_log2e;
    float m_used = -CUDART_INF_F, l = 0.f;
    bool ok = true;
    for (int j = 0; j < T; ++j) {
      const int b = j & 1;
      ok = ok && mbar_wait(bar(S_FULL + b), (j >> 1) & 1, abort_flag);
      ok = __all_sync(0xffffffffu, ok);  // leave the loop as a whole warp
      if (!ok) break;
      tc_fence_after();
      const uint32_t t_s = t_lane + kColS + b * kKeys;
      uint32_t sv[kKeys];
      TSD_TMEM_LD32(sv, 0, t_s);
      TSD_TMEM_LD32(sv, 32, t_s + 32);
      tmem_wait_ld();

      // visibility of this tile's 64 keys for this row
      uint32_t cm[2] = {0xffffffffu, 0xffffffffu};
      bool masked = false;
      if (j < n_ct) {
        const int valid = clen - j * kKeys;  // keys past the sequence's cache length are invisible
        if (valid < kKeys) {
          masked = true;
#pragma unroll
          for (int w = 0; w < 2; ++w) {
            const int v = valid - 32 * w;
            cm[w] = v >= 32 ? 0xffffffffu : (v <= 0 ? 0u : ((1u << v) - 1u));
          }
        }
      } else {
        const int e = j - n_ct;
        const uint32_t nib = ((uint32_t)rec[3 + 2 * (e >> 1)] >> (qs * 4)) & 15u;  // visible key slots
        masked = true;
#pragma unroll
        for (int w = 0; w < 2; ++w) cm[w] = ((nib >> (((e & 1) * kKeys + w * 32) / p.R)) & 1u) ? 0xffffffffu : 0u;
      }
      if (masked) {
#pragma unroll
        for (int i = 0; i < kKeys; ++i)
          if (!((cm[i >> 5] >> (i & 31)) & 1u)) sv[i] = 0xff800000u;  // -inf: weight exactly 0
      }
      float mx4[4] = {-CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F};  // independent chains
#pragma unroll
      for (int i = 0; i < kKeys / 2; ++i)
        mx4[i & 3] = max3(mx4[i & 3], __uint_as_float(sv[2 * i]), __uint_as_float(sv[2 * i + 1]));
      const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
      const float m_new = fmaxf(m_used, mx * c);
      const bool grow = m_new > m_used + 8.f;  // also true for the first finite maximum
      const float alpha = grow ? ex2f(m_used - m_new) : 1.f;
      if (grow) m_used = m_new;
      const float off = (m_used == -CUDART_INF_F) ? 0.f : -m_used;
      const uint64_t c2 = pack2f(c, c), off2 = pack2f(off, off);
      uint64_t rs4[4] = {0ull, 0ull, 0ull, 0ull};
      uint32_t pk[kKeys / 2];
      if (masked) {  // every exponential on the special-function unit: 2^(-inf) is exactly 0
#pragma unroll
        for (int i = 0; i < kKeys / 2; ++i) {
          float t0, t1;
          unpack2(fma2(pack2(sv[2 * i], sv[2 * i + 1]), c2, off2), t0, t1);
          const float p0 = ex2f(t0), p1 = ex2f(t1);
          rs4[i & 3] = add2(rs4[i & 3], pack2f(p0, p1));
          pk[i] = pack_bf16x2(p0, p1);
        }
      } else {
#pragma unroll
        for (int i = 0; i < kKeys / 2; ++i) {
          const uint64_t t2 = fma2(pack2(sv[2 * i], sv[2 * i + 1]), c2, off2);
          float p0, p1;
          if ((i & 7) < kPolyOf8) {
            exp2_poly2(t2, p0, p1);
          } else {
            float t0, t1;
            unpack2(t2, t0, t1);
            p0 = ex2f(t0);
            p1 = ex2f(t1);
          }
          rs4[i & 3] = add2(rs4[i & 3], pack2f(p0, p1));
          pk[i] = pack_bf16x2(p0, p1);
        }
      }
      float r0, r1;
      unpack2(add2(add2(rs4[0], rs4[1]), add2(rs4[2], rs4[3])), r0, r1);
      l = l * alpha + (r0 + r1);

      if (j > 0 && __any_sync(0xffffffffu, alpha != 1.f)) {
        // rare: the exponent offset moved.  O must be at rest: wait for P V of tile j-1 (P V of
        // tile j cannot start before this thread publishes P_j), then rescale the row.
        ok = ok && mbar_wait(bar(PV_DONE + ((j - 1) & 1)), ((j - 1) >> 1) & 1, abort_flag);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        tc_fence_after();
#pragma unroll
        for (int q4 = 0; q4 < 4; ++q4) {
          uint32_t ov[32];
          TSD_TMEM_LD32(ov, 0, t_lane + kColO + q4 * 32);
          tmem_wait_ld();
#pragma unroll
          for (int i = 0; i < 32; ++i) ov[i] = __float_as_uint(__uint_as_float(ov[i]) * alpha);
          TSD_TMEM_ST32(ov, 0, t_lane + kColO + q4 * 32);
        }
      }
      // P (bf16 pairs) over the first 32 columns of this S buffer: column i = keys 2i (low half), 2i+1
      TSD_TMEM_ST32(pk, 0, t_s);
      tmem_wait_st();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(P_FULL + b));
    }
    // epilogue: O / l -> bf16 -> global, lse
    if (ok && T > 0) ok = mbar_wait(bar(PV_DONE + ((T - 1) & 1)), ((T - 1) >> 1) & 1, abort_flag);
    if (ok && hdr_ok) {
      // O / l -> bf16 -> the shared memory that held Q (every Q K^T has completed), in the layout
      // of the output tensor map (128-byte swizzle: 16-byte chunk c of row r sits at chunk c ^ (r & 7)),
      // then one TMA store per half of head_dim: full 128-byte rows instead of 16-byte pieces per
      // thread, and rows past the end of the tensor are clipped by the copy engine.
      tc_fence_after();
      const int i = qt * kTile + r;
      const float inv = l > 0.f ? 1.f / l : 0.f;
#pragma unroll
      for (int q4 = 0; q4 < 4; ++q4) {
        uint32_t ov[32];
        if (T > 0) {
          TSD_TMEM_LD32(ov, 0, t_lane + kColO + q4 * 32);
          tmem_wait_ld();
        } else {
#pragma unroll
          for (int x = 0; x < 32; ++x) ov[x] = 0u;
        }
        const uint32_t row_base = base + kOffQ + (q4 >> 1) * kSub + (uint32_t)r * 128u;
#pragma unroll
        for (int x = 0; x < 4; ++x) {
          uint4 w;
          w.x = pack_bf16x2(__uint_as_float(ov[8 * x + 0]) * inv, __uint_as_float(ov[8 * x + 1]) * inv);
          w.y = pack_bf16x2(__uint_as_float(ov[8 * x + 2]) * inv, __uint_as_float(ov[8 * x + 3]) * inv);
          w.z = pack_bf16x2(__uint_as_float(ov[8 * x + 4]) * inv, __uint_as_float(ov[8 * x + 5]) * inv);
          w.w = pack_bf16x2(__uint_as_float(ov[8 * x + 6]) * inv, __uint_as_float(ov[8 * x + 7]) * inv);
          const uint32_t chunk = (uint32_t)((q4 & 1) * 4 + x) ^ ((uint32_t)r & 7u);
          asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(row_base + (chunk << 4)), "r"(w.x), "r"(w.y),
                       "r"(w.z), "r"(w.w) : "memory");
        }
      }
      if (p.lse && i < p.N) p.lse[((size_t)s * p.Hq + h) * p.N + i] = (m_used + log2f(l)) * kLn2;
      fence_async_smem();
    }
    // the four softmax warps meet (named barrier 1; every thread of them arrives, also after a
    // timeout), then one thread hands the tile to the copy engine and waits until it has been read
    asm volatile("bar.sync 1, 128;" ::: "memory");
    if (tid == 0 && ok && hdr_ok && !*abort_flag) {
      tma_store_4d(&map_o, base + kOffQ, 0, h, qt * kTile, s);
      tma_store_4d(&map_o, base + kOffQ + kSub, 64, h, qt * kTile, s);
      asm volatile("cp.async.bulk.commit_group;" ::: "memory");
      asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
    }
  }

  // ---------------------------------------------------------------- teardown (all threads)
  tc_fence_before();
  __syncthreads();
  if (warp == 5) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 256;" ::"r"(tmem) : "memory");
  }
  if (tid == 0 && *abort_flag && p.status) atomicOr(p.status, TSD_STATUS_TIMEOUT);
}

// ------------------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* f = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(f);
  });
  return fn;
}

// [S, rows, H, 128] bf16 with element strides (sb, sr, sh): box = box_rows x 64 elements, 128B swizzle.
static bool make_map(CUtensorMap* m, const void* ptr, int S, int rows, int H, int64_t sb, int64_t sr, int64_t sh,
                     int box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn || rows < 1) return false;
  cuuint64_t dims[4] = {128, (cuuint64_t)H, (cuuint64_t)rows, (cuuint64_t)S};
  cuuint64_t strides[3] = {(cuuint64_t)sh * 2, (cuuint64_t)sr * 2, (cuuint64_t)sb * 2};
  // a size-1 dimension may carry any stride; give it a harmless valid one
  if (H == 1) strides[0] = 256;
  if (S == 1) strides[2] = strides[1] * (cuuint64_t)rows;
  cuuint32_t box[4] = {64, 1, (cuuint32_t)box_rows, 1};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(ptr), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Per-device facts and one-time setup (a process may drive several GPUs).
constexpr int kMaxDevices = 64;
static int current_device() {
  int dev = 0;
  return cudaGetDevice(&dev) == cudaSuccess && dev >= 0 && dev < kMaxDevices ? dev : -1;
}

static bool device_is_sm100() {
  static std::mutex mu;
  static int cached[kMaxDevices];  // 0 = unknown, 1 = yes, 2 = no
  const int dev = current_device();
  if (dev < 0) return false;
  std::lock_guard<std::mutex> lock(mu);
  if (cached[dev] == 0) {
    int major = 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return false;
    cached[dev] = major == 10 ? 1 : 2;
  }
  return cached[dev] == 1;
}

bool attention_tc_supported(const AttnArgs& a) {
  return a.L.dtype == TSD_BF16 && a.L.head_dim == 128 && a.sm_scale > 0.f && device_is_sm100();
}

size_t attention_tc_workspace_bytes(const tsd_layout&) { return 0; }

int launch_attention_tc(const AttnArgs& a) {
  const tsd_layout& L = a.L;
  const int N = L.n_branches * L.rows_per_branch;
  CUtensorMap mq, mkc, mvc, mkd, mvd, mo;
  bool ok = make_map(&mq, a.q, L.batch, N, L.n_q_heads, a.qs_b, a.qs_r, a.qs_h, kTile) &&
            make_map(&mo, a.out, L.batch, N, L.n_q_heads, a.os_b, a.os_r, a.os_h, kTile) &&
            make_map(&mkd, a.kd, L.batch, N, L.n_kv_heads, a.ds_b, a.ds_r, a.ds_h, kKeys) &&
            make_map(&mvd, a.vd, L.batch, N, L.n_kv_heads, a.ds_b, a.ds_r, a.ds_h, kKeys);
  if (ok && L.n_cache > 0) {
    ok = make_map(&mkc, a.kc, L.batch, L.n_cache, L.n_kv_heads, a.cs_b, a.cs_r, a.cs_h, kKeys) &&
         make_map(&mvc, a.vc, L.batch, L.n_cache, L.n_kv_heads, a.cs_b, a.cs_r, a.cs_h, kKeys);
  } else if (ok) {  // no cache: the cached maps are never dereferenced
    mkc = mkd;
    mvc = mvd;
  }
  if (!ok) return launch_attention_simt(a);  // strides the tensor maps cannot express
  {  // the dynamic shared memory limit is an attribute of the kernel on each device
    static std::mutex mu;
    static bool done[kMaxDevices];
    const int dev = current_device();
    if (dev < 0) return cuda_fail(cudaErrorInvalidDevice, "cudaGetDevice");
    std::lock_guard<std::mutex> lock(mu);
    if (!done[dev]) {
      cudaError_t attr_err =
          cudaFuncSetAttribute(attention_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
      if (attr_err != cudaSuccess) return cuda_fail(attr_err, "cudaFuncSetAttribute(attention_tc_kernel)");
      done[dev] = true;
    }
  }
  TcParams p;
  p.mask = a.mask;
  p.out = static_cast<__nv_bfloat16*>(a.out);
  p.lse = a.lse;
  p.status = a.status;
  p.os_b = a.os_b; p.os_r = a.os_r; p.os_h = a.os_h;
  p.S = L.batch; p.B = L.n_branches; p.R = L.rows_per_branch; p.Nc = L.n_cache; p.N = N;
  p.Hq = L.n_q_heads; p.group = L.n_q_heads / L.n_kv_heads;
  const MaskDims md = mask_dims(L);
  p.recs_off = md.recs_off; p.n_qt = md.n_qt; p.rec_words = md.rec_words;
  p.scale_log2e = a.sm_scale * kLog2e;
  dim3 grid((N + kTile - 1) / kTile, L.n_q_heads, L.batch);
  attention_tc_kernel<<<grid, kTcThreads, kSmemBytes, a.stream>>>(mq, mkc, mvc, mkd, mvd, mo, p);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(e, "attention_tc_kernel");
  return TSD_OK;
}

}  // namespace tsd
