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
//   S = Q K^T : tcgen05.mma, A and B K-major from 128B-swizzled shared memory, fp32 in TMEM (x2 buffers)
//   softmax  : tcgen05.ld S -> registers, running max / sum in the exp2 domain, P -> bf16 -> shared
//   O += P V : tcgen05.mma, A = P (K-major), B = V (MN-major: head_dim contiguous), fp32 in TMEM
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
constexpr uint32_t kOffQ = 0, kOffP = kTileBytes, kOffK = 2 * kTileBytes, kOffV = 4 * kTileBytes;
constexpr uint32_t kOffBar = 6 * kTileBytes;
constexpr uint32_t kSmemBytes = kOffBar + 256 + 1024;  // + barriers + slack to align the base to 1 KB
constexpr uint32_t kSpinLimit = 1u << 21;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

enum Bar { Q_FULL = 0, K_FULL = 1, K_EMPTY = 3, V_FULL = 5, V_EMPTY = 7, S_FULL = 9, S_EMPTY = 11,
           P_FULL = 13, PV_DONE = 14, N_BARS = 15 };

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
// Bounded wait.  Returns false when the block is aborting (this wait or another one ran out).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag) {
  for (uint32_t it = 0; it < kSpinLimit; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
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

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                       uint32_t accumulate) {
  asm volatile("{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\n"
               "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
               ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
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

// Shared-memory matrix descriptor, 128-byte swizzle (descriptor version 1 = this architecture).
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  return (uint64_t)((addr >> 4) & 0x3FFFu) | ((uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16) |
         ((uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32) | (1ull << 46) | (2ull << 61);
}
// Instruction descriptor: fp32 accumulate, bf16 x bf16, M = N = 128; b_mn = 1 when B is MN-major.
__host__ __device__ constexpr uint32_t instr_desc(uint32_t b_mn) {
  return (1u << 4) | (1u << 7) | (1u << 10) | (b_mn << 16) | ((128u >> 3) << 17) | ((128u >> 4) << 24);
}

struct TcParams {
  const int32_t* mask;
  __nv_bfloat16* out;
  float* lse;
  uint32_t* status;
  int64_t os_b, os_r, os_h;
  int S, B, R, Nc, N, Hq, group;
  float scale_log2e;  // sm_scale * log2(e), > 0
};

__global__ void __launch_bounds__(kTcThreads, 1)
attention_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_kc,
                    const __grid_constant__ CUtensorMap map_vc, const __grid_constant__ CUtensorMap map_kd,
                    const __grid_constant__ CUtensorMap map_vd, const TcParams p) {
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

  const int32_t* mask = p.mask;
  const bool hdr_ok = mask[H_MAGIC] == kMaskMagic && mask[H_S] == p.S && mask[H_B] == p.B &&
                      mask[H_R] == p.R && mask[H_NC] == p.Nc;
  if (!hdr_ok) {  // uniform over the block: nothing has been set up yet
    if (tid == 0 && p.status) atomicOr(p.status, TSD_STATUS_BAD_MASK);
    return;
  }
  const int clen = mask[kHdrWords + s];
  const int32_t* rec = mask + mask[H_RECS_OFF] + (size_t)(s * mask[H_NQT] + qt) * mask[H_REC_WORDS];
  const int n_ct = (clen + kTile - 1) / kTile;  // cached tiles
  const int n_dt = rec[0];                      // visible draft tiles
  const int T = n_ct + n_dt;

  if (tid == 0) {
    abort_flag[0] = 0;
    abort_flag[1] = 0;  // scratch flag for the producer's drain waits
    mbar_init(bar(Q_FULL), 1);
    for (int i = 0; i < 2; ++i) {
      mbar_init(bar(K_FULL + i), 1);
      mbar_init(bar(K_EMPTY + i), 1);
      mbar_init(bar(V_FULL + i), 1);
      mbar_init(bar(V_EMPTY + i), 1);
      mbar_init(bar(S_FULL + i), 1);
      mbar_init(bar(S_EMPTY + i), 4);
    }
    mbar_init(bar(P_FULL), 4);
    mbar_init(bar(PV_DONE), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_async_smem();
  }
  if (warp == 5) {  // TMEM: 2 x S (128 columns each) + O (128 columns) -> 512-column allocation
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(bars + 128u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  if (warp == 4) {
    // ------------------------------------------------------------ TMA producer (one lane)
    if (lane == 0) {
      auto load_tile = [&](uint32_t dst, uint32_t full_bar, const CUtensorMap* mc, const CUtensorMap* md, int j) {
        mbar_expect_tx(full_bar, kTileBytes);
        const bool cached = j < n_ct;
        const CUtensorMap* m = cached ? mc : md;
        const int row = cached ? j * kTile : rec[2 + 2 * (j - n_ct)] * kTile;
        tma_load_4d(dst, m, full_bar, 0, g, row, s);
        tma_load_4d(dst + kSub, m, full_bar, 64, g, row, s);
      };
      mbar_expect_tx(bar(Q_FULL), kTileBytes);
      tma_load_4d(base + kOffQ, &map_q, bar(Q_FULL), 0, h, qt * kTile, s);
      tma_load_4d(base + kOffQ + kSub, &map_q, bar(Q_FULL), 64, h, qt * kTile, s);
      bool ok = true;
      int k_issued = 0, v_issued = 0;
      auto load_k = [&](int j) {
        if (j >= 2) ok = ok && mbar_wait(bar(K_EMPTY + (j & 1)), ((j >> 1) - 1) & 1, abort_flag);
        if (ok) { load_tile(base + kOffK + (j & 1) * kTileBytes, bar(K_FULL + (j & 1)), &map_kc, &map_kd, j); k_issued = j + 1; }
      };
      auto load_v = [&](int j) {
        if (j >= 2) ok = ok && mbar_wait(bar(V_EMPTY + (j & 1)), ((j >> 1) - 1) & 1, abort_flag);
        if (ok) { load_tile(base + kOffV + (j & 1) * kTileBytes, bar(V_FULL + (j & 1)), &map_vc, &map_vd, j); v_issued = j + 1; }
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
    // ------------------------------------------------------------ MMA issuer (one lane)
    if (lane == 0) {
      const uint32_t idesc_qk = instr_desc(0), idesc_pv = instr_desc(1);
      bool ok = mbar_wait(bar(Q_FULL), 0, abort_flag);
      for (int j = 0; j <= T && ok; ++j) {
        if (j < T) {  // S[j&1] = Q K_j^T
          const int b = j & 1;
          ok = ok && mbar_wait(bar(K_FULL + b), (j >> 1) & 1, abort_flag);
          if (j >= 2) ok = ok && mbar_wait(bar(S_EMPTY + b), ((j >> 1) - 1) & 1, abort_flag);
          if (!ok) break;
          tc_fence_after();
          const uint32_t qa = base + kOffQ, ka = base + kOffK + b * kTileBytes;
#pragma unroll
          for (int kk = 0; kk < 8; ++kk) {
            const uint32_t off = (kk >> 2) * kSub + (kk & 3) * 32;
            tc_mma(tmem + b * 128, smem_desc(qa + off, 16, 1024), smem_desc(ka + off, 16, 1024), idesc_qk, kk > 0);
          }
          tc_commit(bar(S_FULL + b));
          tc_commit(bar(K_EMPTY + b));
        }
        if (j >= 1) {  // O += P_{j-1} V_{j-1}
          const int jj = j - 1, b = jj & 1;
          ok = ok && mbar_wait(bar(V_FULL + b), (jj >> 1) & 1, abort_flag);
          ok = ok && mbar_wait(bar(P_FULL), jj & 1, abort_flag);
          if (!ok) break;
          tc_fence_after();
          const uint32_t pa = base + kOffP, va = base + kOffV + b * kTileBytes;
#pragma unroll
          for (int kk = 0; kk < 8; ++kk) {
            const uint32_t a_off = (kk >> 2) * kSub + (kk & 3) * 32;
            tc_mma(tmem + 256, smem_desc(pa + a_off, 16, 1024), smem_desc(va + kk * 2048, kSub, 1024), idesc_pv,
                   (jj > 0 || kk > 0));
          }
          tc_commit(bar(PV_DONE));
          tc_commit(bar(V_EMPTY + b));
        }
      }
    }
  } else {
    // ------------------------------------------------------------ softmax, one query row per thread
    const int r = tid;
    const uint32_t t_lane = tmem + ((uint32_t)(warp * 32) << 16);
    const int slots = kTile / p.R, qs = r / p.R;
    const float c = p.scale_log2e;
    float m_used = -CUDART_INF_F, l = 0.f;
    bool ok = true;
    for (int j = 0; j < T; ++j) {
      const int b = j & 1;
      ok = ok && mbar_wait(bar(S_FULL + b), (j >> 1) & 1, abort_flag);
      ok = __all_sync(0xffffffffu, ok);  // leave the loop as a whole warp
      if (!ok) break;
      tc_fence_after();
      uint32_t sv[128];
      TSD_TMEM_LD32(sv, 0, t_lane + b * 128);
      TSD_TMEM_LD32(sv, 32, t_lane + b * 128 + 32);
      TSD_TMEM_LD32(sv, 64, t_lane + b * 128 + 64);
      TSD_TMEM_LD32(sv, 96, t_lane + b * 128 + 96);
      tmem_wait_ld();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(S_EMPTY + b));  // S is in registers: the buffer may be overwritten

      // visibility of this tile's 128 keys for this row
      uint32_t cm[4] = {0xffffffffu, 0xffffffffu, 0xffffffffu, 0xffffffffu};
      bool masked = false;
      if (j < n_ct) {
        const int valid = clen - j * kTile;  // keys past the sequence's cache length are invisible
        if (valid < kTile) {
          masked = true;
#pragma unroll
          for (int w = 0; w < 4; ++w) {
            const int v = valid - 32 * w;
            cm[w] = v >= 32 ? 0xffffffffu : (v <= 0 ? 0u : ((1u << v) - 1u));
          }
        }
      } else {
        const uint32_t nib = ((uint32_t)rec[3 + 2 * (j - n_ct)] >> (qs * 4)) & 15u;
        masked = true;
#pragma unroll
        for (int w = 0; w < 4; ++w) cm[w] = ((nib >> ((w * 32) / p.R)) & 1u) ? 0xffffffffu : 0u;
        (void)slots;
      }
      if (masked) {
#pragma unroll
        for (int i = 0; i < 128; ++i)
          if (!((cm[i >> 5] >> (i & 31)) & 1u)) sv[i] = 0xff800000u;  // -inf: weight exactly 0
      }
      float mx4[4] = {-CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F};  // independent chains
#pragma unroll
      for (int i = 0; i < 128; ++i) mx4[i & 3] = fmaxf(mx4[i & 3], __uint_as_float(sv[i]));
      const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
      const float m_new = fmaxf(m_used, mx * c);
      const bool grow = m_new > m_used + 8.f;  // also true for the first finite maximum
      const float alpha = grow ? ex2f(m_used - m_new) : 1.f;
      if (grow) m_used = m_new;
      const float off = (m_used == -CUDART_INF_F) ? 0.f : -m_used;
      float rs4[4] = {0.f, 0.f, 0.f, 0.f};
      uint32_t pk[64];
#pragma unroll
      for (int i = 0; i < 64; ++i) {
        const float p0 = ex2f(fmaf(__uint_as_float(sv[2 * i]), c, off));
        const float p1 = ex2f(fmaf(__uint_as_float(sv[2 * i + 1]), c, off));
        rs4[i & 3] += p0 + p1;
        pk[i] = pack_bf16x2(p0, p1);
      }
      const float rowsum = (rs4[0] + rs4[1]) + (rs4[2] + rs4[3]);
      l = l * alpha + rowsum;

      if (j > 0) {  // P and O are free once the previous tile's P V has completed
        ok = ok && mbar_wait(bar(PV_DONE), (j - 1) & 1, abort_flag);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        tc_fence_after();
        if (__any_sync(0xffffffffu, alpha != 1.f)) {  // rare: the exponent offset moved, rescale O
#pragma unroll
          for (int q4 = 0; q4 < 4; ++q4) {
            uint32_t ov[32];
            TSD_TMEM_LD32(ov, 0, t_lane + 256 + q4 * 32);
            tmem_wait_ld();
#pragma unroll
            for (int i = 0; i < 32; ++i) ov[i] = __float_as_uint(__uint_as_float(ov[i]) * alpha);
            TSD_TMEM_ST32(ov, 0, t_lane + 256 + q4 * 32);
          }
          tmem_wait_st();
        }
      }
      // P (bf16) into the 128B-swizzled K-major tile: row r, 16-byte chunk cc at position cc ^ (r & 7)
      const uint32_t prow = base + kOffP + (uint32_t)r * 128u;
#pragma unroll
      for (int cc = 0; cc < 16; ++cc) {
        const uint32_t addr = prow + (cc >> 3) * kSub + (((uint32_t)(cc & 7) ^ (uint32_t)(r & 7)) << 4);
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(pk[4 * cc]), "r"(pk[4 * cc + 1]),
                     "r"(pk[4 * cc + 2]), "r"(pk[4 * cc + 3]) : "memory");
      }
      fence_async_smem();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(P_FULL));
    }
    // epilogue: O / l -> bf16 -> global, lse
    if (ok && T > 0) ok = mbar_wait(bar(PV_DONE), (T - 1) & 1, abort_flag);
    if (ok) {
      tc_fence_after();
      const int i = qt * kTile + r;
      const float inv = l > 0.f ? 1.f / l : 0.f;
      __nv_bfloat16* orow = p.out + s * p.os_b + (int64_t)i * p.os_r + h * p.os_h;
#pragma unroll
      for (int q4 = 0; q4 < 4; ++q4) {
        uint32_t ov[32];
        if (T > 0) {
          TSD_TMEM_LD32(ov, 0, t_lane + 256 + q4 * 32);
          tmem_wait_ld();
        } else {
#pragma unroll
          for (int x = 0; x < 32; ++x) ov[x] = 0u;
        }
        if (i < p.N) {
#pragma unroll
          for (int x = 0; x < 4; ++x) {
            uint4 w;
            w.x = pack_bf16x2(__uint_as_float(ov[8 * x + 0]) * inv, __uint_as_float(ov[8 * x + 1]) * inv);
            w.y = pack_bf16x2(__uint_as_float(ov[8 * x + 2]) * inv, __uint_as_float(ov[8 * x + 3]) * inv);
            w.z = pack_bf16x2(__uint_as_float(ov[8 * x + 4]) * inv, __uint_as_float(ov[8 * x + 5]) * inv);
            w.w = pack_bf16x2(__uint_as_float(ov[8 * x + 6]) * inv, __uint_as_float(ov[8 * x + 7]) * inv);
            *reinterpret_cast<uint4*>(orow + q4 * 32 + x * 8) = w;
          }
        }
      }
      if (p.lse && i < p.N) p.lse[((size_t)s * p.Hq + h) * p.N + i] = (m_used + log2f(l)) * kLn2;
    }
  }

  // ---------------------------------------------------------------- teardown (all threads)
  tc_fence_before();
  __syncthreads();
  if (warp == 5) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tmem) : "memory");
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

// [S, rows, H, 128] bf16 with element strides (sb, sr, sh): box = 128 rows x 64 elements, 128B swizzle.
static bool make_map(CUtensorMap* m, const void* ptr, int S, int rows, int H, int64_t sb, int64_t sr, int64_t sh) {
  EncodeTiledFn fn = encode_fn();
  if (!fn || rows < 1) return false;
  cuuint64_t dims[4] = {128, (cuuint64_t)H, (cuuint64_t)rows, (cuuint64_t)S};
  cuuint64_t strides[3] = {(cuuint64_t)sh * 2, (cuuint64_t)sr * 2, (cuuint64_t)sb * 2};
  // a size-1 dimension may carry any stride; give it a harmless valid one
  if (H == 1) strides[0] = 256;
  if (S == 1) strides[2] = strides[1] * (cuuint64_t)rows;
  cuuint32_t box[4] = {64, 1, 128, 1};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(ptr), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

static bool device_is_sm100() {
  static int cached = -1;
  if (cached < 0) {
    int dev = 0, major = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess)
      return false;
    cached = major == 10 ? 1 : 0;
  }
  return cached == 1;
}

bool attention_tc_supported(const AttnArgs& a) {
  return a.L.dtype == TSD_BF16 && a.L.head_dim == 128 && a.sm_scale > 0.f && device_is_sm100();
}

size_t attention_tc_workspace_bytes(const tsd_layout&) { return 0; }

int launch_attention_tc(const AttnArgs& a) {
  const tsd_layout& L = a.L;
  const int N = L.n_branches * L.rows_per_branch;
  CUtensorMap mq, mkc, mvc, mkd, mvd;
  bool ok = make_map(&mq, a.q, L.batch, N, L.n_q_heads, a.qs_b, a.qs_r, a.qs_h) &&
            make_map(&mkd, a.kd, L.batch, N, L.n_kv_heads, a.ds_b, a.ds_r, a.ds_h) &&
            make_map(&mvd, a.vd, L.batch, N, L.n_kv_heads, a.ds_b, a.ds_r, a.ds_h);
  if (ok && L.n_cache > 0) {
    ok = make_map(&mkc, a.kc, L.batch, L.n_cache, L.n_kv_heads, a.cs_b, a.cs_r, a.cs_h) &&
         make_map(&mvc, a.vc, L.batch, L.n_cache, L.n_kv_heads, a.cs_b, a.cs_r, a.cs_h);
  } else if (ok) {  // no cache: the cached maps are never dereferenced
    mkc = mkd;
    mvc = mvd;
  }
  if (!ok) return launch_attention_simt(a);  // strides the tensor maps cannot express
  static std::once_flag once;
  static cudaError_t attr_err = cudaSuccess;
  std::call_once(once, [] {
    attr_err = cudaFuncSetAttribute(attention_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
  });
  if (attr_err != cudaSuccess) return cuda_fail(attr_err, "cudaFuncSetAttribute(attention_tc_kernel)");
  TcParams p;
  p.mask = a.mask;
  p.out = static_cast<__nv_bfloat16*>(a.out);
  p.lse = a.lse;
  p.status = a.status;
  p.os_b = a.os_b; p.os_r = a.os_r; p.os_h = a.os_h;
  p.S = L.batch; p.B = L.n_branches; p.R = L.rows_per_branch; p.Nc = L.n_cache; p.N = N;
  p.Hq = L.n_q_heads; p.group = L.n_q_heads / L.n_kv_heads;
  p.scale_log2e = a.sm_scale * kLog2e;
  dim3 grid((N + kTile - 1) / kTile, L.n_q_heads, L.batch);
  attention_tc_kernel<<<grid, kTcThreads, kSmemBytes, a.stream>>>(mq, mkc, mvc, mkd, mvd, p);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(e, "attention_tc_kernel");
  return TSD_OK;
}

}  // namespace tsd
