// Stage 1b on tensor cores: masked verify attention (paper Section 3.3) for bf16, head_dim 128.
//
// Persistent kernel, one thread block of 20 warps per SM.  A work item is (sequence, query head,
// tile of 128 draft rows = 128/R branches); a block takes items blockIdx.x, blockIdx.x + gridDim.x,
// ...  The key tiles of an item (64 keys each) are the cached prefix/suffix tiles, shared by every
// branch (a dense GEMM), then the draft tiles listed for the query tile in the mask blob; inside a
// draft tile only the (query branch, key branch) pairs whose bit is set are visible, everything
// else gets weight 0.  Tiles of branches a query tile cannot see are never loaded.
//
// Tensor memory (all 512 columns): O (128 columns, fp32), Q of the current and of the next item
// (2 x 64 columns, bf16 pairs), three S buffers (3 x 64) and two P buffers (2 x 32).
//   S = Q K^T : tcgen05.mma with A = Q from TENSOR MEMORY, B = K (K-major) from 128B-swizzled
//               shared memory.  An MMA whose A operand comes from shared memory is limited by
//               shared-memory bandwidth (4 KB of A + 2 KB of B per 128x64x16 step: 48 clocks
//               measured instead of 32); with Q in tensor memory the 64-key steps run at full rate.
//   softmax   : three warpgroups take the key tiles in turn (tile t -> warpgroup t mod 3), one
//               query row per thread (tensor-memory lane = row): tcgen05.ld S, release the S
//               buffer, mask, row maximum, exponentials in the exp2 domain, P -> bf16 ->
//               tcgen05.st into a P buffer.  Three tiles are in the softmax at any time, so one
//               block keeps the tensor pipe fed by itself.
//   O += P V  : tcgen05.mma, A = P from tensor memory, B = V (head_dim contiguous) from shared
//               memory, fp32 accumulation in tensor memory.
// All rows share one O accumulator, so the warpgroups agree on the exponent offset of a row
// through a chain of decisions in tile order: the thread that owns row r in tile t waits for the
// decision of tile t-1 (a per-warp mbarrier and one float per row in shared memory), keeps that
// offset unless the tile's maximum exceeds it by more than 2^8, publishes its decision and only
// then starts on the exponentials.  The chain is short; the expensive part of the tiles overlaps.
// A thread that moves the offset rescales the row of O before it publishes P (the P V of its tile
// cannot start earlier); every thread keeps its own partial row sum on the offset it used last
// and the epilogue brings the partial sums together.  The decisions depend on the row's scores
// only, so results do not depend on timing.
// Warp roles: warp 0 issues Q K^T (and owns the tensor-memory allocation), warp 1 streams K (and Q),
// warp 2 issues P V, warp 3 streams V, warps 4-15 softmax (3 warpgroups), warps 16-19 epilogue
// (wait for the item's last P V, O / l -> bf16 -> staging buffer -> TMA store).  The softmax
// warpgroups take registers from the others (setmaxnreg).
// Items overlap: Q of the next item is loaded into shared memory and copied into the other Q
// buffer during the current item, its first Q K^T are issued while the last softmax tiles of the
// current item run, the softmax warpgroups go on to it without waiting for the epilogue, and its
// first P V waits only until the epilogue has read O into registers.
// Every mbarrier wait is bounded: on expiry the block raises TSD_STATUS_TIMEOUT, stops issuing
// work, waits (bounded) for its copies in flight, frees its tensor memory and returns.
#include <cuda.h>
#include <math_constants.h>
#include <mutex>
#include "tsd_common.cuh"

namespace tsd {

constexpr int kTcThreads = 640;
constexpr int kSoftmaxWarps = 12;              // three warpgroups: warps 4-15
// The issuing roles take the lowest warp indices: the schedulers favour them over the softmax
// warps they share a sub-partition with, and a late MMA or copy stalls the whole pipeline.
constexpr int kQkWarp = 0, kKProducerWarp = 1, kPvWarp = 2, kVProducerWarp = 3, kFirstSoftmaxWarp = 4;
constexpr int kFirstEpilogueWarp = kFirstSoftmaxWarp + kSoftmaxWarps;  // warps 16-19
// Registers per thread after the warpgroups have traded them (the block starts with 96 each):
// what the softmax threads gain (384 x 24) is exactly what the others release (128 x 40 + 128 x 32):
// a warpgroup can only take registers that another one of the block has given back.
constexpr int kRegsService = 56, kRegsEpilogue = 64, kRegsSoftmax = 120;
constexpr int kNSb = 3;                        // S buffers in tensor memory
constexpr int kNK = 5;                         // K stages: a K tile is needed well before its V tile
constexpr int kNV = 4;                         // V stages
constexpr int kNP = 2;                         // P buffers in tensor memory
constexpr int kKeys = 64;                      // keys per tile
constexpr int kMaxItems = 512;                 // work items of one block (their tile counts sit in shared memory)
constexpr uint32_t kSub = 16384;               // bytes of one [128 rows x 64 elements] bf16 sub-tile
constexpr uint32_t kTileBytes = 2 * kSub;      // a [128 x 128] bf16 tile
constexpr uint32_t kSubKV = 8192;              // bytes of one [64 keys x 64 elements] bf16 sub-tile
constexpr uint32_t kKVBytes = 2 * kSubKV;      // a [64 x 128] bf16 K or V tile
constexpr uint32_t kOffQ = 0;                  // Q staging (TMA destination, copied to tensor memory)
constexpr uint32_t kOffO = kTileBytes;         // O staging (TMA store source)
constexpr uint32_t kOffK = 2 * kTileBytes;
constexpr uint32_t kOffV = kOffK + kNK * kKVBytes;
constexpr uint32_t kOffBar = kOffV + kNV * kKVBytes;
constexpr uint32_t kOffMref = kOffBar + 512;   // exponent offset per row (128 floats)
// partial row sums and the exponent offsets they are on, per softmax warpgroup, for three items in
// rotation (3 x 3 x 128 floats each): a softmax warpgroup leaves them for the epilogue and moves on
constexpr uint32_t kOffLpart = kOffMref + 512;
constexpr uint32_t kOffMpart = kOffLpart + 3 * 3 * 128 * 4;
constexpr uint32_t kOffItems = kOffMpart + 3 * 3 * 128 * 4;  // key tiles / cache length per item (2 x kMaxItems int32)
constexpr uint32_t kSmemBytes = kOffItems + 2 * kMaxItems * 4 + 1024;  // + slack to align the base to 1 KB
constexpr uint32_t kColO = 0, kColQ = 128, kColS = 256, kColP = 448;  // tensor-memory columns
constexpr uint32_t kSpinLimit = 1u << 21;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

// Barriers.  Tile t (counted over all items of the block) uses S buffer t mod 3, K stage t mod 5,
// V stage t mod 4 and P buffer t mod 2.  A test of a barrier costs the issuing warps a
// shared-memory round trip in front of every batch of MMAs, so each of them waits on ONE barrier
// per tile: the barrier on which a K (V) tile lands also collects the arrivals that tell that the
// S buffer is free (that P has been written).
enum Bar {
  QS_FULL = 0,    // Q of an item has landed in the staging buffer
  QT_READY = 1,   // [2] Q has been copied into tensor-memory buffer q (and the staging buffer is free)
  QK_GO = 3,      // [5] per K stage: the K tile of tile t has landed (1 arrival + bytes) and the four softmax
                  //     warps of tile t-3 have S in registers, so its buffer can be overwritten (4 arrivals;
                  //     the producer supplies them for the first three tiles)
  K_FREE = 8,     // [5] Q K^T complete: the K stage can be refilled
  PV_GO = 13,     // [4] per V stage: the V tile of tile t has landed (1 arrival + bytes) and the four softmax
                  //     warps have written P of tile t (4 arrivals)
  S_FULL = 17,    // [3] Q K^T complete: S can be read
  PV_DONE = 20,   // [4] P V of a tile (and every MMA before it) complete, per tile mod 4: its V stage and
                  //     its P buffer are free, O is up to date.  Waiters look at most one phase ahead of
                  //     what they know to be complete (a parity wait cannot tell two phases apart), which
                  //     is why this is a ring of four although there are only two P buffers.
  DEC = 24,       // [4][4] exponent offsets of a tile decided, per tile mod 4 and warp quarter
  O_FREE = 40,    // the epilogue has read O into registers
  LPART = 41,     // every softmax warp has published its partial row sums of an item
  STAGED = 42,    // the output tile is complete in the staging buffer
  OS_FREE = 43,   // the previous item's store has read the staging buffer
  N_BARS = 44
};

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
                                          uint32_t sleep_ns = 0, uint32_t limit = kSpinLimit) {
  if (mbar_test_wait(bar, parity)) return true;
  for (uint32_t it = 0; it < limit; ++it) {
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

__device__ __forceinline__ void prefetch_tensormap(const CUtensorMap* map) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(map)) : "memory");
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

#define TSD_R16(a, o) "=r"(a[o+0]), "=r"(a[o+1]), "=r"(a[o+2]), "=r"(a[o+3]), "=r"(a[o+4]), "=r"(a[o+5]), "=r"(a[o+6]), "=r"(a[o+7]), \
  "=r"(a[o+8]), "=r"(a[o+9]), "=r"(a[o+10]), "=r"(a[o+11]), "=r"(a[o+12]), "=r"(a[o+13]), "=r"(a[o+14]), "=r"(a[o+15])
#define TSD_W16(a, o) "r"(a[o+0]), "r"(a[o+1]), "r"(a[o+2]), "r"(a[o+3]), "r"(a[o+4]), "r"(a[o+5]), "r"(a[o+6]), "r"(a[o+7]), \
  "r"(a[o+8]), "r"(a[o+9]), "r"(a[o+10]), "r"(a[o+11]), "r"(a[o+12]), "r"(a[o+13]), "r"(a[o+14]), "r"(a[o+15])
#define TSD_R32(a, o) TSD_R16(a, o), TSD_R16(a, o + 16)
#define TSD_W32(a, o) TSD_W16(a, o), TSD_W16(a, o + 16)

// 32 (16) consecutive 32-bit columns of this thread's tensor-memory lane <-> registers a[o ...]
#define TSD_TMEM_LD32(a, o, taddr)                                                                         \
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "                                                   \
               "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"                                   \
               "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"                  \
               : TSD_R32(a, o) : "r"(taddr) : "memory")
#define TSD_TMEM_LD16(a, o, taddr)                                                                         \
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 "                                                   \
               "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"                           \
               : TSD_R16(a, o) : "r"(taddr) : "memory")
#define TSD_TMEM_ST32(a, o, taddr)                                                                         \
  asm volatile("tcgen05.st.sync.aligned.32x32b.x32.b32 [%32], "                                            \
               "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"                                   \
               "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31};"                         \
               ::TSD_W32(a, o), "r"(taddr) : "memory")
#define TSD_TMEM_ST16(a, o, taddr)                                                                         \
  asm volatile("tcgen05.st.sync.aligned.32x32b.x16.b32 [%16], "                                            \
               "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15};"                                  \
               ::TSD_W16(a, o), "r"(taddr) : "memory")
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ float ex2f(float x) {
#ifdef TSD_EXPERIMENT_NO_EX2  /* timing experiment only: wrong results */
  return x;
#else
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
#endif
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
#ifndef TSD_SM_SLEEP
#define TSD_SM_SLEEP 0
#endif
#ifndef TSD_POLY_OF8
#define TSD_POLY_OF8 0
#endif
constexpr int kPolyOf8 = TSD_POLY_OF8;  // of every 8 score pairs, this many take the polynomial exp2 (unmasked tiles)

// Shared-memory matrix descriptor, 128-byte swizzle (descriptor version 1 = this architecture).
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  return (uint64_t)((addr >> 4) & 0x3FFFu) | ((uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16) |
         ((uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32) | (1ull << 46) | (2ull << 61);
}
// Instruction descriptor: fp32 accumulate, bf16 x bf16, M = 128, N = n; b_mn = 1 when B is MN-major.
__host__ __device__ constexpr uint32_t instr_desc(uint32_t n, uint32_t b_mn) {
  return (1u << 4) | (1u << 7) | (1u << 10) | (b_mn << 16) | ((n >> 3) << 17) | ((128u >> 4) << 24);
}

// Optional clock trace of one block's pipeline (compiled in with -DTSD_ATTN_TRACE only): per key
// tile, when each role passed each of its steps.
#ifdef TSD_ATTN_TRACE
constexpr int kTrTiles = 256, kTrEvents = 16, kTrBlocks = 4;
__device__ long long g_attn_trace[kTrBlocks * kTrTiles * kTrEvents];
#define TSD_TR_ALWAYS(ev, G)                                                               \
  do {                                                                                     \
    if (blockIdx.x < kTrBlocks && (G) < kTrTiles)                                          \
      g_attn_trace[((int)blockIdx.x * kTrTiles + (G)) * kTrEvents + (ev)] = clock64();     \
  } while (0)
#if TSD_ATTN_TRACE >= 2  /* level 2: the block's entry and exit only, which costs nothing per tile */
#define TSD_TR(ev, G) do { } while (0)
#else
#define TSD_TR(ev, G) TSD_TR_ALWAYS(ev, G)
#endif
#define TSD_TR_SUM(ev, G, v)                                                               \
  do {                                                                                     \
    if (blockIdx.x < kTrBlocks) g_attn_trace[((int)blockIdx.x * kTrTiles + (G)) * kTrEvents + (ev)] = (v); \
  } while (0)
#define TSD_CLK() clock64()
#else
#define TSD_TR(ev, G) do { } while (0)
#define TSD_TR_ALWAYS(ev, G) do { } while (0)
#define TSD_TR_SUM(ev, G, v) do { } while (0)
#define TSD_CLK() 0ll
#endif

struct TcParams {
  const int32_t* mask;
  float* lse;
  uint32_t* status;
  int S, B, R, Nc, N, Hq, group;
  int recs_off, n_qt, rec_words;  // layout of the mask blob, computed on the host from the same tsd_layout
  int n_items;                    // S * Hq * n_qt
  float scale_log2e;              // sm_scale * log2(e), > 0
};

// The MMAs of a tile go out as ONE block of instructions: the issuing lane shares its scheduler with
// three softmax warps, so every instruction between two MMAs (a predicate, a 64-bit add for a
// descriptor) is a gap in which the tensor pipe may run dry.  Descriptors are passed as their low
// words (the address field varies, the high word is the same for all of one operand).
//
// One Q K^T: 8 MMAs (K = 16 over head_dim) into the S buffer at tensor-memory address `s_tmem`, Q
// from tensor memory at `q_tmem`, K through the descriptors (lo[kk], hi); then the two commits.
__device__ __forceinline__ void issue_qk_mmas(uint32_t s_tmem, uint32_t q_tmem, const uint32_t (&lo)[8], uint32_t hi,
                                              uint32_t s_full, uint32_t k_free) {
  constexpr uint32_t idesc_qk = instr_desc(kKeys, 0);
  asm volatile(
      "{\n.reg .pred pf, pt;\n.reg .b32 a;\n.reg .b64 dsc;\n"
      "setp.ne.b32 pf, 0, 0;\nsetp.eq.b32 pt, 0, 0;\n"
      "mov.b64 dsc, {%2, %10};\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], dsc, %11, pf;\n"
      "add.u32 a, %1, 8;\nmov.b64 dsc, {%3, %10};\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [a], dsc, %11, pt;\n"
      "add.u32 a, %1, 16;\nmov.b64 dsc, {%4, %10};\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [a], dsc, %11, pt;\n"
      "add.u32 a, %1, 24;\nmov.b64 dsc, {%5, %10};\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [a], dsc, %11, pt;\n"
      "add.u32 a, %1, 32;\nmov.b64 dsc, {%6, %10};\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [a], dsc, %11, pt;\n"
      "add.u32 a, %1, 40;\nmov.b64 dsc, {%7, %10};\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [a], dsc, %11, pt;\n"
      "add.u32 a, %1, 48;\nmov.b64 dsc, {%8, %10};\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [a], dsc, %11, pt;\n"
      "add.u32 a, %1, 56;\nmov.b64 dsc, {%9, %10};\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [a], dsc, %11, pt;\n"
      "tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%12];\n"
      "tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%13];\n}"
      ::"r"(s_tmem), "r"(q_tmem), "r"(lo[0]), "r"(lo[1]), "r"(lo[2]), "r"(lo[3]), "r"(lo[4]), "r"(lo[5]), "r"(lo[6]),
        "r"(lo[7]), "r"(hi), "r"(idesc_qk), "r"(s_full), "r"(k_free) : "memory");
}
// One P V: 4 MMAs (16 keys = 8 packed columns of P each), P from tensor memory at `p_tmem`, V through
// the descriptors (lo[kk], hi), into O at `o_tmem`; `acc` = 0 starts a new accumulation; then the commit.
__device__ __forceinline__ void issue_pv_mmas(uint32_t o_tmem, uint32_t p_tmem, const uint32_t (&lo)[kKeys / 16], uint32_t hi,
                                              uint32_t acc, uint32_t pv_done) {
  constexpr uint32_t idesc_pv = instr_desc(128, 1);
  asm volatile(
      "{\n.reg .pred pa, pt;\n.reg .b32 a;\n.reg .b64 dsc;\n"
      "setp.ne.b32 pa, %7, 0;\nsetp.eq.b32 pt, 0, 0;\n"
      "mov.b64 dsc, {%2, %6};\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], dsc, %8, pa;\n"
      "add.u32 a, %1, 8;\nmov.b64 dsc, {%3, %6};\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [a], dsc, %8, pt;\n"
      "add.u32 a, %1, 16;\nmov.b64 dsc, {%4, %6};\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [a], dsc, %8, pt;\n"
      "add.u32 a, %1, 24;\nmov.b64 dsc, {%5, %6};\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [a], dsc, %8, pt;\n"
      "tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%9];\n}"
      ::"r"(o_tmem), "r"(p_tmem), "r"(lo[0]), "r"(lo[1]), "r"(lo[2]), "r"(lo[3]), "r"(hi), "r"(acc), "r"(idesc_pv),
        "r"(pv_done) : "memory");
}

// Rarely executed pieces of the softmax warps, kept out of line so that the loop over the key
// tiles stays small in the instruction cache.
// One row of O (128 fp32 columns of this thread's tensor-memory lane) times alpha.
__device__ __noinline__ void rescale_o_row(uint32_t t_o, float alpha) {
#pragma unroll 1
  for (int q4 = 0; q4 < 4; ++q4) {
    uint32_t ov[32];
    TSD_TMEM_LD32(ov, 0, t_o + q4 * 32);
    tmem_wait_ld();
#pragma unroll
    for (int i = 0; i < 32; ++i) ov[i] = __float_as_uint(__uint_as_float(ov[i]) * alpha);
    TSD_TMEM_ST32(ov, 0, t_o + q4 * 32);
  }
}
// One row of Q: staging buffer (128-byte swizzle: 16-byte chunk c of row r sits at chunk c ^ (r & 7),
// one sub-tile per half of head_dim) -> 64 columns of this thread's tensor-memory lane, as the A
// operand of Q K^T (32-bit column i = elements 2i, 2i+1).
__device__ __noinline__ void copy_q_row(uint32_t q_smem, int r, uint32_t t_q) {
#pragma unroll 1
  for (int sub = 0; sub < 2; ++sub) {
    uint32_t w[32];
#pragma unroll
    for (int ch = 0; ch < 8; ++ch) {
      const uint32_t a = q_smem + sub * kSub + (uint32_t)r * 128u + ((uint32_t)(ch ^ (r & 7)) << 4);
      asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];"
                   : "=r"(w[ch * 4]), "=r"(w[ch * 4 + 1]), "=r"(w[ch * 4 + 2]), "=r"(w[ch * 4 + 3]) : "r"(a) : "memory");
    }
    TSD_TMEM_ST32(w, 0, t_q + sub * 32);
  }
  tmem_wait_st();
}

__global__ void __launch_bounds__(kTcThreads, 1)
attention_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_kc,
                    const __grid_constant__ CUtensorMap map_vc, const __grid_constant__ CUtensorMap map_kd,
                    const __grid_constant__ CUtensorMap map_vd, const __grid_constant__ CUtensorMap map_o,
                    const TcParams p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* base_ptr = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t bars = base + kOffBar;
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(base_ptr + kOffBar + 448);
  volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(base_ptr + kOffBar + 452);
  float* mref = reinterpret_cast<float*>(base_ptr + kOffMref);
  float* lpart = reinterpret_cast<float*>(base_ptr + kOffLpart);
  float* mpart = reinterpret_cast<float*>(base_ptr + kOffMpart);
  int32_t* item_T = reinterpret_cast<int32_t*>(base_ptr + kOffItems);
  int32_t* item_clen = item_T + kMaxItems;
  auto bar = [&](int i) { return bars + 8u * (uint32_t)i; };

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  if (tid == 0) TSD_TR_ALWAYS(0, 200);
  // The copy engine fetches a tensor map from global memory the first time a copy names it: ask
  // for all six now, so that this overlaps the prologue (no measurable effect where the maps are
  // already cached from the previous launch, as in a replayed graph).
  if (tid == kVProducerWarp * 32) {
    prefetch_tensormap(&map_q);
    prefetch_tensormap(&map_kc);
    prefetch_tensormap(&map_vc);
    prefetch_tensormap(&map_kd);
    prefetch_tensormap(&map_vd);
    prefetch_tensormap(&map_o);
  }
  const int32_t* mask = p.mask;
  const int n_my = (int)blockIdx.x < p.n_items ? (p.n_items - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x : 0;
  // item -> (sequence, query head, query tile); query tiles of a head, then heads, then sequences
  // are neighbours, so that blocks running at the same time share K/V in L2
  auto item_coords = [&](int it, int& s, int& h, int& qt) {
    const int item = (int)blockIdx.x + it * (int)gridDim.x;
    qt = item % p.n_qt;
    h = (item / p.n_qt) % p.Hq;
    s = item / (p.n_qt * p.Hq);
  };

  const int h_magic = mask[H_MAGIC], h_s = mask[H_S], h_b = mask[H_B], h_r = mask[H_R], h_nc = mask[H_NC];
  // tile counts of this block's items (the blob's layout follows from the tsd_layout, so no
  // address depends on a loaded value)
  for (int it = tid; it < n_my; it += kTcThreads) {
    int s, h, qt;
    item_coords(it, s, h, qt);
    const int clen = min(max(mask[kHdrWords + s], 0), p.Nc);
    const int n_dt = min(max(mask[p.recs_off + (size_t)(s * p.n_qt + qt) * p.rec_words], 1), p.n_qt);
    const int n_ct = (clen + kKeys - 1) / kKeys;
    item_clen[it] = clen;
    item_T[it] = n_ct + 2 * n_dt;
  }

  // Coordinates of the block's first item for the two producer lanes: worked out here, while the
  // block is still setting up, so that their first requests after the sync are a few instructions.
  int s_first = 0, g_first = 0;
  if (lane == 0 && (warp == kKProducerWarp || warp == kVProducerWarp) && n_my > 0) {
    int h, qt;
    item_coords(0, s_first, h, qt);
    g_first = h / p.group;
  }
  if (warp == kKProducerWarp && lane == 0) {
    abort_flag[0] = 0;
    abort_flag[1] = 0;  // scratch flag for the drain waits
    mbar_init(bar(QS_FULL), 1);
    mbar_init(bar(QT_READY), 4);
    mbar_init(bar(QT_READY + 1), 4);
    for (int i = 0; i < kNSb; ++i) mbar_init(bar(S_FULL + i), 1);
    for (int i = 0; i < kNK; ++i) {
      mbar_init(bar(QK_GO + i), 5);
      mbar_init(bar(K_FREE + i), 1);
    }
    for (int i = 0; i < kNV; ++i) {
      mbar_init(bar(PV_GO + i), 5);
      mbar_init(bar(PV_DONE + i), 1);
    }
    for (int i = 0; i < 16; ++i) mbar_init(bar(DEC + i), 1);
    mbar_init(bar(O_FREE), 4);
    mbar_init(bar(LPART), kSoftmaxWarps);
    mbar_init(bar(STAGED), 4);
    mbar_init(bar(OS_FREE), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_async_smem();
    if (n_my > 0) {  // Q of the first item: its coordinates need nothing from the blob
      int s, h, qt;
      item_coords(0, s, h, qt);
      mbar_expect_tx(bar(QS_FULL), kTileBytes);
      tma_load_4d(base + kOffQ, &map_q, bar(QS_FULL), 0, h, qt * kTile, s);
      tma_load_4d(base + kOffQ + kSub, &map_q, bar(QS_FULL), 64, h, qt * kTile, s);
    }
  }
  if (warp == kQkWarp) {  // the whole tensor memory of the SM: O, 2 x Q, 3 x S, 2 x P
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(bars + 448u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  // A blob that was built for another layout: report it and run no item (the Q load in flight is
  // still waited for before the block leaves).
  const bool hdr_ok = h_magic == kMaskMagic && h_s == p.S && h_b == p.B && h_r == p.R && h_nc == p.Nc;
  if (!hdr_ok && tid == 0 && blockIdx.x == 0 && p.status) atomicOr(p.status, TSD_STATUS_BAD_MASK);
  const int n_run = hdr_ok ? n_my : 0;

  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  if (tid == 0) TSD_TR_ALWAYS(1, 200);

  // The softmax threads need the registers; the issuing, copying and epilogue warpgroups give theirs
  // up (each warpgroup trades at the top of its own branch).
  if (warp < kFirstSoftmaxWarp) {
  asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kRegsService));
  if (warp == kKProducerWarp || warp == kVProducerWarp) {
    // ------------------------------------------------------------ TMA producers (one lane each)
    // One warp streams the K tiles (and Q of the items to come), the other the V tiles: a lone
    // thread needs several hundred clocks per tile for its waits and copies, and K must run up to
    // four tiles ahead of V.
    if (lane == 0) {
      const bool is_k = warp == kKProducerWarp;
      bool ok = true;
      int issued = 0, q_issued = (is_k && n_my > 0) ? 1 : 0;
      // Q of item x goes to the staging buffer once Q of item x-1 has been copied out of it
      auto issue_q = [&](bool block) {
        if (!ok || q_issued >= n_run) return;
        const int x = q_issued;
        const uint32_t b = bar(QT_READY + ((x - 1) & 1)), ph = ((x - 1) >> 1) & 1;
        if (block) ok = mbar_wait(b, ph, abort_flag, 100);
        else if (!mbar_test_wait(b, ph)) return;
        if (!ok) return;
        int s, h, qt;
        item_coords(x, s, h, qt);
        mbar_expect_tx(bar(QS_FULL), kTileBytes);
        tma_load_4d(base + kOffQ, &map_q, bar(QS_FULL), 0, h, qt * kTile, s);
        tma_load_4d(base + kOffQ + kSub, &map_q, bar(QS_FULL), 64, h, qt * kTile, s);
        q_issued = x + 1;
      };
      const CUtensorMap* mc = is_k ? &map_kc : &map_vc;
      const CUtensorMap* md = is_k ? &map_kd : &map_vd;
      const uint32_t stage0 = base + (is_k ? kOffK : kOffV);
      const int full0 = is_k ? QK_GO : PV_GO, free0 = is_k ? K_FREE : PV_DONE;
      const int n_stage = is_k ? kNK : kNV;
      int G = 0, b = 0;       // tile count, its stage = G mod n_stage
      uint32_t ph = 0;        // phase of that stage's barriers = (G / n_stage) & 1
      // The first cached tiles of the first item, one per stage, go out before the general loop
      // below is entered: on its first pass that loop costs ~1.5 k clocks of instruction fetches and
      // single-lane index arithmetic before its first request (measured), and the whole block
      // waits for these tiles.
      const int n_pre = n_run > 0 ? min(n_stage, (item_clen[0] + kKeys - 1) / kKeys) : 0;
      for (int t = 0; t < n_pre; ++t) {
        const uint32_t dst = stage0 + t * kKVBytes, full_bar = bar(full0 + t);
        mbar_expect_tx(full_bar, kKVBytes);
        if (is_k && t < kNSb) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0], 4;" ::"r"(full_bar) : "memory");
        tma_load_4d(dst, mc, full_bar, 0, g_first, t * kKeys, s_first);
        tma_load_4d(dst + kSubKV, mc, full_bar, 64, g_first, t * kKeys, s_first);
      }
      issued = n_pre;
      for (int it = 0; it < n_run && ok; ++it) {
        // Q of this item must be on its way before its K tiles queue behind it
        while (is_k && ok && q_issued <= it) issue_q(true);
        int s, h, qt;
        item_coords(it, s, h, qt);
        const int g = h / p.group, n_ct = (item_clen[it] + kKeys - 1) / kKeys, T = item_T[it];
        const int32_t* rec = mask + p.recs_off + (size_t)(s * p.n_qt + qt) * p.rec_words;
        for (int j = 0; j < T && ok; ++j, ++G) {
          if (is_k) issue_q(false);
          if (!ok) break;
          // the stage is free once the MMAs that read its previous tile have completed
          if (G >= n_stage) ok = mbar_wait(bar(free0 + b), ph ^ 1u, abort_flag, 100);
          if (!ok) break;
          if (G >= n_pre) {
            const bool cached = j < n_ct;
            const int e = j - n_ct;  // draft key tile e = half (e & 1) of the listed 128-row tile e >> 1
            const int row = cached ? j * kKeys : rec[2 + 2 * (e >> 1)] * kTile + (e & 1) * kKeys;
            const CUtensorMap* m = cached ? mc : md;
            const uint32_t dst = stage0 + b * kKVBytes, full_bar = bar(full0 + b);
            mbar_expect_tx(full_bar, kKVBytes);
            // no softmax has run before the first three tiles: their S buffers are free from the start
            if (is_k && G < kNSb) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0], 4;" ::"r"(full_bar) : "memory");
            tma_load_4d(dst, m, full_bar, 0, g, row, s);
            tma_load_4d(dst + kSubKV, m, full_bar, 64, g, row, s);
            issued = G + 1;
          }
          TSD_TR(is_k ? 0 : 1, G);
          if (++b == n_stage) { b = 0; ph ^= 1u; }
        }
      }
      if (*abort_flag || !hdr_ok) {
        // leaving early: give the copies already issued a bounded time to land before the block exits
        volatile uint32_t* scratch = abort_flag + 1;
        if (q_issued > 0) mbar_wait(bar(QS_FULL), (q_issued - 1) & 1, scratch);
        for (int t = max(0, issued - n_stage); t < issued; ++t)
          mbar_wait(bar(full0 + t % n_stage), (t / n_stage) & 1, scratch);
      }
    }
  } else {
    // ------------------------------------------------------------ MMA issuers
    // Two warps, one for Q K^T and one for P V: the thread that issues an MMA is held until the
    // tensor pipe takes it, so a single issuer would leave the pipe idle during its own waits and
    // bookkeeping; with two, one warp's MMAs run while the other prepares.  Each whole warp walks its
    // loop (uniform control flow, all lanes wait on the barriers); one elected lane issues the
    // MMAs and commits.  Tile counts come through a lane-0 broadcast so that the loop counters, and
    // with them the operands of the MMAs, stay on the uniform datapath.
    bool ok = true;
    const uint32_t ubase = __shfl_sync(0xffffffffu, base, 0);
    const uint32_t utmem = __shfl_sync(0xffffffffu, tmem, 0);
    int G = 0;
    // The test of the next tile's barrier is issued before the MMAs of the current one and its
    // result is read after them, so that its latency (a shared-memory round trip that queues behind
    // the tensor pipe's operand reads, the TMA writes and the softmax warps' tensor-memory
    // traffic: about 200 clocks) passes while the issuing lane is held by the MMAs.
    if (warp == kQkWarp) {
      long long acc_a = 0, acc_c = 0;
      int sb = 0, kb = 0;   // S buffer of tile G = G mod 3, K stage = G mod 5
      uint32_t kph = 0;     // (G / 5) & 1
      uint32_t kd_lo[8];  // low words of the descriptors of K stage 0; the others differ in the address field only
#pragma unroll
      for (int kk = 0; kk < 8; ++kk)
        kd_lo[kk] = (uint32_t)smem_desc(ubase + kOffK + (kk >> 2) * kSubKV + (kk & 3) * 32, 16, 1024);
      const uint32_t kd_hi = (uint32_t)(smem_desc(0, 16, 1024) >> 32);
      bool ready = false;  // the barrier of the tile at hand was seen complete by the early test
      for (int it = 0; it < n_run && ok; ++it) {
        const int T = __shfl_sync(0xffffffffu, item_T[it], 0);
        const uint32_t q_tmem = utmem + kColQ + (uint32_t)(it & 1) * 64u;
        ok = mbar_wait(bar(QT_READY + (it & 1)), (it >> 1) & 1, abort_flag);
        for (int j = 0; j < T; ++j, ++G) {
          if (lane == 0) TSD_TR(2, G);
          const long long c0 = TSD_CLK();
          if (!ready) {
            ok = ok && mbar_wait(bar(QK_GO + kb), kph, abort_flag);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
          }
          tc_fence_after();
          if (lane == 0) TSD_TR(3, G);
          const long long c2 = TSD_CLK();
          const int kb1 = kb + 1 == kNK ? 0 : kb + 1;
          const uint32_t kph1 = kb1 == 0 ? kph ^ 1u : kph;
          const bool seen = mbar_test_wait(bar(QK_GO + kb1), kph1);  // used after the MMAs
          if (elect_one()) {
            const uint32_t k_off = (uint32_t)kb * (kKVBytes >> 4);
            uint32_t lo[8];
#pragma unroll
            for (int kk = 0; kk < 8; ++kk) lo[kk] = kd_lo[kk] + k_off;
            issue_qk_mmas(utmem + kColS + (uint32_t)sb * kKeys, q_tmem, lo, kd_hi, bar(S_FULL + sb), bar(K_FREE + kb));
          }
          __syncwarp();
          ready = seen;
          if (lane == 0) TSD_TR(4, G);
          sb = sb + 1 == kNSb ? 0 : sb + 1;
          kb = kb1; kph = kph1;
          const long long c3 = TSD_CLK();
          acc_a += c2 - c0; acc_c += c3 - c2;
        }
        ready = false;  // the first tile of an item also waits for its Q
      }
      if (lane == 0) { TSD_TR_SUM(0, 201, acc_a); TSD_TR_SUM(2, 201, acc_c); TSD_TR_SUM(3, 201, (long long)G); }
    } else {
      long long acc_a = 0, acc_c = 0;
      uint32_t vd_lo[kKeys / 16];
#pragma unroll
      for (int kk = 0; kk < kKeys / 16; ++kk) vd_lo[kk] = (uint32_t)smem_desc(ubase + kOffV + kk * 2048, kSubKV, 1024);
      const uint32_t vd_hi = (uint32_t)(smem_desc(0, kSubKV, 1024) >> 32);
      bool ready = false;
      for (int it = 0; it < n_run && ok; ++it) {
        const int T = __shfl_sync(0xffffffffu, item_T[it], 0);
        const int clen = __shfl_sync(0xffffffffu, item_clen[it], 0);
        const int n_ct = (clen + kKeys - 1) / kKeys;
        int s, h, qt;
        item_coords(it, s, h, qt);
        const int32_t* rec = mask + p.recs_off + (size_t)(s * p.n_qt + qt) * p.rec_words;
        const unsigned bits0 = (unsigned)__ldg(rec + 3);  // visibility of the first listed draft tile, asked for early
        // the first P V of an item overwrites O: the epilogue of the previous item must have read it
        if (it > 0) ok = mbar_wait(bar(O_FREE), (it - 1) & 1, abort_flag);
        for (int j = 0; j < T; ++j, ++G) {
          const int b = G & 3;  // V stage; P buffer = G & 1
          if (lane == 0) TSD_TR(5, G);
          const long long c0 = TSD_CLK();
          if (!ready) {
            ok = ok && mbar_wait(bar(PV_GO + b), (G >> 2) & 1, abort_flag);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
          }
          // A weight of exactly 0 is not enough where V holds Inf or NaN (0 x NaN = NaN): key rows that
          // no row of the query tile may read are zeroed in shared memory before the MMAs see them.
          // These are the cached rows past the sequence's cache length (whatever the caller left in the
          // unused capacity) and the rows of a draft tile's branches that the query tile cannot see.
          {
            int z0 = kKeys, z1 = kKeys;  // rows [z0, z1) to zero
            unsigned dead = 0;           // bit i: rows [32 i, 32 i + 32) to zero (draft tiles)
            if (j < n_ct) {
              if (j == n_ct - 1) z0 = clen - j * kKeys;  // 1..64 valid rows
            } else {
              const int e = j - n_ct;
              const unsigned bits = e < 2 ? bits0 : (unsigned)__ldg(rec + 3 + 2 * (e >> 1));  // bit qs*4+ks
              unsigned seen_slots = 0;
#pragma unroll
              for (int qs = 0; qs < 4; ++qs) seen_slots |= (bits >> (4 * qs)) & 15u;
#pragma unroll
              for (int w = 0; w < 2; ++w)
                if (!((seen_slots >> (((e & 1) * kKeys + w * 32) / p.R)) & 1u)) dead |= 1u << w;
            }
            if (z0 < z1 || dead) {
              const uint32_t v_stage = base + kOffV + (uint32_t)b * kKVBytes;
              if (dead) { z0 = (dead & 1u) ? 0 : 32; z1 = (dead & 2u) ? kKeys : 32; }
              // 16 chunks of 16 bytes per row (8 per sub-tile): whole rows, so the swizzle does not matter
              for (int idx = lane; idx < (z1 - z0) * 16; idx += 32) {
                const int row = z0 + (idx >> 4), ch = idx & 15;
                const uint32_t a = v_stage + (uint32_t)(ch >> 3) * kSubKV + (uint32_t)row * 128u + (uint32_t)(ch & 7) * 16u;
                asm volatile("st.shared.v4.u32 [%0], {%1, %1, %1, %1};" ::"r"(a), "r"(0u) : "memory");
              }
              fence_async_smem();  // the tensor pipe reads shared memory through the async proxy
              __syncwarp();
            }
          }
          tc_fence_after();
          if (lane == 0) TSD_TR(7, G);
          const long long c2 = TSD_CLK();
          const bool seen = mbar_test_wait(bar(PV_GO + ((G + 1) & 3)), ((G + 1) >> 2) & 1);  // used after the MMAs
          if (elect_one()) {
            const uint32_t v_off = (uint32_t)b * (kKVBytes >> 4);
            uint32_t lo[kKeys / 16];
#pragma unroll
            for (int kk = 0; kk < kKeys / 16; ++kk) lo[kk] = vd_lo[kk] + v_off;
            issue_pv_mmas(utmem + kColO, utmem + kColP + (uint32_t)(b & 1) * 32u, lo, vd_hi, j == 0 ? 0u : 1u, bar(PV_DONE + b));
          }
          __syncwarp();
          ready = seen;
          if (lane == 0) TSD_TR(8, G);
          const long long c3 = TSD_CLK();
          acc_a += c2 - c0; acc_c += c3 - c2;
        }
        ready = false;  // the first tile of an item also waits for O
      }
      if (lane == 0) { TSD_TR_SUM(4, 201, acc_a); TSD_TR_SUM(5, 201, acc_c); }
    }
  }
  } else if (warp < kFirstEpilogueWarp) {
    // ------------------------------------------------------------ softmax, one query row per thread
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kRegsSoftmax));
    const int wg = (warp - kFirstSoftmaxWarp) >> 2, wq = warp & 3;
    const int r = wq * 32 + lane;
    const uint32_t t_lane = tmem + ((uint32_t)(wq * 32) << 16);
    const int qs = r / p.R;
    const float c = p.scale_log2e;
    bool ok = true;
    // Q of item `it`: staging buffer -> tensor-memory buffer it & 1, as the A operand of Q K^T
    // (lane = row, 32-bit column i = elements 2i, 2i+1).  The caller knows that the Q K^T of item
    // it-2, which read this buffer last, are complete.
    auto copy_q = [&](int it) {
      ok = ok && mbar_wait(bar(QS_FULL), it & 1, abort_flag);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) return;
      copy_q_row(base + kOffQ, r, t_lane + kColQ + (uint32_t)(it & 1) * 64u);
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(QT_READY + (it & 1)));
    };
    if (wg == 0 && n_run > 0) copy_q(0);
    int n_tiles = 0;  // key tiles of all items of this block
    for (int i = lane; i < n_run; i += 32) n_tiles += item_T[i];
#pragma unroll
    for (int off = 16; off; off >>= 1) n_tiles += __shfl_xor_sync(0xffffffffu, n_tiles, off);

    int G = 0, n_done = 0;
    for (int it = 0; it < n_run && ok; ++it) {
      int s, h, qt;
      item_coords(it, s, h, qt);
      const int32_t* rec = mask + p.recs_off + (size_t)(s * p.n_qt + qt) * p.rec_words;
      const int clen = item_clen[it];
      const int n_ct = (clen + kKeys - 1) / kKeys, T = item_T[it];
      const int jc = min(4, T - 1);  // the tile at which Q of the next item is copied
      float m_mine = -CUDART_INF_F, l = 0.f;  // the exponent offset this thread used last, its partial row sum
      // tile t goes to warpgroup t mod 3, which is also its S buffer; n_done counts this
      // warpgroup's tiles, so the buffer's barriers are in phase n_done & 1
      for (int j = ((wg - G) % 3 + 3) % 3; j < T; j += 3, ++n_done) {
        const int Gj = G + j, pb = Gj & 1;
        const uint32_t ph = (uint32_t)n_done & 1u;
        if (wq == 0 && lane == 0) TSD_TR(9, Gj);
        ok = ok && mbar_wait(bar(S_FULL + wg), ph, abort_flag, TSD_SM_SLEEP);
        ok = __all_sync(0xffffffffu, ok);  // leave the loop as a whole warp
        if (!ok) break;
        tc_fence_after();
        if (wq == 0 && lane == 0) TSD_TR(10, Gj);
        // S of a tile of this item is complete, so every Q K^T of the previous item is, and the Q
        // buffer they read can take Q of the next item
        if (j == jc && it + 1 < n_run) { copy_q(it + 1); if (!ok) break; }
        const uint32_t t_s = t_lane + kColS + wg * kKeys;
        uint32_t sv[kKeys];
        TSD_TMEM_LD32(sv, 0, t_s);
        TSD_TMEM_LD32(sv, 32, t_s + 32);
        tmem_wait_ld();
        tc_fence_before();
        __syncwarp();
        // S is in registers: the buffer can take the Q K^T of the tile three ahead (if there is one)
        if (lane == 0 && Gj + kNSb < n_tiles) mbar_arrive(bar(QK_GO + (int)((unsigned)(Gj + kNSb) % (unsigned)kNK)));

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
#ifdef TSD_EXPERIMENT_NO_MAX  /* timing experiment only: wrong results */
        const float mx = __uint_as_float(sv[0]);
#else
        const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
#endif

        // the row's exponent offset: the decision of the previous tile, moved only when this tile's
        // maximum exceeds it by more than 2^8 (always for the first finite maximum)
        float m_prev = -CUDART_INF_F;
        if (wq == 0 && lane == 0) TSD_TR(11, Gj);
        if (Gj > 0) {
          // also for the first tile of an item, which takes nothing from the previous item: its
          // write below must not overtake that item's last read of the same word
          ok = ok && mbar_wait(bar(DEC + 4 * ((Gj - 1) & 3) + wq), ((Gj - 1) >> 2) & 1, abort_flag);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          if (j > 0) m_prev = mref[r];
        }
        const float m_new = fmaxf(m_prev, mx * c);
        const bool grow = m_new > m_prev + 8.f;
        const float m_use = grow ? m_new : m_prev;
        mref[r] = m_use;
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(DEC + 4 * (Gj & 3) + wq));
        if (wq == 0 && lane == 0) TSD_TR(12, Gj);
        const float alpha = grow ? ex2f(m_prev - m_new) : 1.f;  // what O has to be multiplied by
        if (m_mine != m_use) {
          l *= (m_mine == -CUDART_INF_F) ? 0.f : ex2f(m_mine - m_use);
          m_mine = m_use;
        }
        const float off = (m_use == -CUDART_INF_F) ? 0.f : -m_use;
        const uint64_t c2 = pack2f(c, c), off2 = pack2f(off, off);
        uint64_t rs4[4] = {0ull, 0ull, 0ull, 0ull};
        uint32_t pk[kKeys / 2];
        if (masked || kPolyOf8 == 0) {  // every exponential on the special-function unit: 2^(-inf) is exactly 0
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
        l += r0 + r1;
        if (wq == 0 && lane == 0) TSD_TR(13, Gj);

        if (j > 0 && __any_sync(0xffffffffu, alpha != 1.f)) {
          // rare: the exponent offset moved.  O must be at rest: wait for P V of tile j-1 (P V of
          // tile j cannot start before this thread publishes P_j), then rescale the row.
          ok = ok && mbar_wait(bar(PV_DONE + ((Gj - 1) & 3)), ((Gj - 1) >> 2) & 1, abort_flag);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          tc_fence_after();
          rescale_o_row(t_lane + kColO, alpha);
        }
        // P (bf16 pairs) into P buffer pb, free once the P V of tile t-2 has completed:
        // column i = keys 2i (low half), 2i+1
        if (Gj >= kNP) {
          ok = ok && mbar_wait(bar(PV_DONE + ((Gj - 2) & 3)), ((Gj - 2) >> 2) & 1, abort_flag);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          tc_fence_after();
        }
        TSD_TMEM_ST32(pk, 0, t_lane + kColP + pb * 32);
        tmem_wait_st();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(PV_GO + (Gj & 3)));
        if (wq == 0 && lane == 0) TSD_TR(14, Gj);
      }
      if (!ok) break;

      // ---- the item's partial row sum of this thread, and the offset it is on, go to the epilogue
      // warpgroup (three sets in rotation: a warpgroup that runs ahead writes the set of item it+3
      // only after a P of item it+1 or later, whose buffer needs a P V that follows the epilogue's read of O)
      lpart[(it % 3) * 384 + wg * kTile + r] = l;
      mpart[(it % 3) * 384 + wg * kTile + r] = m_mine;
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(LPART));
      G += T;
    }
  } else {
    // ------------------------------------------------------------ epilogue, one query row per thread
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kRegsEpilogue));
    // Per item: wait for the softmax warps' partial sums and for the last P V, read O (32 columns
    // at a time), O / l -> bf16 -> staging buffer -> TMA store.  O is released for the next item's
    // first P V as soon as its last columns are in registers.
    const int wq = warp & 3;
    const int r = wq * 32 + lane;
    const uint32_t t_lane = tmem + ((uint32_t)(wq * 32) << 16);
    bool ok = true;
    int G = 0;
    for (int it = 0; it < n_run && ok; ++it) {
      int s, h, qt;
      item_coords(it, s, h, qt);
      const int T = item_T[it], Gl = G + T - 1;
      if (tid == kFirstEpilogueWarp * 32) TSD_TR(5, 255 - it);
      ok = mbar_wait(bar(LPART), it & 1, abort_flag, 200);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      if (tid == kFirstEpilogueWarp * 32) TSD_TR(0, 255 - it);
      // the offsets only grow along the tiles, so the largest is the final one
      const float* lp = lpart + (it % 3) * 384 + r;
      const float* mp = mpart + (it % 3) * 384 + r;
      const float m0 = mp[0], m1 = mp[kTile], m2 = mp[2 * kTile];
      const float m_fin = fmaxf(m0, fmaxf(m1, m2));
      auto on_final = [&](float lg, float mg) { return mg == -CUDART_INF_F ? 0.f : lg * ex2f(mg - m_fin); };
      const float lt = (on_final(lp[0], m0) + on_final(lp[kTile], m1)) + on_final(lp[2 * kTile], m2);
      const float inv = lt > 0.f ? 1.f / lt : 0.f;
      // the previous item's store must have read the staging buffer before it is written again
      if (warp == kFirstEpilogueWarp && lane == 0) {
        asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
        mbar_arrive(bar(OS_FREE));
      }
      ok = mbar_wait(bar(OS_FREE), it & 1, abort_flag);
      // the softmax warps wrote the last P after the P V two tiles earlier had completed, so this
      // barrier is at most one phase behind the one waited for
      ok = ok && mbar_wait(bar(PV_DONE + (Gl & 3)), (Gl >> 2) & 1, abort_flag);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      if (tid == kFirstEpilogueWarp * 32) TSD_TR(1, 255 - it);
      // staging layout = the output tensor map's: 128-byte swizzle, 16-byte chunk c of row r sits at
      // chunk c ^ (r & 7); one sub-tile per half of head_dim; rows past the end of the tensor are
      // clipped by the copy engine
#pragma unroll
      for (int q4 = 0; q4 < 4; ++q4) {
        uint32_t ov[32];
        TSD_TMEM_LD32(ov, 0, t_lane + kColO + q4 * 32);
        tmem_wait_ld();
        if (q4 == 3) {
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(bar(O_FREE));
          if (tid == kFirstEpilogueWarp * 32) TSD_TR(2, 255 - it);
        }
        const uint32_t row_base = base + kOffO + (q4 >> 1) * kSub + (uint32_t)r * 128u;
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
      const int i_row = qt * kTile + r;
      if (p.lse && i_row < p.N) p.lse[((size_t)s * p.Hq + h) * p.N + i_row] = (m_fin + log2f(lt)) * kLn2;
      fence_async_smem();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(STAGED));
      if (tid == kFirstEpilogueWarp * 32) TSD_TR(3, 255 - it);
      if (warp == kFirstEpilogueWarp) {
        ok = mbar_wait(bar(STAGED), it & 1, abort_flag);
        ok = __all_sync(0xffffffffu, ok);
        if (ok && lane == 0) {
          tma_store_4d(&map_o, base + kOffO, 0, h, qt * kTile, s);
          tma_store_4d(&map_o, base + kOffO + kSub, 64, h, qt * kTile, s);
          asm volatile("cp.async.bulk.commit_group;" ::: "memory");
          TSD_TR(4, 255 - it);
        }
        __syncwarp();
        if (!ok) break;
      }
      G += T;
    }
    // the staging buffer must outlive the last store's reads
    if (warp == kFirstEpilogueWarp && lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
  }

  // ---------------------------------------------------------------- teardown (all threads)
  if (tid == 0) TSD_TR_ALWAYS(2, 200);
  tc_fence_before();
  __syncthreads();
  if (tid == 0) TSD_TR_ALWAYS(3, 200);
  if (warp == kQkWarp) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tmem) : "memory");
  }
  if (tid == 0 && *abort_flag && p.status) atomicOr(p.status, TSD_STATUS_TIMEOUT);
}

// The bounded wait of this file on a barrier that nothing ever completes: it gives up after
// `poll_limit` polls, the block notes it and returns by itself, as a block of the attention kernel
// does when one of its waits runs out.
__global__ void bounded_wait_selftest_kernel(uint32_t* status, uint32_t poll_limit) {
  __shared__ uint64_t bar_mem;
  __shared__ uint32_t abort_word;
  const uint32_t b = smem_u32(&bar_mem);
  if (threadIdx.x == 0) {
    abort_word = 0;
    mbar_init(b, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  const bool ok = mbar_wait(b, 0, &abort_word, 0, poll_limit);
  __syncthreads();
  if (threadIdx.x == 0 && (!ok || abort_word) && status) atomicOr(status, TSD_STATUS_TIMEOUT);
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

struct DeviceFacts {
  int state;  // 0 = unknown, 1 = sm_100 family, 2 = something else
  int sms;
};
static DeviceFacts device_facts() {
  static std::mutex mu;
  static DeviceFacts cached[kMaxDevices];
  const int dev = current_device();
  if (dev < 0) return DeviceFacts{2, 0};
  std::lock_guard<std::mutex> lock(mu);
  if (cached[dev].state == 0) {
    int major = 0, sms = 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
      return DeviceFacts{2, 0};
    cached[dev].state = major == 10 ? 1 : 2;
    cached[dev].sms = sms;
  }
  return cached[dev];
}

bool attention_tc_supported(const AttnArgs& a) {
  return a.L.dtype == TSD_BF16 && a.L.head_dim == 128 && a.sm_scale > 0.f && device_facts().state == 1;
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
  const MaskDims md = mask_dims(L);
  const int64_t n_items = (int64_t)L.batch * L.n_q_heads * md.n_qt;
  if (!ok || n_items > 0x7fffffffLL / 4) return launch_attention_simt(a);  // strides the tensor maps cannot express
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
  p.lse = a.lse;
  p.status = a.status;
  p.S = L.batch; p.B = L.n_branches; p.R = L.rows_per_branch; p.Nc = L.n_cache; p.N = N;
  p.Hq = L.n_q_heads; p.group = L.n_q_heads / L.n_kv_heads;
  p.recs_off = md.recs_off; p.n_qt = md.n_qt; p.rec_words = md.rec_words;
  p.n_items = (int)n_items;
  p.scale_log2e = a.sm_scale * kLog2e;
  // one block per SM, each walking its share of the items; more blocks only when a block's share
  // would not fit the per-block item table
  const int sms = std::max(device_facts().sms, 1);
  int64_t grid = std::min<int64_t>(n_items, sms);
  grid = std::max<int64_t>(grid, (n_items + kMaxItems - 1) / kMaxItems);
  attention_tc_kernel<<<(unsigned)grid, kTcThreads, kSmemBytes, a.stream>>>(mq, mkc, mvc, mkd, mvd, mo, p);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(e, "attention_tc_kernel");
  return TSD_OK;
}

}  // namespace tsd

#ifdef TSD_ATTN_TRACE
extern "C" int tsd_attention_trace_read(long long* dst) {
  return (int)cudaMemcpyFromSymbol(dst, tsd::g_attn_trace, sizeof(tsd::g_attn_trace));
}
#endif

extern "C" int tsd_selftest_bounded_wait(uint32_t* status, uint32_t poll_limit, tsd_stream_t stream) {
  if (!status || poll_limit < 1 || poll_limit > (1u << 16)) return TSD_ERR_INVALID_ARG;
  tsd::bounded_wait_selftest_kernel<<<1, 32, 0, stream>>>(status, poll_limit);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return tsd::cuda_fail(e, "bounded_wait_selftest_kernel");
  return TSD_OK;
}

