// Stage 1b on CUDA cores: masked verify attention (paper Section 3.3) for the combinations the
// tensor-core kernel does not serve (fp32 inputs, head_dim 64) and as a cross-check for it.
//
// One thread block per (sequence, query head, branch).  A warp owns a query row at a time; its
// lanes stride over the visible keys (the cached tokens, then the rows of every visible draft
// branch), each lane keeping an online-softmax state (max, sum, weighted value row) in fp32
// registers; the 32 lane states are merged once per row.
#include <limits.h>
#include <math_constants.h>
#include "tsd_common.cuh"

namespace tsd {

constexpr int kSimtWarps = 4;

template <typename T, int D>
__global__ void __launch_bounds__(kSimtWarps * 32)
attention_simt_kernel(int S, int B, int R, int Nc, int Hq, int Hkv, const int32_t* __restrict__ mask,
                      const T* __restrict__ q, const T* __restrict__ kc, const T* __restrict__ vc,
                      const T* __restrict__ kd, const T* __restrict__ vd, T* __restrict__ out,
                      float* __restrict__ lse, int64_t qs_b, int64_t qs_r, int64_t qs_h, int64_t cs_b,
                      int64_t cs_r, int64_t cs_h, int64_t ds_b, int64_t ds_r, int64_t ds_h,
                      int64_t os_b, int64_t os_r, int64_t os_h, float sm_scale,
                      uint32_t* __restrict__ status) {
  __shared__ int s_vis[256];                // visible draft branches of this branch
  __shared__ int s_nvis;
  __shared__ float s_q[kSimtWarps][D];      // the warp's current query row, pre-scaled
  const int b = blockIdx.x, h = blockIdx.y, s = blockIdx.z;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int g = h / (Hq / Hkv);
  const int N = B * R;

  const bool hdr_ok = mask[H_MAGIC] == kMaskMagic && mask[H_S] == S && mask[H_B] == B &&
                      mask[H_R] == R && mask[H_NC] == Nc;
  if (!hdr_ok) {  // a blob built for another layout: report, write nothing
    if (threadIdx.x == 0 && status) atomicOr(status, TSD_STATUS_BAD_MASK);
    return;
  }
  const int n_qt = mask[H_NQT], rec_words = mask[H_REC_WORDS], recs_off = mask[H_RECS_OFF];
  const int clen = mask[kHdrWords + s];
  const int slots = kTile / R;
  if (threadIdx.x == 0) {
    const int32_t* rec = mask + recs_off + (size_t)(s * n_qt + b / slots) * rec_words;
    const int qs = b % slots;
    int n = 0;
    for (int e = 0; e < rec[0]; ++e) {
      const int kt = rec[2 + 2 * e], bits = rec[3 + 2 * e];
      for (int ks = 0; ks < slots; ++ks)
        if ((bits >> (qs * 4 + ks)) & 1) s_vis[n++] = kt * slots + ks;
    }
    s_nvis = n;
  }
  __syncthreads();
  const int n_keys = clen + s_nvis * R;
  const unsigned full = 0xffffffffu;
  constexpr int VEC = 16 / sizeof(T);  // elements per 16-byte load

  for (int r = warp; r < R; r += kSimtWarps) {
    const int i = b * R + r;
    const T* qp = q + s * qs_b + (int64_t)i * qs_r + h * qs_h;
    __syncwarp();
    for (int c = lane; c < D; c += 32) s_q[warp][c] = to_float(qp[c]) * sm_scale;
    __syncwarp();
    float m = -CUDART_INF_F, l = 0.f;
    float acc[D];
#pragma unroll
    for (int c = 0; c < D; ++c) acc[c] = 0.f;
    for (int j = lane; j < n_keys; j += 32) {
      const T *kp, *vp;
      if (j < clen) {
        kp = kc + s * cs_b + (int64_t)j * cs_r + g * cs_h;
        vp = vc + s * cs_b + (int64_t)j * cs_r + g * cs_h;
      } else {
        const int jj = j - clen;
        const int row = s_vis[jj / R] * R + jj % R;
        kp = kd + s * ds_b + (int64_t)row * ds_r + g * ds_h;
        vp = vd + s * ds_b + (int64_t)row * ds_r + g * ds_h;
      }
      float a = 0.f;
#pragma unroll
      for (int c0 = 0; c0 < D; c0 += VEC) {
        const uint4 w = *reinterpret_cast<const uint4*>(kp + c0);
        const T* e = reinterpret_cast<const T*>(&w);
#pragma unroll
        for (int u = 0; u < VEC; ++u) a = fmaf(s_q[warp][c0 + u], to_float(e[u]), a);
      }
      if (a > m) {
        const float f = expf(m - a);  // exp(-inf) = 0 on the first key
        l *= f;
#pragma unroll
        for (int c = 0; c < D; ++c) acc[c] *= f;
        m = a;
      }
      const float p = expf(a - m);
      l += p;
#pragma unroll
      for (int c0 = 0; c0 < D; c0 += VEC) {
        const uint4 w = *reinterpret_cast<const uint4*>(vp + c0);
        const T* e = reinterpret_cast<const T*>(&w);
#pragma unroll
        for (int u = 0; u < VEC; ++u) acc[c0 + u] = fmaf(p, to_float(e[u]), acc[c0 + u]);
      }
    }
    // merge the 32 lane states
    float M = m;
#pragma unroll
    for (int off = 16; off; off >>= 1) M = fmaxf(M, __shfl_xor_sync(full, M, off));
    const float f = (m == -CUDART_INF_F) ? 0.f : expf(m - M);
    float lt = l * f;
#pragma unroll
    for (int off = 16; off; off >>= 1) lt += __shfl_xor_sync(full, lt, off);
    const float inv = 1.f / lt;
    float mine[D / 32];
#pragma unroll
    for (int c = 0; c < D; ++c) {
      float v = acc[c] * f;
#pragma unroll
      for (int off = 16; off; off >>= 1) v += __shfl_xor_sync(full, v, off);
      if (lane == (c & 31)) mine[c >> 5] = v * inv;
    }
    T* op = out + s * os_b + (int64_t)i * os_r + h * os_h;
#pragma unroll
    for (int t = 0; t < D / 32; ++t) from_float(op[t * 32 + lane], mine[t]);
    if (lse && lane == 0) lse[((size_t)s * Hq + h) * N + i] = M + logf(lt);
  }
}

template <typename T, int D>
static cudaError_t launch_simt(const AttnArgs& a) {
  const tsd_layout& L = a.L;
  dim3 grid(L.n_branches, L.n_q_heads, L.batch);
  attention_simt_kernel<T, D><<<grid, kSimtWarps * 32, 0, a.stream>>>(
      L.batch, L.n_branches, L.rows_per_branch, L.n_cache, L.n_q_heads, L.n_kv_heads, a.mask,
      static_cast<const T*>(a.q), static_cast<const T*>(a.kc), static_cast<const T*>(a.vc),
      static_cast<const T*>(a.kd), static_cast<const T*>(a.vd), static_cast<T*>(a.out), a.lse, a.qs_b,
      a.qs_r, a.qs_h, a.cs_b, a.cs_r, a.cs_h, a.ds_b, a.ds_r, a.ds_h, a.os_b, a.os_r, a.os_h,
      a.sm_scale, a.status);
  return cudaGetLastError();
}

int launch_attention_simt(const AttnArgs& a) {
  cudaError_t e;
  const bool f32 = a.L.dtype == TSD_F32;
  if (a.L.head_dim == 64) e = f32 ? launch_simt<float, 64>(a) : launch_simt<__nv_bfloat16, 64>(a);
  else e = f32 ? launch_simt<float, 128>(a) : launch_simt<__nv_bfloat16, 128>(a);
  if (e != cudaSuccess) return cuda_fail(e, "attention_simt_kernel");
  return TSD_OK;
}

}  // namespace tsd
