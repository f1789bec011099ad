// Verify attention over an 8-bit K/V cache.  The paper keeps the dual cache in the model's dtype
// (Section 3.3, App. A); storing it as e4m3 halves its footprint, which is what bounds how many
// sequences a GPU can hold.  A cached value is bf16(decode_e4m3(code) * scale[sequence, kv head])
// (the product and the rounding in fp32 -> bf16).  The cache is expanded into the caller's
// workspace by one streaming launch for both caches (16 codes in, 32 bytes out per thread; grid
// y = sequence, z = K or V, so that the indices stay 32-bit) and the attention kernels then run
// unchanged on the expanded copy; the workspace is transient and can be shared by all layers, the
// persistent cache stays 8-bit.
#include <cuda_fp8.h>
#include "tsd_common.cuh"

namespace tsd {

__global__ void __launch_bounds__(256)
dequant_e4m3_kernel(const uint8_t* __restrict__ k_src, const uint8_t* __restrict__ v_src, int64_t ss_b, int64_t ss_r,
                    int64_t ss_h, const float* __restrict__ k_scale, const float* __restrict__ v_scale,
                    const int32_t* __restrict__ mask_blob, __nv_bfloat16* __restrict__ k_dst,
                    __nv_bfloat16* __restrict__ v_dst, int Nc, int H, int d, uint32_t vec_per_seq) {
  const uint32_t v = blockIdx.x * blockDim.x + threadIdx.x;  // one vector = 16 consecutive codes of sequence s
  if (v >= vec_per_seq) return;
  const uint32_t vec_per_head = (uint32_t)d / 16u, vec_per_row = vec_per_head * (uint32_t)H;
  const uint32_t row = v / vec_per_row, cv = v - row * vec_per_row;
  const uint32_t h = cv / vec_per_head, c = cv - h * vec_per_head;
  const int64_t s = blockIdx.y;
  const bool is_v = blockIdx.z != 0;
  const uint8_t* src = is_v ? v_src : k_src;
  const float* scale = is_v ? v_scale : k_scale;
  __nv_bfloat16* dst = is_v ? v_dst : k_dst;
  uint4* o = reinterpret_cast<uint4*>(dst + (((s * Nc + row) * H + h) * (int64_t)d + c * 16));
  // rows at or past the sequence's cache length (from the mask blob) hold whatever the caller left
  // there, the NaN codes 0x7f / 0xff included: they are written as zeros and never decoded
  if ((int)row >= min(max(mask_blob[kHdrWords + s], 0), Nc)) {
    o[0] = make_uint4(0u, 0u, 0u, 0u);
    o[1] = make_uint4(0u, 0u, 0u, 0u);
    return;
  }
  const uint4 w = *reinterpret_cast<const uint4*>(src + s * ss_b + row * ss_r + h * ss_h + c * 16);
  const float sc = scale ? scale[s * H + h] : 1.f;
  const uint32_t words[4] = {w.x, w.y, w.z, w.w};
  uint32_t out[8];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
#pragma unroll
    for (int j = 0; j < 2; ++j) {
      const __nv_fp8x2_storage_t pair = (__nv_fp8x2_storage_t)((words[i] >> (16 * j)) & 0xffffu);
      const __half2 hv = __half2(__nv_cvt_fp8x2_to_halfraw2(pair, __NV_E4M3));  // exact: e4m3 is a subset of fp16
      const float2 f = __half22float2(hv);
      const __nv_bfloat162 b = __floats2bfloat162_rn(f.x * sc, f.y * sc);
      out[2 * i + j] = *reinterpret_cast<const uint32_t*>(&b);
    }
  }
  o[0] = make_uint4(out[0], out[1], out[2], out[3]);
  o[1] = make_uint4(out[4], out[5], out[6], out[7]);
}

static size_t expanded_bytes(const tsd_layout& L) {
  return (size_t)L.batch * L.n_cache * L.n_kv_heads * L.head_dim * 2;
}

}  // namespace tsd

extern "C" size_t tsd_verify_attention_fp8_cache_workspace_bytes(const tsd_layout* L) {
  if (tsd::validate_layout(L) != TSD_OK) return 0;
  const size_t inner = (tsd_verify_attention_workspace_bytes(L) + 255) / 256 * 256;
  return inner + 2 * tsd::expanded_bytes(*L);
}

extern "C" int tsd_verify_attention_fp8_cache(
    const tsd_layout* L, const void* mask, const void* q, int64_t q_stride_b, int64_t q_stride_row,
    int64_t q_stride_head, const uint8_t* k_cache_e4m3, const uint8_t* v_cache_e4m3, int64_t c_stride_b,
    int64_t c_stride_row, int64_t c_stride_head, const float* k_scale, const float* v_scale, const void* k_draft,
    const void* v_draft, int64_t d_stride_b, int64_t d_stride_row, int64_t d_stride_head, void* out,
    int64_t o_stride_b, int64_t o_stride_row, int64_t o_stride_head, float* lse, float sm_scale, void* workspace,
    size_t workspace_bytes, uint32_t flags, uint32_t* status, tsd_stream_t stream) {
  int rc = tsd::validate_layout(L);
  if (rc != TSD_OK) return rc;
  if (L->dtype != TSD_BF16) return TSD_ERR_UNSUPPORTED;
  if (L->n_cache > 0 && !workspace) return TSD_ERR_INVALID_ARG;
  if (workspace_bytes < tsd_verify_attention_fp8_cache_workspace_bytes(L)) return TSD_ERR_WORKSPACE;
  const size_t inner = (tsd_verify_attention_workspace_bytes(L) + 255) / 256 * 256;
  const size_t half = tsd::expanded_bytes(*L);
  char* ws = static_cast<char*>(workspace);
  const int64_t hs = L->head_dim, rs = (int64_t)L->n_kv_heads * hs, bs = (int64_t)L->n_cache * rs;
  // every check of the attention call that follows, before the first launch: a rejected call launches nothing
  rc = tsd::check_attention_args(L, mask, q, q_stride_b, q_stride_row, q_stride_head,
                                 L->n_cache > 0 ? ws + inner : nullptr, L->n_cache > 0 ? ws + inner + half : nullptr,
                                 bs, rs, hs, k_draft, v_draft, d_stride_b, d_stride_row, d_stride_head, out,
                                 o_stride_b, o_stride_row, o_stride_head, sm_scale, inner ? workspace : nullptr);
  if (rc != TSD_OK) return rc;
  if (L->n_cache > 0) {
    if (!k_cache_e4m3 || !v_cache_e4m3 || !workspace || !tsd::aligned16(workspace) || !tsd::aligned16(k_cache_e4m3) ||
        !tsd::aligned16(v_cache_e4m3))
      return TSD_ERR_INVALID_ARG;
    if (c_stride_b < 0 || c_stride_row < 0 || c_stride_head < L->head_dim || c_stride_b % 16 || c_stride_row % 16 ||
        c_stride_head % 16)
      return TSD_ERR_INVALID_ARG;
    const int64_t vec_per_seq = (int64_t)L->n_cache * L->n_kv_heads * (L->head_dim / 16);
    if (vec_per_seq > 0x7fffff00ll || L->batch > 65535) return TSD_ERR_UNSUPPORTED;  // 32-bit indices, grid y
    const dim3 grid((unsigned)((vec_per_seq + 255) / 256), (unsigned)L->batch, 2);
    tsd::dequant_e4m3_kernel<<<grid, 256, 0, stream>>>(
        k_cache_e4m3, v_cache_e4m3, c_stride_b, c_stride_row, c_stride_head, k_scale, v_scale,
        static_cast<const int32_t*>(mask), reinterpret_cast<__nv_bfloat16*>(ws + inner),
        reinterpret_cast<__nv_bfloat16*>(ws + inner + half), L->n_cache, L->n_kv_heads, L->head_dim,
        (uint32_t)vec_per_seq);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return tsd::cuda_fail(e, "dequant_e4m3_kernel");
  }
  return tsd_verify_attention(L, mask, q, q_stride_b, q_stride_row, q_stride_head,
                              L->n_cache > 0 ? ws + inner : nullptr, L->n_cache > 0 ? ws + inner + half : nullptr, bs, rs,
                              hs, k_draft, v_draft, d_stride_b, d_stride_row, d_stride_head, out, o_stride_b,
                              o_stride_row, o_stride_head, lse, sm_scale, inner ? workspace : nullptr, inner, flags,
                              status, stream);
}
