// Stage 1b entry point: argument checks and the choice between the tensor-core kernel
// (bf16, head_dim 128) and the CUDA-core kernel (everything else).
#include "tsd_common.cuh"

namespace tsd {

// Every host-side check of the attention call, shared by the entry points that end in it: a call
// that is going to be rejected must be rejected before anything has been launched.
int check_attention_args(const tsd_layout* L, const void* mask, const void* q, int64_t q_stride_b,
                         int64_t q_stride_row, int64_t q_stride_head, const void* k_cache, const void* v_cache,
                         int64_t c_stride_b, int64_t c_stride_row, int64_t c_stride_head, const void* k_draft,
                         const void* v_draft, int64_t d_stride_b, int64_t d_stride_row, int64_t d_stride_head,
                         const void* out, int64_t o_stride_b, int64_t o_stride_row, int64_t o_stride_head,
                         float sm_scale, const void* workspace) {
  int rc = validate_layout(L);
  if (rc != TSD_OK) return rc;
  if (!mask || !q || !k_draft || !v_draft || !out) return TSD_ERR_INVALID_ARG;
  if (L->n_cache > 0 && (!k_cache || !v_cache)) return TSD_ERR_INVALID_ARG;
  if (!(sm_scale == sm_scale)) return TSD_ERR_INVALID_ARG;
  const void* ptrs[] = {mask, q, k_cache, v_cache, k_draft, v_draft, out, workspace};
  for (const void* p : ptrs)
    if (p && !aligned16(p)) return TSD_ERR_INVALID_ARG;
  const int esize = L->dtype == TSD_F32 ? 4 : 2;
  const int64_t strides[] = {q_stride_b, q_stride_row, q_stride_head, c_stride_b, c_stride_row,
                             c_stride_head, d_stride_b, d_stride_row, d_stride_head, o_stride_b,
                             o_stride_row, o_stride_head};
  for (int64_t st : strides)
    if (st < 0 || (st * esize) % 16 != 0) return TSD_ERR_INVALID_ARG;
  if (q_stride_head < L->head_dim || c_stride_head < L->head_dim || d_stride_head < L->head_dim ||
      o_stride_head < L->head_dim)
    return TSD_ERR_INVALID_ARG;
  return TSD_OK;
}

}  // namespace tsd

extern "C" {

size_t tsd_verify_attention_workspace_bytes(const tsd_layout* L) {
  if (tsd::validate_layout(L) != TSD_OK) return 0;
  return tsd::attention_tc_workspace_bytes(*L);
}

int tsd_verify_attention(const tsd_layout* L, const void* mask, const void* q, int64_t q_stride_b,
                         int64_t q_stride_row, int64_t q_stride_head, const void* k_cache,
                         const void* v_cache, int64_t c_stride_b, int64_t c_stride_row,
                         int64_t c_stride_head, const void* k_draft, const void* v_draft,
                         int64_t d_stride_b, int64_t d_stride_row, int64_t d_stride_head, void* out,
                         int64_t o_stride_b, int64_t o_stride_row, int64_t o_stride_head, float* lse,
                         float sm_scale, void* workspace, size_t workspace_bytes, uint32_t flags,
                         uint32_t* status, tsd_stream_t stream) {
  int rc = tsd::check_attention_args(L, mask, q, q_stride_b, q_stride_row, q_stride_head, k_cache, v_cache,
                                     c_stride_b, c_stride_row, c_stride_head, k_draft, v_draft, d_stride_b,
                                     d_stride_row, d_stride_head, out, o_stride_b, o_stride_row, o_stride_head,
                                     sm_scale, workspace);
  if (rc != TSD_OK) return rc;

  tsd::AttnArgs a;
  a.L = *L;
  a.mask = static_cast<const int32_t*>(mask);
  a.q = q; a.kc = k_cache; a.vc = v_cache; a.kd = k_draft; a.vd = v_draft; a.out = out; a.lse = lse;
  a.qs_b = q_stride_b; a.qs_r = q_stride_row; a.qs_h = q_stride_head;
  a.cs_b = c_stride_b; a.cs_r = c_stride_row; a.cs_h = c_stride_head;
  a.ds_b = d_stride_b; a.ds_r = d_stride_row; a.ds_h = d_stride_head;
  a.os_b = o_stride_b; a.os_r = o_stride_row; a.os_h = o_stride_head;
  a.sm_scale = sm_scale;
  a.workspace = workspace;
  a.workspace_bytes = workspace_bytes;
  a.status = status;
  a.stream = stream;
  if (!(flags & TSD_ATTN_FORCE_SIMT) && tsd::attention_tc_supported(a)) {
    if (workspace_bytes < tsd::attention_tc_workspace_bytes(*L)) return TSD_ERR_WORKSPACE;
    return tsd::launch_attention_tc(a);
  }
  return tsd::launch_attention_simt(a);
}

}  // extern "C"
