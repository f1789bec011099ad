// Host-side utilities of the C ABI: error text, status decoding, layout checks.
#include <stdio.h>
#include <string.h>
#include "tsd_common.cuh"

namespace tsd {

static thread_local char g_last_cuda_error[256] = "";

int cuda_fail(cudaError_t e, const char* where) {
  snprintf(g_last_cuda_error, sizeof(g_last_cuda_error), "%s: %s (%s)", where,
           cudaGetErrorName(e), cudaGetErrorString(e));
  return TSD_ERR_CUDA;
}

int validate_layout(const tsd_layout* L) {
  if (!L) return TSD_ERR_INVALID_ARG;
  if (L->batch < 1 || L->n_branches < 1 || L->n_branches > 256 || L->n_cache < 0 ||
      L->n_q_heads < 1 || L->n_kv_heads < 1 || L->n_q_heads % L->n_kv_heads != 0)
    return TSD_ERR_INVALID_ARG;
  if (L->rows_per_branch != 32 && L->rows_per_branch != 64 && L->rows_per_branch != 128)
    return TSD_ERR_UNSUPPORTED;
  if (L->head_dim != 64 && L->head_dim != 128) return TSD_ERR_UNSUPPORTED;
  if (L->dtype != TSD_F32 && L->dtype != TSD_BF16) return TSD_ERR_UNSUPPORTED;
  return TSD_OK;
}

}  // namespace tsd

extern "C" {

const char* tsd_strerror(int err) {
  switch (err) {
    case TSD_OK: return "ok";
    case TSD_ERR_INVALID_ARG: return "invalid argument";
    case TSD_ERR_UNSUPPORTED: return "unsupported dtype or shape";
    case TSD_ERR_WORKSPACE: return "caller-provided buffer too small";
    case TSD_ERR_CUDA: return "CUDA runtime error";
    case TSD_ERR_TIMEOUT: return "bounded device wait expired";
    case TSD_ERR_DEVICE_DATA: return "inconsistent device data";
    default: return "unknown error";
  }
}

const char* tsd_last_cuda_error(void) { return tsd::g_last_cuda_error; }

int tsd_check_status(uint32_t w) {
  if (w & TSD_STATUS_TIMEOUT) return TSD_ERR_TIMEOUT;
  if (w & (TSD_STATUS_BAD_PARENT | TSD_STATUS_BAD_MASK | TSD_STATUS_BAD_INDEX)) return TSD_ERR_DEVICE_DATA;
  return TSD_OK;
}

}  // extern "C"
