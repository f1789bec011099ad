// Stage 1a: branch-isolation mask (paper Section 3.3).  Builds the compact per-query-tile
// visibility lists the attention kernels read, and optionally the dense boolean mask.
#include <algorithm>
#include "tsd_common.cuh"

namespace tsd {

__device__ __forceinline__ bool branch_sees(const uint64_t* vis, int s, int B, int words, int bq, int bk) {
  if (bq == bk) return true;  // bidirectional inside the own block
  if (!vis) return false;     // competing branches are mutually invisible
  return (vis[((size_t)s * B + bq) * words + (bk >> 6)] >> (bk & 63)) & 1ull;
}

__global__ void build_mask_kernel(int S, int B, int R, int Nc, int n_qt, int rec_words, int lens_off,
                                  int recs_off, const uint64_t* __restrict__ vis,
                                  const int32_t* __restrict__ cache_lens, int32_t* __restrict__ blob) {
  const int t = blockIdx.x * blockDim.x + threadIdx.x;
  if (t == 0) {
    blob[H_MAGIC] = kMaskMagic; blob[H_S] = S; blob[H_B] = B; blob[H_R] = R; blob[H_NC] = Nc;
    blob[H_NQT] = n_qt; blob[H_REC_WORDS] = rec_words; blob[H_RECS_OFF] = recs_off;
  }
  if (t < S) {
    int len = cache_lens ? cache_lens[t] : Nc;
    blob[lens_off + t] = min(max(len, 0), Nc);
  }
  if (t >= S * n_qt) return;
  const int s = t / n_qt, qt = t % n_qt;
  const int slots = kTile / R, words = (B + 63) / 64;
  int32_t* rec = blob + recs_off + (size_t)t * rec_words;
  int count = 0;
  for (int kt = 0; kt < n_qt; ++kt) {
    int bits = 0;
    for (int qs = 0; qs < slots; ++qs) {
      const int bq = qt * slots + qs;
      if (bq >= B) break;
      for (int ks = 0; ks < slots; ++ks) {
        const int bk = kt * slots + ks;
        if (bk >= B) break;
        if (branch_sees(vis, s, B, words, bq, bk)) bits |= 1 << (qs * 4 + ks);
      }
    }
    if (bits) { rec[2 + 2 * count] = kt; rec[3 + 2 * count] = bits; ++count; }
  }
  rec[0] = count;
  rec[1] = 0;
}

__global__ void dense_mask_kernel(int S, int B, int R, int Nc, const uint64_t* __restrict__ vis,
                                  const int32_t* __restrict__ cache_lens, uint8_t* __restrict__ dense) {
  const int N = B * R, words = (B + 63) / 64;
  const int64_t L = (int64_t)Nc + N, total = (int64_t)S * N * L;
  for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < total;
       t += (int64_t)gridDim.x * blockDim.x) {
    const int64_t j = t % L;
    const int i = (int)((t / L) % N), s = (int)(t / (L * N));
    bool v;
    if (j < Nc) {
      int len = cache_lens ? cache_lens[s] : Nc;
      v = j < min(max(len, 0), Nc);
    } else {
      v = branch_sees(vis, s, B, words, i / R, (int)(j - Nc) / R);
    }
    dense[t] = v ? 1 : 0;
  }
}

}  // namespace tsd

extern "C" {

size_t tsd_branch_mask_bytes(const tsd_layout* L) {
  if (tsd::validate_layout(L) != TSD_OK) return 0;
  return tsd::mask_dims(*L).bytes;
}

int tsd_build_branch_mask(const tsd_layout* L, const uint64_t* vis, const int32_t* cache_lens,
                          void* mask_out, size_t mask_bytes, uint8_t* dense_out, tsd_stream_t stream) {
  int rc = tsd::validate_layout(L);
  if (rc != TSD_OK) return rc;
  if (!mask_out || !tsd::aligned16(mask_out)) return TSD_ERR_INVALID_ARG;
  if (vis && (reinterpret_cast<uintptr_t>(vis) & 7u)) return TSD_ERR_INVALID_ARG;
  if (cache_lens && (reinterpret_cast<uintptr_t>(cache_lens) & 3u)) return TSD_ERR_INVALID_ARG;
  const tsd::MaskDims m = tsd::mask_dims(*L);
  if (mask_bytes < m.bytes) return TSD_ERR_WORKSPACE;
  const int threads = 128;
  const int work = max(L->batch * m.n_qt, L->batch);
  tsd::build_mask_kernel<<<(work + threads - 1) / threads, threads, 0, stream>>>(
      L->batch, L->n_branches, L->rows_per_branch, L->n_cache, m.n_qt, m.rec_words, m.lens_off,
      m.recs_off, vis, cache_lens, static_cast<int32_t*>(mask_out));
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return tsd::cuda_fail(e, "build_mask_kernel");
  if (dense_out) {
    const int64_t N = (int64_t)L->n_branches * L->rows_per_branch;
    const int64_t total = (int64_t)L->batch * N * (L->n_cache + N);
    const int blocks = (int)std::min<int64_t>((total + 255) / 256, 148 * 16);
    tsd::dense_mask_kernel<<<blocks, 256, 0, stream>>>(L->batch, L->n_branches, L->rows_per_branch,
                                                       L->n_cache, vis, cache_lens, dense_out);
    e = cudaGetLastError();
    if (e != cudaSuccess) return tsd::cuda_fail(e, "dense_mask_kernel");
  }
  return TSD_OK;
}

}  // extern "C"
