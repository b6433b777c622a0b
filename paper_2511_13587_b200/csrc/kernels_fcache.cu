// Token-level feature cache (paper Sec. 4.3; Alg. 2 lines 5 and 11): scatter of verified
// features into a per-sequence ring addressed by absolute position, gather of the most recent
// ones for verification-free steps.  Pure data movement with 128-bit accesses; the index
// arithmetic is integer and must match the oracle exactly.
#include "vvs_internal.cuh"

namespace vvs {

__global__ void fcache_reset_kernel(int32_t* fpos, int32_t* newest, int n_slots, int n_rows) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n_slots) fpos[i] = -1;
  if (i < n_rows) newest[i] = -1;
}

void launch_fcache_reset(const vvs_fcache& fc, cudaStream_t s) {
  int n = fc.n_rows * fc.cap;
  fcache_reset_kernel<<<(n + 255) / 256, 256, 0, s>>>(fc.fpos, fc.newest, n, fc.n_rows);
}

// grid (rows_per_seq, n_rows): block (t, r) copies hidden[r, t, :] to the slot of base_pos[r] + t
__global__ void fcache_store_kernel(uint4* __restrict__ feat, int32_t* __restrict__ fpos,
                                    int32_t* __restrict__ newest, const uint4* __restrict__ hidden,
                                    int rows_per_seq, int cap, int row_vecs,
                                    const int32_t* __restrict__ base_pos,
                                    const int32_t* __restrict__ n_store, int32_t* status) {
  int t = blockIdx.x, r = blockIdx.y;
  int n = n_store[r], base = base_pos[r];
  if (n < 0 || n > rows_per_seq || n > cap || base < 0) {
    if (t == 0 && threadIdx.x == 0) atomicOr(status, VVS_DEV_BAD_ARG);
    return;
  }
  if (t >= n) return;
  int pos = base + t;
  int slot = pos % cap;
  const uint4* src = hidden + ((size_t)r * rows_per_seq + t) * row_vecs;
  uint4* dst = feat + ((size_t)r * cap + slot) * row_vecs;
  for (int i = threadIdx.x; i < row_vecs; i += blockDim.x) dst[i] = src[i];
  if (threadIdx.x == 0) {
    fpos[(size_t)r * cap + slot] = pos;
    if (t == n - 1) newest[r] = max(newest[r], pos);  // single writer per sequence
  }
}

void launch_fcache_store(const vvs_fcache& fc, const void* hidden, int rows_per_seq, int d,
                         int elem_bytes, const int32_t* base_pos, const int32_t* n_store,
                         int32_t* status, cudaStream_t s) {
  dim3 grid(rows_per_seq, fc.n_rows);
  fcache_store_kernel<<<grid, 128, 0, s>>>((uint4*)fc.feat, fc.fpos, fc.newest, (const uint4*)hidden,
                                           rows_per_seq, fc.cap, d * elem_bytes / 16, base_pos,
                                           n_store, status);
}

// grid (gamma_max, n_rows): block (j, r) gathers position newest - staleness - gamma + 1 + j
__global__ void fcache_fetch_kernel(const uint4* __restrict__ feat, const int32_t* __restrict__ fpos,
                                    const int32_t* __restrict__ newest,
                                    const uint8_t* __restrict__ skip_mask, int n_images,
                                    const int32_t* __restrict__ gamma, int gamma_max, int staleness,
                                    int cap, int row_vecs, uint4* __restrict__ out,
                                    int32_t* __restrict__ out_pos, int32_t* status) {
  int j = blockIdx.x, r = blockIdx.y;
  if (!skip_mask[r % n_images]) return;
  int g = gamma[r];
  if (g < 0 || g > gamma_max) {
    if (j == 0 && threadIdx.x == 0) atomicOr(status, VVS_DEV_BAD_ARG);
    return;
  }
  if (j >= g) return;
  int nw = newest[r];
  int pos = nw - staleness - g + 1 + j;
  bool hit = nw >= 0 && pos >= 0 && fpos[(size_t)r * cap + (pos % cap)] == pos;
  uint4* dst = out + ((size_t)r * gamma_max + j) * row_vecs;
  if (hit) {
    const uint4* src = feat + ((size_t)r * cap + (pos % cap)) * row_vecs;
    for (int i = threadIdx.x; i < row_vecs; i += blockDim.x) dst[i] = src[i];
  } else {
    for (int i = threadIdx.x; i < row_vecs; i += blockDim.x) dst[i] = make_uint4(0, 0, 0, 0);
  }
  if (threadIdx.x == 0) {
    out_pos[(size_t)r * gamma_max + j] = hit ? pos : -1;
    if (!hit) atomicOr(status, VVS_DEV_FCACHE_MISS);
  }
}

void launch_fcache_fetch(const vvs_fcache& fc, const uint8_t* skip_mask, int n_images,
                         const int32_t* gamma, int gamma_max, int staleness, int d, int elem_bytes,
                         void* out, int32_t* out_pos, int32_t* status, cudaStream_t s) {
  dim3 grid(gamma_max, fc.n_rows);
  fcache_fetch_kernel<<<grid, 128, 0, s>>>((const uint4*)fc.feat, fc.fpos, fc.newest, skip_mask,
                                           n_images, gamma, gamma_max, staleness, fc.cap,
                                           d * elem_bytes / 16, (uint4*)out, out_pos, status);
}

}  // namespace vvs
