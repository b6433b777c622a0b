// Dynamic verification-skipping decision (paper Sec. 4.4, Eq. 2, Alg. 1): for each image, the
// cosine similarity of the latent codebook embeddings of its down-sampled candidate token paths,
// weighted over depth by alpha^l, against a threshold; never two skipped steps in a row.
// One CTA per image.  The work is tiny (tens of paths, a few levels, an 8..256-dim codebook): the
// kernel is latency-bound, its cost is one dependent chain of L2 loads.
#include "vvs_internal.cuh"

namespace vvs {

namespace {

constexpr int kSkipThreads = 128;
constexpr int kSkipMaxKept = 64;    // paths kept after down-sampling
constexpr int kSkipMaxDepth = 16;

__global__ void __launch_bounds__(kSkipThreads)
skip_decide_kernel(const int32_t* __restrict__ paths, const int32_t* __restrict__ path_len,
                   const float* __restrict__ codebook, const uint8_t* __restrict__ last_verified,
                   int n_paths, int max_len, int vocab, int dim, int stride, float alpha, float threshold,
                   uint8_t* __restrict__ decision, float* __restrict__ sim, int32_t* status) {
  __shared__ double s_norm[kSkipMaxKept * kSkipMaxDepth];   // |E[c_i[l]]|, -1 for an invalid token
  __shared__ double s_level[kSkipMaxDepth];
  __shared__ double s_red[kSkipThreads];
  __shared__ int s_depth;
  const int b = blockIdx.x, tid = threadIdx.x;
  const int32_t* pb = paths + (size_t)b * n_paths * max_len;
  const int n_keep = (n_paths + stride - 1) / stride;

  if (tid == 0) {
    int depth = max_len;
    for (int i = 0; i < n_keep; ++i) {
      const int len = path_len ? path_len[(size_t)b * n_paths + i * stride] : max_len;
      depth = len < depth ? len : depth;
    }
    s_depth = depth < 0 ? 0 : depth;
  }
  __syncthreads();
  const int depth = s_depth;
  const bool verified = last_verified ? last_verified[b] != 0 : true;
  if (!verified || depth == 0 || n_keep < 2) {              // Alg. 1 guard and the degenerate cases
    if (tid == 0) {
      const float s = (!verified || depth == 0) ? 0.f : 1.f;
      sim[b] = s;
      decision[b] = (verified && s >= threshold) ? 1 : 0;
    }
    return;
  }
  // norms of the embeddings of every kept (path, level)
  for (int t = tid; t < n_keep * depth; t += kSkipThreads) {
    const int i = t / depth, l = t - i * depth;
    const int tok = pb[(size_t)(i * stride) * max_len + l];
    double nn = -1.0;
    if (tok >= 0 && tok < vocab) {
      const float* e = codebook + (size_t)tok * dim;
      nn = 0.0;
      for (int d = 0; d < dim; ++d) nn += (double)e[d] * (double)e[d];
      nn = sqrt(nn);
    } else {
      atomicOr(status, VVS_DEV_BAD_TOKEN);
    }
    s_norm[i * kSkipMaxDepth + l] = nn;
  }
  __syncthreads();
  // S^(l) = mean over unordered pairs of kept paths of the cosine at depth l
  const int n_pairs = n_keep * (n_keep - 1) / 2;
  for (int l = 0; l < depth; ++l) {
    double acc = 0.0;
    for (int t = tid; t < n_pairs; t += kSkipThreads) {
      // pair index -> (i < j)
      int i = 0, rem = t;
      while (rem >= n_keep - 1 - i) { rem -= n_keep - 1 - i; ++i; }
      const int j = i + 1 + rem;
      const double ni = s_norm[i * kSkipMaxDepth + l], nj = s_norm[j * kSkipMaxDepth + l];
      if (ni > 0.0 && nj > 0.0) {
        const float* x = codebook + (size_t)pb[(size_t)(i * stride) * max_len + l] * dim;
        const float* y = codebook + (size_t)pb[(size_t)(j * stride) * max_len + l] * dim;
        double dot = 0.0;
        for (int d = 0; d < dim; ++d) dot += (double)x[d] * (double)y[d];
        acc += dot / (ni * nj);
      }
    }
    s_red[tid] = acc;
    __syncthreads();
    for (int o = kSkipThreads / 2; o > 0; o >>= 1) {         // fixed-order tree: the same sum every run
      if (tid < o) s_red[tid] += s_red[tid + o];
      __syncthreads();
    }
    if (tid == 0) s_level[l] = s_red[0] / (double)n_pairs;
    __syncthreads();
  }
  if (tid == 0) {
    double wsum = 0.0, w = 1.0, s = 0.0;
    for (int l = 0; l < depth; ++l) {
      s += w * s_level[l];
      wsum += w;
      w *= (double)alpha;
    }
    s /= wsum;
    sim[b] = (float)s;
    decision[b] = s >= (double)threshold ? 1 : 0;
  }
}

// Unverified token selection with truncation (Sec. 4.2, Eq. 3): one warp per image.
__global__ void select_unverified_kernel(const int32_t* __restrict__ paths, const int32_t* __restrict__ path_len,
                                         const float* __restrict__ uniforms, int n_paths, int max_len,
                                         int32_t* __restrict__ out_path, int32_t* __restrict__ out_gamma,
                                         int32_t* __restrict__ out_tokens, int32_t* status) {
  const int b = blockIdx.x, lane = threadIdx.x;
  long long total = 0;
  bool bad = false;
  for (int i = lane; i < n_paths; i += 32) {
    const int len = path_len ? path_len[(size_t)b * n_paths + i] : max_len;
    bad |= len < 0 || len > max_len;
    total += len < 0 ? 0 : (len > max_len ? max_len : len);
  }
  for (int o = 16; o > 0; o >>= 1) total += __shfl_xor_sync(0xffffffffu, total, o);
  if (__any_sync(0xffffffffu, bad) && lane == 0) atomicOr(status, VVS_DEV_BAD_ARG);
  int idx = (int)floorf(uniforms[b] * (float)n_paths);
  idx = idx < 0 ? 0 : (idx > n_paths - 1 ? n_paths - 1 : idx);
  int len_s = path_len ? path_len[(size_t)b * n_paths + idx] : max_len;
  len_s = len_s < 0 ? 0 : (len_s > max_len ? max_len : len_s);
  const int mean_floor = (int)(total / n_paths);
  const int gamma = len_s < mean_floor ? len_s : mean_floor;
  if (lane == 0) {
    out_path[b] = idx;
    out_gamma[b] = gamma;
  }
  for (int t = lane; t < max_len; t += 32)
    out_tokens[(size_t)b * max_len + t] = t < gamma ? paths[((size_t)b * n_paths + idx) * max_len + t] : -1;
}

}  // namespace

int launch_select_unverified(const int32_t* paths, const int32_t* path_len, const float* uniforms, int n_images,
                             int n_paths, int max_len, int32_t* out_path, int32_t* out_gamma, int32_t* out_tokens,
                             int32_t* status, cudaStream_t s) {
  select_unverified_kernel<<<n_images, 32, 0, s>>>(paths, path_len, uniforms, n_paths, max_len, out_path, out_gamma,
                                                   out_tokens, status);
  return cudaGetLastError() == cudaSuccess ? VVS_OK : VVS_ERR_CUDA;
}

int launch_skip_decide(const int32_t* paths, const int32_t* path_len, const float* codebook,
                       const uint8_t* last_verified, int n_images, int n_paths, int max_len, int vocab, int dim,
                       int stride, float alpha, float threshold, uint8_t* decision, float* sim, int32_t* status,
                       cudaStream_t s) {
  if ((n_paths + stride - 1) / stride > kSkipMaxKept || max_len > kSkipMaxDepth) return VVS_ERR_SHAPE;
  skip_decide_kernel<<<n_images, kSkipThreads, 0, s>>>(paths, path_len, codebook, last_verified, n_paths, max_len,
                                                      vocab, dim, stride, alpha, threshold, decision, sim, status);
  return cudaGetLastError() == cudaSuccess ? VVS_OK : VVS_ERR_CUDA;
}

}  // namespace vvs
