// Decision stage of the verify step (paper Sec. 2): acceptance test per drafted token, accepted
// prefix, residual / bonus sample.  Works on softmax statistics plus gathered logits, so the
// same kernels serve the generic path (full logits in scratch) and the fused LM-head path
// (logits never written out).
#include <math_constants.h>

#include "vvs_internal.cuh"

namespace vvs {

__device__ __forceinline__ double warp_sum_d(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ double warp_incl_scan_d(double v, int lane) {
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    double t = __shfl_up_sync(0xffffffffu, v, o);
    if (lane >= o) v += t;
  }
  return v;
}

// Relaxed numerator (Sec. 2): the longest distance-ordered prefix of neighbour entries 1 .. kk-1
// whose cumulative mass stays <= delta.  One warp; pn(j) gives the mass of entry j.  Returns the
// pooled mass (the same value in every lane) and the first entry NOT pooled in *j_end.
template <typename F>
__device__ __forceinline__ double pooled_prefix(int kk, double delta, int lane, F pn_of, int* j_end) {
  double cum = 0.0;
  int end = kk;
  for (int j0 = 1; j0 < kk; j0 += 32) {
    const int j = j0 + lane;
    const double pn = (j < kk) ? pn_of(j) : 0.0;
    const double tot = cum + warp_incl_scan_d(pn, lane);
    const unsigned over = __ballot_sync(0xffffffffu, (j < kk) && (tot > delta));
    if (over) {
      const int first = __ffs(over) - 1;
      const double prev = __shfl_sync(0xffffffffu, tot, first > 0 ? first - 1 : 0);
      if (first > 0) cum = prev;
      end = j0 + first;
      break;
    }
    cum = __shfl_sync(0xffffffffu, tot, 31);
  }
  *j_end = end;
  return cum;
}

// ---------------------------------------------------------------------------------------------
// Combine per-tile softmax partials: M = max_t m_t, S = sum_t s_t exp(m_t - M), fixed order.
__global__ void finalize_stats_kernel(const float* __restrict__ part_m, const float* __restrict__ part_s,
                                      float* __restrict__ stat_m, float* __restrict__ stat_inv,
                                      int n_tiles, int n_rows) {
  int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  int lane = threadIdx.x & 31;
  if (row >= n_rows) return;
  float mx = -CUDART_INF_F;
  for (int t = lane; t < n_tiles; t += 32) mx = fmaxf(mx, part_m[(size_t)t * n_rows + row]);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  float sum = 0.f;
  for (int t = lane; t < n_tiles; t += 32)
    sum += part_s[(size_t)t * n_rows + row] * expf(part_m[(size_t)t * n_rows + row] - mx);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
  if (lane == 0) {
    stat_m[row] = mx;
    stat_inv[row] = 1.f / sum;
  }
}

void launch_finalize_stats(const Workspace& ws, int n_tiles, int n_rows, cudaStream_t s) {
  finalize_stats_kernel<<<(n_rows + 3) / 4, 128, 0, s>>>(ws.part_m, ws.part_s, ws.stat_m, ws.stat_inv,
                                                         n_tiles, n_rows);
}

// ---------------------------------------------------------------------------------------------
// Generic path: pull the logits of each drafted token and of its neighbours out of the
// materialised logits.  grid (K, B).
__global__ void gather_logits_kernel(const float* __restrict__ logits, float* __restrict__ l_tok,
                                     float* __restrict__ l_nbr, DecideParams p, int32_t* status) {
  int i = blockIdx.x, b = blockIdx.y;
  int K = p.n_draft_max, V = p.vocab;
  int x = p.drafts[(size_t)b * p.drafts_ld + i] - p.vocab_offset;
  if (x < 0 || x >= V) return;  // reported by the acceptance kernel
  const float* row = logits + ((size_t)b * p.rows_per_seq + p.first_row + i) * V;
  if (threadIdx.x == 0) l_tok[b * K + i] = row[x];
  if (p.mode != VVS_MODE_RELAXED || p.nbr_k <= 1) return;
  int beg = p.row_ptr[x], len = p.row_ptr[x + 1] - beg;
  int kk = min(p.nbr_k, len);
  float* dst = l_nbr + ((size_t)b * K + i) * p.kmax;
  for (int j = 1 + threadIdx.x; j < kk; j += blockDim.x) {
    int c = p.col[beg + j];
    bool ok = c >= 0 && c < V;
    if (!ok) atomicOr(status, VVS_DEV_BAD_NEIGHBOUR);
    dst[j] = ok ? row[c] : -CUDART_INF_F;
  }
}

void launch_gather_logits(const float* logits, const Workspace& ws, const DecideParams& p, cudaStream_t s) {
  if (p.n_draft_max == 0) return;
  dim3 grid(p.n_draft_max, p.n_images);
  gather_logits_kernel<<<grid, 128, 0, s>>>(logits, ws.l_tok, ws.l_nbr, p, ws.status);
}

// ---------------------------------------------------------------------------------------------
// Acceptance (Sec. 2): draft i passes iff u_i < min(1, P_i / q_i(x_i)) with P_i = p(x_i) (strict)
// or the pooled mass of x_i and the longest distance-ordered neighbour prefix whose own mass
// stays <= delta (relaxed).  Verification stops at the first rejection.  One CTA per image.
__global__ void accept_kernel(Workspace ws, DecideParams p) {
  __shared__ double ratio_s[32];
  int b = blockIdx.x;
  int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = blockDim.x >> 5;
  int K = p.n_draft_max, V = p.vocab;
  int nd = p.n_draft ? p.n_draft[b] : K;
  if (nd < 0 || nd > K) {
    if (threadIdx.x == 0) atomicOr(ws.status, VVS_DEV_BAD_ARG);
    nd = nd < 0 ? 0 : K;
  }
  for (int i = warp; i < K; i += nw) {
    double ratio = 0.0;
    if (i < nd) {
      int x = p.drafts[(size_t)b * p.drafts_ld + i] - p.vocab_offset;
      if (x < 0 || x >= V) {
        if (lane == 0) atomicOr(ws.status, VVS_DEV_BAD_TOKEN);
      } else {
        int drow = b * p.rows_per_seq + p.first_row + i;
        const bool direct = p.direct_probs != nullptr;
        float m = direct ? 0.f : ws.stat_m[drow], inv = direct ? 1.f : ws.stat_inv[drow];
        double mass = (double)(direct ? ws.l_tok[b * K + i] : prob_of(ws.l_tok[b * K + i], m, inv));
        if (p.mode == VVS_MODE_RELAXED && p.nbr_k > 1) {
          int beg = p.row_ptr[x], len = p.row_ptr[x + 1] - beg;
          if (len < 1 && lane == 0) atomicOr(ws.status, VVS_DEV_BAD_NEIGHBOUR);
          int kk = min(p.nbr_k, len);
          const float* ln = ws.l_nbr + ((size_t)b * K + i) * p.kmax;
          int j_end;
          const double cum = pooled_prefix(kk, (double)p.delta, lane, [&](int j) {
            return (double)(direct ? ln[j] : prob_of(ln[j], m, inv)); }, &j_end);
          mass += cum;
        }
        double qx = (double)p.draft_probs[((size_t)b * K + i) * V + x];
        ratio = qx > 0.0 ? fmin(1.0, mass / qx) : (mass > 0.0 ? 1.0 : 0.0);
      }
    }
    if (lane == 0) ratio_s[i] = ratio;
  }
  __syncthreads();
  if (threadIdx.x != 0) return;
  int n = 0;
  bool open = true;
  for (int i = 0; i < K; ++i) {
    float margin = CUDART_INF_F;
    uint8_t bit = 0;
    if (open && i < nd) {
      double u = (double)p.uniforms[(size_t)b * (K + 1) + i];
      margin = (float)fabs(u - ratio_s[i]);
      if (u < ratio_s[i]) {
        bit = 1;
        ++n;
      } else {
        open = false;
      }
    }
    if (p.margins) p.margins[(size_t)b * (K + 1) + i] = margin;
    if (p.accept_mask) p.accept_mask[(size_t)b * K + i] = bit;
  }
  p.accept_len[b] = n;
  if (p.new_len && p.cache_len) {
    for (int c = 0; c < p.n_cfg; ++c) {
      int r = c * p.n_images + b;
      p.new_len[r] = p.cache_len[r] + p.n_forced + n;
    }
  }
  if (p.n_commit) {
    for (int c = 0; c < p.n_cfg; ++c) p.n_commit[c * p.n_images + b] = p.n_forced + n;
  }
  int t_sel = p.first_row + n;
  ws.sel_row[b] = (t_sel < p.rows_per_seq) ? b * p.rows_per_seq + t_sel : -1;
  ws.sel_kind[b] = (n < nd) ? 0 : 1;
}

void launch_accept(const Workspace& ws, const DecideParams& p, cudaStream_t s) {
  accept_kernel<<<p.n_images, 256, 0, s>>>(ws, p);
}

// ---------------------------------------------------------------------------------------------
__global__ void probs_kernel(const float* __restrict__ logits, const float* __restrict__ stat_m,
                             const float* __restrict__ stat_inv, float* __restrict__ probs, int v) {
  size_t row = blockIdx.y;
  float m = stat_m[row], inv = stat_inv[row];
  int j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j < v) probs[row * v + j] = prob_of(logits[row * v + j], m, inv);
}

// probs may alias logits (in-place normalisation)
void launch_probs_from_logits(const float* logits, const Workspace& ws, float* probs, int n_rows,
                              int v, cudaStream_t s) {
  dim3 grid((v + 255) / 256, n_rows);
  probs_kernel<<<grid, 256, 0, s>>>(logits, ws.stat_m, ws.stat_inv, probs, v);
}

// target probabilities of the row each image samples from, out of stored guided logits
__global__ void select_p_row_kernel(const float* __restrict__ logits, Workspace ws, int v) {
  int b = blockIdx.y;
  int j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j >= v) return;
  int row = ws.sel_row[b];
  float pr = 0.f;
  if (row >= 0) pr = prob_of(logits[(size_t)row * v + j], ws.stat_m[row], ws.stat_inv[row]);
  ws.p_row[(size_t)b * v + j] = pr;
}

void launch_select_p_row(const float* logits, const Workspace& ws, int n_images, int v, cudaStream_t s) {
  dim3 grid((v + 255) / 256, n_images);
  select_p_row_kernel<<<grid, 256, 0, s>>>(logits, ws, v);
}

// ---------------------------------------------------------------------------------------------
// Adjusted target of a relaxed rejection (flag adjusted_residual): in the row image b samples
// from, the pooled neighbours of the rejected draft x give their mass to x.  The row lives in
// ws.p_row (copied there first when the caller's probabilities are used directly); the pooled
// prefix is found again from the row's own float32 values, by the rule of accept_kernel.
// grid B, 256 threads.
__global__ void adjust_target_kernel(Workspace ws, DecideParams p) {
  const int b = blockIdx.x, V = p.vocab;
  const int sel = ws.sel_row[b];
  if (sel < 0) return;
  float* row = ws.p_row + (size_t)b * V;
  if (p.direct_probs) {
    const float* src = p.direct_probs + (size_t)sel * V;
    for (int j = threadIdx.x; j < V; j += blockDim.x) row[j] = src[j];
    __syncthreads();
  }
  if (ws.sel_kind[b] != 0 || threadIdx.x >= 32) return;    // bonus row: nothing was rejected
  const int lane = threadIdx.x;
  const int n = p.accept_len[b];
  const int x = p.drafts[(size_t)b * p.drafts_ld + n] - p.vocab_offset;
  if (x < 0 || x >= V) return;                             // reported by the acceptance kernel
  const int beg = p.row_ptr[x], len = p.row_ptr[x + 1] - beg;
  const int kk = min(p.nbr_k, len);
  auto mass_of = [&](int j) {
    const int c = p.col[beg + j];
    return (c >= 0 && c < V) ? (double)row[c] : 0.0;
  };
  int j_end;
  const double cum = pooled_prefix(kk, (double)p.delta, lane, mass_of, &j_end);
  const double mass = (double)row[x] + cum;
  __syncwarp();
  for (int j = 1 + lane; j < j_end; j += 32) {
    const int c = p.col[beg + j];
    if (c >= 0 && c < V) row[c] = 0.f;
  }
  __syncwarp();
  if (lane == 0) row[x] = (float)mass;
}

void launch_adjust_target(const Workspace& ws, const DecideParams& p, cudaStream_t s) {
  adjust_target_kernel<<<p.n_images, 256, 0, s>>>(ws, p);
}

// ---------------------------------------------------------------------------------------------
// Residual distribution (Sec. 2): r = max(0, p - q_n) at the first rejected draft n, or r = p for
// the bonus token; float32 difference, float64 accumulation.
__device__ __forceinline__ float residual_value(float pr, const float* q_row, int j, int kind) {
  if (kind != 0) return pr;
  return fmaxf(0.f, pr - q_row[j]);
}

// grid (n_chunks, B), block kSampleChunk/4 threads
__global__ void residual_mass_kernel(Workspace ws, DecideParams p, int n_chunks) {
  __shared__ double red_r[32], red_p[32];
  int c = blockIdx.x, b = blockIdx.y;
  int V = p.vocab, K = p.n_draft_max;
  int kind = ws.sel_kind[b];
  int n = p.accept_len[b];
  const float* q_row = p.draft_probs + ((size_t)b * K + (kind == 0 ? n : 0)) * V;
  const int sel = ws.sel_row[b];
  if (sel < 0) return;  // no row to sample from: sample_kernel reports -1
  const float* p_row = (p.direct_probs && !p.adjusted) ? p.direct_probs + (size_t)sel * V : ws.p_row + (size_t)b * V;
  double sr = 0.0, sp = 0.0;
  int end = min(V, (c + 1) * kSampleChunk);
  for (int j = c * kSampleChunk + threadIdx.x; j < end; j += blockDim.x) {
    float pr = p_row[j];
    sr += (double)residual_value(pr, q_row, j, kind);
    sp += (double)pr;
  }
  sr = warp_sum_d(sr);
  sp = warp_sum_d(sp);
  int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
  if (lane == 0) {
    red_r[warp] = sr;
    red_p[warp] = sp;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    double tr = 0.0, tp = 0.0;
    for (int w = 0; w < nw; ++w) {
      tr += red_r[w];
      tp += red_p[w];
    }
    ws.r_part[(size_t)b * n_chunks + c] = tr;
    ws.p_part[(size_t)b * n_chunks + c] = tp;
  }
}

// Inverse CDF in ascending token order: smallest j with cumulative mass > u * total.
// grid B, block kSampleChunk threads.
__global__ void sample_kernel(Workspace ws, DecideParams p, int n_chunks) {
  __shared__ double warp_tot[32];
  __shared__ double s_lo, s_t, s_total;
  __shared__ int s_chunk, s_use_p, s_first, s_last;
  int b = blockIdx.x;
  int V = p.vocab, K = p.n_draft_max;
  int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (ws.sel_row[b] < 0) {
    if (threadIdx.x == 0) {
      p.next_token[b] = -1;
      if (p.margins) p.margins[(size_t)b * (K + 1) + K] = CUDART_INF_F;
    }
    return;
  }
  int kind = ws.sel_kind[b];
  if (threadIdx.x == 0) {
    const double* rp = ws.r_part + (size_t)b * n_chunks;
    double total = 0.0;
    for (int c = 0; c < n_chunks; ++c) total += rp[c];
    int use_p = 0;
    if (!(total > 0.0)) {  // p == q numerically: fall back to the target row itself
      use_p = 1;
      rp = ws.p_part + (size_t)b * n_chunks;
      total = 0.0;
      for (int c = 0; c < n_chunks; ++c) total += rp[c];
    }
    double t = (double)p.uniforms[(size_t)b * (K + 1) + K] * total;
    double lo = 0.0;
    int chunk = -1, last_nz = 0;
    double last_lo = 0.0;
    for (int c = 0; c < n_chunks; ++c) {
      if (rp[c] > 0.0) {
        last_nz = c;
        last_lo = lo;
      }
      if (lo + rp[c] > t) {
        chunk = c;
        break;
      }
      lo += rp[c];
    }
    if (chunk < 0) {
      chunk = last_nz;
      lo = last_lo;
    }
    s_lo = lo;
    s_t = t;
    s_total = total;
    s_chunk = chunk;
    s_use_p = use_p;
    s_first = 0x7fffffff;
    s_last = -1;
  }
  __syncthreads();
  int n = p.accept_len[b];
  int eff_kind = s_use_p ? 1 : kind;
  const float* q_row = p.draft_probs + ((size_t)b * K + (eff_kind == 0 ? n : 0)) * V;
  const float* p_row = (p.direct_probs && !p.adjusted) ? p.direct_probs + (size_t)ws.sel_row[b] * V
                                                       : ws.p_row + (size_t)b * V;
  int j = s_chunk * kSampleChunk + threadIdx.x;
  double val = 0.0;
  if (j < V) val = (double)residual_value(p_row[j], q_row, j, eff_kind);
  double inc = warp_incl_scan_d(val, lane);
  if (lane == 31) warp_tot[warp] = inc;
  __syncthreads();
  if (warp == 0) {
    double w = warp_tot[lane];
    double ws_incl = warp_incl_scan_d(w, lane);
    warp_tot[lane] = ws_incl - w;  // exclusive prefix of each warp
  }
  __syncthreads();
  double cdf = s_lo + warp_tot[warp] + inc;
  if (j < V && cdf > s_t) atomicMin(&s_first, j);
  if (j < V && val > 0.0) atomicMax(&s_last, j);
  __syncthreads();
  int pick = (s_first != 0x7fffffff) ? s_first : s_last;
  if (j == pick) {
    p.next_token[b] = p.vocab_offset + j;
    if (p.margins) {
      double a = fabs(s_t - (cdf - val)), c2 = fabs(cdf - s_t);
      p.margins[(size_t)b * (K + 1) + K] = (float)(fmin(a, c2) / s_total);
    }
  }
  if (pick < 0 && threadIdx.x == 0) p.next_token[b] = -1;
}

void launch_residual_mass(const Workspace& ws, const DecideParams& p, cudaStream_t s) {
  int n_chunks = (p.vocab + kSampleChunk - 1) / kSampleChunk;
  dim3 grid(n_chunks, p.n_images);
  residual_mass_kernel<<<grid, kSampleChunk / 4, 0, s>>>(ws, p, n_chunks);
}

void launch_sample(const Workspace& ws, const DecideParams& p, cudaStream_t s) {
  int n_chunks = (p.vocab + kSampleChunk - 1) / kSampleChunk;
  sample_kernel<<<p.n_images, kSampleChunk, 0, s>>>(ws, p, n_chunks);
}

}  // namespace vvs
