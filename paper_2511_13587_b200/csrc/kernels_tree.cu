// Verification of a candidate TREE (the drafter of the paper proposes a token tree, Sec. 5):
// multi-round speculative sampling over the children of the current node, which are taken to be
// independent draws from the drafter's distribution q at that node.  A child x passes iff
// u < min(1, p_res(x) / q(x)); a rejection replaces p_res by norm(max(0, p_res - q)); when no
// child is left the next token is drawn from the last residual.  A chain-shaped tree reduces to
// the chain rule of Sec. 2 bit for bit: the first residual is the float32 difference of the two
// float32 rows, later rounds (which a chain never reaches) work in float64.
// Relaxed mode: the numerator is the pooled mass of x and its neighbours in the current p_res
// (the chain's relaxed rule with p_res in the place of p); with the adjusted-residual flag a
// rejection subtracts q from p_res after the pooled neighbours' mass has been moved onto x.
//
// One CTA per image; the walk is sequential over tree depth and siblings, each residual update
// and the final inverse-CDF draw are block-wide passes over the V codes.  Sums run in a fixed
// order, so a call repeats bit for bit on the same probabilities.
#include <math_constants.h>

#include "vvs_internal.cuh"

namespace vvs {

namespace {

constexpr int kTreeThreads = 1024;

__device__ __forceinline__ double tw_warp_sum(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ double tw_warp_scan(double v, int lane) {
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const double t = __shfl_up_sync(0xffffffffu, v, o);
    if (lane >= o) v += t;
  }
  return v;
}

// Longest distance-ordered prefix of neighbour entries 1 .. kk-1 whose cumulative mass stays
// <= delta (one warp; the pooled mass in every lane, the first entry not pooled in *j_end).
template <typename F>
__device__ __forceinline__ double tw_pooled_prefix(int kk, double delta, int lane, F pn_of, int* j_end) {
  double cum = 0.0;
  int end = kk;
  for (int j0 = 1; j0 < kk; j0 += 32) {
    const int j = j0 + lane;
    const double pn = (j < kk) ? pn_of(j) : 0.0;
    const double tot = cum + tw_warp_scan(pn, lane);
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

// Sum over the block, the same value in every thread (two barriers).
__device__ double tw_block_sum(double v, double* s_warp) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  v = tw_warp_sum(v);
  __syncthreads();
  if (lane == 0) s_warp[warp] = v;
  __syncthreads();
  double tot = 0.0;
  for (int w = 0; w < kTreeThreads / 32; ++w) tot += s_warp[w];
  return tot;
}

__global__ void __launch_bounds__(kTreeThreads) tree_walk_kernel(TreeParams p) {
  __shared__ double s_warp[kTreeThreads / 32];
  __shared__ int s_child[32];
  __shared__ int s_n, s_pass, s_first, s_last, s_jend;
  __shared__ double s_mass;
  const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int F = p.n_forced, K = p.n_draft_max, T = p.t_len, V = p.vocab;
  const int32_t* par = p.parent + (size_t)b * T;
  double* buf[2] = {p.res + (size_t)b * V, p.res + ((size_t)p.n_images + b) * V};

  if (tid == 0) {
    for (int i = 0; i <= K; ++i)
      if (p.margins) p.margins[(size_t)b * (K + 1) + i] = CUDART_INF_F;
    for (int i = 0; i < K; ++i) {
      if (p.accept_mask) p.accept_mask[(size_t)b * K + i] = 0;
      p.accept_path[(size_t)b * K + i] = -1;
    }
  }
  int cur = F - 1, n_acc = 0;
  int src = -1;                 // -1: sample from the float32 row of `cur`; else from buf[src]
  const float* prow = nullptr;
#pragma unroll 1
  for (int level = 0; level <= K; ++level) {
    __syncthreads();
    if (tid == 0) {
      int n = 0;
      for (int c = F; c < T; ++c)
        if (par[c] == cur) s_child[n++] = c;
      s_n = n;
    }
    __syncthreads();
    const int n_child = s_n;
    prow = p.probs + ((size_t)b * T + cur) * V;
    src = -1;
    if (n_child == 0) break;                      // leaf: the bonus token comes from its own row
    bool first_round = true;
    double z = 1.0;
    int accepted = -1;
#pragma unroll 1
    for (int ci = 0; ci < n_child; ++ci) {
      const int c = s_child[ci], i = c - F;
      const float* qrow = p.draft_probs + ((size_t)b * K + i) * V;
      const int x = p.drafts[(size_t)b * p.drafts_ld + i] - p.vocab_offset;
      const bool x_ok = x >= 0 && x < V;
      if (warp == 0) {
        int pass = 0;
        if (!x_ok) {
          if (lane == 0) atomicOr(p.status, VVS_DEV_BAD_TOKEN);
        } else {
          double px = first_round ? (double)prow[x] : buf[src][x] / z;
          int j_end = 1;
          if (p.relaxed) {
            const int beg = p.row_ptr[x], len = p.row_ptr[x + 1] - beg;
            if (len < 1 && lane == 0) atomicOr(p.status, VVS_DEV_BAD_NEIGHBOUR);
            const int kk = min(p.nbr_k, len);
            const double* cur_res = first_round ? nullptr : buf[src];
            px += tw_pooled_prefix(kk, (double)p.delta, lane, [&](int j) {
              const int cc = p.col[beg + j];
              if (cc < 0 || cc >= V) return 0.0;
              return cur_res ? cur_res[cc] / z : (double)prow[cc]; }, &j_end);
          }
          const double qx = (double)qrow[x];
          const double ratio = qx > 0.0 ? fmin(1.0, px / qx) : (px > 0.0 ? 1.0 : 0.0);
          const double u = (double)p.uniforms[(size_t)b * (K + 1) + i];
          if (lane == 0 && p.margins) p.margins[(size_t)b * (K + 1) + i] = (float)fabs(u - ratio);
          pass = u < ratio ? 1 : 0;
          if (lane == 0) {
            s_mass = px;
            s_jend = j_end;
          }
        }
        if (lane == 0) s_pass = pass;
      }
      __syncthreads();
      const int pass = s_pass;
      __syncthreads();
      if (pass) {
        accepted = c;
        break;
      }
      if (!x_ok) continue;
      // rejected: residual of this round
      double* dst = buf[src < 0 ? 0 : (src ^ 1)];
      double local = 0.0;
      if (first_round) {
        for (int v = tid; v < V; v += kTreeThreads) {
          const double r = (double)fmaxf(0.f, __fsub_rn(prow[v], qrow[v]));
          dst[v] = r;
          local += r;
        }
      } else {
        const double* cur_res = buf[src];
        for (int v = tid; v < V; v += kTreeThreads) {
          const double r = fmax(0.0, __dsub_rn(cur_res[v] / z, (double)qrow[v]));
          dst[v] = r;
          local += r;
        }
      }
      if (p.adjusted) {
        // adjusted target of the rejected child: its pooled neighbours carry no mass, the child
        // carries the pooled mass; the touched entries are rewritten and the sum is taken again
        __syncthreads();
        const int beg = p.row_ptr[x];
        const int j_end = s_jend;
        for (int j = 1 + tid; j < j_end; j += kTreeThreads) {
          const int cc = p.col[beg + j];
          if (cc >= 0 && cc < V) dst[cc] = 0.0;
        }
        __syncthreads();
        if (tid == 0)
          dst[x] = first_round ? (double)fmaxf(0.f, __fsub_rn((float)s_mass, qrow[x]))
                               : fmax(0.0, __dsub_rn(s_mass, (double)qrow[x]));
        __syncthreads();
        local = 0.0;
        for (int v = tid; v < V; v += kTreeThreads) local += dst[v];
      }
      const double z_new = tw_block_sum(local, s_warp);
      if (z_new > 0.0) {                          // else p_res == q numerically: keep p_res
        src = src < 0 ? 0 : (src ^ 1);
        z = z_new;
        first_round = false;
      }
    }
    if (accepted < 0) break;
    if (tid == 0) {
      p.accept_path[(size_t)b * K + n_acc] = accepted;
      if (p.accept_mask) p.accept_mask[(size_t)b * K + (accepted - F)] = 1;
    }
    ++n_acc;
    cur = accepted;
  }
  __syncthreads();

  // ---- inverse-CDF draw from the un-normalised source, ascending index ----
  const int seg = (V + kTreeThreads - 1) / kTreeThreads;
  const int v0 = tid * seg, v1 = min(V, v0 + seg);
  const double* dsrc = src < 0 ? nullptr : buf[src];
  double local = 0.0;
  for (int v = v0; v < v1; ++v) local += dsrc ? dsrc[v] : (double)prow[v];
  double incl = tw_warp_scan(local, lane);
  if (lane == 31) s_warp[warp] = incl;
  if (tid == 0) {
    s_first = 0x7fffffff;
    s_last = -1;
  }
  __syncthreads();
  double before = 0.0, total = 0.0;
  for (int w = 0; w < kTreeThreads / 32; ++w) {
    const double t = s_warp[w];
    if (w < warp) before += t;
    total += t;
  }
  const double excl = before + incl - local;
  const double target = (double)p.uniforms[(size_t)b * (K + 1) + K] * total;
  {
    double c = excl;
    int first = 0x7fffffff, last = -1;
    for (int v = v0; v < v1; ++v) {
      const double r = dsrc ? dsrc[v] : (double)prow[v];
      c += r;
      if (r > 0.0) last = v;
      if (first == 0x7fffffff && c > target) first = v;
    }
    if (first != 0x7fffffff) atomicMin(&s_first, first);
    if (last >= 0) atomicMax(&s_last, last);
  }
  __syncthreads();
  const int pick = s_first != 0x7fffffff ? s_first : s_last;
  if (pick >= v0 && pick < v1) {
    double c = excl;
    for (int v = v0; v < pick; ++v) c += dsrc ? dsrc[v] : (double)prow[v];
    const double hi = c + (dsrc ? dsrc[pick] : (double)prow[pick]);
    p.next_token[b] = p.vocab_offset + pick;
    if (p.margins) p.margins[(size_t)b * (K + 1) + K] = (float)(fmin(fabs(target - c), fabs(hi - target)) / total);
  }
  if (tid == 0) {
    if (pick < 0) {                               // an all-zero source: no token can be drawn
      p.next_token[b] = -1;
      atomicOr(p.status, VVS_DEV_BAD_ARG);
    }
    p.accept_len[b] = n_acc;
    for (int c = 0; c < p.n_cfg; ++c) {
      const int r = c * p.n_images + b;
      if (p.new_len && p.cache_len) p.new_len[r] = p.cache_len[r] + F + n_acc;
      if (p.n_commit) p.n_commit[r] = F + n_acc;
    }
  }
}

// K/V of the accepted nodes move from their block slots fill + node to fill + F + i (i-th
// accepted node): the cache is contiguous again and the rejected branches fall behind new_len.
// node_i >= F + i and the nodes ascend, so moving in path order never overwrites a later source.
template <typename T>
__global__ void tree_commit_kernel(T* __restrict__ kv_k, T* __restrict__ kv_v, const int32_t* __restrict__ cache_len,
                                   const int32_t* __restrict__ accept_len, const int32_t* __restrict__ accept_path,
                                   int n_heads, int hd, int s_max, int kv_rows, int n_images, int n_forced,
                                   int n_draft_max) {
  const int h = blockIdx.x, r = blockIdx.y, layer = blockIdx.z;
  const int b = r % n_images;
  const int fill = cache_len[r];
  if (fill < 0 || fill + n_forced + n_draft_max > s_max) return;
  const int n = accept_len[b];
  const int vecs = hd * (int)sizeof(T) / 16;          // 16-byte vectors per row
  T* base = (threadIdx.x < (unsigned)vecs ? kv_k : kv_v) + (((size_t)layer * kv_rows + r) * n_heads + h) * s_max * hd;
  const int vec = threadIdx.x < (unsigned)vecs ? threadIdx.x : threadIdx.x - vecs;
  if (vec >= vecs) return;
  for (int i = 0; i < n; ++i) {
    const int node = accept_path[(size_t)b * n_draft_max + i];
    if (node < n_forced + i || node >= n_forced + n_draft_max || node == n_forced + i) continue;
    const uint4 val = reinterpret_cast<const uint4*>(base + (size_t)(fill + node) * hd)[vec];
    reinterpret_cast<uint4*>(base + (size_t)(fill + n_forced + i) * hd)[vec] = val;
  }
}

}  // namespace

void launch_tree_walk(const TreeParams& p, cudaStream_t s) {
  tree_walk_kernel<<<p.n_images, kTreeThreads, 0, s>>>(p);
}

void launch_tree_commit(void* kv_k, void* kv_v, const int32_t* cache_len, const int32_t* accept_len,
                        const int32_t* accept_path, const vvs_model_desc& md, int kv_rows, int n_images, int n_cfg,
                        int n_forced, int n_draft_max, cudaStream_t s) {
  if (md.n_layers < 1) return;
  using T = __nv_bfloat16;
  const int vecs = md.head_dim * (int)sizeof(T) / 16;
  dim3 grid(md.n_heads, n_images * n_cfg, md.n_layers);
  tree_commit_kernel<T><<<grid, 2 * vecs, 0, s>>>(static_cast<T*>(kv_k), static_cast<T*>(kv_v), cache_len, accept_len,
                                                  accept_path, md.n_heads, md.head_dim, md.s_max, kv_rows, n_images,
                                                  n_forced, n_draft_max);
}

}  // namespace vvs
