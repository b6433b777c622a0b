// Storage-type-generic kernels of the verify step: embedding gather, RMSNorm, a warp-per-output
// projection kernel, RoPE + KV append, block-vs-cache attention, SwiGLU gating, guidance and
// softmax statistics.  They serve float32 contexts (which have no tensor-core path) and are the
// in-library cross-check of the bf16 tensor-core kernels.
#include <math_constants.h>

#include "vvs_internal.cuh"

namespace vvs {

template <typename T> struct VecOf;
template <> struct VecOf<float> { static constexpr int n = 4; };
template <> struct VecOf<__nv_bfloat16> { static constexpr int n = 8; };

__device__ __forceinline__ float to_f(float v) { return v; }
__device__ __forceinline__ float to_f(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f(float v);
template <> __device__ __forceinline__ float from_f<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f<__nv_bfloat16>(float v) {
  return __float2bfloat16_rn(v);
}

// 16-byte vector load widened to float
__device__ __forceinline__ void load_vec(const float* p, float* o) {
  float4 v = *reinterpret_cast<const float4*>(p);
  o[0] = v.x; o[1] = v.y; o[2] = v.z; o[3] = v.w;
}
__device__ __forceinline__ void load_vec(const __nv_bfloat16* p, float* o) {
  uint4 u = *reinterpret_cast<const uint4*>(p);
  const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&u);
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    float2 f = __bfloat1622float2(h[j]);
    o[2 * j] = f.x;
    o[2 * j + 1] = f.y;
  }
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// block-wide reductions for blockDim.x <= 1024 (multiple of 32); `red` holds 32 floats
__device__ float block_sum(float v, float* red) {
  int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
  v = warp_sum(v);
  __syncthreads();
  if (lane == 0) red[warp] = v;
  __syncthreads();
  float t = (lane < nw) ? red[lane] : 0.f;
  return warp_sum(t);
}
__device__ float block_max(float v, float* red) {
  int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
  v = warp_max(v);
  __syncthreads();
  if (lane == 0) red[warp] = v;
  __syncthreads();
  float t = (lane < nw) ? red[lane] : -CUDART_INF_F;
  return warp_max(t);
}

// ---------------------------------------------------------------------------------------------
// x0[r, t, :] = tok_emb[block[b, t]]  (cond and uncond sequences of an image share the block)
template <typename T>
__global__ void embed_kernel(const T* __restrict__ tok_emb, const int32_t* __restrict__ block,
                             float* __restrict__ x, int n_images, int t_len, int d, int tok_rows,
                             int32_t* status) {
  int m = blockIdx.x;
  int r = m / t_len, t = m % t_len;
  int b = r % n_images;
  int tok = block[b * t_len + t];
  bool ok = tok >= 0 && tok < tok_rows;
  if (!ok && threadIdx.x == 0) atomicOr(status, VVS_DEV_BAD_TOKEN);
  const T* src = tok_emb + (size_t)(ok ? tok : 0) * d;
  float* dst = x + (size_t)m * d;
  for (int i = threadIdx.x; i < d; i += blockDim.x) dst[i] = ok ? to_f(src[i]) : 0.f;
}

template <typename T>
void launch_embed(const T* tok_emb, const int32_t* block, float* x, int n_images, int n_cfg,
                  int t_len, int d, int tok_rows, int32_t* status, cudaStream_t s) {
  embed_kernel<T><<<n_images * n_cfg * t_len, 256, 0, s>>>(tok_emb, block, x, n_images, t_len, d,
                                                           tok_rows, status);
}

// ---------------------------------------------------------------------------------------------
// out[m, :] = x[m, :] * rsqrt(mean(x^2) + eps) * scale
template <typename T>
__global__ void rmsnorm_kernel(const float* __restrict__ x, const T* __restrict__ scale,
                               T* __restrict__ out, int d, float eps) {
  __shared__ float red[32];
  const float* row = x + (size_t)blockIdx.x * d;
  float ss = 0.f;
  for (int i = threadIdx.x; i < d; i += blockDim.x) ss += row[i] * row[i];
  ss = block_sum(ss, red);
  float rs = rsqrtf(ss / (float)d + eps);
  T* o = out + (size_t)blockIdx.x * d;
  for (int i = threadIdx.x; i < d; i += blockDim.x) o[i] = from_f<T>(row[i] * rs * to_f(scale[i]));
}

// The same for many rows of a bf16 context: one warp per row, 16-byte loads, no shared memory; as a
// programmatic dependent of the projection before it (the row is read after griddepcontrol.wait).
__global__ void __launch_bounds__(128) rmsnorm_rows_kernel(const float* __restrict__ x,
                                                           const __nv_bfloat16* __restrict__ scale,
                                                           __nv_bfloat16* __restrict__ out, int m, int d, float eps) {
  constexpr int kKeep = 12;            // 16-byte pieces of the row a lane keeps in registers (d <= 1536)
  const int lane = threadIdx.x & 31, row_i = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
  if (row_i >= m) return;
  const float* row = x + (size_t)row_i * d;
  float4 keep[kKeep];
#pragma unroll
  for (int u = 0; u < kKeep; ++u) {
    const int i = lane * 4 + u * 128;
    keep[u] = i < d ? *reinterpret_cast<const float4*>(row + i) : make_float4(0.f, 0.f, 0.f, 0.f);
  }
  float ss = 0.f;
#pragma unroll
  for (int u = 0; u < kKeep; ++u)
    ss += keep[u].x * keep[u].x + keep[u].y * keep[u].y + keep[u].z * keep[u].z + keep[u].w * keep[u].w;
  for (int i = lane * 4 + kKeep * 128; i < d; i += 128) {
    const float4 v = *reinterpret_cast<const float4*>(row + i);
    ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
  const float rs = rsqrtf(ss / (float)d + eps);
  __nv_bfloat16* o = out + (size_t)row_i * d;
  auto emit = [&](int i, const float4& v) {
    const uint2 g = *reinterpret_cast<const uint2*>(scale + i);
    const __nv_bfloat162 g0 = *reinterpret_cast<const __nv_bfloat162*>(&g.x);
    const __nv_bfloat162 g1 = *reinterpret_cast<const __nv_bfloat162*>(&g.y);
    __nv_bfloat162 r0 = __floats2bfloat162_rn(v.x * rs * __bfloat162float(g0.x), v.y * rs * __bfloat162float(g0.y));
    __nv_bfloat162 r1 = __floats2bfloat162_rn(v.z * rs * __bfloat162float(g1.x), v.w * rs * __bfloat162float(g1.y));
    uint2 pk;
    pk.x = *reinterpret_cast<uint32_t*>(&r0);
    pk.y = *reinterpret_cast<uint32_t*>(&r1);
    *reinterpret_cast<uint2*>(o + i) = pk;
  };
#pragma unroll
  for (int u = 0; u < kKeep; ++u) {
    const int i = lane * 4 + u * 128;
    if (i < d) emit(i, keep[u]);
  }
  for (int i = lane * 4 + kKeep * 128; i < d; i += 128) emit(i, *reinterpret_cast<const float4*>(row + i));
}

// Few rows: one CTA of 128 threads per row (every thread holds at most kKeepB 16-byte pieces), so the
// row's loads are all in flight at once and the kernel is two dependent memory round trips long.
__global__ void __launch_bounds__(128) rmsnorm_row_block_kernel(const float* __restrict__ x,
                                                                const __nv_bfloat16* __restrict__ scale,
                                                                __nv_bfloat16* __restrict__ out, int d, float eps) {
  constexpr int kKeepB = 8;            // d <= 4096
  __shared__ float red[4];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  uint2 g[kKeepB];
#pragma unroll
  for (int u = 0; u < kKeepB; ++u) {                  // the scale is an input of the whole step: before the wait
    const int i = tid * 4 + u * 512;
    g[u] = i < d ? *reinterpret_cast<const uint2*>(scale + i) : make_uint2(0u, 0u);
  }
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const float* row = x + (size_t)blockIdx.x * d;
  float4 keep[kKeepB];
  float ss = 0.f;
#pragma unroll
  for (int u = 0; u < kKeepB; ++u) {
    const int i = tid * 4 + u * 512;
    keep[u] = i < d ? *reinterpret_cast<const float4*>(row + i) : make_float4(0.f, 0.f, 0.f, 0.f);
  }
#pragma unroll
  for (int u = 0; u < kKeepB; ++u)
    ss += keep[u].x * keep[u].x + keep[u].y * keep[u].y + keep[u].z * keep[u].z + keep[u].w * keep[u].w;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
  if (lane == 0) red[warp] = ss;
  __syncthreads();
  const float rs = rsqrtf((red[0] + red[1] + red[2] + red[3]) / (float)d + eps);
  __nv_bfloat16* o = out + (size_t)blockIdx.x * d;
#pragma unroll
  for (int u = 0; u < kKeepB; ++u) {
    const int i = tid * 4 + u * 512;
    if (i < d) {
      const __nv_bfloat162 g0 = *reinterpret_cast<const __nv_bfloat162*>(&g[u].x);
      const __nv_bfloat162 g1 = *reinterpret_cast<const __nv_bfloat162*>(&g[u].y);
      __nv_bfloat162 r0 = __floats2bfloat162_rn(keep[u].x * rs * __bfloat162float(g0.x), keep[u].y * rs * __bfloat162float(g0.y));
      __nv_bfloat162 r1 = __floats2bfloat162_rn(keep[u].z * rs * __bfloat162float(g1.x), keep[u].w * rs * __bfloat162float(g1.y));
      uint2 pk;
      pk.x = *reinterpret_cast<uint32_t*>(&r0);
      pk.y = *reinterpret_cast<uint32_t*>(&r1);
      *reinterpret_cast<uint2*>(o + i) = pk;
    }
  }
}

template <typename T>
void launch_rmsnorm(const float* x, const T* scale, T* out, int m, int d, float eps, cudaStream_t s) {
  rmsnorm_kernel<T><<<m, 256, 0, s>>>(x, scale, out, d, eps);
}

static cudaError_t launch_dependent(const void* fn, dim3 grid, dim3 block, void** args, bool pdl, cudaStream_t s) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl ? 1 : 0;
  return cudaLaunchKernelExC(&cfg, fn, args);
}

void launch_rmsnorm_rows(const float* x, const __nv_bfloat16* scale, __nv_bfloat16* out, int m, int d, float eps,
                         bool pdl, cudaStream_t s) {
  if (m <= 64 && d <= 4096) {          // few rows: a CTA per row
    void* args1[] = {&x, &scale, &out, &d, &eps};
    launch_dependent(reinterpret_cast<const void*>(rmsnorm_row_block_kernel), dim3(m), dim3(128), args1, pdl, s);
    return;
  }
  void* args[] = {&x, &scale, &out, &m, &d, &eps};
  launch_dependent(reinterpret_cast<const void*>(rmsnorm_rows_kernel), dim3((m + 3) / 4), dim3(128), args, pdl, s);
}

// ---------------------------------------------------------------------------------------------
// c[m, n] (+)= sum_k a[m, k] * w[n, k].  One warp per weight row n, MT activation rows per pass.
template <typename T, int MT>
__global__ void gemm_nt_kernel(const T* __restrict__ a, const T* __restrict__ w,
                               float* __restrict__ c, int m, int n, int k, int ldc, int accumulate) {
  constexpr int VEC = VecOf<T>::n;
  int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  int col = blockIdx.x * (blockDim.x >> 5) + warp;
  int m0 = blockIdx.y * MT;
  if (col >= n) return;
  float acc[MT];
#pragma unroll
  for (int i = 0; i < MT; ++i) acc[i] = 0.f;
  const T* wrow = w + (size_t)col * k;
  for (int k0 = lane * VEC; k0 < k; k0 += 32 * VEC) {
    float wv[VEC];
    load_vec(wrow + k0, wv);
#pragma unroll
    for (int i = 0; i < MT; ++i) {
      if (m0 + i < m) {
        float av[VEC];
        load_vec(a + (size_t)(m0 + i) * k + k0, av);
#pragma unroll
        for (int j = 0; j < VEC; ++j) acc[i] = fmaf(av[j], wv[j], acc[i]);
      }
    }
  }
#pragma unroll
  for (int i = 0; i < MT; ++i) {
    float v = warp_sum(acc[i]);
    if (lane == 0 && m0 + i < m) {
      float* dst = c + (size_t)(m0 + i) * ldc + col;
      *dst = accumulate ? (*dst + v) : v;
    }
  }
}

template <typename T>
void launch_gemm_nt(const T* a, const T* w, float* c, int m, int n, int k, int ldc, bool accumulate,
                    cudaStream_t s) {
  constexpr int MT = 8;
  dim3 grid((n + 3) / 4, (m + MT - 1) / MT);
  gemm_nt_kernel<T, MT><<<grid, 128, 0, s>>>(a, w, c, m, n, k, ldc, accumulate ? 1 : 0);
}

// ---------------------------------------------------------------------------------------------
// RoPE on q and k of the block rows, k/v appended to the cache at slots L_r + t.
template <typename T>
__global__ void rope_append_kernel(float* __restrict__ qkv, const float* __restrict__ inv_freq,
                                   T* __restrict__ q, T* __restrict__ kv_k, T* __restrict__ kv_v,
                                   const int32_t* __restrict__ cache_len, int d, int n_heads, int hd,
                                   int s_max, int rope_mode, int grid_w, int n_prefix, int layer,
                                   int kv_rows, int t_len, int32_t* status,
                                   const float* __restrict__ tab_cos, const float* __restrict__ tab_sin,
                                   int clear_src) {
  int m = blockIdx.x;
  int r = m / t_len, t = m % t_len;
  int fill = cache_len[r];
  bool ok = fill >= 0 && fill + t_len <= s_max;
  if (!ok && threadIdx.x == 0) atomicOr(status, VVS_DEV_CACHE_OVERFLOW);
  int pos = fill + t;
  float c_lo = 0.f, c_hi = 0.f;  // coordinate driving the pairs of the first / second head half
  if (rope_mode == VVS_ROPE_1D) {
    c_lo = c_hi = (float)pos;
  } else if (rope_mode == VVS_ROPE_2D_GRID && pos >= n_prefix) {
    int n = pos - n_prefix;
    c_lo = (float)(n / grid_w);
    c_hi = (float)(n % grid_w);
  }
  float* src = qkv + (size_t)m * 3 * d;
  int half = hd / 2;
  for (int p = threadIdx.x; p < d / 2; p += blockDim.x) {
    int h = p / half, i = p % half;
    float sn, cs;
    if (tab_cos) {                        // rotation tables of the step (tree calls: position = fill + depth)
      cs = tab_cos[(size_t)m * half + i];
      sn = tab_sin[(size_t)m * half + i];
    } else {
      sincosf(((i < half / 2) ? c_lo : c_hi) * inv_freq[i], &sn, &cs);
    }
    int e = h * hd + 2 * i;
    float q0 = src[e], q1 = src[e + 1];
    q[(size_t)m * d + e] = from_f<T>(q0 * cs - q1 * sn);
    q[(size_t)m * d + e + 1] = from_f<T>(q0 * sn + q1 * cs);
    if (ok) {
      size_t slot = ((((size_t)layer * kv_rows + r) * n_heads + h) * s_max + pos) * hd + 2 * i;
      float k0 = src[d + e], k1 = src[d + e + 1];
      kv_k[slot] = from_f<T>(k0 * cs - k1 * sn);
      kv_k[slot + 1] = from_f<T>(k0 * sn + k1 * cs);
      kv_v[slot] = from_f<T>(src[2 * d + e]);
      kv_v[slot + 1] = from_f<T>(src[2 * d + e + 1]);
    }
    if (clear_src) {                           // split-K sums are added into this buffer: leave it zero
      const float2 z = make_float2(0.f, 0.f);
      *reinterpret_cast<float2*>(src + e) = z;
      *reinterpret_cast<float2*>(src + d + e) = z;
      *reinterpret_cast<float2*>(src + 2 * d + e) = z;
    }
  }
}

template <typename T>
void launch_rope_append(float* qkv, const float* inv_freq, T* q, T* kv_k, T* kv_v,
                        const int32_t* cache_len, const vvs_model_desc& md, int layer, int kv_rows,
                        int n_rows, int t_len, int32_t* status, cudaStream_t s, const float* tab_cos,
                        const float* tab_sin, bool clear_src) {
  rope_append_kernel<T><<<n_rows * t_len, 256, 0, s>>>(
      qkv, inv_freq, q, kv_k, kv_v, cache_len, md.d_model, md.n_heads, md.head_dim, md.s_max,
      md.rope_mode, md.rope_grid_w, md.n_prefix, layer, kv_rows, t_len, status, tab_cos, tab_sin, clear_src ? 1 : 0);
}

// ---------------------------------------------------------------------------------------------
// Block-vs-cache attention: query row t of sequence r sees cache slots [0, L_r + t].
// One CTA per (head, sequence); each warp owns query rows t = warp, warp + nwarps, ...
template <typename T>
__global__ void attention_kernel(const T* __restrict__ q, const T* __restrict__ kv_k,
                                 const T* __restrict__ kv_v, const int32_t* __restrict__ cache_len,
                                 T* __restrict__ out, int d, int n_heads, int hd, int s_max, int layer,
                                 int kv_rows, int t_len) {
  extern __shared__ float sm[];
  constexpr int VEC = VecOf<T>::n;
  int h = blockIdx.x, r = blockIdx.y;
  int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = blockDim.x >> 5;
  float* sc = sm + (size_t)warp * (s_max + hd);
  float* qv = sc + s_max;
  int fill = cache_len[r];
  bool ok = fill >= 0 && fill + t_len <= s_max;
  size_t base = (((size_t)layer * kv_rows + r) * n_heads + h) * (size_t)s_max * hd;
  const T* kb = kv_k + base;
  const T* vb = kv_v + base;
  float scale = rsqrtf((float)hd);
  for (int t = warp; t < t_len; t += nw) {
    size_t o = ((size_t)r * t_len + t) * d + (size_t)h * hd;
    if (!ok) {
      for (int i = lane; i < hd; i += 32) out[o + i] = from_f<T>(0.f);
      continue;
    }
    for (int i = lane; i < hd; i += 32) qv[i] = to_f(q[o + i]);
    __syncwarp();
    int nk = fill + t + 1;
    float mx = -CUDART_INF_F;
    for (int j = lane; j < nk; j += 32) {
      const T* kr = kb + (size_t)j * hd;
      float s = 0.f;
      for (int i = 0; i < hd; i += VEC) {
        float kv[VEC];
        load_vec(kr + i, kv);
#pragma unroll
        for (int e = 0; e < VEC; ++e) s = fmaf(qv[i + e], kv[e], s);
      }
      s *= scale;
      sc[j] = s;
      mx = fmaxf(mx, s);
    }
    mx = warp_max(mx);
    float sum = 0.f;
    for (int j = lane; j < nk; j += 32) {
      float e = expf(sc[j] - mx);
      sc[j] = e;
      sum += e;
    }
    sum = warp_sum(sum);
    __syncwarp();
    float inv = 1.f / sum;
    for (int i = lane; i < hd; i += 32) {
      float acc = 0.f;
      for (int j = 0; j < nk; ++j) acc = fmaf(sc[j], to_f(vb[(size_t)j * hd + i]), acc);
      out[o + i] = from_f<T>(acc * inv);
    }
    __syncwarp();
  }
}

template <typename T>
void launch_attention(const T* q, const T* kv_k, const T* kv_v, const int32_t* cache_len, T* out,
                      const vvs_model_desc& md, int layer, int kv_rows, int n_rows, int t_len,
                      cudaStream_t s) {
  constexpr int kWarps = 4;
  size_t smem = (size_t)kWarps * (md.s_max + md.head_dim) * sizeof(float);
  if (smem > 48 * 1024) ensure_dynamic_smem(reinterpret_cast<const void*>(attention_kernel<T>), (int)smem);
  dim3 grid(md.n_heads, n_rows);
  attention_kernel<T><<<grid, kWarps * 32, smem, s>>>(q, kv_k, kv_v, cache_len, out, md.d_model,
                                                      md.n_heads, md.head_dim, md.s_max, layer,
                                                      kv_rows, t_len);
}

// ---------------------------------------------------------------------------------------------
// act[m, j] = silu(gate[m, j]) * up[m, j]; grid (column chunks of 1024, rows), 4 columns per thread
template <typename T>
__global__ void silu_mul_kernel(float* __restrict__ gu, T* __restrict__ act, int ff, int clear_src) {
  float* row = gu + (size_t)blockIdx.y * 2 * ff;
  T* o = act + (size_t)blockIdx.y * ff;
  const int j = (blockIdx.x * blockDim.x + threadIdx.x) * 4;
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");   // returns at once unless launched as a programmatic dependent
  if (j >= ff) return;                       // ff is a multiple of 8
  const float4 g = *reinterpret_cast<const float4*>(row + j);
  const float4 u = *reinterpret_cast<const float4*>(row + ff + j);
  o[j] = from_f<T>(g.x / (1.f + expf(-g.x)) * u.x);
  o[j + 1] = from_f<T>(g.y / (1.f + expf(-g.y)) * u.y);
  o[j + 2] = from_f<T>(g.z / (1.f + expf(-g.z)) * u.z);
  o[j + 3] = from_f<T>(g.w / (1.f + expf(-g.w)) * u.w);
  if (clear_src) {                             // split-K sums are added into this buffer: leave it zero
    const float4 z = make_float4(0.f, 0.f, 0.f, 0.f);
    *reinterpret_cast<float4*>(row + j) = z;
    *reinterpret_cast<float4*>(row + ff + j) = z;
  }
}

template <typename T>
void launch_silu_mul(float* gu, T* act, int m, int ff, cudaStream_t s, bool clear_src, bool pdl) {
  int clear = clear_src ? 1 : 0;
  void* args[] = {&gu, &act, &ff, &clear};
  launch_dependent(reinterpret_cast<const void*>(silu_mul_kernel<T>), dim3((ff + 1023) / 1024, m), dim3(256), args,
                   pdl, s);
}

// ---------------------------------------------------------------------------------------------
// guided logits / temperature:  l = l_u + s (l_c - l_u)  (or l_c without guidance)
__global__ void guide_kernel(const float* __restrict__ raw, float* __restrict__ logits, int n_images,
                             int n_cfg, int rows_per_seq, int v, float cfg_scale, float inv_temp) {
  int row = blockIdx.x;  // b * rows_per_seq + t
  const float* lc = raw + (size_t)row * v;
  const float* lu = raw + ((size_t)n_images * rows_per_seq + row) * v;
  float* o = logits + (size_t)row * v;
  for (int j = threadIdx.x; j < v; j += blockDim.x) {
    float l = lc[j];
    if (n_cfg == 2) {
      float u = lu[j];
      l = u + cfg_scale * (l - u);
    }
    o[j] = l * inv_temp;
  }
}

void launch_guide(const float* raw, float* logits, int n_images, int n_cfg, int rows_per_seq, int v,
                  float cfg_scale, float inv_temp, cudaStream_t s) {
  guide_kernel<<<n_images * rows_per_seq, 256, 0, s>>>(raw, logits, n_images, n_cfg, rows_per_seq, v,
                                                       cfg_scale, inv_temp);
}

// per-row max and sum of exp(l - max) as a single "tile" of softmax partials
__global__ void row_stats_kernel(const float* __restrict__ logits, float* __restrict__ part_m,
                                 float* __restrict__ part_s, int v) {
  __shared__ float red[32];
  const float* row = logits + (size_t)blockIdx.x * v;
  float mx = -CUDART_INF_F;
  for (int j = threadIdx.x; j < v; j += blockDim.x) mx = fmaxf(mx, row[j]);
  mx = block_max(mx, red);
  float sum = 0.f;
  for (int j = threadIdx.x; j < v; j += blockDim.x) sum += expf(row[j] - mx);
  sum = block_sum(sum, red);
  if (threadIdx.x == 0) {
    part_m[blockIdx.x] = mx;
    part_s[blockIdx.x] = sum;
  }
}

void launch_row_stats(const float* logits, float* part_m, float* part_s, int n_rows, int v,
                      cudaStream_t s) {
  row_stats_kernel<<<n_rows, 256, 0, s>>>(logits, part_m, part_s, v);
}

// explicit instantiations
#define VVS_INSTANTIATE(T)                                                                          \
  template void launch_embed<T>(const T*, const int32_t*, float*, int, int, int, int, int, int32_t*, \
                                cudaStream_t);                                                       \
  template void launch_rmsnorm<T>(const float*, const T*, T*, int, int, float, cudaStream_t);        \
  template void launch_gemm_nt<T>(const T*, const T*, float*, int, int, int, int, bool, cudaStream_t); \
  template void launch_rope_append<T>(float*, const float*, T*, T*, T*, const int32_t*,              \
                                      const vvs_model_desc&, int, int, int, int, int32_t*,           \
                                      cudaStream_t, const float*, const float*, bool);               \
  template void launch_attention<T>(const T*, const T*, const T*, const int32_t*, T*,                \
                                    const vvs_model_desc&, int, int, int, int, cudaStream_t);        \
  template void launch_silu_mul<T>(float*, T*, int, int, cudaStream_t, bool, bool);
VVS_INSTANTIATE(float)
VVS_INSTANTIATE(__nv_bfloat16)

}  // namespace vvs
