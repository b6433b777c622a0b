// Block-vs-cache attention of the verify step on the 5th-generation tensor cores (bf16).
//
// Sequence r, head h: the T <= 32 block rows (queries) attend cache slots [0, L_r + t].  The key
// range is cut into chunks of 128 keys, one CTA per (chunk, head, sequence) (flash-decoding
// style split-KV), so a batch-1 step still fills the GPU and every CTA is a single shot:
//   1. TMA stages the K chunk [128 keys x hd], the V chunk and the Q rows in 128-byte-swizzled
//      shared memory (chunks that lie entirely in the old cache are requested before
//      griddepcontrol.wait, i.e. while the QKV projection is still running).
//   2. S^T = K Q^T  (tcgen05.mma, M = 128 keys, N = 16/32 queries) into TMEM.
//   3. Each thread owns one key: scale, causal mask, per-query max / sum over the 128 keys by
//      warp shuffles + shared memory, P = exp(S - max) written as bf16 into swizzled shared
//      memory.  V rows of masked-out keys are zeroed so stale cache contents cannot leak.
//   4. O^T = V^T P^T  (tcgen05.mma, M = 128 head-dimension rows (rows >= hd are don't-care), N = 16/32
//      queries, V as MN-major A operand, P as K-major B operand of only 16/32 rows: the P tile is
//      4-8 KB instead of the 32 KB a 128-row A operand would take, which is what lets four CTAs
//      share an SM).
//   5. Query rows write (max, sum, O) partials; the CTA that arrives last for (r, h) merges the
//      chunks (exact softmax re-normalisation) and writes the bf16 attention output.  No CTA
//      waits for another.
#include <math_constants.h>

#include "tc_common.cuh"
#include "vvs_internal.cuh"

namespace vvs {

using namespace tc;

namespace {

constexpr int kChunkKeys = 128;

struct AttnParams {
  const int32_t* cache_len;
  const uint32_t* anc_mask;  // [M] block rows visible to each block row (chain or tree)
  __nv_bfloat16* out;     // [M, d]
  float* part_o;          // [R*H, n_chunks_max, T, hd]
  float* part_ml;         // [R*H, n_chunks_max, T, 2]
  int* counters;          // [R*H]
  int32_t* status;
  int d, n_heads, hd, s_max, layer, kv_rows, t_len, tq, n_chunks_max;
  uint32_t tmem_cols;
  float scale;
};

__device__ __forceinline__ bool wait_bounded(uint64_t* bar, uint32_t parity) { return mbar_wait(bar, parity); }

__device__ __forceinline__ float warp_max_f(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ float warp_sum_f(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

template <int HD>
__global__ void __launch_bounds__(128)
attention_tc_kernel(const AttnParams p, const __grid_constant__ CUtensorMap tm_q,
                    const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v) {
  constexpr int NC = HD / 64;                       // 64-column chunks of the head dimension
  constexpr uint32_t kKVBytes = kChunkKeys * 128;   // one 64-column chunk of a K or V tile
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bar_kq, bar_v, bar_s, bar_o;
  __shared__ uint32_t tmem_slot;
  __shared__ float red_max[4][32];
  __shared__ float red_sum[4][32];
  __shared__ int s_last;

  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sK = smem;
  uint8_t* sV = sK + NC * kKVBytes;
  const uint32_t q_chunk_bytes = (uint32_t)p.tq * 128u;
  uint8_t* sP = sV + NC * kKVBytes;                 // 2 chunks of 64 keys: [tq rows x 128 B] each
  uint8_t* sQ = sP + 2 * q_chunk_bytes;             // NC chunks: [tq rows x 128 B]
  float* sS = reinterpret_cast<float*>(sQ + NC * q_chunk_bytes);   // scores, [tq queries][128 keys] fp32

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, tid = threadIdx.x;
  const int c = blockIdx.x, h = blockIdx.y, r = blockIdx.z;
  const int T = p.t_len;

  {
    // chunks beyond this sequence's keys have nothing to do: leave before any set-up (the grid is
    // sized for the longest possible sequence)
    const int fill0 = p.cache_len[r];
    if (fill0 >= 0 && fill0 + T <= p.s_max && c * kChunkKeys >= fill0 + T) return;
  }
  if (tid == 0) {
    mbar_init(&bar_kq, 1);
    mbar_init(&bar_v, 1);
    mbar_init(&bar_s, 1);
    mbar_init(&bar_o, 1);
    fence_barrier_init();
    tma_prefetch_desc(&tm_q);
    tma_prefetch_desc(&tm_k);
    tma_prefetch_desc(&tm_v);
  }
  if (warp == 1) {
    tmem_alloc(&tmem_slot, p.tmem_cols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_slot;
  pdl_launch_dependents();

  const int fill = p.cache_len[r];                  // written by earlier steps, not by the previous kernel
  const bool ok = fill >= 0 && fill + T <= p.s_max;
  const int n_keys = fill + T;
  const int n_chunks = ok ? (n_keys + kChunkKeys - 1) / kChunkKeys : 0;
  const int key0 = c * kChunkKeys;
  bool active = ok && c < n_chunks;
  const int row_base = ((p.layer * p.kv_rows + r) * p.n_heads + h) * p.s_max + key0;
  const bool old_only = key0 + kChunkKeys <= fill;  // chunk holds no row written by this step

  if (!ok && c == 0) {                              // overflowing sequence: defined (zero) output
    pdl_wait();
    for (int i = tid; i < T * HD; i += blockDim.x)
      p.out[((size_t)r * T + i / HD) * p.d + (size_t)h * HD + i % HD] = __float2bfloat16_rn(0.f);
  }

  bool alive = active;
  if (active && tid == 0) {
    mbar_expect_tx(&bar_kq, NC * kKVBytes + NC * q_chunk_bytes);
    mbar_expect_tx(&bar_v, NC * kKVBytes);
    if (old_only) {
      for (int j = 0; j < NC; ++j) tma_load_2d(sK + j * kKVBytes, &tm_k, &bar_kq, j * 64, row_base);
      for (int j = 0; j < NC; ++j) tma_load_2d(sV + j * kKVBytes, &tm_v, &bar_v, j * 64, row_base);
    }
    pdl_wait();
    for (int j = 0; j < NC; ++j) tma_load_2d(sQ + j * q_chunk_bytes, &tm_q, &bar_kq, h * HD + j * 64, r * T);
    if (!old_only) {
      for (int j = 0; j < NC; ++j) tma_load_2d(sK + j * kKVBytes, &tm_k, &bar_kq, j * 64, row_base);
      for (int j = 0; j < NC; ++j) tma_load_2d(sV + j * kKVBytes, &tm_v, &bar_v, j * 64, row_base);
    }
  }
  if (active && warp == 1 && lane == 0) {
    // S^T[key, query] = sum_e K[key, e] Q[query, e]
    if (wait_bounded(&bar_kq, 0)) {
      tc_fence_after();
      const uint32_t idesc = idesc_bf16_f32(128, (uint32_t)p.tq);
#pragma unroll
      for (int k16 = 0; k16 < HD / 16; ++k16) {
        const uint32_t a = smem_u32(sK + (k16 / 4) * kKVBytes) + (k16 % 4) * 32;
        const uint32_t b = smem_u32(sQ + (k16 / 4) * q_chunk_bytes) + (k16 % 4) * 32;
        mma_bf16(tmem_base, smem_desc_sw128(a), smem_desc_sw128(b), idesc, k16 > 0 ? 1u : 0u);
      }
      mma_commit(&bar_s);
    } else {
      atomicOr(p.status, VVS_DEV_TIMEOUT);
    }
  }
  __syncwarp();
  pdl_wait();

  if (active) {
    const bool got = wait_bounded(&bar_s, 0);
    if (__syncthreads_or(got ? 0 : 1)) {
      if (tid == 0) atomicOr(p.status, VVS_DEV_TIMEOUT);
      alive = false;
    }
  }
  if (alive) {
    tc_fence_after();
    const int key = key0 + tid;
    const uint32_t t_row = tmem_base + ((uint32_t)(warp * 32) << 16);
    {
      // scores of this key for all queries -> shared memory, transposed ([query][key], fp32)
      float sc[32];
      tmem_ld16(t_row, sc);
      if (p.tq > 16) tmem_ld16(t_row + 16, sc + 16);
#pragma unroll
      for (int t = 0; t < 32; ++t)
        if (t < p.tq) sS[t * 128 + tid] = sc[t];
    }
    // visibility masks of this sequence's block rows, one per lane (written by the table kernel
    // at the start of the step, several launches ago)
    const uint32_t anc_l = lane < T ? p.anc_mask[r * T + lane] : 0u;
    __syncthreads();
    // eight lanes per query row (16 keys each), sixteen rows per pass: mask, max, exp, sum.
    // Visible: a cache key (kj < 0) or block row kj with its bit set in the row's mask.
#pragma unroll 1
    for (int t0 = 0; t0 < T; t0 += 16) {
      const int t = t0 + warp * 4 + (lane >> 3), sub = lane & 7;
      const bool live = t < T;
      const uint32_t anc = __shfl_sync(0xffffffffu, anc_l, t & 31);
      float sv[16];
      float mx = -CUDART_INF_F;
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        const int cc = (c + (sub >> 1)) & 3;          // rotation: conflict-free 128-bit loads
        float4 s4 = make_float4(0.f, 0.f, 0.f, 0.f);
        if (live) s4 = reinterpret_cast<const float4*>(sS)[t * 32 + sub * 4 + cc];
        const float in[4] = {s4.x, s4.y, s4.z, s4.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const int kj = key0 + sub * 16 + cc * 4 + j - fill;
          const uint32_t vis = (kj < 0 ? 1u : 0u) | (((uint32_t)kj < 32u ? 1u : 0u) & (anc >> (kj & 31)));
          sv[c * 4 + j] = (live && (vis & 1u)) ? in[j] * p.scale : -CUDART_INF_F;
          mx = fmaxf(mx, sv[c * 4 + j]);
        }
      }
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 4));
      float sum = 0.f;
#pragma unroll
      for (int i = 0; i < 16; ++i) {
        sv[i] = (sv[i] == -CUDART_INF_F) ? 0.f : __expf(sv[i] - mx);
        sum += sv[i];
      }
      sum += __shfl_xor_sync(0xffffffffu, sum, 1);
      sum += __shfl_xor_sync(0xffffffffu, sum, 2);
      sum += __shfl_xor_sync(0xffffffffu, sum, 4);
      if (live && sub == 0) {
        red_max[0][t] = mx;
        red_sum[0][t] = sum;
      }
      if (live) {
        // P[t, key] as bf16, K-major rows of 64 keys with the 128-byte swizzle
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          const int cc = (c + (sub >> 1)) & 3;
          const int k4 = sub * 16 + cc * 4;
          uint2 pk;
          *reinterpret_cast<__nv_bfloat162*>(&pk.x) = __floats2bfloat162_rn(sv[c * 4], sv[c * 4 + 1]);
          *reinterpret_cast<__nv_bfloat162*>(&pk.y) = __floats2bfloat162_rn(sv[c * 4 + 2], sv[c * 4 + 3]);
          uint8_t* dst = sP + (k4 >> 6) * q_chunk_bytes + t * 128 + (((((k4 & 63) >> 3) ^ (t & 7)) << 4) | ((k4 & 7) << 1));
          *reinterpret_cast<uint2*>(dst) = pk;
        }
      }
    }
    // V rows of keys that no query may see: cleared, so unwritten cache slots cannot inject NaN
    if (!wait_bounded(&bar_v, 0)) atomicOr(p.status, VVS_DEV_TIMEOUT);
    if (key >= n_keys) {
#pragma unroll
      for (int j = 0; j < NC; ++j) {
        uint4* row = reinterpret_cast<uint4*>(sV + j * kKVBytes + tid * 128);
#pragma unroll
        for (int i = 0; i < 8; ++i) row[i] = make_uint4(0, 0, 0, 0);
      }
    }
    fence_proxy_async();      // generic-proxy writes of P and V visible to the tensor core
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (warp == 1 && lane == 0) {
      // O^T[e, query] = sum_key V[key, e] P[query, key]; with hd = 64 the rows 64..127 of the A operand
      // come from whatever follows the V tile in shared memory and land in TMEM lanes nobody reads
      const uint32_t idesc = idesc_bf16_f32(128, (uint32_t)p.tq) | (1u << 15);  // A is MN-major
#pragma unroll
      for (int k16 = 0; k16 < kChunkKeys / 16; ++k16) {
        const uint32_t a = smem_u32(sV) + k16 * 2048;
        const uint32_t b = smem_u32(sP + (k16 / 4) * q_chunk_bytes) + (k16 % 4) * 32;
        mma_bf16(tmem_base + 32, smem_desc_mn_sw128(a, kKVBytes), smem_desc_sw128(b), idesc, k16 > 0 ? 1u : 0u);
      }
      mma_commit(&bar_o);
    }
    __syncwarp();
    const bool got = wait_bounded(&bar_o, 0);
    if (__syncthreads_or(got ? 0 : 1)) {
      if (tid == 0) atomicOr(p.status, VVS_DEV_TIMEOUT);
      alive = false;
    }
  }
  if (alive) {
    tc_fence_after();
    const size_t rh = (size_t)r * p.n_heads + h;
    if (warp * 32 < HD) {                             // TMEM lane = head-dimension index e
      const int e = warp * 32 + lane;
      const uint32_t t_row = tmem_base + ((uint32_t)(warp * 32) << 16) + 32;
      float o[32];
      tmem_ld16(t_row, o);
      if (p.tq > 16) tmem_ld16(t_row + 16, o + 16);
#pragma unroll
      for (int t = 0; t < 32; ++t) {
        if (t < T) {                                  // chunk-wide max / sum of query t are in red_max / red_sum
          if (n_chunks == 1)
            p.out[((size_t)r * T + t) * p.d + (size_t)h * HD + e] = __float2bfloat16_rn(o[t] / red_sum[0][t]);
          else
            p.part_o[((rh * p.n_chunks_max + c) * T + t) * HD + e] = o[t];
        }
      }
    }
    if (tid < T && n_chunks > 1) {
      float* ml = p.part_ml + ((rh * p.n_chunks_max + c) * T + tid) * 2;
      ml[0] = red_max[0][tid];
      ml[1] = red_sum[0][tid];
    }
    if (n_chunks > 1) {
      __threadfence();
      __syncthreads();
      if (tid == 0) {
        const int prev = atomicAdd(&p.counters[rh], 1);
        s_last = (prev == n_chunks - 1) ? 1 : 0;
      }
      __syncthreads();
      if (s_last) {
        __threadfence();
        for (int i = tid; i < T * HD; i += blockDim.x) {
          const int t = i / HD, e = i - t * HD;
          float m = -CUDART_INF_F;
          for (int cc = 0; cc < n_chunks; ++cc)
            m = fmaxf(m, __ldcg(p.part_ml + ((rh * p.n_chunks_max + cc) * T + t) * 2));
          float num = 0.f, den = 0.f;
          for (int cc = 0; cc < n_chunks; ++cc) {
            const float* ml = p.part_ml + ((rh * p.n_chunks_max + cc) * T + t) * 2;
            const float mc = __ldcg(ml);
            const float w = (mc == -CUDART_INF_F) ? 0.f : expf(mc - m);
            den += w * __ldcg(ml + 1);
            num += w * __ldcg(p.part_o + ((rh * p.n_chunks_max + cc) * T + t) * HD + e);
          }
          p.out[((size_t)r * T + t) * p.d + (size_t)h * HD + e] = __float2bfloat16_rn(num / den);
        }
        if (tid == 0) p.counters[rh] = 0;
      }
    }
  }
  // ---- teardown ---------------------------------------------------------------------------------
  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_base, p.tmem_cols);
}

}  // namespace

int launch_attention_tc(const AttentionTcArgs& a, cudaStream_t s) {
  AttnParams p{};
  p.cache_len = a.cache_len; p.anc_mask = a.anc_mask; p.out = a.out; p.part_o = a.part_o; p.part_ml = a.part_ml;
  p.counters = a.counters; p.status = a.status;
  p.d = a.d; p.n_heads = a.n_heads; p.hd = a.hd; p.s_max = a.s_max; p.layer = a.layer;
  p.kv_rows = a.kv_rows; p.t_len = a.t_len; p.tq = a.t_len <= 16 ? 16 : 32;
  p.n_chunks_max = (a.s_max + kChunkKeys - 1) / kChunkKeys;
  p.tmem_cols = 64u;                                  // scores at column 0, O^T at column 32 (16 or 32 wide each)
  p.scale = 1.0f / sqrtf((float)a.hd);
  const int nc = a.hd / 64;
  // K and V chunk tiles, P (2 key chunks) and Q (nc chunks) of tq rows, transposed scores, alignment slack
  // With hd = 64 the 128-row A operand of O^T = V^T P^T reaches one V tile (16 KB) past the V tile:
  // what follows it must be at least that large, whatever it holds.
  auto tail_bytes = [&](int tq) {
    const int t = (2 + nc) * tq * 128 + tq * 512;
    return (a.hd == 64 && t < kChunkKeys * 128) ? kChunkKeys * 128 : t;
  };
  const int smem = nc * 2 * kChunkKeys * 128 + tail_bytes(p.tq) + 1024;

  const int smem_max = nc * 2 * kChunkKeys * 128 + tail_bytes(32) + 1024;

  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(p.n_chunks_max, a.n_heads, a.n_rows);
  cfg.blockDim = dim3(128, 1, 1);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = a.pdl ? 1 : 0;
  cudaError_t e;
  if (a.hd == 64) {
    if (ensure_dynamic_smem(reinterpret_cast<const void*>(attention_tc_kernel<64>), smem_max) != cudaSuccess)
      return VVS_ERR_CUDA;
    e = cudaLaunchKernelEx(&cfg, attention_tc_kernel<64>, p, *a.tm_q, *a.tm_k, *a.tm_v);
  } else {
    if (ensure_dynamic_smem(reinterpret_cast<const void*>(attention_tc_kernel<128>), smem_max) != cudaSuccess)
      return VVS_ERR_CUDA;
    e = cudaLaunchKernelEx(&cfg, attention_tc_kernel<128>, p, *a.tm_q, *a.tm_k, *a.tm_v);
  }
  return e == cudaSuccess ? VVS_OK : VVS_ERR_CUDA;
}

}  // namespace vvs
