// The decoder chain of the verify step as ONE persistent kernel (bf16, at most 32 block tokens).
//
// Status: previous generation.  The per-projection kernels (gemm_tc.cu, attention_rows.cu) with
// programmatic dependent launch were measured faster at both benchmark shapes and are the default;
// this kernel runs only in contexts created under the debug switch VVS_DEBUG_CHAIN_KERNELS with
// arrival-order sums, and stays parity-tested.
//
// A batch-1 verify step is a chain of ~180 dependent small projections: run as separate kernels
// it is bound by launch, fill and drain latency, not by the weight stream.  Here one CTA per SM
// stays resident for the whole chain and the work of every phase is cut into fixed shares:
//
//   warp 0      weight producer: walks the CTA's share of every projection of every layer, in
//               order, and streams 128-row x 64-column weight slabs through a TMA ring.  It waits
//               for nothing but a free ring slot, so the HBM stream runs ahead of the dependency
//               chain by the depth of the ring (all SMs together hold most of a layer).
//   warp 1      MMA issuer (tcgen05.mma, weights on the M = 128 side, the <= 32 tokens on N;
//               accumulators in TMEM), also for the attention products.
//   warps 6-9   operand builders: turn the fp32 results of the previous phase into the bf16
//               token operand of this phase, directly in 128-byte-swizzled shared memory:
//               x * norm scale (the 1/rms factor is applied to the product afterwards), merged
//               split-KV attention output, silu(gate) * up.
//   warps 2-5   epilogue: read accumulators (tcgen05.ld) and add them into fp32 accumulators in
//               L2 (split-K by red.global.add), the residual stream for o / down projections.
//
// Phases of a layer: QKV projection | attention | output projection | gate+up | down, separated
// by grid barriers (an arrival counter in global memory; every wait in this file is bounded and
// falls through once the abort flag is raised, so a broken schedule ends as VVS_DEV_TIMEOUT).
// Attention: work items (sequence, head, 128-key chunk); K / V chunks come by TMA (the first
// item of the next layer is requested a whole layer ahead), the block's own K / V rows are
// rotated, written to the cache and patched into the staged tiles, S^T = K Q^T and O = P V run
// on the tensor cores, partial (max, sum, O) go to global memory and are merged by the builders
// of the output projection.
#include <math_constants.h>

#include "tc_common.cuh"
#include "vvs_internal.cuh"

// Event trace hooks: empty unless a profiling build defines them before this point.
#ifndef VVS_TRACE
#define VVS_TRACE_DECL
#define VVS_TRACE(tag) ((void)0)
#define VVS_TRACE_MMA(tag) ((void)0)   // inside the MMA warp's layer loop (layer index `l` in scope)
#define VVS_TRACE_END ((void)0)
#endif

namespace vvs {

using namespace tc;

namespace {

constexpr int kThreads = 320;
constexpr int kWorkers = 256;          // warps 2-9
constexpr int kGroup = 128;
constexpr int kSlabBytes = 16384;      // 128 weight rows x 64 bf16
constexpr int kTokSlabBytes = 4096;    // 32 tokens x 64 bf16
constexpr int kStageBytes = kSlabBytes + kTokSlabBytes;   // one ring stage: weight slab + token slab
constexpr int kAccSlots = 4;           // TMEM accumulator slots of 64 columns
constexpr int kMaxStages = 10;
constexpr int kMaxSeq = 32;
constexpr int kMaxLayers = 64;
constexpr uint32_t kColS = 256, kColO = 320, kTmemCols = 512;
constexpr uint32_t kGridSpinLimit = 1u << 21;
constexpr uint32_t kParkNs = 4000;          // a parked wait answers after at most this long
constexpr uint32_t kParkedPolls = 1u << 19;  // ~2 s before a wait gives up
enum { BAR_W = 1, BAR_E = 2, BAR_D = 3 };
enum { PH_QKV = 0, PH_O = 1, PH_GU = 2, PH_DOWN = 3 };

struct ChainParams {
  int n_layers, d, n_heads, hd, ff, s_max, kv_rows;
  int m, t_len, tq, n_rows, n_images, tok_rows;
  int n_stages, n_chunks_max;
  float eps, scale;
  const CUtensorMap* wmaps;            // device [n_layers][5]: qkv, o, gate, up, down
  const __nv_bfloat16* tok_emb;
  const int32_t* block;
  float* x;                            // [m, d] residual stream
  float* qkv_acc;                      // [2][m, 3d]
  float* gu_acc;                       // [2][m, 2ff]
  float* ss;                           // [2 * n_layers][32] sums of squares of x rows
  const int32_t* cache_len;
  const uint32_t* anc_mask;            // [m] block rows visible to each block row (chain or tree)
  __nv_bfloat16* kv_k;
  __nv_bfloat16* kv_v;
  const float* rope_cos;
  const float* rope_sin;
  float* part_o;
  float* part_ml;
  unsigned* sync_words;                // [0] arrivals, [1] epoch base, [2] abort
  int32_t* status;
  const __nv_bfloat16* norms[2 * kMaxLayers];   // norm scales, read through the constant bank
};

struct Phase {
  int tiles, kbs, dual, map0;
};

__device__ __forceinline__ Phase phase_of(const ChainParams& p, int ph) {
  Phase f;
  if (ph == PH_QKV) {
    f.tiles = (3 * p.d + 127) >> 7; f.kbs = (p.d + 63) >> 6; f.dual = 0; f.map0 = 0;
  } else if (ph == PH_O) {
    f.tiles = (p.d + 127) >> 7; f.kbs = (p.d + 63) >> 6; f.dual = 0; f.map0 = 1;
  } else if (ph == PH_GU) {
    f.tiles = (p.ff + 127) >> 7; f.kbs = (p.d + 63) >> 6; f.dual = 1; f.map0 = 2;
  } else {
    f.tiles = (p.d + 127) >> 7; f.kbs = (p.ff + 63) >> 6; f.dual = 0; f.map0 = 4;
  }
  return f;
}

// Share of a projection owned by this CTA: a contiguous range of (tile, k-block) units in
// tile-major order; the rotation moves the CTAs that get one unit more from phase to phase.
// (tiles * k-blocks * grid stays far below 2^32 for every supported shape.)
__device__ __forceinline__ void unit_range(const Phase& f, int layer, int ph, int& lo, int& hi) {
  const unsigned G = gridDim.x, S = (unsigned)(f.tiles * f.kbs);
  const unsigned v = (blockIdx.x + (unsigned)(layer * 4 + ph) * 53u) % G;
  lo = (int)(v * S / G);
  hi = (int)((v + 1) * S / G);
}

// Bounded wait; falls through at once when the CTA is in abort mode.
__device__ __noinline__ bool wait_bar(uint64_t* bar, uint32_t parity, volatile int* s_abort, int32_t* status) {
  if (*s_abort) return false;
  for (uint32_t i = 0; i < kParkedPolls; ++i) {
    if (mbar_try_wait_parked(bar, parity, kParkNs)) return true;
    if ((i & 15u) == 15u && *s_abort) return false;
  }
  *s_abort = 1;
  atomicOr(status, VVS_DEV_TIMEOUT);
  return false;
}

__device__ __forceinline__ void unpack8(const uint4& u, float* o) {
  const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&u);
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const float2 f = __bfloat1622float2(h[j]);
    o[2 * j] = f.x;
    o[2 * j + 1] = f.y;
  }
}
__device__ __forceinline__ uint4 pack8(const float* v) {
  uint4 u;
  __nv_bfloat162* h = reinterpret_cast<__nv_bfloat162*>(&u);
#pragma unroll
  for (int j = 0; j < 4; ++j) h[j] = __floats2bfloat162_rn(v[2 * j], v[2 * j + 1]);
  return u;
}
__device__ __forceinline__ void ldcg8(const float* p, float* o) {
  const float4 a = __ldcg(reinterpret_cast<const float4*>(p));
  const float4 b = __ldcg(reinterpret_cast<const float4*>(p) + 1);
  o[0] = a.x; o[1] = a.y; o[2] = a.z; o[3] = a.w;
  o[4] = b.x; o[5] = b.y; o[6] = b.z; o[7] = b.w;
}
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

// Rotate the consecutive pairs of 8 values (elements e .. e+7 of a head) of token `tok`.
__device__ __forceinline__ void rope8(const ChainParams& p, int tok, int e, float* v) {
  const float* cs = p.rope_cos + (size_t)tok * (p.hd >> 1) + (e >> 1);
  const float* sn = p.rope_sin + (size_t)tok * (p.hd >> 1) + (e >> 1);
  const float4 c4 = __ldcg(reinterpret_cast<const float4*>(cs));
  const float4 s4 = __ldcg(reinterpret_cast<const float4*>(sn));
  const float c[4] = {c4.x, c4.y, c4.z, c4.w}, s[4] = {s4.x, s4.y, s4.z, s4.w};
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const float a = v[2 * j], b = v[2 * j + 1];
    v[2 * j] = a * c[j] - b * s[j];
    v[2 * j + 1] = b * c[j] + a * s[j];
  }
}

// The MMA warp runs its loop with all 32 lanes (so that descriptors and addresses stay warp-uniform
// values); the lane elected once at the start of the role issues, as a predicated instruction
// (an election per instruction cost ~0.2 us per layer, a lone lane running the loop far more).
__device__ __forceinline__ void mma_pred(uint32_t leader, uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                         uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred pe, pa;\n\t"
      "setp.ne.b32 pe, %5, 0;\n\t"
      "setp.ne.b32 pa, %4, 0;\n\t"
      "@pe tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, pa;\n\t}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(leader)
      : "memory");
}
__device__ __forceinline__ void commit_pred(uint32_t leader, uint64_t* bar) {
  asm volatile(
      "{\n\t.reg .pred pe;\n\t"
      "setp.ne.b32 pe, %1, 0;\n\t"
      "@pe tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n\t}"
      ::"r"(smem_u32(bar)), "r"(leader)
      : "memory");
}

// Fast path of a wait: one poll, inline.
__device__ __forceinline__ bool wait_fast(uint64_t* bar, uint32_t parity, volatile int* s_abort, int32_t* status) {
  if (mbar_try_wait(bar, parity)) return true;
  return wait_bar(bar, parity, s_abort, status);
}

// x / d for 0 <= x < 2^21 and d >= 1 through the float unit (a handful of instructions; an integer
// division is a dependent chain of ~30).  (x + 0.5) / d is at least 1 / (2d) away from every
// integer; reciprocal and product are each rounded once, an error below (x / d) * 2^-23 < 1 / (4d).
__device__ __forceinline__ int div_small(int x, int d) {
  return (int)(((float)x + 0.5f) * __frcp_rn((float)d));
}

// One round of token-operand building by the 256 worker threads: nb <= (1 << lg) units,
// 256 >> lg threads per unit.  A unit's slab is m rows x 8 groups of 8 columns (one 16-byte
// swizzle chunk each); thread j of the unit takes group j & 7 of rows (j >> 3) + k * (tpu >> 3),
// so eight consecutive lanes read one row's 256 contiguous bytes and every load of the round is
// in flight before the first use (MAXI = rows per thread; 32 rows need MAXI = 1 << lg).
//   DOWN == false: slab = bf16(x * norm scale); the CTAs that own tile 0 also add the row sums
//                  of squares into ss_out
//   DOWN == true : slab = bf16(silu(gate / rms) * (up / rms)), rms from ss_in
template <int MAXI, bool DOWN>
__device__ __noinline__ void build_round(const ChainParams& p, uint8_t* ring, uint64_t* empty, volatile int* s_abort,
                                         int tid_w, int nb, int lg, uint32_t it0, uint32_t per_unit, int s0, int kbs,
                                         const float* src, const __nv_bfloat16* gsc, const float* ss_in,
                                         float* ss_out) {
  const uint32_t NS = (uint32_t)p.n_stages;
  const int tpu = 256 >> lg, u = tid_w >> (8 - lg), j = tid_w & (tpu - 1);
  if (u >= nb) return;                                   // uniform per warp (tpu >= 32)
  const uint32_t it = it0 + (uint32_t)u * per_unit;
  const uint32_t use = (uint32_t)div_small((int)it, (int)NS), st = it - use * NS;
  if (use > 0) wait_fast(&empty[st], (use - 1) & 1, s_abort, p.status);
  const int s = s0 + u, tile = div_small(s, kbs), kb = s - tile * kbs;
  const int m = p.m, ff = p.ff;
  const int q = j & 7, row0 = j >> 3, rstep = tpu >> 3;
  const int col = kb * 64 + q * 8;
  const int ld = DOWN ? 2 * ff : p.d;
  const float* sp = src + (size_t)row0 * ld + col;
  const size_t sstep = (size_t)rstep * ld;
  const bool col_ok = !DOWN || col < ff;
  const float4 z4 = make_float4(0.f, 0.f, 0.f, 0.f);
  float4 a0[MAXI], a1[MAXI];
  float4 b0[DOWN ? MAXI : 1], b1[DOWN ? MAXI : 1];
  float sv[DOWN ? MAXI : 1];
  uint4 g = make_uint4(0u, 0u, 0u, 0u);
  if (!DOWN) g = __ldg(reinterpret_cast<const uint4*>(gsc + col));
#pragma unroll
  for (int k = 0; k < MAXI; ++k) {
    a0[k] = z4;
    a1[k] = z4;
    if (DOWN) { b0[k] = z4; b1[k] = z4; sv[k] = 1.f; }
    if (row0 + k * rstep < m) {
      if (col_ok) {
        a0[k] = __ldcg(reinterpret_cast<const float4*>(sp));
        a1[k] = __ldcg(reinterpret_cast<const float4*>(sp) + 1);
        if (DOWN) {
          b0[k] = __ldcg(reinterpret_cast<const float4*>(sp + ff));
          b1[k] = __ldcg(reinterpret_cast<const float4*>(sp + ff) + 1);
        }
      }
      if (DOWN) sv[k] = __ldcg(ss_in + row0 + k * rstep);
    }
    sp += sstep;
  }
  float gv[8];
  unpack8(g, gv);
  const float inv_d = 1.f / (float)p.d, eps = p.eps;
  uint8_t* out = ring + (size_t)st * kStageBytes + kSlabBytes;
#pragma unroll
  for (int k = 0; k < MAXI; ++k) {
    const int row = row0 + k * rstep;
    float v[8] = {a0[k].x, a0[k].y, a0[k].z, a0[k].w, a1[k].x, a1[k].y, a1[k].z, a1[k].w};
    if (DOWN) {
      const float rinv = rsqrtf(fmaf(sv[k], inv_d, eps));
      const float w[8] = {b0[k].x, b0[k].y, b0[k].z, b0[k].w, b1[k].x, b1[k].y, b1[k].z, b1[k].w};
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const float t = v[e] * rinv;
        v[e] = __fdividef(t, 1.f + __expf(-t)) * (w[e] * rinv);
      }
    } else {
      if (tile == 0) {                                   // uniform per warp
        float ssq = 0.f;
#pragma unroll
        for (int e = 0; e < 8; ++e) ssq = fmaf(v[e], v[e], ssq);
        ssq += __shfl_xor_sync(0xffffffffu, ssq, 4);     // 8 lanes = one row
        ssq += __shfl_xor_sync(0xffffffffu, ssq, 2);
        ssq += __shfl_xor_sync(0xffffffffu, ssq, 1);
        if (q == 0 && row < m) atomicAdd(ss_out + row, ssq);
      }
#pragma unroll
      for (int e = 0; e < 8; ++e) v[e] *= gv[e];
    }
    if (row < m) *reinterpret_cast<uint4*>(out + row * 128 + ((q ^ (row & 7)) << 4)) = pack8(v);
  }
}

__global__ void __launch_bounds__(kThreads, 1)
fused_chain_kernel(const __grid_constant__ ChainParams p, const __grid_constant__ CUtensorMap tm_k,
                   const __grid_constant__ CUtensorMap tm_v) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t full[kMaxStages], empty[kMaxStages];
  __shared__ __align__(8) uint64_t acc_full[kAccSlots], acc_empty[kAccSlots];
  __shared__ __align__(8) uint64_t att_kv_full, att_q_ready, att_s_full, att_p_ready, att_o_full;
  __shared__ uint32_t tmem_slot;
  __shared__ volatile int s_abort;
  __shared__ int s_fill[kMaxSeq], s_nch[kMaxSeq], s_prefix[kMaxSeq + 1];
  __shared__ uint32_t s_anc[32];
  __shared__ float row_max[32], row_sum[32];
  VVS_TRACE_DECL

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int G = (int)gridDim.x;
  const int NC = p.hd >> 6;                       // 64-column chunks of a head
  const uint32_t NS = (uint32_t)p.n_stages;
  const int T = p.t_len, H = p.n_heads, L = p.n_layers;

  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* ring = smem;                           // n_stages x [weight slab | token slab]
  uint8_t* sK = ring + (size_t)NS * kStageBytes;
  uint8_t* sV = sK + NC * kSlabBytes;
  uint8_t* sP = sV + NC * kSlabBytes;             // 2 x [128 rows x 128 B]
  uint8_t* sQ = sP + 2 * kSlabBytes;              // NC x [tq rows x 128 B]
  const uint32_t q_chunk_bytes = (uint32_t)p.tq * 128u;

  // ---- set-up ------------------------------------------------------------------------------------
  if (tid == 0) {
    for (uint32_t i = 0; i < NS; ++i) { mbar_init(&full[i], 2); mbar_init(&empty[i], 1); }   // TMA + builders
    for (int i = 0; i < kAccSlots; ++i) { mbar_init(&acc_full[i], 1); mbar_init(&acc_empty[i], 1); }
    mbar_init(&att_kv_full, 1);
    mbar_init(&att_q_ready, 2);   // the Q builders and the K / V row builders
    mbar_init(&att_s_full, 1);
    mbar_init(&att_p_ready, 1);
    mbar_init(&att_o_full, 1);
    s_abort = 0;
    fence_barrier_init();
    tma_prefetch_desc(&tm_k);
    tma_prefetch_desc(&tm_v);
    // sequences: fill level, number of 128-key chunks, prefix of chunk counts
    int acc = 0;
    for (int r = 0; r < p.n_rows; ++r) {
      const int fill = p.cache_len[r];
      const bool ok = fill >= 0 && fill + T <= p.s_max;
      s_fill[r] = fill;
      s_nch[r] = ok ? (fill + T + 127) >> 7 : 0;
      s_prefix[r] = acc;
      acc += s_nch[r];
    }
    s_prefix[p.n_rows] = acc;
  }
  if (tid >= 32 && tid < 64) s_anc[tid - 32] = (int)(tid - 32) < p.m ? p.anc_mask[tid - 32] : 0u;
  // token operands: rows of tokens that do not exist stay zero for the whole kernel
  for (uint32_t i = tid; i < NS * (kTokSlabBytes / 16); i += kThreads)
    reinterpret_cast<uint4*>(ring + (size_t)(i / (kTokSlabBytes / 16)) * kStageBytes + kSlabBytes)[i % (kTokSlabBytes / 16)] =
        make_uint4(0, 0, 0, 0);
  for (int i = tid; i < (int)(NC * q_chunk_bytes) / 16; i += kThreads)
    reinterpret_cast<uint4*>(sQ)[i] = make_uint4(0, 0, 0, 0);
  if (warp == 1) {
    tmem_alloc(&tmem_slot, kTmemCols);
    tmem_relinquish();
  }
  fence_proxy_async();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_slot;
  const unsigned epoch = *reinterpret_cast<volatile unsigned*>(p.sync_words + 1);
  const int n_items = s_prefix[p.n_rows] * H;     // attention items of one layer, all CTAs

  auto decode_item = [&](int i, int& r, int& h, int& c) {
    const int rc = div_small(i, H);
    h = i - rc * H;
    r = 0;
    while (r + 1 < p.n_rows && s_prefix[r + 1] <= rc) ++r;
    c = rc - s_prefix[r];
  };
  auto kv_row_base = [&](int layer, int r, int h, int c) {
    return ((layer * p.kv_rows + r) * H + h) * p.s_max + c * 128;
  };

  if (warp == 0) {
    // =================================== weight producer ===========================================
    if (lane == 0) {
      uint32_t st = 0, round = 0;
      bool alive = true;
#pragma unroll 1
      for (int l = 0; l < L && alive; ++l) {
#pragma unroll 1
        for (int ph = 0; ph < 4 && alive; ++ph) {
          const Phase f = phase_of(p, ph);
          int lo, hi;
          unit_range(f, l, ph, lo, hi);
          int tile = lo / f.kbs, kb = lo - tile * f.kbs;
          const CUtensorMap* map = &p.wmaps[l * 5 + f.map0];
#pragma unroll 1
          for (int s = lo; s < hi && alive; ++s) {
            for (int j = 0; j <= f.dual; ++j) {
              if (round > 0 && !wait_bar(&empty[st], (round - 1) & 1, &s_abort, p.status)) { alive = false; break; }
              mbar_expect_tx(&full[st], kSlabBytes);
              tma_load_2d(ring + (size_t)st * kStageBytes, map + j, &full[st], kb * 64, tile * 128);
              VVS_TRACE(0x100 | (ph << 4) | ((s - lo) & 15));
              if (++st == NS) { st = 0; ++round; }
            }
            if (++kb == f.kbs) { kb = 0; ++tile; }
          }
        }
      }
      // In abort mode loads may still be in flight with nobody waiting for them: let them land.
      if (s_abort) __nanosleep(200000);
    }
  } else if (warp == 1) {
    // =================================== MMA issuer ==================================================
    {
      uint32_t st = 0, par = 0, ita = 0, iatt = 0;
      // one lane is elected once; every MMA and commit below is predicated on it, so the whole
      // warp runs the loop and its waits without diverging
      uint32_t leader;
      asm volatile("{\n\t.reg .pred pe;\n\telect.sync _|pe, 0xffffffff;\n\tselp.u32 %0, 1, 0, pe;\n\t}" : "=r"(leader));
      bool alive = true;
      const uint32_t idesc_gemm = idesc_bf16_f32(128, 32);
      const uint64_t desc0 = smem_desc_sw128(smem_u32(ring));   // + (byte offset >> 4) selects a slab
#pragma unroll 1
      for (int l = 0; l < L && alive; ++l) {
#pragma unroll 1
        for (int ph = 0; ph < 4 && alive; ++ph) {
          if (ph == PH_O) {
            // ---- attention products of this CTA's items ----
#pragma unroll 1
            for (int i = blockIdx.x; i < n_items && alive; i += G, ++iatt) {
              const uint32_t apar = iatt & 1;
              if (!wait_bar(&att_kv_full, apar, &s_abort, p.status) ||
                  !wait_bar(&att_q_ready, apar, &s_abort, p.status)) { alive = false; break; }
              __syncwarp();
              tc_fence_after();
              VVS_TRACE_MMA(0x2F1);
              const uint32_t idesc_s = idesc_bf16_f32(128, (uint32_t)p.tq);
              for (int k16 = 0; k16 < p.hd / 16; ++k16) {
                const uint32_t a = smem_u32(sK + (k16 >> 2) * kSlabBytes) + (k16 & 3) * 32;
                const uint32_t b = smem_u32(sQ + (k16 >> 2) * q_chunk_bytes) + (k16 & 3) * 32;
                mma_pred(leader, tmem_base + kColS, smem_desc_sw128(a), smem_desc_sw128(b), idesc_s, k16 > 0 ? 1u : 0u);
              }
              commit_pred(leader, &att_s_full);
              VVS_TRACE_MMA(0x2F2);
              if (!wait_bar(&att_p_ready, apar, &s_abort, p.status)) { alive = false; break; }
              __syncwarp();
              tc_fence_after();
              VVS_TRACE_MMA(0x2F3);
              const uint32_t idesc_o = idesc_bf16_f32(128, (uint32_t)p.hd) | (1u << 16);  // B is MN-major
              for (int k16 = 0; k16 < 8; ++k16) {
                const uint32_t a = smem_u32(sP + (k16 >> 2) * kSlabBytes) + (k16 & 3) * 32;
                const uint32_t b = smem_u32(sV) + k16 * 2048;
                mma_pred(leader, tmem_base + kColO, smem_desc_sw128(a), smem_desc_mn_sw128(b, kSlabBytes), idesc_o,
                         k16 > 0 ? 1u : 0u);
              }
              commit_pred(leader, &att_o_full);
              VVS_TRACE_MMA(0x2F4);
            }
            if (!alive) break;
          }
          const Phase f = phase_of(p, ph);
          int lo, hi;
          unit_range(f, l, ph, lo, hi);
          int kb = lo % f.kbs;
          uint32_t slot = 0;
#pragma unroll 1
          for (int s = lo; s < hi; ++s) {
            const bool first = (s == lo) || (kb == 0);
            if (first) {
              if (s != lo) commit_pred(leader, &acc_full[slot]);
              slot = ita % kAccSlots;
              const uint32_t use = ita / kAccSlots;
              if (use > 0 && !wait_bar(&acc_empty[slot], (use - 1) & 1, &s_abort, p.status)) { alive = false; break; }
              ++ita;
            }
            if (!wait_fast(&full[st], par, &s_abort, p.status)) { alive = false; break; }
            const uint64_t a_desc = desc0 + (uint64_t)(st * (kStageBytes >> 4));
            const uint64_t b_desc = a_desc + (kSlabBytes >> 4);
            const uint32_t st_a = st;
            if (++st == NS) { st = 0; par ^= 1; }
            uint64_t a2_desc = 0;
            uint32_t st_b = 0;
            if (f.dual) {
              if (!wait_fast(&full[st], par, &s_abort, p.status)) { alive = false; break; }
              a2_desc = desc0 + (uint64_t)(st * (kStageBytes >> 4));
              st_b = st;
              if (++st == NS) { st = 0; par ^= 1; }
            }
            __syncwarp();
            tc_fence_after();
            VVS_TRACE_MMA(0x200 | (ph << 4) | ((s - lo) & 15));
            const uint32_t acc = tmem_base + slot * 64;
            mma_pred(leader, acc, a_desc, b_desc, idesc_gemm, first ? 0u : 1u);
            mma_pred(leader, acc, a_desc + 2, b_desc + 2, idesc_gemm, 1u);
            mma_pred(leader, acc, a_desc + 4, b_desc + 4, idesc_gemm, 1u);
            mma_pred(leader, acc, a_desc + 6, b_desc + 6, idesc_gemm, 1u);
            if (f.dual) {
              // the second weight slab multiplies the token slab of the FIRST stage: that stage is
              // released only after these have been issued as well
              mma_pred(leader, acc + 32, a2_desc, b_desc, idesc_gemm, first ? 0u : 1u);
              mma_pred(leader, acc + 32, a2_desc + 2, b_desc + 2, idesc_gemm, 1u);
              mma_pred(leader, acc + 32, a2_desc + 4, b_desc + 4, idesc_gemm, 1u);
              mma_pred(leader, acc + 32, a2_desc + 6, b_desc + 6, idesc_gemm, 1u);
              commit_pred(leader, &empty[st_a]);
              commit_pred(leader, &empty[st_b]);
            } else {
              commit_pred(leader, &empty[st_a]);
            }
            VVS_TRACE_MMA(0x280 | (ph << 4) | ((s - lo) & 15));
            if (++kb == f.kbs) kb = 0;
          }
          if (alive && hi > lo) commit_pred(leader, &acc_full[slot]);
        }
      }
    }
  } else {
    // =================================== workers (warps 2-9) =========================================
    const bool grp_e = warp < 6;
    const int tid_w = tid - 64;
    const int tid_g = grp_e ? tid - 64 : tid - 192;   // index inside the group of 128
    const int quarter = warp & 3;                     // TMEM lane quarter this warp may read
    unsigned target = epoch;
    uint32_t it_slab = 0, ita = 0, iatt = 0;         // ring position at the start of the phase, items, att items

    // Plan of the projection that follows the next grid barrier (its share of units): worked out
    // between the arrival at the barrier and the first poll, where its integer divisions cost
    // nothing, instead of after the release, where they sat on every phase's critical path.
    Phase f = phase_of(p, PH_QKV);
    int lo = 0, hi = 0;
    auto grid_sync = [&](int next_l, int next_ph) {
      if (tid_w == 0) VVS_TRACE(0x900);
      named_bar_sync(BAR_W, kWorkers);
      target += (unsigned)G;
      if (tid_w == 0) VVS_TRACE(0x901);
      const bool poll = tid_w == 0 && !s_abort;
      if (poll) {
        __threadfence();
        atomicAdd(p.sync_words, 1u);
      }
      if (next_ph >= 0) {
        f = phase_of(p, next_ph);
        unit_range(f, next_l, next_ph, lo, hi);
      }
      if (poll) {
        bool ok = false;
        for (uint32_t i = 0; i < kGridSpinLimit; ++i) {
          if ((int)(ld_acquire_gpu(p.sync_words) - target) >= 0) { ok = true; break; }
          if ((i & 63u) == 63u && *reinterpret_cast<volatile unsigned*>(p.sync_words + 2)) break;
        }
        if (!ok) {
          s_abort = 1;
          *reinterpret_cast<volatile unsigned*>(p.sync_words + 2) = 1u;
          atomicOr(p.status, VVS_DEV_TIMEOUT);
        }
        VVS_TRACE(0x902);
      }
      named_bar_sync(BAR_W, kWorkers);
    };
    auto issue_kv = [&](int layer, int item) {   // one thread
      int r, h, c;
      decode_item(item, r, h, c);
      const int row = kv_row_base(layer, r, h, c);
      mbar_expect_tx(&att_kv_full, (uint32_t)(2 * NC * kSlabBytes));
      for (int j = 0; j < NC; ++j) tma_load_2d(sK + j * kSlabBytes, &tm_k, &att_kv_full, j * 64, row);
      for (int j = 0; j < NC; ++j) tma_load_2d(sV + j * kSlabBytes, &tm_v, &att_kv_full, j * 64, row);
    };
    // A CTA's second item of a layer: its K tile is requested as soon as the first item's score MMA
    // has read the staging buffer, its V tile once the output MMA has; the K request only raises
    // the byte count of the barrier's next phase, the V request also arrives on it.
    auto issue_next_k = [&](int layer, int item) {   // one thread
      int r, h, c;
      decode_item(item, r, h, c);
      const int row = kv_row_base(layer, r, h, c);
      mbar_expect_tx_only(&att_kv_full, (uint32_t)(NC * kSlabBytes));
      for (int j = 0; j < NC; ++j) tma_load_2d(sK + j * kSlabBytes, &tm_k, &att_kv_full, j * 64, row);
    };
    auto issue_next_v = [&](int layer, int item) {   // one thread
      int r, h, c;
      decode_item(item, r, h, c);
      const int row = kv_row_base(layer, r, h, c);
      mbar_expect_tx(&att_kv_full, (uint32_t)(NC * kSlabBytes));
      for (int j = 0; j < NC; ++j) tma_load_2d(sV + j * kSlabBytes, &tm_v, &att_kv_full, j * 64, row);
    };

    // ---- phase 0: clear the accumulators, gather the embeddings ----
    {
      const int gtid = blockIdx.x * kWorkers + tid_w, gstride = G * kWorkers;
      const float4 z = make_float4(0.f, 0.f, 0.f, 0.f);
      const int nq = (2 * p.m * 3 * p.d) >> 2, ng = (2 * p.m * 2 * p.ff) >> 2, ns = (2 * L * 32) >> 2;
#pragma unroll 1
      for (int i = gtid; i < nq; i += gstride) reinterpret_cast<float4*>(p.qkv_acc)[i] = z;
#pragma unroll 1
      for (int i = gtid; i < ng; i += gstride) reinterpret_cast<float4*>(p.gu_acc)[i] = z;
#pragma unroll 1
      for (int i = gtid; i < ns; i += gstride) reinterpret_cast<float4*>(p.ss)[i] = z;
      const int per_row = p.d >> 3;
#pragma unroll 1
      for (int i = gtid; i < p.m * per_row; i += gstride) {
        const int tok = i / per_row, ch = i - tok * per_row;
        const int r = tok / T, t = tok - r * T, b = r % p.n_images;
        const int token = p.block[b * T + t];
        const bool ok = token >= 0 && token < p.tok_rows;
        float v[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
        if (ok) unpack8(__ldg(reinterpret_cast<const uint4*>(p.tok_emb + (size_t)token * p.d) + ch), v);
        else if (ch == 0) atomicOr(p.status, VVS_DEV_BAD_TOKEN);
        float4* dst = reinterpret_cast<float4*>(p.x + (size_t)tok * p.d) + 2 * ch;
        dst[0] = make_float4(v[0], v[1], v[2], v[3]);
        dst[1] = make_float4(v[4], v[5], v[6], v[7]);
      }
      if (!grp_e && tid_g == 0 && (int)blockIdx.x < n_items) issue_kv(0, blockIdx.x);
      grid_sync(0, PH_QKV);
    }

    // per-thread constants of the merge builders (128 threads per unit: token, 16 columns)
    const int b_tok = tid_g >> 2, b_qtr = tid_g & 3;
    const int b_r = b_tok / T, b_t = b_tok - b_r * T;

#pragma unroll 1
    for (int l = 0; l < L; ++l) {
      const int par_l = l & 1;
      float* qkv = p.qkv_acc + (size_t)par_l * p.m * 3 * p.d;
      float* gu = p.gu_acc + (size_t)par_l * p.m * 2 * p.ff;
      // The norm scales of a layer are first touched by its builders, right after a grid barrier:
      // a miss to HBM there sits on the critical path, so the next layer's are pulled into L2 now.
      if (l + 1 < L && tid_w < 2 * ((p.d + 63) >> 6)) {
        const int which = tid_w & 1, line = tid_w >> 1;
        const __nv_bfloat16* nx = p.norms[(l + 1) * 2 + which] + line * 64;
        asm volatile("prefetch.global.L2 [%0];" ::"l"(nx));
      }
#pragma unroll 1
      for (int ph = 0; ph < 4; ++ph) {
        if (ph == PH_O) {
          // ================================ attention ================================================
          int n_mine = 0;
#pragma unroll 1
          for (int i = blockIdx.x; i < n_items; i += G, ++iatt, ++n_mine) {
            int r, h, c;
            decode_item(i, r, h, c);
            const uint32_t par = iatt & 1;
            const int fill = s_fill[r], n_keys = fill + T, key0 = c * 128;
            const int row_base = kv_row_base(l, r, h, c);
            const int per_head = p.hd >> 3;
            const int ph_sh = p.hd == 64 ? 3 : 4;            // head_dim is 64 or 128: shifts, not divisions
            const float inv_d = 1.f / (float)p.d;
            if (!grp_e) {
              // Q operand: q * (1/rms) rotated, bf16, K-major with the 128-byte swizzle
#pragma unroll 1
              for (int idx = tid_g; idx < T * per_head; idx += kGroup) {
                const int t = idx >> ph_sh, ch = idx - (t << ph_sh), e = ch << 3, tok = r * T + t;
                const float ssv = __ldcg(p.ss + (2 * l) * 32 + tok);
                float v[8];
                ldcg8(qkv + (size_t)tok * 3 * p.d + h * p.hd + e, v);
                const float rinv = rsqrtf(fmaf(ssv, inv_d, p.eps));
#pragma unroll
                for (int j = 0; j < 8; ++j) v[j] *= rinv;
                rope8(p, tok, e, v);
                uint8_t* dst = sQ + (e >> 6) * q_chunk_bytes + t * 128 + ((((e & 63) >> 3) ^ (t & 7)) << 4);
                *reinterpret_cast<uint4*>(dst) = pack8(v);
              }
              fence_proxy_async();
              if (tid_g == 0) VVS_TRACE(0x3F1);
              named_bar_sync(BAR_D, kGroup);
              if (tid_g == 0 && !s_abort) mbar_arrive(&att_q_ready);
            } else {
              // the block's own K / V rows inside this chunk: cache append + patch of the staged tiles
              const int new_lo = fill > key0 ? fill : key0;
              const int new_hi = n_keys < key0 + 128 ? n_keys : key0 + 128;
              if (new_lo < new_hi) {
                wait_bar(&att_kv_full, par, &s_abort, p.status);
                const int n_new = new_hi - new_lo;
#pragma unroll 1
                for (int idx = tid_g; idx < n_new * per_head * 2; idx += kGroup) {
                  const int which = idx >= n_new * per_head ? 1 : 0;   // 0 = K, 1 = V
                  const int rem = idx - which * n_new * per_head;
                  const int kk = rem >> ph_sh, ch = rem - (kk << ph_sh), e = ch << 3;
                  const int key = new_lo + kk, t = key - fill, tok = r * T + t;
                  const float ssv = __ldcg(p.ss + (2 * l) * 32 + tok);
                  float v[8];
                  ldcg8(qkv + (size_t)tok * 3 * p.d + (which + 1) * p.d + h * p.hd + e, v);
                  const float rinv = rsqrtf(fmaf(ssv, inv_d, p.eps));
#pragma unroll
                  for (int j = 0; j < 8; ++j) v[j] *= rinv;
                  if (which == 0) rope8(p, tok, e, v);
                  const uint4 u = pack8(v);
                  const int row = key - key0;
                  uint8_t* tile = (which == 0 ? sK : sV) + (e >> 6) * kSlabBytes;
                  *reinterpret_cast<uint4*>(tile + row * 128 + ((((e & 63) >> 3) ^ (row & 7)) << 4)) = u;
                  __nv_bfloat16* cache = which == 0 ? p.kv_k : p.kv_v;
                  *reinterpret_cast<uint4*>(cache + ((size_t)row_base + row) * p.hd + e) = u;
                }
              }
              fence_proxy_async();
              if (tid_g == 0) VVS_TRACE(0x4F1);
              named_bar_sync(BAR_E, kGroup);
              if (tid_g == 0 && !s_abort) mbar_arrive(&att_q_ready);
              // scores: this thread owns key (quarter * 32 + lane) of the chunk
              wait_bar(&att_s_full, par, &s_abort, p.status);
              tc_fence_after();
              if (tid_g == 0 && i + G < n_items && !s_abort) issue_next_k(l, i + G);
              if (tid_g == 0) VVS_TRACE(0x4F2);
              const int kl = quarter * 32 + lane;
              const uint32_t t_row = tmem_base + ((uint32_t)(quarter * 32) << 16) + kColS;
              {
                // scores of this key for all queries -> shared memory, transposed ([query][key], fp32;
                // kept in rows of the P tiles that belong to no query)
                float sc[32];
                tmem_ld16(t_row, sc);
                if (p.tq > 16) tmem_ld16(t_row + 16, sc + 16);
#pragma unroll
                for (int t = 0; t < 32; ++t)
                  if (t < p.tq) reinterpret_cast<float*>(sP + (t >> 4) * kSlabBytes + 4096)[(t & 15) * 128 + kl] = sc[t];
              }
              named_bar_sync(BAR_E, kGroup);
              // eight lanes per query row (16 keys each), sixteen rows per pass: mask, max, exp, sum.
              // Visible: a cache key (kj < 0) or block row kj with its bit set in the row's mask;
              // written without branches (a short-circuit form of the test cost 1 us per layer).
#pragma unroll 1
              for (int t0 = 0; t0 < T; t0 += 16) {
                const int t = t0 + quarter * 4 + (lane >> 3), sub = lane & 7;
                const bool live = t < T;
                const uint32_t anc = live ? s_anc[r * T + t] : 0u;
                float sv[16];
                float mx = -CUDART_INF_F;
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                  const int cc = (c + (sub >> 1)) & 3;          // rotation: conflict-free 128-bit loads
                  float4 s4 = make_float4(0.f, 0.f, 0.f, 0.f);
                  if (live) s4 = reinterpret_cast<const float4*>(sP + (t >> 4) * kSlabBytes + 4096)[(t & 15) * 32 + sub * 4 + cc];
                  const float in[4] = {s4.x, s4.y, s4.z, s4.w};
#pragma unroll
                  for (int j = 0; j < 4; ++j) {
                    const int kj = key0 + sub * 16 + cc * 4 + j - fill;
                    const uint32_t vis = (kj < 0 ? 1u : 0u) | (((uint32_t)kj < 32u ? 1u : 0u) & (anc >> (kj & 31)));
                    sv[c * 4 + j] = (vis & 1u) ? in[j] * p.scale : -CUDART_INF_F;
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
                  row_max[t] = mx;
                  row_sum[t] = sum;
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
                    uint8_t* dst = sP + (k4 >> 6) * kSlabBytes + t * 128 + (((((k4 & 63) >> 3) ^ (t & 7)) << 4) | ((k4 & 7) << 1));
                    *reinterpret_cast<uint2*>(dst) = pk;
                  }
                }
              }
              if (key0 + kl >= n_keys) {   // slots no query may see: cleared so stale contents cannot inject NaN
                for (int j = 0; j < NC; ++j) {
                  uint4* row = reinterpret_cast<uint4*>(sV + j * kSlabBytes + kl * 128);
#pragma unroll
                  for (int q = 0; q < 8; ++q) row[q] = make_uint4(0, 0, 0, 0);
                }
              }
              fence_proxy_async();
              tc_fence_before();
              if (tid_g == 0) VVS_TRACE(0x4F3);
              named_bar_sync(BAR_E, kGroup);
              if (tid_g == 0 && !s_abort) mbar_arrive(&att_p_ready);
            }
            wait_bar(&att_o_full, par, &s_abort, p.status);
            tc_fence_after();
            if (tid_w == 0 && i + G < n_items && !s_abort) issue_next_v(l, i + G);
            if (tid_w == 0) VVS_TRACE(0x4F4);
            if (grp_e && quarter == 0) {                  // TMEM lanes 0..31 = query rows
              const size_t rh = (size_t)r * H + h;
              const size_t slot = (rh * p.n_chunks_max + c) * T + lane;
#pragma unroll 1
              for (int e0 = 0; e0 < p.hd; e0 += 32) {
                float o[32];
                tmem_ld32(tmem_base + kColO + e0, o);
                if (lane < T) {
                  float4* dst = reinterpret_cast<float4*>(p.part_o + slot * p.hd + e0);
#pragma unroll
                  for (int q = 0; q < 8; ++q) dst[q] = make_float4(o[4 * q], o[4 * q + 1], o[4 * q + 2], o[4 * q + 3]);
                }
              }
              if (lane < T) {
                p.part_ml[slot * 2] = row_max[lane];
                p.part_ml[slot * 2 + 1] = row_sum[lane];
              }
            }
            tc_fence_before();
            if (tid_w == 64) VVS_TRACE(0x4F5);
            named_bar_sync(BAR_W, kWorkers);
          }
          if (!grp_e && tid_g == 0 && l + 1 < L && (int)blockIdx.x < n_items) issue_kv(l + 1, blockIdx.x);
          grid_sync(l, PH_O);
        }

        // ================================ projection phase ==========================================
        // (f, lo, hi were set inside the grid barrier that precedes this phase)
        const int n_units = hi - lo;
        const uint32_t per_unit = 1u + (uint32_t)f.dual;

        // ---- token operands of this CTA's units, built by all eight worker warps at once ----
        if (ph == PH_O) {
          // merge of the split-KV attention partials: one group of 128 threads per unit
          // (thread = token, 16 columns), two units per round
#pragma unroll 1
          for (int b0 = 0; b0 < n_units; b0 += 2) {
            const int k = b0 + (grp_e ? 1 : 0);
            if (k < n_units) {
              const uint32_t it = it_slab + (uint32_t)k;
              const uint32_t use = (uint32_t)div_small((int)it, (int)NS), st = it - use * NS;
              if (use > 0) wait_bar(&empty[st], (use - 1) & 1, &s_abort, p.status);
              if (b_tok < p.m) {
                const int kb = (lo + k) - div_small(lo + k, f.kbs) * f.kbs;
                const int k0 = kb * 64 + b_qtr * 16;
                const int hd_sh = p.hd == 64 ? 6 : 7;
                const int h = k0 >> hd_sh, e = k0 - (h << hd_sh);
                const int nch = s_nch[b_r];
                const size_t base = (((size_t)b_r * H + h) * p.n_chunks_max) * T + b_t;
                float v[16];
#pragma unroll
                for (int j = 0; j < 16; ++j) v[j] = 0.f;
                float mrun = -CUDART_INF_F, den = 0.f;
#pragma unroll 1
                for (int c0 = 0; c0 < nch; c0 += 4) {   // four chunks in flight at once
                  float mc[4], lc[4], o[4][16];
#pragma unroll
                  for (int j = 0; j < 4; ++j) {
                    if (c0 + j < nch) {
                      const size_t slot = base + (size_t)(c0 + j) * T;
                      const float2 ml = __ldcg(reinterpret_cast<const float2*>(p.part_ml + slot * 2));
                      mc[j] = ml.x;
                      lc[j] = ml.y;
                      ldcg8(p.part_o + slot * p.hd + e, o[j]);
                      ldcg8(p.part_o + slot * p.hd + e + 8, o[j] + 8);
                    } else {
                      mc[j] = -CUDART_INF_F;
                      lc[j] = 0.f;
#pragma unroll
                      for (int q = 0; q < 16; ++q) o[j][q] = 0.f;
                    }
                  }
                  const float mnew = fmaxf(fmaxf(mrun, mc[0]), fmaxf(fmaxf(mc[1], mc[2]), mc[3]));
                  if (mnew == -CUDART_INF_F) continue;
                  const float keep = (mrun == -CUDART_INF_F) ? 0.f : __expf(mrun - mnew);
                  den *= keep;
#pragma unroll
                  for (int q = 0; q < 16; ++q) v[q] *= keep;
#pragma unroll
                  for (int j = 0; j < 4; ++j) {
                    const float w = (mc[j] == -CUDART_INF_F) ? 0.f : __expf(mc[j] - mnew);
                    den = fmaf(w, lc[j], den);
#pragma unroll
                    for (int q = 0; q < 16; ++q) v[q] = fmaf(w, o[j][q], v[q]);
                  }
                  mrun = mnew;
                }
                const float inv = den > 0.f ? 1.f / den : 0.f;
#pragma unroll
                for (int q = 0; q < 16; ++q) v[q] *= inv;
                uint8_t* row = ring + (size_t)st * kStageBytes + kSlabBytes + b_tok * 128;
                *reinterpret_cast<uint4*>(row + (((2 * b_qtr) ^ (b_tok & 7)) << 4)) = pack8(v);
                *reinterpret_cast<uint4*>(row + (((2 * b_qtr + 1) ^ (b_tok & 7)) << 4)) = pack8(v + 8);
              }
            }
            fence_proxy_async();
            if (tid_w == 0) VVS_TRACE(0x300 | (ph << 4) | (b0 & 15));
            named_bar_sync(BAR_W, kWorkers);
            if (tid_w == 0) VVS_TRACE(0x380 | (ph << 4) | (b0 & 15));
            if (tid_w < 2 && b0 + tid_w < n_units && !s_abort) {
              const uint32_t it = it_slab + (uint32_t)(b0 + tid_w);
              mbar_arrive(&full[it - (uint32_t)div_small((int)it, (int)NS) * NS]);
            }
          }
        } else {
          // x * norm scale (QKV, gate/up) or silu(gate) * up (down): up to four units per round
          // (64 threads per unit), up to eight (32 threads per unit) for the norm operands
          const int which = ph == PH_GU ? 1 : 0;
          const __nv_bfloat16* gsc = p.norms[l * 2 + which];
          int b0 = 0;
#pragma unroll 1
          while (b0 < n_units) {
            const int left = n_units - b0;
            // A round may not reach around the ring: its threads wait for the slot of their own
            // unit to be free before any of them reports a unit of the round as built, so two
            // units of one round must never share a slot.
            const int ring_cap = ((int)NS + f.dual) >> f.dual;            // ceil(NS / per_unit), per_unit = 1 or 2
            int cap = (ph != PH_DOWN && left > 4) ? 8 : 4;
            if (cap > ring_cap) cap = ring_cap;
            const int nb = left < cap ? left : cap;
            const int lg = nb <= 1 ? 0 : nb <= 2 ? 1 : nb <= 4 ? 2 : 3;
            const uint32_t it0 = it_slab + (uint32_t)b0 * per_unit;
            if (ph == PH_DOWN)
              build_round<4, true>(p, ring, empty, &s_abort, tid_w, nb, lg, it0, per_unit, lo + b0, f.kbs, gu, nullptr,
                                   p.ss + (2 * l + 1) * 32, nullptr);
            else if (lg == 3)
              build_round<8, false>(p, ring, empty, &s_abort, tid_w, nb, lg, it0, per_unit, lo + b0, f.kbs, p.x, gsc,
                                     nullptr, p.ss + (2 * l + which) * 32);
            else
              build_round<4, false>(p, ring, empty, &s_abort, tid_w, nb, lg, it0, per_unit, lo + b0, f.kbs, p.x, gsc,
                                    nullptr, p.ss + (2 * l + which) * 32);
            fence_proxy_async();
            if (tid_w == 0) VVS_TRACE(0x300 | (ph << 4) | (b0 & 15));
            named_bar_sync(BAR_W, kWorkers);
            if (tid_w == 0) VVS_TRACE(0x380 | (ph << 4) | (b0 & 15));
            if (tid_w < nb && !s_abort) {
              const uint32_t it = it0 + (uint32_t)tid_w * per_unit;
              const uint32_t use1 = (uint32_t)div_small((int)it, (int)NS);
              mbar_arrive(&full[it - use1 * NS]);
              if (f.dual) {
                // the second stage of the unit holds no token slab, but its barrier must be in the
                // phase of this use before it takes the arrival
                const uint32_t it2 = it + 1, use2 = (uint32_t)div_small((int)it2, (int)NS), st2 = it2 - use2 * NS;
                if (use2 > 0) wait_fast(&empty[st2], (use2 - 1) & 1, &s_abort, p.status);
                if (!s_abort) mbar_arrive(&full[st2]);
              }
            }
            b0 += nb;
          }
        }
        it_slab += (uint32_t)n_units * per_unit;

        if (!grp_e) {
          if (ph == PH_O && l + 1 < L) {
            // clear the accumulators the next layer adds into (last read one layer ago)
            const int gtid = blockIdx.x * kGroup + tid_g, gstride = G * kGroup;
            const float4 z = make_float4(0.f, 0.f, 0.f, 0.f);
            float4* q4 = reinterpret_cast<float4*>(p.qkv_acc + (size_t)(par_l ^ 1) * p.m * 3 * p.d);
            float4* g4 = reinterpret_cast<float4*>(p.gu_acc + (size_t)(par_l ^ 1) * p.m * 2 * p.ff);
#pragma unroll 1
            for (int i = gtid; i < (p.m * 3 * p.d) >> 2; i += gstride) q4[i] = z;
#pragma unroll 1
            for (int i = gtid; i < (p.m * 2 * p.ff) >> 2; i += gstride) g4[i] = z;
          }
        } else {
          // ---- epilogue: accumulators -> fp32 sums in L2 ----
          int s = lo;
#pragma unroll 1
          while (s < hi) {
            const int tile = div_small(s, f.kbs);
            int next = (tile + 1) * f.kbs;
            s = next < hi ? next : hi;
            const uint32_t slot = ita % kAccSlots;
            wait_fast(&acc_full[slot], (ita / kAccSlots) & 1, &s_abort, p.status);
            tc_fence_after();
            if (tid_g == 0) VVS_TRACE(0x400 | (ph << 4));
            const int n = tile * 128 + quarter * 32 + lane;
            const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + slot * 64;
            float* dst;
            int ld, nlim;
            if (ph == PH_QKV) { dst = qkv; ld = 3 * p.d; nlim = 3 * p.d; }
            else if (ph == PH_GU) { dst = gu; ld = 2 * p.ff; nlim = p.ff; }
            else { dst = p.x; ld = p.d; nlim = p.d; }
            float v[32];
            tmem_ld32(taddr, v);
            if (n < nlim) {
              float* ptr = dst + n;
#pragma unroll
              for (int tok = 0; tok < 32; ++tok) {
                if (tok < p.m) red_add_f32(ptr, v[tok]);
                ptr += ld;
              }
            }
            if (f.dual) {
              tmem_ld32(taddr + 32, v);
              if (n < nlim) {
                float* ptr = dst + p.ff + n;
#pragma unroll
                for (int tok = 0; tok < 32; ++tok) {
                  if (tok < p.m) red_add_f32(ptr, v[tok]);
                  ptr += ld;
                }
              }
            }
            tc_fence_before();
            if (tid_g == 0) VVS_TRACE(0x480 | (ph << 4));
            named_bar_sync(BAR_E, kGroup);
            if (tid_g == 0 && !s_abort) mbar_arrive(&acc_empty[slot]);
            ++ita;
          }
        }
        // what follows: the attention items (no projection plan), or the next projection
        if (!(l == L - 1 && ph == PH_DOWN)) {
          if (ph == PH_QKV) grid_sync(l, -1);
          else if (ph == PH_DOWN) grid_sync(l + 1, PH_QKV);
          else grid_sync(l, ph + 1);
        }
      }
    }
    if (blockIdx.x == 0 && tid_w == 0 && !s_abort)
      *reinterpret_cast<volatile unsigned*>(p.sync_words + 1) = target;
  }

  // ---- teardown ---------------------------------------------------------------------------------
  VVS_TRACE_END;
  __syncwarp();
  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_base, kTmemCols);
}

}  // namespace

bool fused_chain_applicable(const vvs_model_desc& md, int n_rows, int t_len) {
  if (md.dtype != VVS_DTYPE_BF16 || md.n_layers < 1) return false;
  if (n_rows * t_len > 32 || n_rows > kMaxSeq || md.n_layers > kMaxLayers) return false;
  if (md.d_model % 64 != 0 || md.d_ff % 8 != 0) return false;
  return true;
}

size_t fused_chain_smem_bytes(const vvs_model_desc& md, int t_len, int* n_stages) {
  const int nc = md.head_dim / 64, tq = t_len <= 16 ? 16 : 32;
  const size_t fixed = 1024 + (size_t)2 * nc * kSlabBytes + 2 * kSlabBytes + (size_t)nc * tq * 128;
  const size_t budget = 226 * 1024;   // leaves room for the static barriers and tables
  int stages = (int)((budget - fixed) / kStageBytes);
  if (stages > kMaxStages) stages = kMaxStages;
  if (n_stages) *n_stages = stages;
  return fixed + (size_t)stages * kStageBytes;
}

int launch_fused_chain(const FusedChainArgs& a, cudaStream_t s) {
  ChainParams p{};
  const vvs_model_desc& md = *a.md;
  p.n_layers = md.n_layers; p.d = md.d_model; p.n_heads = md.n_heads; p.hd = md.head_dim; p.ff = md.d_ff;
  p.s_max = md.s_max; p.kv_rows = a.kv_rows;
  p.m = a.n_rows * a.t_len; p.t_len = a.t_len; p.tq = a.t_len <= 16 ? 16 : 32;
  p.n_rows = a.n_rows; p.n_images = a.n_images; p.tok_rows = md.tok_rows;
  p.n_chunks_max = (md.s_max + 127) / 128;
  p.eps = md.rms_eps; p.scale = 1.0f / sqrtf((float)md.head_dim);
  p.wmaps = a.wmaps; p.tok_emb = a.tok_emb; p.block = a.block;
  for (int i = 0; i < 2 * md.n_layers; ++i) p.norms[i] = a.norms_host[i];
  p.x = a.x; p.qkv_acc = a.qkv_acc; p.gu_acc = a.gu_acc; p.ss = a.ss;
  p.cache_len = a.cache_len; p.anc_mask = a.anc_mask; p.kv_k = a.kv_k; p.kv_v = a.kv_v;
  p.rope_cos = a.rope_cos; p.rope_sin = a.rope_sin;
  p.part_o = a.part_o; p.part_ml = a.part_ml; p.sync_words = a.sync_words; p.status = a.status;
  int stages = 0;
  const size_t smem = fused_chain_smem_bytes(md, a.t_len, &stages);
  if (stages < 3) return VVS_ERR_SHAPE;
  p.n_stages = stages;
  if (ensure_dynamic_smem(reinterpret_cast<const void*>(fused_chain_kernel), (int)smem) != cudaSuccess) return VVS_ERR_CUDA;
  CUtensorMap tk = *a.tm_k, tv = *a.tm_v;
  void* args[] = {&p, &tk, &tv};
  // cooperative launch: all CTAs are resident together, which the grid barriers rely on
  cudaError_t e = cudaLaunchCooperativeKernel(reinterpret_cast<const void*>(fused_chain_kernel), dim3(a.n_sms),
                                              dim3(kThreads), args, smem, s);
  return e == cudaSuccess ? VVS_OK : VVS_ERR_CUDA;
}

}  // namespace vvs
