// The decoder chain of the verify step as ONE persistent kernel (bf16, at most 32 block tokens).
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

namespace vvs {

using namespace tc;

namespace {

constexpr int kThreads = 320;
constexpr int kWorkers = 256;          // warps 2-9
constexpr int kGroup = 128;
constexpr int kSlabBytes = 16384;      // 128 weight rows x 64 bf16
constexpr int kTokSlabBytes = 4096;    // 32 tokens x 64 bf16
constexpr int kTokStages = 4;
constexpr int kAccSlots = 4;           // TMEM accumulator slots of 64 columns
constexpr int kMaxWStages = 12;
constexpr int kMaxSeq = 32;
constexpr uint32_t kColS = 256, kColO = 320, kTmemCols = 512;
constexpr uint32_t kGridSpinLimit = 1u << 21;
enum { BAR_W = 1, BAR_E = 2, BAR_D = 3 };
enum { PH_QKV = 0, PH_O = 1, PH_GU = 2, PH_DOWN = 3 };

struct ChainParams {
  int n_layers, d, n_heads, hd, ff, s_max, kv_rows;
  int m, t_len, tq, n_rows, n_images, tok_rows;
  int w_stages, n_chunks_max;
  float eps, scale;
  const CUtensorMap* wmaps;            // device [n_layers][5]: qkv, o, gate, up, down
  const __nv_bfloat16* const* norms;   // device [n_layers][2]
  const __nv_bfloat16* tok_emb;
  const int32_t* block;
  float* x;                            // [m, d] residual stream
  float* qkv_acc;                      // [2][m, 3d]
  float* gu_acc;                       // [2][m, 2ff]
  float* ss;                           // [2 * n_layers][32] sums of squares of x rows
  const int32_t* cache_len;
  __nv_bfloat16* kv_k;
  __nv_bfloat16* kv_v;
  const int32_t* slot_pos;
  const float* rope_cos;
  const float* rope_sin;
  float* part_o;
  float* part_ml;
  unsigned* sync_words;                // [0] arrivals, [1] epoch base, [2] abort
  int32_t* status;
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
__device__ __forceinline__ void unit_range(const Phase& f, int layer, int ph, int& lo, int& hi) {
  const int G = (int)gridDim.x, S = f.tiles * f.kbs;
  const int v = (int)((blockIdx.x + (unsigned)(layer * 4 + ph) * 53u) % (unsigned)G);
  lo = (int)(((long long)v * S) / G);
  hi = (int)(((long long)(v + 1) * S) / G);
}

// Bounded wait; falls through at once when the CTA is in abort mode.
__device__ __forceinline__ bool wait_bar(uint64_t* bar, uint32_t parity, volatile int* s_abort, int32_t* status) {
  if (*s_abort) return false;
  for (uint32_t i = 0; i < kSpinLimit; ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((i & 255u) == 255u && *s_abort) return false;
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

__global__ void __launch_bounds__(kThreads, 1)
fused_chain_kernel(const ChainParams p, const __grid_constant__ CUtensorMap tm_k,
                   const __grid_constant__ CUtensorMap tm_v) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t w_full[kMaxWStages], w_empty[kMaxWStages];
  __shared__ __align__(8) uint64_t b_full[kTokStages], b_empty[kTokStages];
  __shared__ __align__(8) uint64_t acc_full[kAccSlots], acc_empty[kAccSlots];
  __shared__ __align__(8) uint64_t att_kv_full, att_q_ready, att_s_full, att_p_ready, att_o_full;
  __shared__ uint32_t tmem_slot;
  __shared__ volatile int s_abort;
  __shared__ int s_fill[kMaxSeq], s_nch[kMaxSeq], s_prefix[kMaxSeq + 1];
  __shared__ float red_max[4][32], red_sum[4][32];

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int G = (int)gridDim.x;
  const int NC = p.hd >> 6;                       // 64-column chunks of a head
  const int NS = p.w_stages;
  const int T = p.t_len, H = p.n_heads, L = p.n_layers;

  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* ring = smem;
  uint8_t* tokring = ring + (size_t)NS * kSlabBytes;
  uint8_t* sK = tokring + kTokStages * kTokSlabBytes;
  uint8_t* sV = sK + NC * kSlabBytes;
  uint8_t* sP = sV + NC * kSlabBytes;             // 2 x [128 rows x 128 B]
  uint8_t* sQ = sP + 2 * kSlabBytes;              // NC x [tq rows x 128 B]
  const uint32_t q_chunk_bytes = (uint32_t)p.tq * 128u;

  // ---- set-up ------------------------------------------------------------------------------------
  if (tid == 0) {
    for (int i = 0; i < NS; ++i) { mbar_init(&w_full[i], 1); mbar_init(&w_empty[i], 1); }
    for (int i = 0; i < kTokStages; ++i) { mbar_init(&b_full[i], 1); mbar_init(&b_empty[i], 1); }
    for (int i = 0; i < kAccSlots; ++i) { mbar_init(&acc_full[i], 1); mbar_init(&acc_empty[i], 1); }
    mbar_init(&att_kv_full, 1);
    mbar_init(&att_q_ready, 1);
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
  // token operands: rows of tokens that do not exist stay zero for the whole kernel
  for (int i = tid; i < (kTokStages * kTokSlabBytes) / 16; i += kThreads)
    reinterpret_cast<uint4*>(tokring)[i] = make_uint4(0, 0, 0, 0);
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
  const uint32_t idesc_gemm = idesc_bf16_f32(128, 32);

  auto decode_item = [&](int i, int& r, int& h, int& c) {
    const int rc = i / H;
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
      uint32_t it = 0;
      bool alive = true;
      for (int l = 0; l < L && alive; ++l) {
        for (int ph = 0; ph < 4 && alive; ++ph) {
          const Phase f = phase_of(p, ph);
          int lo, hi;
          unit_range(f, l, ph, lo, hi);
          for (int s = lo; s < hi && alive; ++s) {
            const int tile = s / f.kbs, kb = s - tile * f.kbs;
            for (int j = 0; j <= f.dual; ++j, ++it) {
              const uint32_t stage = it % NS, use = it / NS;
              if (use > 0 && !wait_bar(&w_empty[stage], (use - 1) & 1, &s_abort, p.status)) { alive = false; break; }
              mbar_expect_tx(&w_full[stage], kSlabBytes);
              tma_load_2d(ring + (size_t)stage * kSlabBytes, &p.wmaps[l * 5 + f.map0 + j], &w_full[stage],
                          kb * 64, tile * 128);
            }
          }
        }
      }
      // every load that was issued must have landed before the CTA may exit
      for (uint32_t stage = 0; stage < (uint32_t)NS; ++stage) {
        if (it > stage) mbar_wait(&w_full[stage], ((it - 1 - stage) / NS) & 1);
      }
    }
  } else if (warp == 1) {
    // =================================== MMA issuer ==================================================
    if (lane == 0) {
      uint32_t itw = 0, itb = 0, ita = 0, iatt = 0;
      bool alive = true;
      for (int l = 0; l < L && alive; ++l) {
        for (int ph = 0; ph < 4 && alive; ++ph) {
          if (ph == PH_O) {
            // ---- attention products of this CTA's items ----
            for (int i = blockIdx.x; i < n_items && alive; i += G, ++iatt) {
              const uint32_t par = iatt & 1;
              if (!wait_bar(&att_kv_full, par, &s_abort, p.status) ||
                  !wait_bar(&att_q_ready, par, &s_abort, p.status)) { alive = false; break; }
              tc_fence_after();
              const uint32_t idesc_s = idesc_bf16_f32(128, (uint32_t)p.tq);
              for (int k16 = 0; k16 < p.hd / 16; ++k16) {
                const uint32_t a = smem_u32(sK + (k16 >> 2) * kSlabBytes) + (k16 & 3) * 32;
                const uint32_t b = smem_u32(sQ + (k16 >> 2) * q_chunk_bytes) + (k16 & 3) * 32;
                mma_bf16(tmem_base + kColS, smem_desc_sw128(a), smem_desc_sw128(b), idesc_s, k16 > 0 ? 1u : 0u);
              }
              mma_commit(&att_s_full);
              if (!wait_bar(&att_p_ready, par, &s_abort, p.status)) { alive = false; break; }
              tc_fence_after();
              const uint32_t idesc_o = idesc_bf16_f32(128, (uint32_t)p.hd) | (1u << 16);  // B is MN-major
              for (int k16 = 0; k16 < 8; ++k16) {
                const uint32_t a = smem_u32(sP + (k16 >> 2) * kSlabBytes) + (k16 & 3) * 32;
                const uint32_t b = smem_u32(sV) + k16 * 2048;
                mma_bf16(tmem_base + kColO, smem_desc_sw128(a), smem_desc_mn_sw128(b, kSlabBytes), idesc_o,
                         k16 > 0 ? 1u : 0u);
              }
              mma_commit(&att_o_full);
            }
            if (!alive) break;
          }
          const Phase f = phase_of(p, ph);
          int lo, hi;
          unit_range(f, l, ph, lo, hi);
          int cur_tile = -1;
          uint32_t slot = 0;
          for (int s = lo; s < hi; ++s, ++itb) {
            const int tile = s / f.kbs;
            const bool first = tile != cur_tile;
            if (first) {
              if (cur_tile >= 0) mma_commit(&acc_full[slot]);
              slot = ita % kAccSlots;
              const uint32_t use = ita / kAccSlots;
              if (use > 0 && !wait_bar(&acc_empty[slot], (use - 1) & 1, &s_abort, p.status)) { alive = false; break; }
              cur_tile = tile;
              ++ita;
            }
            const uint32_t bst = itb % kTokStages, st = itw % NS, st2 = (itw + 1) % NS;
            if (!wait_bar(&b_full[bst], (itb / kTokStages) & 1, &s_abort, p.status) ||
                !wait_bar(&w_full[st], (itw / NS) & 1, &s_abort, p.status) ||
                (f.dual && !wait_bar(&w_full[st2], ((itw + 1) / NS) & 1, &s_abort, p.status))) { alive = false; break; }
            tc_fence_after();
            const uint32_t a_addr = smem_u32(ring + (size_t)st * kSlabBytes);
            const uint32_t a2_addr = smem_u32(ring + (size_t)st2 * kSlabBytes);
            const uint32_t b_addr = smem_u32(tokring + bst * kTokSlabBytes);
            const uint32_t acc = tmem_base + slot * 64;
#pragma unroll
            for (uint32_t k16 = 0; k16 < 4; ++k16) {
              const uint32_t accum = (!first || k16 > 0) ? 1u : 0u;
              const uint64_t bd = smem_desc_sw128(b_addr + k16 * 32);
              mma_bf16(acc, smem_desc_sw128(a_addr + k16 * 32), bd, idesc_gemm, accum);
              if (f.dual) mma_bf16(acc + 32, smem_desc_sw128(a2_addr + k16 * 32), bd, idesc_gemm, accum);
            }
            mma_commit(&w_empty[st]);
            if (f.dual) mma_commit(&w_empty[st2]);
            mma_commit(&b_empty[bst]);
            itw += 1 + f.dual;
          }
          if (alive && cur_tile >= 0) mma_commit(&acc_full[slot]);
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
    uint32_t itb = 0, ita = 0, iatt = 0;

    auto grid_sync = [&]() {
      named_bar_sync(BAR_W, kWorkers);
      target += (unsigned)G;
      if (tid_w == 0 && !s_abort) {
        __threadfence();
        atomicAdd(p.sync_words, 1u);
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

    // ---- phase 0: clear the accumulators, gather the embeddings ----
    {
      const int gtid = blockIdx.x * kWorkers + tid_w, gstride = G * kWorkers;
      const float4 z = make_float4(0.f, 0.f, 0.f, 0.f);
      const int nq = (2 * p.m * 3 * p.d) >> 2, ng = (2 * p.m * 2 * p.ff) >> 2, ns = (2 * L * 32) >> 2;
      for (int i = gtid; i < nq; i += gstride) reinterpret_cast<float4*>(p.qkv_acc)[i] = z;
      for (int i = gtid; i < ng; i += gstride) reinterpret_cast<float4*>(p.gu_acc)[i] = z;
      for (int i = gtid; i < ns; i += gstride) reinterpret_cast<float4*>(p.ss)[i] = z;
      const int per_row = p.d >> 3;
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
      grid_sync();
    }

    // per-thread constants of the operand builders
    const int b_tok = tid_g >> 2, b_qtr = tid_g & 3;
    const int b_r = b_tok / T, b_t = b_tok - b_r * T;

    for (int l = 0; l < L; ++l) {
      const int par_l = l & 1;
      float* qkv = p.qkv_acc + (size_t)par_l * p.m * 3 * p.d;
      float* gu = p.gu_acc + (size_t)par_l * p.m * 2 * p.ff;
      for (int ph = 0; ph < 4; ++ph) {
        if (ph == PH_O) {
          // ================================ attention ================================================
          int n_mine = 0;
          for (int i = blockIdx.x; i < n_items; i += G, ++iatt, ++n_mine) {
            int r, h, c;
            decode_item(i, r, h, c);
            const uint32_t par = iatt & 1;
            const int fill = s_fill[r], n_keys = fill + T, key0 = c * 128;
            const int row_base = kv_row_base(l, r, h, c);
            if (!grp_e) {
              if (tid_g == 0 && n_mine > 0) issue_kv(l, i);   // the first item was requested a layer ahead
              // Q operand: q * (1/rms) rotated, bf16, K-major with the 128-byte swizzle
              const int per_head = p.hd >> 3;
              for (int idx = tid_g; idx < T * per_head; idx += kGroup) {
                const int t = idx / per_head, ch = idx - t * per_head, e = ch << 3, tok = r * T + t;
                const float rinv = rsqrtf(__ldcg(p.ss + (2 * l) * 32 + tok) / (float)p.d + p.eps);
                float v[8];
                ldcg8(qkv + (size_t)tok * 3 * p.d + h * p.hd + e, v);
#pragma unroll
                for (int j = 0; j < 8; ++j) v[j] *= rinv;
                rope8(p, tok, e, v);
                uint8_t* dst = sQ + (e >> 6) * q_chunk_bytes + t * 128 + ((((e & 63) >> 3) ^ (t & 7)) << 4);
                *reinterpret_cast<uint4*>(dst) = pack8(v);
              }
              // the block's own K / V rows inside this chunk: cache append + patch of the staged tiles
              const int new_lo = fill > key0 ? fill : key0;
              const int new_hi = n_keys < key0 + 128 ? n_keys : key0 + 128;
              if (new_lo < new_hi) {
                wait_bar(&att_kv_full, par, &s_abort, p.status);
                const int n_new = new_hi - new_lo;
                for (int idx = tid_g; idx < n_new * per_head * 2; idx += kGroup) {
                  const int which = idx / (n_new * per_head);       // 0 = K, 1 = V
                  const int rem = idx - which * n_new * per_head;
                  const int kk = rem / per_head, ch = rem - kk * per_head, e = ch << 3;
                  const int key = new_lo + kk, t = key - fill, tok = r * T + t;
                  const float rinv = rsqrtf(__ldcg(p.ss + (2 * l) * 32 + tok) / (float)p.d + p.eps);
                  float v[8];
                  ldcg8(qkv + (size_t)tok * 3 * p.d + (which + 1) * p.d + h * p.hd + e, v);
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
              named_bar_sync(BAR_D, kGroup);
              if (tid_g == 0) mbar_arrive(&att_q_ready);
            } else {
              // scores: this thread owns key (quarter * 32 + lane) of the chunk
              wait_bar(&att_s_full, par, &s_abort, p.status);
              tc_fence_after();
              const int kl = quarter * 32 + lane, key = key0 + kl;
              const uint32_t t_row = tmem_base + ((uint32_t)(quarter * 32) << 16) + kColS;
              float s[32];
              tmem_ld16(t_row, s);
              if (p.tq > 16) tmem_ld16(t_row + 16, s + 16);
#pragma unroll
              for (int t = 0; t < 32; ++t) {
                if (t < T) {
                  s[t] = (key <= fill + t) ? s[t] * p.scale : -CUDART_INF_F;
                  const float wm = warp_max_f(s[t]);
                  if (lane == 0) red_max[quarter][t] = wm;
                }
              }
              named_bar_sync(BAR_E, kGroup);
#pragma unroll
              for (int t = 0; t < 32; ++t) {
                if (t < T) {
                  const float mx = fmaxf(fmaxf(red_max[0][t], red_max[1][t]), fmaxf(red_max[2][t], red_max[3][t]));
                  const float e = (s[t] == -CUDART_INF_F) ? 0.f : expf(s[t] - mx);
                  const float ws = warp_sum_f(e);
                  if (lane == 0) red_sum[quarter][t] = ws;
                  uint8_t* dst = sP + (kl >> 6) * kSlabBytes + t * 128 + (((((kl & 63) >> 3) ^ (t & 7)) << 4) | ((kl & 7) << 1));
                  *reinterpret_cast<__nv_bfloat16*>(dst) = __float2bfloat16_rn(e);
                }
              }
              if (key >= n_keys) {   // slots no query may see: cleared so stale contents cannot inject NaN
                for (int j = 0; j < NC; ++j) {
                  uint4* row = reinterpret_cast<uint4*>(sV + j * kSlabBytes + kl * 128);
#pragma unroll
                  for (int q = 0; q < 8; ++q) row[q] = make_uint4(0, 0, 0, 0);
                }
              }
              fence_proxy_async();
              tc_fence_before();
              named_bar_sync(BAR_E, kGroup);
              if (tid_g == 0) mbar_arrive(&att_p_ready);
            }
            wait_bar(&att_o_full, par, &s_abort, p.status);
            tc_fence_after();
            if (grp_e && quarter == 0) {                  // TMEM lanes 0..31 = query rows
              const size_t rh = (size_t)r * H + h;
              const size_t slot = (rh * p.n_chunks_max + c) * T + lane;
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
                p.part_ml[slot * 2] = fmaxf(fmaxf(red_max[0][lane], red_max[1][lane]), fmaxf(red_max[2][lane], red_max[3][lane]));
                p.part_ml[slot * 2 + 1] = red_sum[0][lane] + red_sum[1][lane] + red_sum[2][lane] + red_sum[3][lane];
              }
            }
            tc_fence_before();
            named_bar_sync(BAR_W, kWorkers);
          }
          if (!grp_e && tid_g == 0 && l + 1 < L && (int)blockIdx.x < n_items) issue_kv(l + 1, blockIdx.x);
          grid_sync();
        }

        // ================================ projection phase ==========================================
        const Phase f = phase_of(p, ph);
        int lo, hi;
        unit_range(f, l, ph, lo, hi);
        if (!grp_e) {
          // ---- operand builders ----
          for (int s = lo; s < hi; ++s, ++itb) {
            const int tile = s / f.kbs, kb = s - tile * f.kbs;
            const uint32_t bst = itb % kTokStages, use = itb / kTokStages;
            if (use > 0) wait_bar(&b_empty[bst], (use - 1) & 1, &s_abort, p.status);
            uint8_t* slab = tokring + bst * kTokSlabBytes;
            const int k0 = kb * 64 + b_qtr * 16;
            float v[16];
#pragma unroll
            for (int j = 0; j < 16; ++j) v[j] = 0.f;
            float ssq = 0.f;
            if (b_tok < p.m) {
              if (ph == PH_QKV || ph == PH_GU) {
                const int which = ph == PH_GU ? 1 : 0;
                float xv[16], gv[16];
                ldcg8(p.x + (size_t)b_tok * p.d + k0, xv);
                ldcg8(p.x + (size_t)b_tok * p.d + k0 + 8, xv + 8);
                const uint4* g = reinterpret_cast<const uint4*>(p.norms[l * 2 + which] + k0);
                unpack8(__ldg(g), gv);
                unpack8(__ldg(g + 1), gv + 8);
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                  ssq = fmaf(xv[j], xv[j], ssq);
                  v[j] = xv[j] * gv[j];
                }
              } else if (ph == PH_O) {
                const int h = k0 / p.hd, e = k0 - h * p.hd;
                const int nch = s_nch[b_r];
                const size_t base = (((size_t)b_r * H + h) * p.n_chunks_max) * T + b_t;
                float mx = -CUDART_INF_F;
                for (int c = 0; c < nch; ++c) mx = fmaxf(mx, __ldcg(p.part_ml + (base + (size_t)c * T) * 2));
                float den = 0.f;
                for (int c = 0; c < nch; ++c) {
                  const size_t slot = base + (size_t)c * T;
                  const float mc = __ldcg(p.part_ml + slot * 2);
                  const float w = (mc == -CUDART_INF_F) ? 0.f : expf(mc - mx);
                  den = fmaf(w, __ldcg(p.part_ml + slot * 2 + 1), den);
                  float o[16];
                  ldcg8(p.part_o + slot * p.hd + e, o);
                  ldcg8(p.part_o + slot * p.hd + e + 8, o + 8);
#pragma unroll
                  for (int j = 0; j < 16; ++j) v[j] = fmaf(w, o[j], v[j]);
                }
                const float inv = den > 0.f ? 1.f / den : 0.f;
#pragma unroll
                for (int j = 0; j < 16; ++j) v[j] *= inv;
              } else {
                const float rinv = rsqrtf(__ldcg(p.ss + (2 * l + 1) * 32 + b_tok) / (float)p.d + p.eps);
                const float* gp = gu + (size_t)b_tok * 2 * p.ff + k0;
#pragma unroll
                for (int c8 = 0; c8 < 2; ++c8) {
                  if (k0 + c8 * 8 < p.ff) {
                    float gt[8], up[8];
                    ldcg8(gp + c8 * 8, gt);
                    ldcg8(gp + p.ff + c8 * 8, up);
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                      const float a = gt[j] * rinv;
                      v[c8 * 8 + j] = a / (1.f + expf(-a)) * (up[j] * rinv);
                    }
                  }
                }
              }
              uint8_t* row = slab + b_tok * 128;
              *reinterpret_cast<uint4*>(row + (((2 * b_qtr) ^ (b_tok & 7)) << 4)) = pack8(v);
              *reinterpret_cast<uint4*>(row + (((2 * b_qtr + 1) ^ (b_tok & 7)) << 4)) = pack8(v + 8);
            }
            if ((ph == PH_QKV || ph == PH_GU) && tile == 0) {
              // sum of squares of the row, once per k-block (the CTAs that own tile 0)
              ssq += __shfl_xor_sync(0xffffffffu, ssq, 1);
              ssq += __shfl_xor_sync(0xffffffffu, ssq, 2);
              if (b_qtr == 0 && b_tok < p.m) atomicAdd(p.ss + (2 * l + (ph == PH_GU ? 1 : 0)) * 32 + b_tok, ssq);
            }
            fence_proxy_async();
            named_bar_sync(BAR_D, kGroup);
            if (tid_g == 0) mbar_arrive(&b_full[bst]);
          }
          if (ph == PH_O && l + 1 < L) {
            // clear the accumulators the next layer adds into (last read one layer ago)
            const int gtid = blockIdx.x * kGroup + tid_g, gstride = G * kGroup;
            const float4 z = make_float4(0.f, 0.f, 0.f, 0.f);
            float4* q4 = reinterpret_cast<float4*>(p.qkv_acc + (size_t)(par_l ^ 1) * p.m * 3 * p.d);
            float4* g4 = reinterpret_cast<float4*>(p.gu_acc + (size_t)(par_l ^ 1) * p.m * 2 * p.ff);
            for (int i = gtid; i < (p.m * 3 * p.d) >> 2; i += gstride) q4[i] = z;
            for (int i = gtid; i < (p.m * 2 * p.ff) >> 2; i += gstride) g4[i] = z;
          }
        } else {
          // ---- epilogue: accumulators -> fp32 sums in L2 ----
          int s = lo;
          while (s < hi) {
            const int tile = s / f.kbs;
            int next = (tile + 1) * f.kbs;
            s = next < hi ? next : hi;
            const uint32_t slot = ita % kAccSlots;
            wait_bar(&acc_full[slot], (ita / kAccSlots) & 1, &s_abort, p.status);
            tc_fence_after();
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
#pragma unroll
              for (int tok = 0; tok < 32; ++tok)
                if (tok < p.m) red_add_f32(dst + (size_t)tok * ld + n, v[tok]);
            }
            if (f.dual) {
              tmem_ld32(taddr + 32, v);
              if (n < nlim) {
#pragma unroll
                for (int tok = 0; tok < 32; ++tok)
                  if (tok < p.m) red_add_f32(dst + (size_t)tok * ld + p.ff + n, v[tok]);
              }
            }
            tc_fence_before();
            named_bar_sync(BAR_E, kGroup);
            if (tid_g == 0) mbar_arrive(&acc_empty[slot]);
            ++ita;
          }
        }
        if (!(l == L - 1 && ph == PH_DOWN)) grid_sync();
      }
    }
    if (blockIdx.x == 0 && tid_w == 0 && !s_abort)
      *reinterpret_cast<volatile unsigned*>(p.sync_words + 1) = target;
  }

  // ---- teardown ---------------------------------------------------------------------------------
  __syncwarp();
  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_base, kTmemCols);
}

}  // namespace

bool fused_chain_applicable(const vvs_model_desc& md, int n_rows, int t_len) {
  if (md.dtype != VVS_DTYPE_BF16 || md.n_layers < 1) return false;
  if (n_rows * t_len > 32 || n_rows > kMaxSeq) return false;
  if (md.d_model % 64 != 0 || md.d_ff % 8 != 0) return false;
  return true;
}

size_t fused_chain_smem_bytes(const vvs_model_desc& md, int t_len, int* w_stages) {
  const int nc = md.head_dim / 64, tq = t_len <= 16 ? 16 : 32;
  const size_t fixed = 1024 + (size_t)kTokStages * kTokSlabBytes + (size_t)2 * nc * kSlabBytes +
                       2 * kSlabBytes + (size_t)nc * tq * 128;
  const size_t budget = 226 * 1024;   // leaves room for the static barriers and tables
  int stages = (int)((budget - fixed) / kSlabBytes);
  if (stages > kMaxWStages) stages = kMaxWStages;
  if (w_stages) *w_stages = stages;
  return fixed + (size_t)stages * kSlabBytes;
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
  p.wmaps = a.wmaps; p.norms = a.norms; p.tok_emb = a.tok_emb; p.block = a.block;
  p.x = a.x; p.qkv_acc = a.qkv_acc; p.gu_acc = a.gu_acc; p.ss = a.ss;
  p.cache_len = a.cache_len; p.kv_k = a.kv_k; p.kv_v = a.kv_v;
  p.slot_pos = a.slot_pos; p.rope_cos = a.rope_cos; p.rope_sin = a.rope_sin;
  p.part_o = a.part_o; p.part_ml = a.part_ml; p.sync_words = a.sync_words; p.status = a.status;
  int stages = 0;
  const size_t smem = fused_chain_smem_bytes(md, a.t_len, &stages);
  if (stages < 3) return VVS_ERR_SHAPE;
  p.w_stages = stages;
  static size_t configured = 0;
  if (configured < smem) {
    if (cudaFuncSetAttribute(fused_chain_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
      return VVS_ERR_CUDA;
    configured = smem;
  }
  CUtensorMap tk = *a.tm_k, tv = *a.tm_v;
  void* args[] = {&p, &tk, &tv};
  // cooperative launch: all CTAs are resident together, which the grid barriers rely on
  cudaError_t e = cudaLaunchCooperativeKernel(reinterpret_cast<const void*>(fused_chain_kernel), dim3(a.n_sms),
                                              dim3(kThreads), args, smem, s);
  return e == cudaSuccess ? VVS_OK : VVS_ERR_CUDA;
}

}  // namespace vvs
