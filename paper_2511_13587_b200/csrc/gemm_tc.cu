// Weight-streaming projection GEMM for small token counts on the 5th-generation tensor cores.
//
//   out[tok, n] = sum_k act[tok, k] * w[n, k]          (w is [out_features, in_features])
//
// The roles are swapped relative to a textbook GEMM: the 128 weight rows of a tile sit on the
// MMA's M side (tcgen05.mma, M = 128), the tokens on its N side (N = tokens rounded up to 16,
// at most 256 per pass), so a batch-1 verify step (18 tokens) wastes no weight bandwidth and
// little tensor-core work.  Per CTA: one weight tile x one K slice (split-K).  Weight and
// activation tiles are staged by TMA into 128-byte-swizzled shared memory, one elected thread
// issues the MMAs, accumulators live in TMEM, and the four warps read them back (tcgen05.ld) for
// a fused epilogue:
//   ADD     out[tok, n] += acc                     (every projection of the default path: fp32 sums that
//                                                   the next kernel rotates / gates / normalises)
//   ADD2    the same for two weight matrices sharing the activation tile (gate and up as one launch)
//   QKV     rotate q, k pairs, write q and append k, v to the KV cache      (debug-switch path, 33-64 tokens)
//   SWIGLU  act[tok, n] = silu(gate) * up          (two weight tiles, two accumulators; same path)
//   STORE   out[tok, n] = acc
// How the split-K sums of ADD meet: (a) scalar reductions into L2 in arrival order (at most 32 tokens
// per pass); (b) above that the accumulator tile is staged token-major in shared memory and every
// thread adds four consecutive columns with one vector reduction; (c) in fixed-order contexts the
// K splits of a tile are the CTAs of one thread-block cluster: each rank sums its share of the token
// rows over all ranks' staged tiles in rank order through distributed shared memory and is the only
// writer of those outputs (no atomics, repeatable bits).
// Planning: two CTAs per SM when the tokens need several passes, up to five small CTAs (two stages
// each) for a single pass: more independent weight streams per SM.
// Split-K partial sums of the non-linear epilogues are added into a zeroed fp32 scratch; the CTA
// that arrives last on the tile's counter applies the epilogue and re-zeroes what it read, so no
// CTA ever waits for another.  Weight tiles are requested before griddepcontrol.wait, i.e. while
// the previous kernel of the stream is still running (programmatic dependent launch).
#include "tc_common.cuh"
#include "vvs_internal.cuh"

namespace vvs {

using namespace tc;

namespace {

constexpr int kMaxStages = 10;
constexpr uint32_t kTileRows = 128;       // weight rows per tile = MMA M
constexpr uint32_t kBlockK = 64;          // bf16 elements per smem row = one 128-byte swizzle row
constexpr uint32_t kATileBytes = kTileRows * kBlockK * 2;

struct KernelParams {
  int m, n, k;
  int nt, passes, kb_total, splits, stages, wide_add, cluster_mode;
  uint32_t tmem_cols;
  float* scratch;
  int ld_scratch;
  int* counters;
  int32_t* status;
  float* out;
  int ldo;
  __nv_bfloat16* q;
  __nv_bfloat16* kv_k;
  __nv_bfloat16* kv_v;
  const int32_t* slot_pos;
  const float* rope_cos;
  const float* rope_sin;
  int d, n_heads, hd, s_max, layer, kv_rows, t_len;
  __nv_bfloat16* act;
  int ff;
};

// bounded wait that also gives up when another role of the CTA already did
__device__ __forceinline__ bool wait_or_abort(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
  for (uint32_t i = 0; i < kSpinLimit; ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((i & 1023u) == 1023u && *abort_flag) return false;
  }
  return false;
}

template <int EPI>
__device__ __forceinline__ void final_chunk(const KernelParams& p, int n, int tok_base, const float* v,
                                            const float* v2) {
  // v[j] (and v2[j]) belong to weight row n and token tok_base + j
#pragma unroll
  for (int j = 0; j < 16; ++j) {
    const int tok = tok_base + j;
    if (tok >= p.m) break;  // uniform across the warp
    if constexpr (EPI == GEMM_EPI_STORE) {
      if (n < p.n) p.out[(size_t)tok * p.ldo + n] = v[j];
    } else if constexpr (EPI == GEMM_EPI_ADD) {
      if (n < p.n) atomicAdd(&p.out[(size_t)tok * p.ldo + n], v[j]);
    } else if constexpr (EPI == GEMM_EPI_ADD2) {          // two matrices, sums added side by side: out[tok, n], out[tok, ff + n]
      if (n < p.n) {
        atomicAdd(&p.out[(size_t)tok * p.ldo + n], v[j]);
        atomicAdd(&p.out[(size_t)tok * p.ldo + p.ff + n], v2[j]);
      }
    } else if constexpr (EPI == GEMM_EPI_SWIGLU) {
      if (n < p.n) {
        const float g = v[j];
        p.act[(size_t)tok * p.ff + n] = __float2bfloat16_rn(g / (1.f + expf(-g)) * v2[j]);
      }
    } else {  // GEMM_EPI_QKV
      const float val = v[j];
      const float other = __shfl_xor_sync(0xffffffffu, val, 1);  // the pair partner (row n ^ 1)
      if (n < p.n) {
        const int sec = n / p.d, e = n - sec * p.d;
        const int h = e / p.hd, i = e - h * p.hd;
        float y = val;
        if (sec < 2) {
          const float cs = p.rope_cos[(size_t)tok * (p.hd / 2) + (i >> 1)];
          const float sn = p.rope_sin[(size_t)tok * (p.hd / 2) + (i >> 1)];
          y = (i & 1) ? (other * sn + val * cs) : (val * cs - other * sn);
        }
        if (sec == 0) {
          p.q[(size_t)tok * p.d + e] = __float2bfloat16_rn(y);
        } else {
          const int slot = p.slot_pos[tok];
          if (slot >= 0) {
            const int r = tok / p.t_len;
            const size_t idx =
                ((((size_t)p.layer * p.kv_rows + r) * p.n_heads + h) * p.s_max + slot) * p.hd + i;
            (sec == 1 ? p.kv_k : p.kv_v)[idx] = __float2bfloat16_rn(y);
          }
        }
      }
    }
  }
}

__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ float4 ld_cluster_f4(uint32_t local_addr, uint32_t rank) {
  uint32_t remote;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local_addr), "r"(rank));
  float4 v;
  asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];"
               : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(remote) : "memory");
  return v;
}

template <int EPI>
__global__ void __launch_bounds__(128, 1)
gemm_tc_kernel(const KernelParams p, const __grid_constant__ CUtensorMap tm_a,
               const __grid_constant__ CUtensorMap tm_a2, const __grid_constant__ CUtensorMap tm_b) {
  constexpr bool DUAL = (EPI == GEMM_EPI_SWIGLU || EPI == GEMM_EPI_ADD2);
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t full_bar[kMaxStages];
  __shared__ __align__(8) uint64_t empty_bar[kMaxStages];
  __shared__ __align__(8) uint64_t acc_bar;
  __shared__ uint32_t tmem_slot;
  __shared__ int s_last;
  __shared__ volatile int s_abort;

  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int tile = blockIdx.x, split = blockIdx.y;
  const int kb0 = (int)(((long long)split * p.kb_total) / p.splits);
  const int kb1 = (int)(((long long)(split + 1) * p.kb_total) / p.splits);
  const int nkb = kb1 - kb0;
  const uint32_t a_bytes = kATileBytes * (DUAL ? 2u : 1u);
  const uint32_t b_bytes = (uint32_t)p.nt * kBlockK * 2u;
  const uint32_t stage_bytes = a_bytes + b_bytes;

  if (threadIdx.x == 0) {
    for (int i = 0; i < p.stages; ++i) {
      mbar_init(&full_bar[i], 1);
      mbar_init(&empty_bar[i], 1);
    }
    mbar_init(&acc_bar, 1);
    s_abort = 0;
    fence_barrier_init();
    tma_prefetch_desc(&tm_a);
    if (DUAL) tma_prefetch_desc(&tm_a2);
    tma_prefetch_desc(&tm_b);
  }
  if (warp == 1) {
    tmem_alloc(&tmem_slot, p.tmem_cols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_slot;
  pdl_launch_dependents();  // after this CTA holds its TMEM: a dependent grid cannot take it first

  const uint32_t idesc = idesc_bf16_f32(kTileRows, (uint32_t)p.nt);
  uint32_t it_p = 0, it_c = 0;
  bool alive = true;

  // One token pass per CTA (blockIdx.z): with more than 256 tokens the passes of a tile run as
  // separate CTAs, two to an SM, so that one's epilogue overlaps the other's loads and MMAs.
  const int pass0 = blockIdx.z;
  for (int pass = pass0; pass < pass0 + 1 && alive; ++pass) {
    const int tok0 = pass * p.nt;
    if (warp == 0 && lane == 0) {
      // ---- TMA producer ------------------------------------------------------------------
      int kb = kb0;
      {
        const int n_pre = nkb < p.stages ? nkb : p.stages;  // all stages are free: weights first
        for (int i = 0; i < n_pre; ++i) {
          uint8_t* st = smem + (size_t)i * stage_bytes;
          mbar_expect_tx(&full_bar[i], stage_bytes);
          tma_load_2d(st, &tm_a, &full_bar[i], (kb0 + i) * (int)kBlockK, tile * (int)kTileRows);
          if (DUAL) tma_load_2d(st + kATileBytes, &tm_a2, &full_bar[i], (kb0 + i) * (int)kBlockK, tile * (int)kTileRows);
        }
        pdl_wait();  // activations come from the previous kernel
        for (int i = 0; i < n_pre; ++i)
          tma_load_2d(smem + (size_t)i * stage_bytes + a_bytes, &tm_b, &full_bar[i], (kb0 + i) * (int)kBlockK, tok0);
        it_p = n_pre;
        kb = kb0 + n_pre;
      }
      for (; kb < kb1; ++kb, ++it_p) {
        const uint32_t stage = it_p % p.stages, use = it_p / p.stages;
        if (use > 0 && !wait_or_abort(&empty_bar[stage], (use - 1) & 1, &s_abort)) {
          atomicOr(p.status, VVS_DEV_TIMEOUT);
          s_abort = 1;
          break;
        }
        uint8_t* st = smem + (size_t)stage * stage_bytes;
        mbar_expect_tx(&full_bar[stage], stage_bytes);
        tma_load_2d(st, &tm_a, &full_bar[stage], kb * (int)kBlockK, tile * (int)kTileRows);
        if (DUAL) tma_load_2d(st + kATileBytes, &tm_a2, &full_bar[stage], kb * (int)kBlockK, tile * (int)kTileRows);
        tma_load_2d(st + a_bytes, &tm_b, &full_bar[stage], kb * (int)kBlockK, tok0);
      }
    } else if (warp == 1 && lane == 0) {
      // ---- MMA issuer --------------------------------------------------------------------
      bool ok = true;
      for (int kb = kb0; kb < kb1; ++kb, ++it_c) {
        const uint32_t stage = it_c % p.stages, use = it_c / p.stages;
        if (!wait_or_abort(&full_bar[stage], use & 1, &s_abort)) {
          atomicOr(p.status, VVS_DEV_TIMEOUT);
          s_abort = 1;
          ok = false;
          break;
        }
        tc_fence_after();
        const uint32_t a_addr = smem_u32(smem + (size_t)stage * stage_bytes);
        const uint32_t b_addr = a_addr + a_bytes;
#pragma unroll
        for (uint32_t k16 = 0; k16 < kBlockK / 16; ++k16) {
          const uint32_t acc = (kb > kb0 || k16 > 0) ? 1u : 0u;
          const uint64_t bd = smem_desc_sw128(b_addr + k16 * 32);
          mma_bf16(tmem_base, smem_desc_sw128(a_addr + k16 * 32), bd, idesc, acc);
          if (DUAL) mma_bf16(tmem_base + (uint32_t)p.nt, smem_desc_sw128(a_addr + kATileBytes + k16 * 32), bd, idesc, acc);
        }
        mma_commit(&empty_bar[stage]);  // frees the stage once these MMAs have read it
      }
      if (ok) mma_commit(&acc_bar);
    }
    __syncwarp();
    pdl_wait();
    // ---- epilogue: all four warps ----------------------------------------------------------
    bool got = wait_or_abort(&acc_bar, 0, &s_abort);
    if (!got) s_abort = 1;
    if (__syncthreads_or(got ? 0 : 1)) {
      if (threadIdx.x == 0) atomicOr(p.status, VVS_DEV_TIMEOUT);
      if (EPI == GEMM_EPI_ADD && p.cluster_mode) {   // the other CTAs of the cluster wait on these two barriers
        cluster_sync_all();
        cluster_sync_all();
      }
      alive = false;
      break;
    }
    tc_fence_after();

    const int n = tile * (int)kTileRows + warp * 32 + lane;  // weight row of this thread = TMEM lane
    const uint32_t t_row = tmem_base + ((uint32_t)(warp * 32) << 16);
    const bool fixup = (EPI != GEMM_EPI_ADD && EPI != GEMM_EPI_ADD2) && p.splits > 1;
    bool do_final = true;
    if (fixup) {
      for (int c0 = 0; c0 < p.nt && tok0 + c0 < p.m; c0 += 16) {
        float v[16], v2[16];
        tmem_ld16(t_row + c0, v);
        if (DUAL) tmem_ld16(t_row + (uint32_t)p.nt + c0, v2);
        if (n < p.n) {
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const int tok = tok0 + c0 + j;
            if (tok < p.m) {
              atomicAdd(&p.scratch[(size_t)tok * p.ld_scratch + n], v[j]);
              if (DUAL) atomicAdd(&p.scratch[(size_t)tok * p.ld_scratch + p.ff + n], v2[j]);
            }
          }
        }
      }
      __threadfence();
      __syncthreads();
      if (threadIdx.x == 0) {
        const int prev = atomicAdd(&p.counters[pass * gridDim.x + tile], 1);
        s_last = (prev == p.splits - 1) ? 1 : 0;
      }
      __syncthreads();
      do_final = s_last != 0;
      if (do_final) __threadfence();
    }
    if (EPI == GEMM_EPI_ADD && p.wide_add) {
      // Many tokens: the tile goes through shared memory (token-major, the ring is free once the
      // accumulator is complete) so that each thread adds four consecutive output columns of one
      // token with ONE vector reduction: a quarter of the reduction instructions, 512 contiguous
      // bytes per warp.
      float* sT = reinterpret_cast<float*>(smem);
      constexpr int kLd = (int)kTileRows + 4;
      const int ntok = min(p.nt, p.m - tok0);
      for (int c0 = 0; c0 < ntok; c0 += 16) {
        float v[16];
        tmem_ld16(t_row + c0, v);
#pragma unroll
        for (int j = 0; j < 16; ++j) sT[(c0 + j) * kLd + (int)threadIdx.x] = v[j];
      }
      __syncthreads();
      const int n_base = tile * (int)kTileRows;
      if (p.cluster_mode) {
        // The K splits of this (tile, token pass) are the CTAs of one cluster (cluster rank = split).
        // Rank r sums token rows r, r + splits, ... over all ranks' staged tiles in rank order and is
        // the only writer of those outputs.
        cluster_sync_all();
        const uint32_t rank = (uint32_t)split, nrank = (uint32_t)p.splits;
        const int mine = ntok > (int)rank ? (ntok - (int)rank + (int)nrank - 1) / (int)nrank : 0;
        const uint32_t sT_addr = smem_u32(sT);
        for (int idx = threadIdx.x; idx < mine * (int)(kTileRows / 4); idx += blockDim.x) {
          const int tk = (int)rank + (idx >> 5) * (int)nrank, g4 = (idx & 31) * 4;
          float4 part[8];                                   // all remote loads in flight, then summed in rank order
#pragma unroll
          for (uint32_t q = 0; q < 8; ++q)
            if (q < nrank) part[q] = ld_cluster_f4(sT_addr + (uint32_t)(tk * kLd + g4) * 4u, q);
          float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
          for (uint32_t q = 0; q < 8; ++q)
            if (q < nrank) { acc.x += part[q].x; acc.y += part[q].y; acc.z += part[q].z; acc.w += part[q].w; }
          float* dst = p.out + (size_t)(tok0 + tk) * p.ldo + n_base + g4;
          if (n_base + g4 + 3 < p.n) {
            if (p.cluster_mode == 2) {
              const float4 o = *reinterpret_cast<const float4*>(dst);
              acc.x += o.x; acc.y += o.y; acc.z += o.z; acc.w += o.w;
            }
            *reinterpret_cast<float4*>(dst) = acc;
          } else {
            const float a4[4] = {acc.x, acc.y, acc.z, acc.w};
            for (int e = 0; e < 4; ++e)
              if (n_base + g4 + e < p.n) dst[e] = (p.cluster_mode == 2 ? dst[e] : 0.f) + a4[e];
          }
        }
        cluster_sync_all();      // nobody leaves while its tile may still be read
      } else
      for (int idx = threadIdx.x; idx < ntok * (int)(kTileRows / 4); idx += blockDim.x) {
        const int tk = idx >> 5, g4 = (idx & 31) * 4;
        const float4 val = *reinterpret_cast<const float4*>(sT + tk * kLd + g4);
        float* dst = p.out + (size_t)(tok0 + tk) * p.ldo + n_base + g4;
        if (n_base + g4 + 3 < p.n) {
          asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(dst), "f"(val.x), "f"(val.y), "f"(val.z),
                       "f"(val.w) : "memory");
        } else {
          if (n_base + g4 < p.n) atomicAdd(dst, val.x);
          if (n_base + g4 + 1 < p.n) atomicAdd(dst + 1, val.y);
          if (n_base + g4 + 2 < p.n) atomicAdd(dst + 2, val.z);
        }
      }
    } else if (do_final) {
      for (int c0 = 0; c0 < p.nt && tok0 + c0 < p.m; c0 += 16) {
        float v[16], v2[16];
        if (fixup) {
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const int tok = tok0 + c0 + j;
            v[j] = 0.f;
            v2[j] = 0.f;
            if (tok < p.m && n < p.n) {
              float* s1 = &p.scratch[(size_t)tok * p.ld_scratch + n];
              v[j] = __ldcg(s1);
              *s1 = 0.f;
              if (DUAL) {
                float* s2 = &p.scratch[(size_t)tok * p.ld_scratch + p.ff + n];
                v2[j] = __ldcg(s2);
                *s2 = 0.f;
              }
            }
          }
        } else {
          tmem_ld16(t_row + c0, v);
          if (DUAL) tmem_ld16(t_row + (uint32_t)p.nt + c0, v2);
        }
        final_chunk<EPI>(p, n, tok0 + c0, v, v2);
      }
      if (fixup && threadIdx.x == 0) p.counters[pass * gridDim.x + tile] = 0;
    }
    tc_fence_before();
    __syncthreads();
  }

  // ---- teardown ---------------------------------------------------------------------------------
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_base, p.tmem_cols);
}

// ---------------------------------------------------------------------------------------------
// positions, validity, visibility and rotation tables of the block rows: the same for every
// layer of a call.  Chain: row t sits at position fill + t and sees block rows 0..t.  Tree
// (tree_parent given): row t sits at fill + depth(t) and sees its ancestors and itself; its K/V
// still go to cache slot fill + t.
__global__ void rope_table_kernel(const int32_t* __restrict__ cache_len, const float* __restrict__ inv_freq,
                                  const int32_t* __restrict__ tree_parent, int n_images, int n_forced,
                                  int32_t* __restrict__ slot_pos, int32_t* __restrict__ seq_order,
                                  uint32_t* __restrict__ anc_mask,
                                  float* __restrict__ rope_cos, float* __restrict__ rope_sin, int t_len, int hd,
                                  int s_max, int rope_mode, int grid_w, int n_prefix, int32_t* status,
                                  unsigned* clear_words, int n_clear) {
  __shared__ int s_depth;
  const int m = blockIdx.x, r = m / t_len, t = m % t_len;
  // the stage counters of the chain kernel that follows in the stream start from zero
  if (blockIdx.x == 0) {
    for (int i = threadIdx.x; i < n_clear; i += blockDim.x) clear_words[i] = 0u;
    // sequences by descending fill level (ties by index): the row-batched attention starts its longest
    // (sequence, head) items first, so that the short ones fill the tail of the grid
    const int n_rows = gridDim.x / t_len;
    for (int i = threadIdx.x; i < n_rows; i += blockDim.x) {
      const int fi = cache_len[i];
      int rank = 0;
      for (int j = 0; j < n_rows; ++j) {
        const int fj = cache_len[j];
        rank += (fj > fi || (fj == fi && j < i)) ? 1 : 0;
      }
      seq_order[rank] = i;
    }
  }
  const int fill = cache_len[r];
  const bool ok = fill >= 0 && fill + t_len <= s_max;
  if (!ok && threadIdx.x == 0) atomicOr(status, VVS_DEV_CACHE_OVERFLOW);
  if (threadIdx.x == 0) {
    int depth = t;
    uint32_t mask = t >= 31 ? 0xffffffffu : ((2u << t) - 1u);
    if (tree_parent) {
      const int32_t* par = tree_parent + (size_t)(r % n_images) * t_len;
      bool bad = false;
      depth = 0;
      mask = 1u << t;
      for (int c = t, steps = 0; c > 0 && steps < 32; ++steps) {
        const int q = par[c];
        // forced rows form a chain; a draft node hangs below the last forced row or a draft node
        if (q < 0 || q >= c || (c < n_forced && q != c - 1) || (c >= n_forced && q < n_forced - 1)) {
          bad = true;
          break;
        }
        mask |= 1u << q;
        ++depth;
        c = q;
      }
      if (par[0] != -1) bad = true;
      if (bad) {
        atomicOr(status, VVS_DEV_BAD_ARG);
        depth = t;
        mask = t >= 31 ? 0xffffffffu : ((2u << t) - 1u);
      }
    }
    s_depth = depth;
    slot_pos[m] = ok ? fill + t : -1;
    anc_mask[m] = mask;
  }
  __syncthreads();
  const int pos = fill + s_depth;
  float c_lo = 0.f, c_hi = 0.f;
  if (rope_mode == VVS_ROPE_1D) {
    c_lo = c_hi = (float)pos;
  } else if (rope_mode == VVS_ROPE_2D_GRID && pos >= n_prefix) {
    const int n = pos - n_prefix;
    c_lo = (float)(n / grid_w);
    c_hi = (float)(n % grid_w);
  }
  const int half = hd / 2;
  for (int i = threadIdx.x; i < half; i += blockDim.x) {
    float sn, cs;
    sincosf(((i < half / 2) ? c_lo : c_hi) * inv_freq[i], &sn, &cs);
    rope_cos[(size_t)m * half + i] = cs;
    rope_sin[(size_t)m * half + i] = sn;
  }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

template <int EPI>
cudaError_t launch_one(const GemmTcPlan& plan, const KernelParams& kp, const CUtensorMap& a, const CUtensorMap& a2,
                       const CUtensorMap& b, int tiles, bool pdl, cudaStream_t s) {
  {
    cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(gemm_tc_kernel<EPI>), 200 * 1024 + 1024);
    if (e != cudaSuccess) return e;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(tiles, plan.splits, plan.passes);
  cfg.blockDim = dim3(128, 1, 1);
  cfg.dynamicSmemBytes = plan.smem_bytes;
  cfg.stream = s;
  cudaLaunchAttribute attr[2];
  int na = 0;
  if (pdl) {
    attr[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[na].val.programmaticStreamSerializationAllowed = 1;
    ++na;
  }
  if (kp.cluster_mode && plan.splits > 1) {          // the K splits of a tile: one cluster along grid y
    attr[na].id = cudaLaunchAttributeClusterDimension;
    attr[na].val.clusterDim.x = 1;
    attr[na].val.clusterDim.y = (unsigned)plan.splits;
    attr[na].val.clusterDim.z = 1;
    ++na;
  }
  cfg.attrs = attr;
  cfg.numAttrs = na;
  return cudaLaunchKernelEx(&cfg, gemm_tc_kernel<EPI>, kp, a, a2, b);
}

}  // namespace

// ---------------------------------------------------------------------------------------------
// host side

int make_tmap_bf16_2d(CUtensorMap* out, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return VVS_ERR_CUDA;
  cuuint64_t dims[2] = {cols, rows};
  cuuint64_t strides[1] = {cols * 2};
  cuuint32_t box[2] = {kBlockK, box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? VVS_OK : VVS_ERR_CUDA;
}

int make_weight_tmap(CUtensorMap* out, const void* w, int rows, int cols) {
  return make_tmap_bf16_2d(out, w, (uint64_t)rows, (uint64_t)cols, kTileRows);
}

GemmTcPlan plan_gemm_tc(int m, int n, int k, bool dual, bool allow_split, int n_sms, int split_cap) {
  GemmTcPlan pl{};
  pl.passes = (m + 255) / 256;
  const int per = (m + pl.passes - 1) / pl.passes;
  pl.nt = ((per + 15) / 16) * 16;
  pl.tiles = (n + (int)kTileRows - 1) / (int)kTileRows;
  pl.kb_total = (k + (int)kBlockK - 1) / (int)kBlockK;
  // split K so that one wave of CTAs covers the SMs with as few K blocks per CTA as possible
  int best = 1;
  long long best_cost = -1;
  const int cap = split_cap < 32 ? split_cap : 32;
  const int max_splits = allow_split ? (pl.kb_total < cap ? pl.kb_total : cap) : 1;
  // CTAs per SM the plan counts on.  Several token passes: two (one's epilogue overlaps the other's loads).
  // One pass of a single weight matrix: up to five small CTAs of at least two stages each -- more
  // independent weight streams per SM (measured at 18 tokens: 1.27 -> 1.09 ms per step at the XL shape,
  // 4.87 -> 4.06 ms at the 7B shape; three to eight per SM are within 3 % of one another).
  const uint32_t stage_b = kATileBytes * (dual ? 2u : 1u) + (uint32_t)pl.nt * kBlockK * 2u;
  int cps = 1;
  if (pl.passes > 1) {
    cps = 2;
  } else if (allow_split) {
    cps = (int)(218u * 1024u / (2u * stage_b));
    cps = cps > 5 ? 5 : cps < 1 ? 1 : cps;
    if (split_cap <= 8 && cps > 2) cps = 2;   // cluster reduction: fewer, longer CTAs (1.52 / 4.42 ms against 1.68 / 4.8 at five)
  }
  const long long slots = (long long)n_sms * cps;
  for (int s = 1; s <= max_splits; ++s) {
    const long long per_cta = (pl.kb_total + s - 1) / s;
    const long long waves = ((long long)pl.tiles * s * pl.passes + slots - 1) / slots;
    // mild preference for fewer splits.  (Measured at 288 tokens: charging a split for its extra atomic
    // adds, i.e. fewer and longer CTAs, made every projection slower, not faster.)
    const long long cost = per_cta * waves * 64 + s;
    if (best_cost < 0 || cost < best_cost) {
      best_cost = cost;
      best = s;
    }
  }
  pl.splits = best;
  const uint32_t stage_bytes = kATileBytes * (dual ? 2u : 1u) + (uint32_t)pl.nt * kBlockK * 2u;
  const int per_cta = (pl.kb_total + pl.splits - 1) / pl.splits;
  int stages = ((cps == 1 ? 200 : cps == 2 ? 110 : 218 / cps) * 1024) / (int)stage_bytes;
  if (stages > kMaxStages) stages = kMaxStages;
  if (stages > per_cta) stages = per_cta;
  if (stages < 1) stages = 1;
  pl.stages = stages;
  pl.smem_bytes = stages * (int)stage_bytes;
  // calls of many tokens stage the accumulator tile for vector reductions: nt rows of 132 floats
  if (!dual && pl.smem_bytes < pl.nt * ((int)kTileRows + 4) * 4) pl.smem_bytes = pl.nt * ((int)kTileRows + 4) * 4;
  pl.smem_bytes += 1024;
  uint32_t cols = 32;
  while (cols < (uint32_t)pl.nt * (dual ? 2u : 1u)) cols <<= 1;
  pl.tmem_cols = (int)cols;
  return pl;
}

int launch_gemm_tc(int epi, const GemmTcPlan& plan, const GemmTcArgs& g, cudaStream_t s) {
  KernelParams kp{};
  kp.m = g.m; kp.n = g.n; kp.k = g.k;
  kp.nt = plan.nt; kp.passes = plan.passes; kp.kb_total = plan.kb_total; kp.splits = plan.splits;
  kp.stages = plan.stages; kp.tmem_cols = (uint32_t)plan.tmem_cols;
  // (at 32 tokens and fewer the staged vector reductions were measured no faster than scalar ones)
  kp.wide_add = (epi == GEMM_EPI_ADD && (plan.nt > 32 || g.cluster_mode) && g.ldo % 4 == 0 &&
                 (reinterpret_cast<uintptr_t>(g.out) & 15) == 0) ? 1 : 0;
  kp.cluster_mode = (kp.wide_add && plan.splits <= 8) ? g.cluster_mode : 0;
  if (g.cluster_mode && !kp.cluster_mode) return VVS_ERR_SHAPE;   // the caller planned for a cluster
  kp.scratch = g.scratch; kp.ld_scratch = g.ld_scratch; kp.counters = g.counters; kp.status = g.status;
  kp.out = g.out; kp.ldo = g.ldo;
  kp.q = g.q; kp.kv_k = g.kv_k; kp.kv_v = g.kv_v; kp.slot_pos = g.slot_pos;
  kp.rope_cos = g.rope_cos; kp.rope_sin = g.rope_sin;
  kp.d = g.d; kp.n_heads = g.n_heads; kp.hd = g.hd; kp.s_max = g.s_max; kp.layer = g.layer;
  kp.kv_rows = g.kv_rows; kp.t_len = g.t_len;
  kp.act = g.act; kp.ff = g.ff;
  const CUtensorMap& a2 = g.tm_a2 ? *g.tm_a2 : *g.tm_a;
  cudaError_t e;
  switch (epi) {
    case GEMM_EPI_STORE: e = launch_one<GEMM_EPI_STORE>(plan, kp, *g.tm_a, a2, *g.tm_b, plan.tiles, g.pdl, s); break;
    case GEMM_EPI_ADD: e = launch_one<GEMM_EPI_ADD>(plan, kp, *g.tm_a, a2, *g.tm_b, plan.tiles, g.pdl, s); break;
    case GEMM_EPI_QKV: e = launch_one<GEMM_EPI_QKV>(plan, kp, *g.tm_a, a2, *g.tm_b, plan.tiles, g.pdl, s); break;
    case GEMM_EPI_SWIGLU: e = launch_one<GEMM_EPI_SWIGLU>(plan, kp, *g.tm_a, a2, *g.tm_b, plan.tiles, g.pdl, s); break;
    case GEMM_EPI_ADD2: e = launch_one<GEMM_EPI_ADD2>(plan, kp, *g.tm_a, a2, *g.tm_b, plan.tiles, g.pdl, s); break;
    default: return VVS_ERR_INVALID_ARG;
  }
  return e == cudaSuccess ? VVS_OK : VVS_ERR_CUDA;
}

void launch_rope_table(const int32_t* cache_len, const int32_t* tree_parent, int n_images, int n_forced,
                       const Workspace& ws, const vvs_model_desc& md, int n_rows, int t_len, cudaStream_t s,
                       unsigned* clear_words, int n_clear) {
  rope_table_kernel<<<n_rows * t_len, 64, 0, s>>>(cache_len, ws.rope_inv_freq, tree_parent, n_images, n_forced,
                                                  ws.slot_pos, ws.seq_order, ws.anc_mask, ws.rope_cos, ws.rope_sin, t_len,
                                                  md.head_dim, md.s_max, md.rope_mode, md.rope_grid_w, md.n_prefix,
                                                  ws.status, clear_words, n_clear);
}

}  // namespace vvs
