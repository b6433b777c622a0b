// LM head with the decision epilogue fused in (bf16, tensor cores): logits over the codebook are
// never written to global memory unless the caller asked for target_probs.
//
// Roles as in the projection GEMM: the 128 codebook rows of a tile sit on the MMA's M side, the
// feature rows on N.  One pass covers up to 128 DECISION rows (image, block position); with
// guidance the conditional and the unconditional feature rows of the same decision row are loaded
// as two TMA boxes into one token tile, so both logits of a pair are columns of one accumulator.
// Epilogue of a pass, straight from TMEM:
//   1. l = l_u + s (l_c - l_u), divided by the temperature          (the guided logit)
//   2. the [128 codes x rows] tile goes to shared memory; one thread per decision row reduces it
//      to the tile's (max, sum exp) softmax partial
//   3. the guided logits of each drafted token and of its first nbr_k CSR neighbours are picked
//      out of the tile (whatever part of them lies in this tile)
//   4. only on request: the guided logits are stored, to be normalised in place afterwards
// Row mode (second launch, after acceptance): the feature rows are the one row per image the
// next token is sampled from; the epilogue turns the guided logits into probabilities with that
// row's statistics and writes one V-row per image.  The sums are the same tensor-core sums as in
// the first launch, so decided and sampled probabilities agree bit for bit.
#include <math_constants.h>

#include "tc_common.cuh"
#include "vvs_internal.cuh"

namespace vvs {

using namespace tc;

namespace {

constexpr int kMaxStages = 10;
constexpr uint32_t kTileRows = 128;
constexpr uint32_t kBlockK = 64;
constexpr uint32_t kATileBytes = kTileRows * kBlockK * 2;
constexpr int kTileLd = 129;   // padded row length of the logit tile in shared memory

struct LmParams {
  int v, k, bt;                // codebook size, d_model, decision rows (B * rows_per_seq)
  int n_cfg, nd_pad, passes, kb_total, stages;
  uint32_t tmem_cols;
  float cfg_scale, inv_temp;
  float* part_m; float* part_s;     // [n_tiles, bt]
  float* logits_out;                // optional [bt, v]
  int32_t* status;
  // gathers
  int rows_per_seq, first_row, n_draft_max, vocab_offset, relaxed, nbr_k, kmax, drafts_ld;
  const int32_t* drafts; const int32_t* row_ptr; const int32_t* col;
  float* l_tok; float* l_nbr;
  // row mode
  int row_mode;
  const int32_t* sel_row; const float* stat_m; const float* stat_inv; float* p_row;
};

__device__ __forceinline__ bool wait_or_abort(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
  for (uint32_t i = 0; i < kSpinLimit; ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((i & 1023u) == 1023u && *abort_flag) return false;
  }
  return false;
}

// NM = codebook tiles of 128 rows per CTA.  With NM = 2 the feature tile of a k-block is read from L2
// once for 256 codes (two MMAs on one B operand, two accumulators side by side in TMEM): half the
// feature traffic per flop, which is what bounds the kernel at large batch; used when the codebook
// still gives every SM a CTA.  The logit tile then reuses the (idle) pipeline stages.
template <int NM>
__global__ void __launch_bounds__(128, 1)
lmhead_tc_kernel(const LmParams p, const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t full_bar[kMaxStages];
  __shared__ __align__(8) uint64_t empty_bar[kMaxStages];
  __shared__ __align__(8) uint64_t acc_bar;
  __shared__ uint32_t tmem_slot;
  __shared__ volatile int s_abort;

  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, tid = threadIdx.x;
  const int tile0 = blockIdx.y * NM;
  const int C = p.n_cfg;
  const uint32_t half_bytes = (uint32_t)p.nd_pad * kBlockK * 2u;     // one box of feature rows
  const uint32_t b_bytes = half_bytes * (uint32_t)C;
  constexpr uint32_t a_bytes = kATileBytes * NM;
  const uint32_t stage_bytes = a_bytes + b_bytes;
  // [nd_pad][kTileLd]; with two tiles per CTA it lies over the stages, which are idle during an epilogue
  float* sL = reinterpret_cast<float*>(NM == 2 ? smem : smem + (size_t)p.stages * stage_bytes);
  const int nt = p.nd_pad * C;

  if (tid == 0) {
    for (int i = 0; i < p.stages; ++i) {
      mbar_init(&full_bar[i], 1);
      mbar_init(&empty_bar[i], 1);
    }
    mbar_init(&acc_bar, 1);
    s_abort = 0;
    fence_barrier_init();
    tma_prefetch_desc(&tm_a);
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
  pdl_launch_dependents();

  const uint32_t idesc = idesc_bf16_f32(kTileRows, (uint32_t)nt);
  uint32_t it_p = 0, it_c = 0;
  bool alive = true;

  // The CTAs of one codebook tile sit next to each other on grid x and deal the passes among
  // themselves: they stream the same weight rows at the same time, so all but one of them find
  // those rows in L2, and the work comes in units of one pass instead of one whole tile.
  int iter = 0;
  for (int pass = blockIdx.x; pass < p.passes && alive; pass += gridDim.x, ++iter) {
    const int row0 = pass * 128;                                  // first decision row of the pass
    const int nd = p.bt - row0 < 128 ? p.bt - row0 : 128;
    if (warp == 0 && lane == 0) {
      // ---- TMA producer: weights may be requested before the features exist ------------------
      int kb = 0;
      if (iter == 0) {
        const int n_pre = p.kb_total < p.stages ? p.kb_total : p.stages;
        for (int i = 0; i < n_pre; ++i) {
          mbar_expect_tx(&full_bar[i], stage_bytes);
#pragma unroll
          for (int m = 0; m < NM; ++m)
            tma_load_2d(smem + (size_t)i * stage_bytes + m * kATileBytes, &tm_a, &full_bar[i], i * (int)kBlockK,
                        (tile0 + m) * (int)kTileRows);
        }
        pdl_wait();
        for (int i = 0; i < n_pre; ++i) {
          uint8_t* b = smem + (size_t)i * stage_bytes + a_bytes;
          tma_load_2d(b, &tm_b, &full_bar[i], i * (int)kBlockK, row0);
          if (C == 2) tma_load_2d(b + half_bytes, &tm_b, &full_bar[i], i * (int)kBlockK, p.bt + row0);
        }
        it_p = n_pre;
        kb = n_pre;
      }
      for (; kb < p.kb_total; ++kb, ++it_p) {
        const uint32_t stage = it_p % p.stages, use = it_p / p.stages;
        if (use > 0 && !wait_or_abort(&empty_bar[stage], (use - 1) & 1, &s_abort)) {
          atomicOr(p.status, VVS_DEV_TIMEOUT);
          s_abort = 1;
          break;
        }
        uint8_t* st = smem + (size_t)stage * stage_bytes;
        mbar_expect_tx(&full_bar[stage], stage_bytes);
#pragma unroll
        for (int m = 0; m < NM; ++m)
          tma_load_2d(st + m * kATileBytes, &tm_a, &full_bar[stage], kb * (int)kBlockK, (tile0 + m) * (int)kTileRows);
        tma_load_2d(st + a_bytes, &tm_b, &full_bar[stage], kb * (int)kBlockK, row0);
        if (C == 2) tma_load_2d(st + a_bytes + half_bytes, &tm_b, &full_bar[stage], kb * (int)kBlockK, p.bt + row0);
      }
    } else if (warp == 1 && lane == 0) {
      // ---- MMA issuer --------------------------------------------------------------------------
      bool ok = true;
      for (int kb = 0; kb < p.kb_total; ++kb, ++it_c) {
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
          const uint64_t bd = smem_desc_sw128(b_addr + k16 * 32);
#pragma unroll
          for (uint32_t m = 0; m < (uint32_t)NM; ++m)
            mma_bf16(tmem_base + m * (uint32_t)nt, smem_desc_sw128(a_addr + m * kATileBytes + k16 * 32), bd, idesc,
                     (kb > 0 || k16 > 0) ? 1u : 0u);
        }
        mma_commit(&empty_bar[stage]);
      }
      if (ok) mma_commit(&acc_bar);
    }
    __syncwarp();
    pdl_wait();
    bool got = wait_or_abort(&acc_bar, iter & 1, &s_abort);
    if (!got) s_abort = 1;
    if (__syncthreads_or(got ? 0 : 1)) {
      if (tid == 0) atomicOr(p.status, VVS_DEV_TIMEOUT);
      alive = false;
      break;
    }
    tc_fence_after();

    for (int mt = 0; mt < NM; ++mt) {
    const int tile = tile0 + mt;
    if (tile * (int)kTileRows >= p.v) break;                        // the codebook ends before this tile
    // ---- 1. guided logits of this thread's codebook row, for every decision row of the pass ------
    const int n = tile * (int)kTileRows + tid;
    const bool n_ok = n < p.v;
    const uint32_t t_row = tmem_base + (uint32_t)(mt * nt) + ((uint32_t)(warp * 32) << 16);
    for (int c0 = 0; c0 < p.nd_pad && c0 < nd; c0 += 16) {
      float lc[16], lu[16];
      tmem_ld16(t_row + c0, lc);
      if (C == 2) tmem_ld16(t_row + (uint32_t)p.nd_pad + c0, lu);
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        const int r = c0 + j;
        if (r < nd) {
          float l = lc[j];
          if (C == 2) l = lu[j] + p.cfg_scale * (l - lu[j]);
          l *= p.inv_temp;
          if (p.row_mode) {
            const int sel = p.sel_row[row0 + r];
            if (n_ok) p.p_row[(size_t)(row0 + r) * p.v + n] = sel >= 0 ? prob_of(l, p.stat_m[sel], p.stat_inv[sel]) : 0.f;
          } else {
            sL[r * kTileLd + tid] = n_ok ? l : -CUDART_INF_F;
            if (p.logits_out && n_ok) p.logits_out[(size_t)(row0 + r) * p.v + n] = l;
          }
        }
      }
    }
    if (!p.row_mode) {
      __syncthreads();
      // ---- 2. softmax partial of the tile, one thread per decision row ---------------------------
      if (tid < nd) {
        const float* row = sL + tid * kTileLd;
        float mx = -CUDART_INF_F;
        for (int i = 0; i < 128; ++i) mx = fmaxf(mx, row[i]);
        float sum = 0.f;
        if (mx > -CUDART_INF_F)
          for (int i = 0; i < 128; ++i) sum += expf(row[i] - mx);
        p.part_m[(size_t)tile * p.bt + row0 + tid] = mx;
        p.part_s[(size_t)tile * p.bt + row0 + tid] = sum;
      }
      // ---- 3. logits of the drafted tokens and of their neighbours that live in this tile --------
      // One warp per (image, draft) pair of the pass; its lanes walk the draft's neighbour row (one
      // coalesced load of the column indices per 32 neighbours) and pick the entries of this tile.
      if (p.n_draft_max > 0) {
        const int kk_max = p.relaxed ? p.nbr_k : 1;
        const int b0 = row0 / p.rows_per_seq, b1 = (row0 + nd - 1) / p.rows_per_seq;
        const int n_pairs = (b1 - b0 + 1) * p.n_draft_max;
        if (kk_max <= 1) {                                  // strict: one thread per pair
          for (int pr = tid; pr < n_pairs; pr += 128) {
            const int b = b0 + pr / p.n_draft_max, i = pr % p.n_draft_max;
            const int r = b * p.rows_per_seq + p.first_row + i - row0;
            if (r < 0 || r >= nd) continue;
            const int x = p.drafts[(size_t)b * p.drafts_ld + i] - p.vocab_offset;
            if (x >= 0 && x < p.v && (x >> 7) == tile) p.l_tok[b * p.n_draft_max + i] = sL[r * kTileLd + (x & 127)];
          }
        } else
        for (int pr = warp; pr < n_pairs; pr += 4) {
          const int b = b0 + pr / p.n_draft_max, i = pr % p.n_draft_max;
          const int r = b * p.rows_per_seq + p.first_row + i - row0;   // decision row inside the pass
          if (r < 0 || r >= nd) continue;
          const int x = p.drafts[(size_t)b * p.drafts_ld + i] - p.vocab_offset;
          if (x < 0 || x >= p.v) continue;                            // reported by the acceptance kernel
          if (lane == 0 && (x >> 7) == tile) p.l_tok[b * p.n_draft_max + i] = sL[r * kTileLd + (x & 127)];
          const int beg = p.row_ptr[x], len = p.row_ptr[x + 1] - beg;
          const int kk = kk_max < len ? kk_max : len;
          float* dst = p.l_nbr + ((size_t)b * p.n_draft_max + i) * p.kmax;
          for (int jj = 1 + lane; jj < kk; jj += 32) {
            const int c = p.col[beg + jj];
            if (c < 0 || c >= p.v) {
              atomicOr(p.status, VVS_DEV_BAD_NEIGHBOUR);
              if (tile == 0) dst[jj] = -CUDART_INF_F;
            } else if ((c >> 7) == tile) {
              dst[jj] = sL[r * kTileLd + (c & 127)];
            }
          }
        }
      }
    }
    if (NM == 2) __syncthreads();                                 // the logit tile is reused by the next codebook tile
    }
    tc_fence_before();
    __syncthreads();
  }

  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_base, p.tmem_cols);
}

}  // namespace

int launch_lmhead_tc(const LmHeadArgs& a, cudaStream_t s) {
  LmParams p{};
  p.v = a.v; p.k = a.k; p.bt = a.bt; p.n_cfg = a.n_cfg;
  const int rows = a.bt < 128 ? a.bt : 128;
  p.nd_pad = ((rows + 15) / 16) * 16;
  p.passes = (a.bt + 127) / 128;
  p.kb_total = (a.k + (int)kBlockK - 1) / (int)kBlockK;
  p.cfg_scale = a.cfg_scale; p.inv_temp = a.inv_temp;
  p.part_m = a.part_m; p.part_s = a.part_s; p.logits_out = a.logits_out; p.status = a.status;
  p.rows_per_seq = a.rows_per_seq; p.first_row = a.first_row; p.n_draft_max = a.n_draft_max;
  p.vocab_offset = a.vocab_offset; p.relaxed = a.relaxed; p.nbr_k = a.nbr_k; p.kmax = a.kmax;
  p.drafts_ld = a.drafts_ld; p.drafts = a.drafts; p.row_ptr = a.row_ptr; p.col = a.col;
  p.l_tok = a.l_tok; p.l_nbr = a.l_nbr;
  p.row_mode = a.row_mode; p.sel_row = a.sel_row; p.stat_m = a.stat_m; p.stat_inv = a.stat_inv; p.p_row = a.p_row;
  const int nt = p.nd_pad * a.n_cfg;
  // two codebook tiles per CTA when 256-row tiles still give every SM a CTA (the feature tile is then
  // read once per 256 codes); the logit tile lies over the stages in that case
  const int n_sms_hint = 120;
  // (row mode streams the codebook once for a few feature rows: single tiles, and where the codebook
  // has two of them for every SM, CTAs small enough to sit two to an SM, so that one CTA's fill and
  // epilogue hide behind the other's stream)
  const bool two = !a.row_mode && a.v >= 2 * (int)kTileRows * n_sms_hint && 2 * nt <= 512;
  const uint32_t stage_bytes = kATileBytes * (two ? 2u : 1u) + (uint32_t)nt * kBlockK * 2u;
  const size_t tile_bytes = a.row_mode ? 0 : (size_t)p.nd_pad * kTileLd * 4;
  const int n_sms = a.n_sms > 0 ? a.n_sms : 148;
  const bool small_ctas = a.row_mode && nt <= 256 && (a.v + 127) / 128 >= 2 * n_sms;
  const size_t smem_budget = small_ctas ? 108 * 1024 : 220 * 1024;
  int stages = (int)((smem_budget - (two ? 0 : tile_bytes)) / stage_bytes);
  if (stages > kMaxStages) stages = kMaxStages;
  if (stages > p.kb_total) stages = p.kb_total;
  if (stages < 1) return VVS_ERR_SHAPE;
  p.stages = stages;
  uint32_t cols = 32;
  while (cols < (uint32_t)nt * (two ? 2u : 1u)) cols <<= 1;
  p.tmem_cols = cols;
  size_t smem = (size_t)stages * stage_bytes + (two ? 0 : tile_bytes);
  if (two && smem < tile_bytes) smem = tile_bytes;
  smem += 1024;
  if (smem > 226 * 1024) return VVS_ERR_SHAPE;
  const void* fn = two ? reinterpret_cast<const void*>(lmhead_tc_kernel<2>) : reinterpret_cast<const void*>(lmhead_tc_kernel<1>);
  if (ensure_dynamic_smem(fn, 226 * 1024) != cudaSuccess) return VVS_ERR_CUDA;
  cudaLaunchConfig_t cfg = {};
  const int rows_per_cta = (int)kTileRows * (two ? 2 : 1);
  const int tiles = (a.v + rows_per_cta - 1) / rows_per_cta;
  // CTAs per codebook tile: the count that needs the fewest rounds of (one pass on every SM); the
  // smaller count on a tie (fewer pipeline fills)
  int share = 1;
  long best = -1;
  for (int g = 1; g <= p.passes; ++g) {
    const long rounds = (long)((tiles * g + n_sms - 1) / n_sms) * ((p.passes + g - 1) / g);
    if (best < 0 || rounds < best) { best = rounds; share = g; }
  }
  cfg.gridDim = dim3(share, tiles, 1);
  cfg.blockDim = dim3(128, 1, 1);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = a.pdl ? 1 : 0;
  const cudaError_t e = two ? cudaLaunchKernelEx(&cfg, lmhead_tc_kernel<2>, p, *a.tm_a, *a.tm_b)
                            : cudaLaunchKernelEx(&cfg, lmhead_tc_kernel<1>, p, *a.tm_a, *a.tm_b);
  return e == cudaSuccess ? VVS_OK : VVS_ERR_CUDA;
}

int lmhead_box_rows(int bt) {
  const int rows = bt < 128 ? bt : 128;
  return ((rows + 15) / 16) * 16;
}

// Copies the feature rows of the decision row each image samples from (cond rows, then uncond
// rows) into a compact [n_cfg * B, d] matrix; images without such a row get zeros.
__global__ void gather_sel_rows_kernel(const uint4* __restrict__ hid, const int32_t* __restrict__ sel_row,
                                       uint4* __restrict__ out, int n_images, int bt, int vec_per_row) {
  const int b = blockIdx.x, c = blockIdx.y;
  const int sel = sel_row[b];
  for (int i = threadIdx.x; i < vec_per_row; i += blockDim.x)
    out[((size_t)c * n_images + b) * vec_per_row + i] =
        sel >= 0 ? hid[((size_t)c * bt + sel) * vec_per_row + i] : make_uint4(0, 0, 0, 0);
}

void launch_gather_sel_rows(const void* hid, const int32_t* sel_row, void* out, int n_images, int n_cfg, int bt,
                            int d, cudaStream_t s) {
  gather_sel_rows_kernel<<<dim3(n_images, n_cfg), 128, 0, s>>>(static_cast<const uint4*>(hid), sel_row,
                                                               static_cast<uint4*>(out), n_images, bt, d / 8);
}

}  // namespace vvs
