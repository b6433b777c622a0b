// The decoder chain of the verify step (embedding + every layer) as ONE persistent dataflow kernel
// for calls of at most 32 block tokens (bf16).
//
// Status: previous generation.  The per-projection kernels (gemm_tc.cu, attention_rows.cu) with
// programmatic dependent launch were measured faster at both benchmark shapes and are the default;
// this kernel runs only in contexts created under the debug switch VVS_DEBUG_CHAIN_KERNELS with
// fixed-order sums, and stays parity-tested.
//
// At this size the step is a chain of ~180 dependent small projections that together stream the
// whole model once: the HBM stream and the latency of the dependency chain both matter.  Design:
//
//   * Every projection is cut by OUTPUT rows: a CTA owns whole 16-row tiles of a weight matrix over
//     the full reduction length, so every sum is finished inside one CTA, in a fixed order
//     (bitwise repeatable; nothing is accumulated with atomics), and its epilogue (1/rms scaling,
//     rotation, cache append, SiLU gating, residual add, next norm's operand) runs on final values.
//   * The weights are re-packed once, when they are bound: per CTA one contiguous stream per layer,
//     in the order that CTA consumes it, each 16 x 32 piece already in the register layout of
//     mma.sync.m16n8k16 (so a fragment is one conflict-free 128-bit shared-memory load).  It is
//     streamed through a ring of shared-memory slots with bulk TMA copies issued by a producer
//     warp that waits for nothing but a free slot, so HBM runs ahead of the dependency chain by the
//     ring depth.  (Every instruction a lone thread executes costs ~5 cycles: bookkeeping of a few
//     hundred instructions per block on a computing warp's path cost more than the MMAs.)
//     The old K / V rows of an attention item travel through the same ring as 2-D TMA tiles.
//   * The <= 32 tokens are the N side of the MMAs (8 per n-tile).  The activations a stage reads
//     (a few tens of KB, in L2) are kept in global memory in B-fragment order (span of 32 k, n-tile,
//     lane: 16 bytes each; the k order inside a span is permuted, identically in the packed weights,
//     so that a lane's share is contiguous); each CTA pulls the k group it works on into shared
//     memory with one bulk TMA copy (the load/store units sustain far fewer requests in flight than
//     the copy engine: register-staged loads of the same bytes took three times as long).
//   * Stages of a layer: QKV | attention | O | gate+up | down.  There is no grid barrier: each
//     (layer, stage) has an arrival counter in global memory, a CTA with work in a stage waits until
//     the producers of the previous stage have all arrived (release / acquire), CTAs without work in
//     a stage do not take part.  A sequencer warp follows the CTA's program: it polls the counter,
//     starts the activation copies, tells the computing warps to go, and after their epilogue makes
//     the CTA's own arrival; the computing warps only ever wait on shared-memory barriers.
//     Every wait is bounded; one that runs out raises VVS_DEV_TIMEOUT, after which all waits fall
//     through and the kernel drains.
//   * Attention: one CTA per (sequence, head), keys split over the warps (16-key slices, online
//     softmax in registers, QK^T and PV as mma.sync with ldmatrix on 128-byte-swizzled tiles), the
//     block's own rows are read back from the cache after the QKV stage; warps merge through
//     shared memory in a fixed tree.
//
// Tensor cores: warp-level mma.sync on purpose.  At <= 32 tokens a tcgen05.mma (M = 128) issued by
// one thread every ~68 cycles does no more work per cycle than the four sub-cores' warp MMAs, and
// its TMEM round trip and operand staging sit on the critical path of every stage.
#include <math_constants.h>

#include <algorithm>
#include <cstdio>
#include <cstdlib>
#include <numeric>
#include <vector>

#include "att_mma.cuh"
#include "tc_common.cuh"
#include "vvs_internal.cuh"

#ifndef VVS_CS_TRACE
#define VVS_CS_TRACE(tag) ((void)0)
#define VVS_CS_TRACE_DECL
#define VVS_CS_TRACE_END ((void)0)
#define VVS_CS_TRACE_SEQ(tag) ((void)0)
#endif

namespace vvs {

using namespace tc;
using namespace attmma;

namespace {

using bf16 = __nv_bfloat16;

constexpr int kCW = 8;                      // warps
constexpr int kCT = kCW * 32;
constexpr int kThreads = kCT + 128;         // + one warp group: weight producer warp, sequencer warp, two idle
constexpr int kTP = 4;                      // weight tiles per sub-panel (accumulators held at once)
constexpr int kGroupSpans = 20;             // 32-wide k spans per k group (one ring slot per tile and group)
constexpr int kMaxSpw = (kGroupSpans + kCW - 1) / kCW;   // spans of a group per warp
constexpr int kSlotBytes = kGroupSpans * 1024;
constexpr int kMaxSlots = 8;
constexpr int kActSlots = 2;                  // (the sequencer toggles between exactly two)
constexpr int kNewBytes = 16384;            // the block's own K and V rows (32 x 256 B each)
constexpr int kMergeBytes = 34816;          // attention merge
constexpr int kRopeUnits = 8;               // QKV tiles of a CTA whose rotation table is cached in shared memory
constexpr int kMiscBytes = kRopeUnits * 32 * 8 * 8 + 256;   // rotation cache (cos, sin) + cache slot per token
constexpr int kMaxLayers = 64;
constexpr int kMaxSeq = 32;
constexpr int kMaxBlocks = 1024;             // ring blocks of one layer of one CTA
constexpr int kMaxOwn = 2;                   // 16-column tiles of the residual stream a CTA may own
constexpr uint32_t kParkNs = 4000;
constexpr uint32_t kParkedPolls = 1u << 19;   // ~2 s
constexpr uint32_t kSpinPolls = 1u << 24;
constexpr uint32_t kFlagPolls = 1u << 22;
enum { ST_QKV = 0, ST_ATT = 1, ST_O = 2, ST_GU = 3, ST_DOWN = 4, N_ST = 5 };
enum { G_QKV = 0, G_O = 1, G_GU = 2, G_DOWN = 3 };
enum { BAR_C = 1 };

__host__ __device__ constexpr int act_slot_bytes(int nt) { return kGroupSpans * nt * 512; }
__host__ __device__ constexpr int ring_slots(int nt) { return nt <= 3 ? 7 : 5; }
__host__ __device__ constexpr size_t smem_bytes(int nt) {
  return 1024 + (size_t)ring_slots(nt) * kSlotBytes + (size_t)kActSlots * act_slot_bytes(nt) + kMiscBytes;
}

struct StreamParams {
  int n_layers, d, n_heads, hd, ff, s_max, kv_rows;
  int m, t_len, n_rows, n_images, tok_rows;
  int spans[2], gsz[2], ngroups[2];       // reduction geometry: [0] K = d, [1] K = ff
  int n_prod[N_ST + 1];                   // CTAs that arrive on each stage's counter (+ the embedding stage)
  int kb;                                 // keys per attention block in the ring
  int span_bytes;                         // bytes of one 32-wide k span of an activation buffer (all tokens)
  float eps, sl2, inv_d;                  // sl2 = log2(e) / sqrt(head_dim); inv_d = 1 / d_model
  unsigned long long layer_bytes;
  const uint8_t* packed;
  const ChainCtaPlan* plan;
  const bf16* tok_emb;
  const int32_t* block;
  float* x;
  bf16 *xn1, *xn2, *attn, *act;           // stage inputs in B-fragment order (see frag_off)
  bf16* qbuf;                             // [m, d] rotated queries, row-major
  float *ss1, *ss2;                       // [d / 16][32] sums of squares per 16-column tile and token
  const int32_t* cache_len;
  const int32_t* slot_pos;
  const uint32_t* anc_mask;
  bf16* kv_k;
  bf16* kv_v;
  const float* rope_cos;
  const float* rope_sin;
  unsigned* flags;                        // [n_layers * 5] stage counters, then embedding counter, abort word
  int32_t* status;
  const bf16* norms[2 * kMaxLayers];
};

// ---- small helpers ------------------------------------------------------------------------------------
__device__ __forceinline__ void bulk_load(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar))
               : "memory");
}
// Element offset of activation (token, k) in a B-fragment-ordered buffer: spans of 32 k; inside a
// span one 512-byte piece per n-tile of 8 tokens (the last n-tile only as many 64-byte token rows as
// there are tokens); inside a piece lane (token % 8) * 4 + (k / 8) % 4 holds k % 8 .. of its 8 values.
__device__ __forceinline__ size_t frag_off(int tok, int k, int span_bytes) {
  return ((size_t)(k >> 5) * span_bytes + (size_t)(tok >> 3) * 512 + (size_t)(((tok & 7) << 2) | ((k >> 3) & 3)) * 16) / 2 +
         (k & 7);
}

// Bounded wait on an mbarrier phase; once the CTA is in abort mode every wait falls through.
__device__ __noinline__ void wait_slow(uint64_t* bar, uint32_t parity, volatile int* s_abort, int32_t* status,
                                       uint32_t limit = kParkedPolls) {
  if (*s_abort) return;
  for (uint32_t i = 0; i < limit; ++i) {
    if (mbar_try_wait_parked(bar, parity, kParkNs)) return;
    if ((i & 15u) == 15u && *s_abort) return;
  }
  *s_abort = 1;
  atomicOr(status, VVS_DEV_TIMEOUT);
}
__device__ __forceinline__ void wait_bar(uint64_t* bar, uint32_t parity, volatile int* s_abort, int32_t* status) {
  if (mbar_try_wait(bar, parity)) return;
  wait_slow(bar, parity, s_abort, status);
}
// The same for a whole warp: one lane polls (256 polling threads slow down every arrival on the
// barrier they poll), the warp barrier passes its observation on to the others.
__device__ __forceinline__ void wait_bar_warp(uint64_t* bar, uint32_t parity, volatile int* s_abort, int32_t* status) {
  wait_bar(bar, parity, s_abort, status);
}

// The sequencer waits until `target` producers have arrived on a stage counter.
__device__ __noinline__ void wait_flag(const unsigned* flag, unsigned target, volatile int* s_abort, unsigned* abort_word,
                                       int32_t* status) {
  if (*s_abort) return;
  for (uint32_t i = 0; i < kFlagPolls; ++i) {
    if (ld_acquire_gpu(flag) >= target) return;
    if ((i & 63u) == 63u && *reinterpret_cast<volatile unsigned*>(abort_word)) break;
  }
  *s_abort = 1;
  *reinterpret_cast<volatile unsigned*>(abort_word) = 1u;
  atomicOr(status, VVS_DEV_TIMEOUT);
}

struct RingPos {
  uint32_t slot = 0, par = 0;
  __device__ __forceinline__ void next(uint32_t n) {
    if (++slot == n) { slot = 0; par ^= 1u; }
  }
};

struct ProdState {   // thread 0 only
  const uint8_t* src;
  int layer, pos, n_entries;
  int it, blk, nb, nb_valid;
  uint32_t slot, par, issued;
  int done;
};

struct Shared {
  uint64_t full[kMaxSlots], empty[kMaxSlots];
  uint64_t act_full[kActSlots], act_empty[kActSlots];
  uint64_t go, epi_done;            // sequencer -> computing warps: stage inputs ready; and back: epilogue finished
  volatile int abort;
  int n_slots;
  int fill[kMaxSeq];
  int ok[kMaxSeq];
  float rinv[32];
  ChainCtaPlan plan;
  float x_own[kMaxOwn * 32 * 16];   // this CTA's 16-column tiles of the residual stream, [tile][token][column]
  ProdState prod;
  uint8_t blk_kb[kMaxBlocks];       // sizes of a layer's weight blocks in KB, 0 = the attention blocks go here
};

// Reduction geometry of a projection: k spans, spans per group, groups.
struct Geom {
  int spans, gsz, ngroups;
};
__device__ __forceinline__ Geom geom_of(const StreamParams& p, int which) {
  return Geom{p.spans[which], p.gsz[which], p.ngroups[which]};
}
__device__ __forceinline__ int group_spans(const Geom& g, int grp) {
  const int left = g.spans - grp * g.gsz;
  return left < g.gsz ? left : g.gsz;
}

// ---- producer: thread 0's second job ---------------------------------------------------------------------
// The blocks this CTA consumes, in order: per layer the QKV tiles, the old K / V rows of its
// attention items, then the O, gate / up and down tiles (sub-panel, k group, tile).  The weight
// blocks of a layer are contiguous in the packed copy and the same in every layer: their sizes (KB)
// are listed once in shared memory, a zero entry marks where the attention blocks go.
struct ProdEnv {
  const StreamParams* p;
  Shared* sh;
  uint8_t* ring;
  const CUtensorMap* tm_k;
  const CUtensorMap* tm_v;
  int grid;
};

// Thread 0, once: the block list of a layer and the start state.
__device__ __noinline__ void prod_init(const ProdEnv& e) {
  const StreamParams& p = *e.p;
  Shared& sh = *e.sh;
  const ChainCtaPlan& pl = sh.plan;
  int n = 0;
  auto add_task = [&](int kind) {
    const int count = pl.n[kind];
    const Geom ge = geom_of(p, kind == G_DOWN ? 1 : 0);
    const int units = kind == G_GU ? kTP / 2 : kTP, per = kind == G_GU ? 2 : 1;
    for (int u0 = 0; u0 < count; u0 += units) {
      const int nt_sub = (count - u0 < units ? count - u0 : units) * per;
      for (int grp = 0; grp < ge.ngroups; ++grp)
        for (int t = 0; t < nt_sub; ++t)
          if (n < kMaxBlocks) sh.blk_kb[n++] = (uint8_t)group_spans(ge, grp);
    }
  };
  add_task(G_QKV);
  if (pl.att_rank < p.n_rows * p.n_heads && n < kMaxBlocks) sh.blk_kb[n++] = 0;
  add_task(G_O);
  add_task(G_GU);
  add_task(G_DOWN);
  ProdState& st = sh.prod;
  st.src = p.packed + pl.off;
  st.layer = 0; st.pos = 0; st.n_entries = n;
  st.it = pl.att_rank; st.blk = 0; st.nb = 0; st.nb_valid = 0;
  st.slot = 0; st.par = 0; st.issued = 0;
  st.done = n == 0 ? 1 : 0;
}

// The weight producer (one thread): issues every block of the CTA's program as ring slots free up.
__device__ __noinline__ void producer_loop(const ProdEnv& e) {
  const StreamParams& p = *e.p;
  Shared& sh = *e.sh;
  ProdState& st = sh.prod;
  const int n_items = p.n_rows * p.n_heads;
  while (!st.done) {
    if (sh.abort) return;
    if (st.pos == st.n_entries) {   // next layer
      st.pos = 0;
      if (++st.layer >= p.n_layers) return;
      st.src = p.packed + (size_t)st.layer * p.layer_bytes + sh.plan.off;
      st.it = sh.plan.att_rank;
      st.nb_valid = 0;
    }
    const uint32_t kb = sh.blk_kb[st.pos];
    int r = 0, h = 0;
    if (!kb) {
      // old K / V rows of this CTA's attention items, one block of p.kb keys at a time
      if (st.it >= n_items) { ++st.pos; continue; }
      r = st.it / p.n_heads;
      h = st.it - r * p.n_heads;
      if (!st.nb_valid) {
        st.nb = sh.ok[r] ? (sh.fill[r] + p.kb - 1) / p.kb : 0;
        st.blk = 0;
        st.nb_valid = 1;
      }
      if (st.blk >= st.nb) { st.it += e.grid; st.nb_valid = 0; continue; }
    }
    if (st.issued >= (uint32_t)sh.n_slots) wait_bar(&sh.empty[st.slot], st.par ^ 1u, &sh.abort, p.status);
    uint8_t* dst = e.ring + (size_t)st.slot * kSlotBytes;
    uint64_t* bar = &sh.full[st.slot];
    if (kb) {
      mbar_expect_tx(bar, kb * 1024u);
      bulk_load(dst, st.src, kb * 1024u, bar);
      st.src += kb * 1024u;
      ++st.pos;
    } else {
      const int nc = p.hd >> 6;
      const int row = ((st.layer * p.kv_rows + r) * p.n_heads + h) * p.s_max + st.blk * p.kb;
      mbar_expect_tx(bar, (uint32_t)(2 * nc * p.kb * 128));
#pragma unroll 1
      for (int j = 0; j < nc; ++j) {
        tma_load_2d(dst + j * p.kb * 128, e.tm_k, bar, j * 64, row);
        tma_load_2d(dst + (nc + j) * p.kb * 128, e.tm_v, bar, j * 64, row);
      }
      ++st.blk;
    }
    if (++st.slot == (uint32_t)sh.n_slots) { st.slot = 0; st.par ^= 1u; }
    ++st.issued;
  }
}

// ---- B operand from the activation ring ------------------------------------------------------------------
// Span s of the group belongs to warp s % 8.  For n-tile j the lane's 16 bytes feed the two k16 steps
// of the span: (x, y) the first, (z, w) the second (the packed weights use the same k permutation).
template <int NT>
__device__ __forceinline__ void mma_block(float (&acc)[NT][4], const uint8_t* blk, const uint8_t* act, int span_bytes,
                                          int nsp, int warp, int lane) {
  // kept as a loop on purpose: unrolled or register-staged variants of this body were slower (the
  // kernel is bound by instruction issue, not by this loop's latency)
  const uint8_t* ap = blk + (size_t)warp * 1024 + lane * 16;
  const uint8_t* bp = act + (size_t)warp * span_bytes + lane * 16;
#pragma unroll 1
  for (int s = warp; s < nsp; s += kCW) {
    const uint4 a0 = *reinterpret_cast<const uint4*>(ap);
    const uint4 a1 = *reinterpret_cast<const uint4*>(ap + 512);
#pragma unroll
    for (int j = 0; j < NT; ++j) {
      const uint4 b = *reinterpret_cast<const uint4*>(bp + j * 512);
      mma16816(acc[j], a0.x, a0.y, a0.z, a0.w, b.x, b.y);
      mma16816(acc[j], a1.x, a1.y, a1.z, a1.w, b.z, b.w);
    }
    ap += kCW * 1024;
    bp += (size_t)kCW * span_bytes;
  }
}

// 1 / rms of every token from the per-tile sums of squares, into shared memory.  Warp w takes tokens
// 4w .. 4w+3: every lane adds its tiles (lane, lane + 32, ..) in ascending order, then a butterfly
// over the lanes: a fixed order.  The loads are issued when a task starts and used after its
// reduction, so that their latency is hidden behind it.
struct RinvLoads {
  float4 v[3];
};
__device__ __forceinline__ void rinv_load(const StreamParams& p, const float* ss, int warp, int lane, RinvLoads& r) {
  const int n_dt = p.d >> 4, tok0 = warp * 4;
#pragma unroll
  for (int k = 0; k < 3; ++k) {
    const int i = lane + 32 * k;
    r.v[k] = (ss && tok0 < p.m && i < n_dt) ? __ldcg(reinterpret_cast<const float4*>(ss + (size_t)i * 32 + tok0))
                                           : make_float4(0.f, 0.f, 0.f, 0.f);
  }
}
__device__ __noinline__ void rinv_finish(const StreamParams& p, Shared& sh, const float* ss, int warp, int lane,
                                         const RinvLoads& r) {
  const int n_dt = p.d >> 4, tok0 = warp * 4;
  if (tok0 >= p.m) return;
  float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
  for (int k = 0; k < 3; ++k) { s.x += r.v[k].x; s.y += r.v[k].y; s.z += r.v[k].z; s.w += r.v[k].w; }
#pragma unroll 1
  for (int i = lane + 96; i < n_dt; i += 32) {   // wider models: the tiles beyond the prefetched ones
    const float4 v = __ldcg(reinterpret_cast<const float4*>(ss + (size_t)i * 32 + tok0));
    s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    s.x += __shfl_xor_sync(0xffffffffu, s.x, o);
    s.y += __shfl_xor_sync(0xffffffffu, s.y, o);
    s.z += __shfl_xor_sync(0xffffffffu, s.z, o);
    s.w += __shfl_xor_sync(0xffffffffu, s.w, o);
  }
  if (lane < 4 && tok0 + lane < p.m) {
    const float t = lane == 0 ? s.x : lane == 1 ? s.y : lane == 2 ? s.z : s.w;
    sh.rinv[tok0 + lane] = rsqrtf(fmaf(t, p.inv_d, p.eps));
  }
}

// Arrival on a stage counter: every thread's global writes happen before it.
__device__ __forceinline__ void signal_stage(unsigned* flag, int tid) {
  named_bar_sync(BAR_C, kCT);
  if (tid == 0) red_release_add(flag, 1u);
}

// ---- the reduction of one sub-panel (shared by the four projections) ---------------------------------------
// nt_sub <= kTP weight tiles over the whole reduction length: the activations come group by group
// through the two-slot activation ring (bulk copies issued by the sequencer), the weight blocks (one per
// tile and group) through the weight ring; accumulators stay in registers.  On return the partial
// sums of the eight warps lie in shared memory, [warp][tile][token][row (+1 pad)], at the start of
// the activation area (whose contents are dead by then), and all threads have passed a barrier.
template <int NT>
__device__ __noinline__ void gemm_main(const StreamParams& p, Shared& sh, const uint8_t* ring, uint8_t* act_area,
                                       RingPos& rp, RingPos& ap, int which, int nt_sub, const float* ss, int tid) {
  const int warp = tid >> 5, lane = tid & 31;
  const Geom ge = geom_of(p, which);
  const int sb = p.span_bytes;
  constexpr int NTOK = 8 * NT;
  constexpr int kAct = act_slot_bytes(NT);

  RinvLoads rl;
  rinv_load(p, ss, warp, lane, rl);

  float acc[kTP][NT][4];
#pragma unroll
  for (int t = 0; t < kTP; ++t)
#pragma unroll
    for (int j = 0; j < NT; ++j)
#pragma unroll
      for (int e = 0; e < 4; ++e) acc[t][j][e] = 0.f;

#pragma unroll 1
  for (int grp = 0; grp < ge.ngroups; ++grp) {
    const int nsp = group_spans(ge, grp);
    wait_bar_warp(&sh.act_full[ap.slot], ap.par, &sh.abort, p.status);
    if (tid == 0) VVS_CS_TRACE(0x52);
    const uint8_t* act = act_area + (size_t)ap.slot * kAct;
#pragma unroll
    for (int t = 0; t < kTP; ++t) {
      if (t < nt_sub) {
        wait_bar_warp(&sh.full[rp.slot], rp.par, &sh.abort, p.status);
        if (tid == 0) VVS_CS_TRACE(0x53);
        mma_block<NT>(acc[t], ring + (size_t)rp.slot * kSlotBytes, act, sb, nsp, warp, lane);
        __syncwarp();
        if (lane == 0) mbar_arrive(&sh.empty[rp.slot]);
        rp.next((uint32_t)sh.n_slots);
        if (tid == 0) VVS_CS_TRACE(0x54);
      }
    }
    // this group's activations are done with; its slot takes the group after the next one
    __syncwarp();
    if (lane == 0) mbar_arrive(&sh.act_empty[ap.slot]);
    ap.next(kActSlots);
  }
  if (ss) rinv_finish(p, sh, ss, warp, lane, rl);
  // every warp has passed its last read of the activation ring before the sums overwrite it
  if (tid == 0) VVS_CS_TRACE(0x20);
  named_bar_sync(BAR_C, kCT);
  if (tid == 0) VVS_CS_TRACE(0x21);
  {
    float* red = reinterpret_cast<float*>(act_area);
    const int g = lane >> 2, c = lane & 3;
#pragma unroll
    for (int t = 0; t < kTP; ++t) {
      if (t < nt_sub) {
        float* base = red + (size_t)((warp * kTP + t) * NTOK) * 17;
#pragma unroll
        for (int j = 0; j < NT; ++j) {
          const int tok = 8 * j + 2 * c;
          base[tok * 17 + g] = acc[t][j][0];
          base[(tok + 1) * 17 + g] = acc[t][j][1];
          base[tok * 17 + g + 8] = acc[t][j][2];
          base[(tok + 1) * 17 + g + 8] = acc[t][j][3];
        }
      }
    }
  }
  named_bar_sync(BAR_C, kCT);
}

// ---- one projection task of this CTA ---------------------------------------------------------------------
// `count` tiles (gate / up: pairs of tiles) starting at `first`, in sub-panels of at most kTP tiles.
// Epilogue on final sums: item = (unit, token, row), 16 consecutive threads = the 16 rows of one token.
//   QKV : scale by 1 / rms, rotate q and k pairs, q -> buffer, k / v -> the cache slot of the token
//   GU  : silu(gate / rms) * (up / rms) -> the down projection's operand
//   O, DOWN : residual add (the CTA's 16-column tiles of the residual stream live in its shared
//             memory for the whole kernel), operand of the next norm, sums of squares per tile
// One copy of the code serves the four projections (the kind is uniform over the CTA): the kernel's
// instruction footprint per layer has to stay inside the instruction cache.
template <int NT>
__device__ __noinline__ void gemm_task(const StreamParams& p, Shared& sh, const uint8_t* ring, uint8_t* act_area,
                                       const float2* rope_c, const int* slot_c, RingPos& rp, RingPos& ap, int kind,
                                       int layer, int first, int count, int tid) {
  const int m = p.m, d = p.d, sb = p.span_bytes;
  const int k_units = kind == G_GU ? kTP / 2 : kTP;
  const float* red = reinterpret_cast<const float*>(act_area);
  const bool last = kind == G_DOWN && layer + 1 >= p.n_layers;
  const bf16* gsc = nullptr;
  bf16* xn = nullptr;
  float* ssq = nullptr;
  if (kind == G_O) { gsc = p.norms[2 * layer + 1]; xn = p.xn2; ssq = p.ss2; }
  if (kind == G_DOWN && !last) { gsc = p.norms[2 * (layer + 1)]; xn = p.xn1; ssq = p.ss1; }

#pragma unroll 1
  for (int unit0 = first; unit0 < first + count; unit0 += k_units) {
    const int units = first + count - unit0 < k_units ? first + count - unit0 : k_units;
    const float* ss = unit0 > first ? nullptr : kind == G_QKV ? p.ss1 : kind == G_GU ? p.ss2 : nullptr;
    const int per_unit = m * 16, n_items = units * per_unit;
    // norm scales of the first two epilogue rounds (residual epilogues), requested before the reduction
    float g_pre[2] = {0.f, 0.f};
    if (gsc) {
#pragma unroll
      for (int k = 0; k < 2; ++k) {
        const int idx = tid + k * kCT;
        if (idx < n_items) {
          int u = 0, rem = idx;
          while (rem >= per_unit) { rem -= per_unit; ++u; }
          g_pre[k] = __bfloat162float(gsc[(unit0 + u) * 16 + (rem & 15)]);
        }
      }
    }
    gemm_main<NT>(p, sh, ring, act_area, rp, ap, kind == G_DOWN ? 1 : 0, kind == G_GU ? 2 * units : units, ss, tid);
    if (tid == 0) VVS_CS_TRACE(0x28 + kind);

#pragma unroll 1
    for (int base = 0; base < n_items; base += kCT) {
      const int idx = base + tid;
      const bool valid = idx < n_items;
      int u = 0, rem = valid ? idx : 0;
      while (rem >= per_unit) { rem -= per_unit; ++u; }
      const int tok = rem >> 4, row = rem & 15;
      const int n = (unit0 + u) * 16 + row;
      const int t0 = kind == G_GU ? 2 * u : u;
      float s0 = 0.f, s1 = 0.f;
      if (valid) {
        const float* rp0 = red + (size_t)(t0 * 8 * NT + tok) * 17 + row;
#pragma unroll
        for (int w = 0; w < kCW; ++w) s0 += rp0[(size_t)w * kTP * 8 * NT * 17];
        if (kind == G_GU) {
#pragma unroll
          for (int w = 0; w < kCW; ++w) s1 += rp0[(size_t)(w * kTP + 1) * 8 * NT * 17];
        }
      }
      if (kind == G_QKV) {
        const float v = s0 * sh.rinv[tok];
        const float other = __shfl_xor_sync(0xffffffffu, v, 1);
        if (valid && !(row & 1)) {
          const int sect = n >= 2 * d ? 2 : n >= d ? 1 : 0;
          const int nn = n - sect * d, h = nn / p.hd, e = nn - h * p.hd;
          float a = v, b = other;
          if (sect < 2) {
            const int uq = unit0 - first + u;
            float2 cs;
            if (uq < kRopeUnits) cs = rope_c[(uq * 32 + tok) * 8 + (row >> 1)];
            else cs = make_float2(__ldg(p.rope_cos + (size_t)tok * (p.hd >> 1) + (e >> 1)),
                                  __ldg(p.rope_sin + (size_t)tok * (p.hd >> 1) + (e >> 1)));
            a = v * cs.x - other * cs.y;
            b = other * cs.x + v * cs.y;
          }
          const uint32_t pk = pack2(a, b);
          if (sect == 0) {
            *reinterpret_cast<uint32_t*>(p.qbuf + (size_t)tok * d + nn) = pk;
          } else {
            const int slot = slot_c[tok];
            if (slot >= 0) {
              const int r = tok / p.t_len;
              bf16* cache = sect == 1 ? p.kv_k : p.kv_v;
              const size_t rowi = ((size_t)(layer * p.kv_rows + r) * p.n_heads + h) * p.s_max + slot;
              *reinterpret_cast<uint32_t*>(cache + rowi * p.hd + e) = pk;
            }
          }
        }
      } else if (kind == G_GU) {
        if (valid) {
          const float ri = sh.rinv[tok];
          const float gt = s0 * ri, up = s1 * ri;
          p.act[frag_off(tok, n, sb)] = __float2bfloat16(__fdividef(gt, 1.f + __expf(-gt)) * up);
        }
      } else {
        float* xs = sh.x_own + (size_t)((unit0 + u - sh.plan.t0[G_DOWN]) * 32 + tok) * 16 + row;
        const float xv = valid ? *xs + s0 : 0.f;
        float sq = xv * xv;
        sq += __shfl_xor_sync(0xffffffffu, sq, 8);
        sq += __shfl_xor_sync(0xffffffffu, sq, 4);
        sq += __shfl_xor_sync(0xffffffffu, sq, 2);
        sq += __shfl_xor_sync(0xffffffffu, sq, 1);
        if (valid) {
          *xs = xv;
          if (last) {
            p.x[(size_t)tok * d + n] = xv;
          } else {
            const float gv = base == 0 ? g_pre[0] : base == kCT ? g_pre[1] : __bfloat162float(gsc[n]);
            xn[frag_off(tok, n, sb)] = __float2bfloat16(xv * gv);
            if (row == 0) ssq[(size_t)(unit0 + u) * 32 + tok] = sq;
          }
        }
      }
    }
    // the sums are read and this sub-panel's global writes are issued: the sequencer may overwrite the
    // activation area and, after the last sub-panel, make the CTA's arrival on the stage counter
    fence_proxy_async();   // the sums were written with ordinary stores; the next writer is the copy engine
    named_bar_sync(BAR_C, kCT);
    if (tid == 0) mbar_arrive(&sh.epi_done);
  }
  if (tid == 0) VVS_CS_TRACE(0x30 + kind);
}

// ---- attention of one (sequence, head) item ---------------------------------------------------------------
template <int HD>
__device__ __noinline__ void attention_item(const StreamParams& p, Shared& sh, const uint8_t* ring, uint8_t* s_new,
                                            float* scratch, RingPos& rp, int layer, int r, int h, int tid) {
  constexpr int NC = HD / 64;
  constexpr int NJ = HD / 8;
  const int warp = tid >> 5, lane = tid & 31, g = lane >> 2, c = lane & 3;
  const int T = p.t_len, d = p.d, KB = p.kb;
  const int fill = sh.fill[r];
  const bool ok = sh.ok[r] != 0;
  const int n_mt = T > 16 ? 2 : 1;
  const int wpm = kCW / n_mt;                     // warps per m-tile
  const int mt = warp / wpm, kg = warp - mt * wpm;
  const int nslices = KB >> 4;
  const int nb = ok ? (fill + KB - 1) / KB : 0;
  const size_t row_base = ((size_t)(layer * p.kv_rows + r) * p.n_heads + h) * p.s_max;

  // the block's own K / V rows (written by the QKV stage of this layer) -> swizzled tiles
  {
    const int per_row = HD >> 3, n_chunks = T * per_row;
    for (int idx = tid; idx < 2 * n_chunks; idx += kCT) {
      const int which = idx >= n_chunks ? 1 : 0;
      const int rem = idx - which * n_chunks, jj = rem / per_row, ch = rem - jj * per_row;
      uint4 v = make_uint4(0u, 0u, 0u, 0u);
      if (ok) v = __ldcg(reinterpret_cast<const uint4*>((which ? p.kv_v : p.kv_k) + (row_base + fill + jj) * HD + ch * 8));
      *reinterpret_cast<uint4*>(s_new + which * (NC * 4096) + (ch >> 3) * 4096 + jj * 128 + (((ch & 7) ^ (jj & 7)) << 4)) = v;
    }
  }
  // query fragments of this warp's m-tile
  uint32_t qa[HD / 16][4];
  {
    const int t0 = mt * 16 + g, t1 = t0 + 8;
    const bf16* q0 = p.qbuf + (size_t)(r * T + t0) * d + h * HD + 2 * c;
    const bf16* q1 = p.qbuf + (size_t)(r * T + t1) * d + h * HD + 2 * c;
#pragma unroll
    for (int kk = 0; kk < HD / 16; ++kk) {
      qa[kk][0] = t0 < T ? __ldcg(reinterpret_cast<const unsigned*>(q0 + 16 * kk)) : 0u;
      qa[kk][1] = t1 < T ? __ldcg(reinterpret_cast<const unsigned*>(q1 + 16 * kk)) : 0u;
      qa[kk][2] = t0 < T ? __ldcg(reinterpret_cast<const unsigned*>(q0 + 16 * kk + 8)) : 0u;
      qa[kk][3] = t1 < T ? __ldcg(reinterpret_cast<const unsigned*>(q1 + 16 * kk + 8)) : 0u;
    }
  }
  uint32_t anc[2];
  {
    const int t0 = mt * 16 + g, t1 = t0 + 8;
    anc[0] = t0 < T ? __ldcg(p.anc_mask + r * T + t0) : 0u;
    anc[1] = t1 < T ? __ldcg(p.anc_mask + r * T + t1) : 0u;
  }
  if (tid == 0) VVS_CS_TRACE(0x70);
  AttState<HD> st;
  st.m[0] = st.m[1] = -CUDART_INF_F;
  st.l[0] = st.l[1] = 0.f;
#pragma unroll
  for (int j = 0; j < NJ; ++j)
#pragma unroll
    for (int e = 0; e < 4; ++e) st.o[j][e] = 0.f;

  // cached keys: blocks of KB keys through the ring, 16-key slices dealt round-robin to the warps
  // of each m-tile; then (blk == nb) the block's own keys from the tiles staged above: ancestors and
  // the row itself, taken by the last warp of each m-tile
  const int n_new = ok ? (T + 15) >> 4 : 0;
#pragma unroll 1
  for (int blk = 0; blk <= nb; ++blk) {
    const bool own = blk == nb;
    uint32_t k_base, v_base, stride;
    int ns;
    if (!own) {
      if (tid == 0) VVS_CS_TRACE(0x72);
      wait_bar_warp(&sh.full[rp.slot], rp.par, &sh.abort, p.status);
      if (tid == 0) VVS_CS_TRACE(0x73);
      k_base = smem_u32(ring + (size_t)rp.slot * kSlotBytes);
      v_base = k_base + NC * KB * 128;
      stride = (uint32_t)KB * 128u;
      ns = nslices;
    } else {
      if (tid == 0) VVS_CS_TRACE(0x71);
      named_bar_sync(BAR_C, kCT);
      k_base = smem_u32(s_new);
      v_base = k_base + NC * 4096;
      stride = 4096u;
      ns = n_new;
    }
#pragma unroll 1
    for (int sl = 0; sl < ns; ++sl) {
      uint32_t vis[2], vmem;
      if (!own) {
        if (((blk * nslices + sl) & (wpm - 1)) != kg) continue;
        const int left = fill - (blk * KB + sl * 16);
        if (left <= 0) continue;
        vmem = left >= 16 ? 0xffffu : ((1u << left) - 1u);
        vis[0] = vis[1] = vmem;
      } else {
        if (kg != wpm - 1 || sl > mt) continue;
        vis[0] = (anc[0] >> (16 * sl)) & 0xffffu;
        vis[1] = (anc[1] >> (16 * sl)) & 0xffffu;
        vmem = T - 16 * sl >= 16 ? 0xffffu : ((1u << (T - 16 * sl)) - 1u);   // rows >= T were never staged
      }
      att_slice<HD>(st, qa, k_base, v_base, stride, sl * 16, lane, p.sl2, vis, vmem);
    }
    if (!own) {
      __syncwarp();
      if (lane == 0) mbar_arrive(&sh.empty[rp.slot]);
      rp.next((uint32_t)sh.n_slots);
    }
  }
#pragma unroll
  for (int i = 0; i < 2; ++i) {
    st.l[i] += __shfl_xor_sync(0xffffffffu, st.l[i], 1);
    st.l[i] += __shfl_xor_sync(0xffffffffu, st.l[i], 2);
  }
  if (tid == 0) VVS_CS_TRACE(0x74);
  // merge the warps of each m-tile in a fixed tree
  constexpr int kRegs = NJ * 4 + 4;
#pragma unroll 1
  for (int stp = wpm >> 1; stp >= 1; stp >>= 1) {
    if (kg >= stp && kg < 2 * stp) {
      float* slot = scratch + (size_t)(mt * stp + kg - stp) * kRegs * 32;
#pragma unroll
      for (int j = 0; j < NJ; ++j)
#pragma unroll
        for (int e = 0; e < 4; ++e) slot[(j * 4 + e) * 32 + lane] = st.o[j][e];
      slot[(NJ * 4 + 0) * 32 + lane] = st.m[0];
      slot[(NJ * 4 + 1) * 32 + lane] = st.m[1];
      slot[(NJ * 4 + 2) * 32 + lane] = st.l[0];
      slot[(NJ * 4 + 3) * 32 + lane] = st.l[1];
    }
    named_bar_sync(BAR_C, kCT);
    if (kg < stp) {
      const float* slot = scratch + (size_t)(mt * stp + kg) * kRegs * 32;
#pragma unroll
      for (int i = 0; i < 2; ++i) {
        const float mo = slot[(NJ * 4 + i) * 32 + lane], lo = slot[(NJ * 4 + 2 + i) * 32 + lane];
        const float m_new = fmaxf(st.m[i], mo);
        const float m_safe = m_new == -CUDART_INF_F ? 0.f : m_new;
        const float a = ex2(st.m[i] - m_safe), b = ex2(mo - m_safe);
        st.m[i] = m_new;
        st.l[i] = st.l[i] * a + lo * b;
#pragma unroll
        for (int j = 0; j < NJ; ++j) {
          st.o[j][2 * i] = st.o[j][2 * i] * a + slot[(j * 4 + 2 * i) * 32 + lane] * b;
          st.o[j][2 * i + 1] = st.o[j][2 * i + 1] * a + slot[(j * 4 + 2 * i + 1) * 32 + lane] * b;
        }
      }
    }
    named_bar_sync(BAR_C, kCT);
  }
  if (kg == 0) {
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      const int t = mt * 16 + g + 8 * i;
      if (t < T) {
        const float inv = st.l[i] > 0.f ? 1.f / st.l[i] : 0.f;
#pragma unroll
        for (int j = 0; j < NJ; ++j)
          *reinterpret_cast<uint32_t*>(p.attn + frag_off(r * T + t, h * HD + 8 * j + 2 * c, p.span_bytes)) =
              pack2(st.o[j][2 * i] * inv, st.o[j][2 * i + 1] * inv);
      }
    }
  }
}

// ---- the sequencer (one thread) ---------------------------------------------------------------------------
// Follows the CTA's program stage by stage: waits for the producers of the stage before, starts the
// bulk copies of the stage's activations (two k groups ahead of the computing warps), releases the
// computing warps, and when they report their epilogue done makes the CTA's arrival on the stage
// counter (their writes happen before the barrier they arrive on; this thread's fence then orders
// them before the arrival for every other CTA).
template <int NT>
__device__ __noinline__ void sequencer_loop(const StreamParams& p, Shared& sh, uint8_t* act_area, int grid) {
  const ChainCtaPlan& pl = sh.plan;
  const int L = p.n_layers, sb = p.span_bytes;
  const bool has_att = pl.att_rank < p.n_rows * p.n_heads;
  unsigned* abort_word = p.flags + L * N_ST + 1;
  constexpr int kAct = act_slot_bytes(NT);
  uint32_t a_slot = 0, a_par = 0, a_issued = 0, epi_par = 0;
#pragma unroll 1
  for (int l = 0; l < L; ++l) {
    unsigned* fl = p.flags + l * N_ST;
#pragma unroll 1
    for (int st = 0; st < N_ST; ++st) {
      const int kind = st == ST_QKV ? G_QKV : st == ST_O ? G_O : st == ST_GU ? G_GU : G_DOWN;
      if (st == ST_ATT ? !has_att : pl.n[kind] == 0) continue;
      // the stage before: the embedding stage for the first projection of the first layer, the
      // previous layer's down projection for the first projection of the others
      const unsigned* prev = st > 0 ? fl + st - 1 : l > 0 ? fl - N_ST + ST_DOWN : p.flags + L * N_ST;
      const int n_prev = st > 0 ? p.n_prod[st - 1] : l > 0 ? p.n_prod[ST_DOWN] : p.n_prod[N_ST];
      VVS_CS_TRACE_SEQ(0x68);
      wait_flag(prev, (unsigned)n_prev, &sh.abort, abort_word, p.status);
      VVS_CS_TRACE_SEQ(0x60 + st);
      if (st == ST_ATT) {
        mbar_arrive(&sh.go);
        wait_bar(&sh.epi_done, epi_par, &sh.abort, p.status);
        epi_par ^= 1u;
      } else {
        const Geom ge = geom_of(p, kind == G_DOWN ? 1 : 0);
        const uint8_t* src0 = reinterpret_cast<const uint8_t*>(kind == G_QKV ? p.xn1 : kind == G_O ? p.attn
                                                              : kind == G_GU ? p.xn2 : p.act);
        const int k_units = kind == G_GU ? kTP / 2 : kTP;
        const uint32_t full_bytes = (uint32_t)(ge.gsz * sb), last_bytes = (uint32_t)(group_spans(ge, ge.ngroups - 1) * sb);
        bool first = true;
#pragma unroll 1
        for (int u0 = 0; u0 < pl.n[kind]; u0 += k_units) {
          const uint8_t* src = src0;
#pragma unroll 1
          for (int grp = 0; grp < ge.ngroups; ++grp) {
            if (a_issued >= (uint32_t)kActSlots) wait_bar(&sh.act_empty[a_slot], a_par ^ 1u, &sh.abort, p.status);
            const uint32_t bytes = grp + 1 == ge.ngroups ? last_bytes : full_bytes;
            mbar_expect_tx(&sh.act_full[a_slot], bytes);
            bulk_load(act_area + (a_slot ? kAct : 0), src, bytes, &sh.act_full[a_slot]);
            if (first) { mbar_arrive(&sh.go); first = false; }
            src += full_bytes;
            a_slot ^= 1u;
            a_par ^= a_slot ^ 1u;   // flips when the slot index wraps to 0
            ++a_issued;
          }
          VVS_CS_TRACE_SEQ(0x69);
          wait_bar(&sh.epi_done, epi_par, &sh.abort, p.status);
          epi_par ^= 1u;
          VVS_CS_TRACE_SEQ(0x6a);
        }
      }
      if (sh.abort) return;
      red_release_add(fl + st, 1u);
      VVS_CS_TRACE_SEQ(0x78 + st);
    }
  }
  (void)grid;
}

// ---- the kernel ---------------------------------------------------------------------------------------------
template <int NT>
__global__ void __launch_bounds__(kThreads, 1)
chain_stream_kernel(const __grid_constant__ StreamParams p, const __grid_constant__ CUtensorMap tm_k,
                    const __grid_constant__ CUtensorMap tm_v) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(16) Shared sh;
  VVS_CS_TRACE_DECL

  const int tid = threadIdx.x, warp = tid >> 5;
  const int G = (int)gridDim.x, L = p.n_layers, T = p.t_len, H = p.n_heads;
  constexpr int kSlots = ring_slots(NT);
  uint8_t* ring = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* act_area = ring + (size_t)kSlots * kSlotBytes;     // activation ring; attention: own rows + merge
  uint8_t* s_new = act_area;
  float* scratch = reinterpret_cast<float*>(act_area + kNewBytes);
  float2* rope_c = reinterpret_cast<float2*>(act_area + (size_t)kActSlots * act_slot_bytes(NT));   // [unit][token][pair]
  int* slot_c = reinterpret_cast<int*>(rope_c + kRopeUnits * 32 * 8);                              // [token]
  static_assert(kNewBytes + kMergeBytes <= kActSlots * act_slot_bytes(NT), "attention scratch fits the activation ring");
  static_assert(kCW * kTP * 8 * NT * 17 * 4 <= kActSlots * act_slot_bytes(NT), "cross-warp sums fit the activation ring");

  if (tid == 0) {
    for (int i = 0; i < kSlots; ++i) { mbar_init(&sh.full[i], 1); mbar_init(&sh.empty[i], kCW); }
    for (int i = 0; i < kActSlots; ++i) { mbar_init(&sh.act_full[i], 1); mbar_init(&sh.act_empty[i], kCW); }
    mbar_init(&sh.go, 1);
    mbar_init(&sh.epi_done, 1);
    sh.abort = 0;
    sh.n_slots = kSlots;
    fence_barrier_init();
    tma_prefetch_desc(&tm_k);
    tma_prefetch_desc(&tm_v);
    sh.plan = p.plan[blockIdx.x];
  }
  if (tid < kMaxSeq) {
    int fill = 0, ok = 0;
    if (tid < p.n_rows) {
      fill = p.cache_len[tid];
      ok = fill >= 0 && fill + T <= p.s_max;
    }
    sh.fill[tid] = fill;
    sh.ok[tid] = ok;
  }
  __syncthreads();
  const ChainCtaPlan& pl = sh.plan;
  const int n_items = p.n_rows * H;

  if (warp >= kCW) {
    // ---- the two service threads; the other lanes of their warp group leave at once ----
    if (tid == kCT) {
      ProdEnv env{&p, &sh, ring, &tm_k, &tm_v, G};
      prod_init(env);
      producer_loop(env);
    } else if (tid == kCT + 32) {
      sequencer_loop<NT>(p, sh, act_area, G);
    }
    if ((tid == kCT || tid == kCT + 32) && sh.abort) {
      // copies may still be in flight with nobody waiting for them: let them land before the CTA
      // gives its shared memory back
      for (int i = 0; i < 128; ++i) __nanosleep(2000);
    }
    return;
  }

  // ================================ computing warps ==================================================
  RingPos rp, ap;
  uint32_t go_par = 0;
  // rotation factors of this CTA's q / k tiles and the cache slot of every token: the same in every layer
  {
    const int nq = pl.n[G_QKV] < kRopeUnits ? pl.n[G_QKV] : kRopeUnits;
    for (int i = tid; i < nq * 32 * 8; i += kCT) {
      const int uq = i >> 8, tok = (i >> 3) & 31, pr = i & 7;
      const int n0 = (pl.t0[G_QKV] + uq) * 16;
      const int sect = n0 >= 2 * p.d ? 2 : n0 >= p.d ? 1 : 0;
      float2 cs = make_float2(1.f, 0.f);
      if (sect < 2 && tok < p.m) {
        const int e = (n0 - sect * p.d) % p.hd + 2 * pr;
        cs = make_float2(p.rope_cos[(size_t)tok * (p.hd >> 1) + (e >> 1)], p.rope_sin[(size_t)tok * (p.hd >> 1) + (e >> 1)]);
      }
      rope_c[i] = cs;
    }
    if (tid < 32) slot_c[tid] = tid < p.m ? p.slot_pos[tid] : -1;
  }
  named_bar_sync(BAR_C, kCT);
  // embedding stage, by the owners of the down-projection tiles: x, first norm operand, sums of squares
  if (pl.n[G_DOWN]) {
    const int per_tile = p.m * 16, total = pl.n[G_DOWN] * per_tile;
    const bf16* gs = p.norms[0];
    for (int base = 0; base < total; base += kCT) {
      const int idx = base + tid;
      const bool valid = idx < total;
      const int t = valid ? idx / per_tile : 0, rem = valid ? idx - t * per_tile : 0, tok = rem >> 4, row = rem & 15;
      const int n = (pl.t0[G_DOWN] + t) * 16 + row;
      float xv = 0.f;
      if (valid) {
        const int r = tok / T, tt = tok - r * T, b = r % p.n_images;
        const int token = p.block[b * T + tt];
        if (token >= 0 && token < p.tok_rows) xv = __bfloat162float(p.tok_emb[(size_t)token * p.d + n]);
        else if (n == 0) atomicOr(p.status, VVS_DEV_BAD_TOKEN);
      }
      float sq = xv * xv;
      sq += __shfl_xor_sync(0xffffffffu, sq, 8);
      sq += __shfl_xor_sync(0xffffffffu, sq, 4);
      sq += __shfl_xor_sync(0xffffffffu, sq, 2);
      sq += __shfl_xor_sync(0xffffffffu, sq, 1);
      if (valid) {
        sh.x_own[(size_t)(t * 32 + tok) * 16 + row] = xv;
        p.xn1[frag_off(tok, n, p.span_bytes)] = __float2bfloat16(xv * __bfloat162float(gs[n]));
        if (row == 0) p.ss1[(size_t)(pl.t0[G_DOWN] + t) * 32 + tok] = sq;
      }
    }
    signal_stage(p.flags + L * N_ST, tid);
  }
  const bool has_att = pl.att_rank < n_items;
#pragma unroll 1
  for (int l = 0; l < L; ++l) {
#pragma unroll 1
    for (int st = 0; st < N_ST; ++st) {
      const int kind = st == ST_QKV ? G_QKV : st == ST_O ? G_O : st == ST_GU ? G_GU : G_DOWN;
      if (st == ST_ATT ? !has_att : pl.n[kind] == 0) continue;
      wait_bar_warp(&sh.go, go_par, &sh.abort, p.status);
      go_par ^= 1u;
      if (tid == 0) VVS_CS_TRACE(0x10 + st);
      if (st != ST_ATT) {
        gemm_task<NT>(p, sh, ring, act_area, rope_c, slot_c, rp, ap, kind, l, pl.t0[kind], pl.n[kind], tid);
        continue;
      }
      // rows of the own-keys tiles that no item writes stay zero (the sums of the last projection
      // may have been here)
      for (int i = tid; i < kNewBytes / 16; i += kCT) reinterpret_cast<uint4*>(s_new)[i] = make_uint4(0u, 0u, 0u, 0u);
      named_bar_sync(BAR_C, kCT);
#pragma unroll 1
      for (int it = pl.att_rank; it < n_items; it += G) {
        const int r = it / H, h = it - r * H;
        if (p.hd == 64) attention_item<64>(p, sh, ring, s_new, scratch, rp, l, r, h, tid);
        else attention_item<128>(p, sh, ring, s_new, scratch, rp, l, r, h, tid);
      }
      if (tid == 0) VVS_CS_TRACE(0x31);
      fence_proxy_async();
      named_bar_sync(BAR_C, kCT);
      if (tid == 0) mbar_arrive(&sh.epi_done);
    }
  }
  VVS_CS_TRACE_END;
}

// ---- one-time re-packing of a layer's weights -----------------------------------------------------------
struct PackLayer {
  const bf16* w[5];   // qkv, o, gate, up, down
};

__global__ void __launch_bounds__(256)
chain_pack_kernel(PackLayer wl, const ChainCtaPlan* plans, uint8_t* out_layer, int d, int ff, int spans_d, int gsz_d,
                  int ngroups_d, int spans_f, int gsz_f, int ngroups_f) {
  const ChainCtaPlan pl = plans[blockIdx.x];
  uint8_t* out = out_layer + pl.off;
  auto pack_task = [&](int kind, int first, int count) {
    const bool down = kind == G_DOWN, pairs = kind == G_GU;
    const int spans = down ? spans_f : spans_d, gsz = down ? gsz_f : gsz_d, ngroups = down ? ngroups_f : ngroups_d;
    const int K = down ? ff : d;
    const int per_sub = pairs ? kTP / 2 : kTP;
    const int nsub = (count + per_sub - 1) / per_sub;
    for (int sub = 0; sub < nsub; ++sub) {
      const int nt_sub = (count - sub * per_sub < per_sub ? count - sub * per_sub : per_sub) * (pairs ? 2 : 1);
      for (int grp = 0; grp < ngroups; ++grp) {
        const int left = spans - grp * gsz, nsp = left < gsz ? left : gsz;
        for (int t = 0; t < nt_sub; ++t) {
          const bf16* W;
          int row0;
          if (kind == G_QKV) { W = wl.w[0]; row0 = (first + sub * kTP + t) * 16; }
          else if (kind == G_O) { W = wl.w[1]; row0 = (first + sub * kTP + t) * 16; }
          else if (kind == G_GU) { W = wl.w[2 + (t & 1)]; row0 = (first + sub * per_sub + (t >> 1)) * 16; }
          else { W = wl.w[4]; row0 = (first + sub * kTP + t) * 16; }
          for (int u = threadIdx.x; u < nsp * 64; u += blockDim.x) {
            const int s = u >> 6, step = (u >> 5) & 1, lane = u & 31, g = lane >> 2, c = lane & 3;
            const size_t k0 = (size_t)(grp * gsz + s) * 32 + 8 * c + 4 * step;
            const bf16* ra = W + (size_t)(row0 + g) * K + k0;
            const bf16* rb = W + (size_t)(row0 + g + 8) * K + k0;
            uint4 v;
            v.x = *reinterpret_cast<const uint32_t*>(ra);
            v.y = *reinterpret_cast<const uint32_t*>(rb);
            v.z = *reinterpret_cast<const uint32_t*>(ra + 2);
            v.w = *reinterpret_cast<const uint32_t*>(rb + 2);
            *reinterpret_cast<uint4*>(out + (size_t)(2 * s + step) * 512 + lane * 16) = v;
          }
          out += (size_t)nsp * 1024;
        }
      }
    }
  };
  if (pl.n[G_QKV]) pack_task(G_QKV, pl.t0[G_QKV], pl.n[G_QKV]);
  if (pl.n[G_O]) pack_task(G_O, pl.t0[G_O], pl.n[G_O]);
  if (pl.n[G_GU]) pack_task(G_GU, pl.t0[G_GU], pl.n[G_GU]);
  if (pl.n[G_DOWN]) pack_task(G_DOWN, pl.t0[G_DOWN], pl.n[G_DOWN]);
}

// Self-test of the bounded waits: one thread waits, with a limit of a few hundred polls, on barriers
// on which nobody ever arrives.  Both helpers must give up, record VVS_DEV_TIMEOUT and return.
__global__ void bounded_wait_selftest_kernel(int32_t* status, int32_t* report) {
  __shared__ __align__(8) uint64_t bar[2];
  __shared__ volatile int s_abort;
  if (threadIdx.x == 0) {
    mbar_init(&bar[0], 1);
    mbar_init(&bar[1], 1);
    s_abort = 0;
    fence_barrier_init();
    const bool got0 = mbar_wait_limited(&bar[0], 0u, 256u);   // the helper of the tcgen05 kernels
    if (!got0) atomicOr(status, VVS_DEV_TIMEOUT);
    wait_slow(&bar[1], 0u, &s_abort, status, 64u);            // the helper of the streaming chain kernel
    report[0] = got0 ? 1 : 0;
    report[1] = s_abort;
  }
}

void geometry(int K, int& spans, int& gsz, int& ngroups) {
  spans = K / 32;
  ngroups = (spans + kGroupSpans - 1) / kGroupSpans;
  gsz = (spans + ngroups - 1) / ngroups;
}


}  // namespace

bool chain_stream_applicable(const vvs_model_desc& md, int n_rows, int t_len) {
  if (md.dtype != VVS_DTYPE_BF16 || md.n_layers < 1 || md.n_layers > kMaxLayers) return false;
  if (n_rows * t_len > 32 || n_rows > kMaxSeq || t_len > 32) return false;
  if (md.d_model % 32 != 0 || md.d_ff % 32 != 0) return false;
  if (md.head_dim != 64 && md.head_dim != 128) return false;
  return true;
}

// Splits the tiles of every projection over the CTAs (contiguous ranges, the least loaded CTAs take
// the extra tiles; largest tiles first) and lays the per-CTA streams out back to back.
bool chain_stream_plan(const vvs_model_desc& md, int grid, ChainStreamPlan& out) {
  const int d = md.d_model, ff = md.d_ff;
  if (grid < 1 || (d / 16 + grid - 1) / grid > kMaxOwn) return false;   // residual tiles per CTA kept in shared memory
  out.grid = grid;
  out.cta.assign((size_t)grid, ChainCtaPlan{});
  std::vector<unsigned long long> load((size_t)grid, 0ull);
  const int counts[4] = {3 * d / 16, d / 16, ff / 16, d / 16};
  const unsigned long long bytes[4] = {16ull * d * 2, 16ull * d * 2, 2 * 16ull * d * 2, 16ull * ff * 2};
  // the output and the down projection share their split: the CTA that owns 16 columns of the
  // residual stream adds both results into them
  const int order[3] = {G_DOWN, G_GU, G_QKV};
  for (int oi = 0; oi < 3; ++oi) {
    const int k = order[oi];
    std::vector<int> idx((size_t)grid);
    std::iota(idx.begin(), idx.end(), 0);
    std::stable_sort(idx.begin(), idx.end(), [&](int a, int b) { return load[a] < load[b]; });
    const int base = counts[k] / grid, extra = counts[k] % grid;
    int next = 0, prod = 0;
    for (int i = 0; i < grid; ++i) {
      const int c = idx[i], n = base + (i < extra ? 1 : 0);
      out.cta[c].t0[k] = next;
      out.cta[c].n[k] = n;
      next += n;
      load[c] += bytes[k] * n;
      if (k == G_DOWN) {
        out.cta[c].t0[G_O] = out.cta[c].t0[G_DOWN];
        out.cta[c].n[G_O] = n;
        load[c] += bytes[G_O] * n;
      }
      if (n) ++prod;
    }
    out.n_prod[k == G_QKV ? ST_QKV : k == G_GU ? ST_GU : ST_DOWN] = prod;
    if (k == G_DOWN) out.n_prod[ST_O] = prod;
  }
  std::vector<int> idx((size_t)grid);
  std::iota(idx.begin(), idx.end(), 0);
  std::stable_sort(idx.begin(), idx.end(), [&](int a, int b) { return load[a] < load[b]; });
  for (int i = 0; i < grid; ++i) out.cta[idx[i]].att_rank = i;
  unsigned long long off = 0;
  for (int c = 0; c < grid; ++c) {
    out.cta[c].off = off;
    off += load[c];
  }
  out.layer_bytes = off;
  return true;
}

size_t chain_stream_packed_bytes(const vvs_model_desc& md, const ChainStreamPlan& plan) {
  return (size_t)plan.layer_bytes * md.n_layers;
}

int chain_stream_pack(const vvs_model_desc& md, const ChainStreamPlan& plan, const ChainCtaPlan* d_plan,
                      const Layer* layers, void* packed, cudaStream_t s) {
  int sd, gd, nd, sf, gf, nf;
  geometry(md.d_model, sd, gd, nd);
  geometry(md.d_ff, sf, gf, nf);
  for (int l = 0; l < md.n_layers; ++l) {
    PackLayer wl;
    wl.w[0] = static_cast<const bf16*>(layers[l].w_qkv);
    wl.w[1] = static_cast<const bf16*>(layers[l].w_o);
    wl.w[2] = static_cast<const bf16*>(layers[l].w_gate);
    wl.w[3] = static_cast<const bf16*>(layers[l].w_up);
    wl.w[4] = static_cast<const bf16*>(layers[l].w_down);
    chain_pack_kernel<<<plan.grid, 256, 0, s>>>(wl, d_plan, static_cast<uint8_t*>(packed) + (size_t)l * plan.layer_bytes,
                                                md.d_model, md.d_ff, sd, gd, nd, sf, gf, nf);
  }
  return cudaGetLastError() == cudaSuccess ? VVS_OK : VVS_ERR_CUDA;
}

// keys per attention block: K and V of a block share one 20 KB ring slot (8 KB each)
void launch_bounded_wait_selftest(int32_t* status, int32_t* report, cudaStream_t s) {
  bounded_wait_selftest_kernel<<<1, 32, 0, s>>>(status, report);
}

int chain_stream_kb(const vvs_model_desc& md) { return md.head_dim == 64 ? 64 : 32; }
size_t chain_stream_flag_words(const vvs_model_desc& md) { return (size_t)md.n_layers * N_ST + 2; }

int chain_stream_configure() {
  if (ensure_dynamic_smem(reinterpret_cast<const void*>(chain_stream_kernel<3>), (int)smem_bytes(3)) != cudaSuccess ||
      ensure_dynamic_smem(reinterpret_cast<const void*>(chain_stream_kernel<4>), (int)smem_bytes(4)) != cudaSuccess)
    return VVS_ERR_CUDA;
  return VVS_OK;
}

int launch_chain_stream(const ChainStreamArgs& a, cudaStream_t s) {
  StreamParams p{};
  const vvs_model_desc& md = *a.md;
  p.n_layers = md.n_layers; p.d = md.d_model; p.n_heads = md.n_heads; p.hd = md.head_dim; p.ff = md.d_ff;
  p.s_max = md.s_max; p.kv_rows = a.kv_rows;
  p.m = a.n_rows * a.t_len; p.t_len = a.t_len; p.n_rows = a.n_rows; p.n_images = a.n_images; p.tok_rows = md.tok_rows;
  geometry(md.d_model, p.spans[0], p.gsz[0], p.ngroups[0]);
  geometry(md.d_ff, p.spans[1], p.gsz[1], p.ngroups[1]);
  const ChainStreamPlan& plan = *a.plan;
  for (int i = 0; i < N_ST; ++i) p.n_prod[i] = plan.n_prod[i];
  const int n_items = a.n_rows * md.n_heads;
  p.n_prod[ST_ATT] = n_items < plan.grid ? n_items : plan.grid;
  p.n_prod[N_ST] = plan.n_prod[ST_DOWN];
  p.kb = chain_stream_kb(md);
  p.eps = md.rms_eps;
  p.inv_d = 1.0f / (float)md.d_model;
  p.sl2 = 1.4426950408889634f / sqrtf((float)md.head_dim);
  p.layer_bytes = plan.layer_bytes;
  p.packed = static_cast<const uint8_t*>(a.packed);
  p.plan = a.d_plan;
  p.tok_emb = a.tok_emb; p.block = a.block;
  p.x = a.x; p.xn1 = a.xn1; p.xn2 = a.xn2; p.qbuf = a.qbuf; p.attn = a.attn; p.act = a.act;
  p.ss1 = a.ss1; p.ss2 = a.ss2;
  {
    const int nt_eff = (p.m + 7) / 8, vl = p.m - 8 * (nt_eff - 1);
    p.span_bytes = (nt_eff - 1) * 512 + vl * 64;
  }
  p.cache_len = a.cache_len; p.slot_pos = a.slot_pos; p.anc_mask = a.anc_mask;
  p.kv_k = a.kv_k; p.kv_v = a.kv_v; p.rope_cos = a.rope_cos; p.rope_sin = a.rope_sin;
  p.flags = a.flags; p.status = a.status;
  for (int i = 0; i < 2 * md.n_layers; ++i) p.norms[i] = a.norms_host[i];
  CUtensorMap tk = *a.tm_k, tv = *a.tm_v;
  void* args[] = {&p, &tk, &tv};
  const void* fn = p.m > 24 ? reinterpret_cast<const void*>(chain_stream_kernel<4>)
                            : reinterpret_cast<const void*>(chain_stream_kernel<3>);
  // cooperative launch: every CTA is resident, which the stage counters rely on
  cudaError_t e = cudaLaunchCooperativeKernel(fn, dim3(plan.grid), dim3(kThreads), args, smem_bytes(p.m > 24 ? 4 : 3), s);
  if (e != cudaSuccess && std::getenv("VVS_DEBUG_VERBOSE"))
    std::fprintf(stderr, "chain_stream launch: %s\n", cudaGetErrorString(e));
  return e == cudaSuccess ? VVS_OK : VVS_ERR_CUDA;
}

}  // namespace vvs
