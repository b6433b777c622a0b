// Block-vs-cache attention of the per-projection path (calls of more than 32 block tokens), with the
// rotation of q / k and the cache append of the block's own K / V rows folded in (Alg. 2 line 9: the
// target forward over the block; Sec. 4.1: the call restores the block's KV entries).
//
// One CTA per (sequence, head).  It streams the head's cached rows [0, fill) -- one contiguous run of
// fill * head_dim bf16 -- through a ring of 64-key blocks in shared memory (16-byte asynchronous
// copies, three blocks in flight), and the request for the first blocks goes out BEFORE
// griddepcontrol.wait, i.e. while the QKV projection that precedes this kernel is still running.
// After the wait the CTA reads the fp32 split-K sums of its head's q, k, v for the block rows,
// rotates q and k with the step's rotation table, rounds to bf16, writes k and v to their cache
// slots and keeps q, k, v of the block in shared memory (the block's own keys are then attended
// from there under the ancestor mask), and clears the sums it read for the next layer.
// The four warps deal the 16-key slices among themselves (two m-tiles of 16 query rows when the
// block has more than 16 rows), keep running maximum / normaliser / output in registers and merge
// once at the end in a fixed order, so the result does not depend on timing.
//
// Roofline: the K and V rows of every (sequence, head) are read exactly once -- 2 * head_dim * 2
// bytes per cached position -- against a few hundred flops per position: HBM-bound, and at 9 query
// rows per sequence far from the tensor roofline whichever MMA is used.
#include "att_mma.cuh"
#include "tc_common.cuh"
#include "vvs_internal.cuh"

namespace vvs {

using namespace attmma;

namespace {

using bf16 = __nv_bfloat16;

// Measured on the 32-sequence LlamaGen-XL workload: 4 warps x 64-key blocks x 3 ring slots (three CTAs
// per SM) and 8 warps or 2 slots are within 2 % of one another; 32-key blocks are 5 % slower.
constexpr int kWarps = 4;
constexpr int kThreads = 32 * kWarps;
constexpr int kStages = 3;
constexpr int kMaxT = 32;      // block rows per sequence

template <int HD>
struct Layout {
  static constexpr int kKB = HD == 64 ? 64 : 32;       // cached keys per staged block (16 KB of K + V either way)
  static constexpr int NC = HD / 64;                   // 128-byte column groups per K / V row
  static constexpr int kTile = kKB * 128;              // one column group of a staged block
  static constexpr int kStage = 2 * NC * kTile;        // K then V
  static constexpr int kNewTile = kMaxT * 128;
  static constexpr int kOffNew = kStages * kStage;     // block's own K tiles, then V tiles
  static constexpr int kOffQ = kOffNew + 2 * NC * kNewTile;
  static constexpr int kRegs = (HD / 8) * 4 + 4;
  static constexpr int kOffScratch = 0;                // the merge buffers reuse the ring once it has drained
  static constexpr int kBytes = kOffQ + kMaxT * HD * 2;
  static_assert((kWarps / 2 + 2) * kRegs * 32 * 4 <= kStages * kStage, "merge buffers must fit in the ring");
};

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ float ld_cluster_f32(uint32_t local_addr, uint32_t rank) {
  uint32_t remote;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local_addr), "r"(rank));
  float v;
  asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(remote) : "memory");
  return v;
}

template <int HD>
__global__ void __launch_bounds__(kThreads) attention_rows_kernel(AttentionRowsArgs a) {
  using L = Layout<HD>;
  constexpr int NC = L::NC, NJ = HD / 8, HALF = HD / 2, kKB = L::kKB;
  extern __shared__ __align__(1024) uint8_t smem[];
  const int h = blockIdx.x, r = a.seq_order[blockIdx.y];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, c = lane & 3;
  const int T = a.t_len, d = a.d;
  const int fill = a.cache_len[r];
  const bool ok = fill >= 0 && fill + T <= a.s_max;
  const size_t row_base = ((size_t)(a.layer * a.kv_rows + r) * a.n_heads + h) * a.s_max;
  // Few (sequence, head) items: the key blocks of an item are dealt to the S CTAs of a cluster (rank =
  // blockIdx.z takes blocks rank, rank + S, ...; the last rank also the block's own keys); rank 0 merges
  // the partial results in rank order through distributed shared memory and writes the output.
  const int S = (int)gridDim.z, rank = (int)blockIdx.z;
  const int nb_all = ok ? (fill + kKB - 1) / kKB : 0;
  const int nb = nb_all > rank ? (nb_all - rank + S - 1) / S : 0;      // this CTA's blocks
  const bool own_keys = rank == S - 1;
  const uint32_t s_base = tc::smem_u32(smem);

  // 16-byte chunks of block `blk` (keys blk*64 .. ), K and V, into its ring slot; rows at or beyond
  // `fill` are not requested (the slices mask them)
  auto request = [&](int j) {
    if (j < nb) {
      const int blk = rank + j * S;
      const uint32_t stage = s_base + (uint32_t)(j % kStages) * L::kStage;
      const int rows = min(kKB, fill - blk * kKB);
      const int per_row = HD / 8, n = rows * per_row;
      const bf16* k_src = a.kv_k + (row_base + (size_t)blk * kKB) * HD;
      const bf16* v_src = a.kv_v + (row_base + (size_t)blk * kKB) * HD;
      for (int idx = tid; idx < 2 * n; idx += kThreads) {
        const int which = idx >= n ? 1 : 0;
        const int rem = idx - which * n, key = rem / per_row, ch = rem - key * per_row;
        const uint32_t dst = stage + (uint32_t)(which * NC + (ch >> 3)) * L::kTile + key * 128 +
                             (((ch & 7) ^ (key & 7)) << 4);
        cp_async16(dst, (which ? v_src : k_src) + (size_t)key * HD + ch * 8);
      }
    }
    cp_async_commit();
  };
  for (int s = 0; s < kStages - 1; ++s) request(s);
  tc::pdl_launch_dependents();      // the projection after this kernel may start fetching its weights

  // ---- the block's own rows: rotate, round, append, stage -------------------------------------------
  // (the rotation table is an input of the whole step: its loads go out before the wait)
  constexpr int kPro = (kMaxT * HALF + kThreads - 1) / kThreads;
  uint8_t* s_new = smem + L::kOffNew;
  bf16* s_q = reinterpret_cast<bf16*>(smem + L::kOffQ);
  float cs[kPro], sn[kPro];
#pragma unroll
  for (int u = 0; u < kPro; ++u) {
    const int idx = tid + u * kThreads;
    if (idx < T * HALF) {
      const int t = idx / HALF, i = idx - t * HALF;
      cs[u] = a.rope_cos[(size_t)(r * T + t) * HALF + i];
      sn[u] = a.rope_sin[(size_t)(r * T + t) * HALF + i];
    }
  }
  tc::pdl_wait();
  float2 q2[kPro], k2[kPro], v2[kPro];
#pragma unroll
  for (int u = 0; u < kPro; ++u) {
    const int idx = tid + u * kThreads;
    if (idx < T * HALF) {
      const int t = idx / HALF, i = idx - t * HALF;
      const float* src = a.qkv + (size_t)(r * T + t) * 3 * d + h * HD + 2 * i;
      q2[u] = __ldcg(reinterpret_cast<const float2*>(src));
      k2[u] = __ldcg(reinterpret_cast<const float2*>(src + d));
      v2[u] = __ldcg(reinterpret_cast<const float2*>(src + 2 * d));
    }
  }
#pragma unroll
  for (int u = 0; u < kPro; ++u) {
    const int idx = tid + u * kThreads;
    if (idx < T * HALF) {
      const int t = idx / HALF, i = idx - t * HALF;
      float* src = a.qkv + (size_t)(r * T + t) * 3 * d + h * HD + 2 * i;
      if (S == 1) {                                          // (a cluster clears after every rank has read)
        const float2 z = make_float2(0.f, 0.f);              // split-K sums are added into this buffer:
        *reinterpret_cast<float2*>(src) = z;                 // leave it zero for the next layer
        *reinterpret_cast<float2*>(src + d) = z;
        *reinterpret_cast<float2*>(src + 2 * d) = z;
      }
      const uint32_t qp = pack2(q2[u].x * cs[u] - q2[u].y * sn[u], q2[u].x * sn[u] + q2[u].y * cs[u]);
      const uint32_t kp = pack2(k2[u].x * cs[u] - k2[u].y * sn[u], k2[u].x * sn[u] + k2[u].y * cs[u]);
      const uint32_t vp = pack2(v2[u].x, v2[u].y);
      *reinterpret_cast<uint32_t*>(s_q + t * HD + 2 * i) = qp;
      const int col = 2 * i, cg = col >> 6, ch = (col & 63) >> 3;
      const uint32_t off = (uint32_t)cg * L::kNewTile + t * 128 + (((ch ^ (t & 7))) << 4) + (col & 7) * 2;
      *reinterpret_cast<uint32_t*>(s_new + off) = kp;
      *reinterpret_cast<uint32_t*>(s_new + NC * L::kNewTile + off) = vp;
      if (ok && own_keys) {
        const size_t slot = (row_base + fill + t) * HD + col;
        *reinterpret_cast<uint32_t*>(a.kv_k + slot) = kp;
        *reinterpret_cast<uint32_t*>(a.kv_v + slot) = vp;
      }
    }
  }
  __syncthreads();

  const int n_mt = T > 16 ? 2 : 1;
  const int wpm = kWarps / n_mt;                  // warps per m-tile
  const int mt = warp / wpm, kg = warp - mt * wpm;
  uint32_t qa[HD / 16][4];
  uint32_t anc[2];
  {
    const int t0 = mt * 16 + g, t1 = t0 + 8;
    const bf16* q0 = s_q + t0 * HD + 2 * c;
    const bf16* q1 = s_q + t1 * HD + 2 * c;
#pragma unroll
    for (int kk = 0; kk < HD / 16; ++kk) {
      qa[kk][0] = t0 < T ? *reinterpret_cast<const uint32_t*>(q0 + 16 * kk) : 0u;
      qa[kk][1] = t1 < T ? *reinterpret_cast<const uint32_t*>(q1 + 16 * kk) : 0u;
      qa[kk][2] = t0 < T ? *reinterpret_cast<const uint32_t*>(q0 + 16 * kk + 8) : 0u;
      qa[kk][3] = t1 < T ? *reinterpret_cast<const uint32_t*>(q1 + 16 * kk + 8) : 0u;
    }
    anc[0] = t0 < T ? a.anc_mask[r * T + t0] : 0u;
    anc[1] = t1 < T ? a.anc_mask[r * T + t1] : 0u;
  }
  AttState<HD> st;
  st.m[0] = st.m[1] = -CUDART_INF_F;
  st.l[0] = st.l[1] = 0.f;
#pragma unroll
  for (int j = 0; j < NJ; ++j)
#pragma unroll
    for (int e = 0; e < 4; ++e) st.o[j][e] = 0.f;
  const float sl2 = rsqrtf((float)HD) * 1.4426950408889634f;

  // ---- cached keys ---------------------------------------------------------------------------------
#pragma unroll 1
  for (int j = 0; j < nb; ++j) {
    const int blk = rank + j * S;
    request(j + kStages - 1);
    cp_async_wait<kStages - 1>();
    __syncthreads();
    const uint32_t k_base = s_base + (uint32_t)(j % kStages) * L::kStage;
    const uint32_t v_base = k_base + NC * L::kTile;
#pragma unroll 1
    for (int sl = 0; sl < kKB / 16; ++sl) {
      if (((j * (kKB / 16) + sl) & (wpm - 1)) != kg) continue;
      const int left = fill - (blk * kKB + sl * 16);
      if (left <= 0) break;
      uint32_t vis[2];
      const uint32_t vmem = left >= 16 ? 0xffffu : ((1u << left) - 1u);
      vis[0] = vis[1] = vmem;
      att_slice<HD>(st, qa, k_base, v_base, (uint32_t)L::kTile, sl * 16, lane, sl2, vis, vmem);
    }
    __syncthreads();                              // the slot is requested again two iterations on
  }
  cp_async_wait<0>();
  // ---- the block's own keys: ancestors and the row itself, by the last warp of each m-tile ----------
  if (ok && own_keys && kg == wpm - 1) {
    const uint32_t k_base = tc::smem_u32(s_new), v_base = k_base + NC * L::kNewTile;
    for (int sl = 0; sl <= mt && sl * 16 < T; ++sl) {
      uint32_t vis[2];
      vis[0] = (anc[0] >> (16 * sl)) & 0xffffu;
      vis[1] = (anc[1] >> (16 * sl)) & 0xffffu;
      const uint32_t vmem = T - 16 * sl >= 16 ? 0xffffu : ((1u << (T - 16 * sl)) - 1u);
      att_slice<HD>(st, qa, k_base, v_base, (uint32_t)L::kNewTile, sl * 16, lane, sl2, vis, vmem);
    }
  }
#pragma unroll
  for (int i = 0; i < 2; ++i) {
    st.l[i] += __shfl_xor_sync(0xffffffffu, st.l[i], 1);
    st.l[i] += __shfl_xor_sync(0xffffffffu, st.l[i], 2);
  }
  // ---- merge the warps of each m-tile in a fixed tree ------------------------------------------------
  float* scratch = reinterpret_cast<float*>(smem + L::kOffScratch);
  constexpr int kRegs = L::kRegs;
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
    __syncthreads();
    if (kg < stp) {
      const float* slot = scratch + (size_t)(mt * stp + kg) * kRegs * 32;
#pragma unroll
      for (int i = 0; i < 2; ++i) {
        const float mo = slot[(NJ * 4 + i) * 32 + lane], lo = slot[(NJ * 4 + 2 + i) * 32 + lane];
        const float m_new = fmaxf(st.m[i], mo);
        const float m_safe = m_new == -CUDART_INF_F ? 0.f : m_new;
        const float aa = ex2(st.m[i] - m_safe), bb = ex2(mo - m_safe);
        st.m[i] = m_new;
        st.l[i] = st.l[i] * aa + lo * bb;
#pragma unroll
        for (int j = 0; j < NJ; ++j) {
          st.o[j][2 * i] = st.o[j][2 * i] * aa + slot[(j * 4 + 2 * i) * 32 + lane] * bb;
          st.o[j][2 * i + 1] = st.o[j][2 * i + 1] * aa + slot[(j * 4 + 2 * i + 1) * 32 + lane] * bb;
        }
      }
    }
    __syncthreads();
  }
  if (S > 1) {
    // ---- merge the ranks of the cluster: every rank publishes its m-tiles' state, rank 0 folds them in
    float* xslot = scratch + (size_t)(kWarps / 2 + mt) * kRegs * 32;
    if (kg == 0 && rank != 0) {
#pragma unroll
      for (int j = 0; j < NJ; ++j)
#pragma unroll
        for (int e = 0; e < 4; ++e) xslot[(j * 4 + e) * 32 + lane] = st.o[j][e];
      xslot[(NJ * 4 + 0) * 32 + lane] = st.m[0];
      xslot[(NJ * 4 + 1) * 32 + lane] = st.m[1];
      xslot[(NJ * 4 + 2) * 32 + lane] = st.l[0];
      xslot[(NJ * 4 + 3) * 32 + lane] = st.l[1];
    }
    cluster_sync_all();
    if (rank == 0) {
      // every rank has read its q / k / v sums long ago: clear them for the next layer
      for (int idx = tid; idx < T * HALF; idx += kThreads) {
        const int t = idx / HALF, i = idx - t * HALF;
        float* src = a.qkv + (size_t)(r * T + t) * 3 * d + h * HD + 2 * i;
        const float2 z = make_float2(0.f, 0.f);
        *reinterpret_cast<float2*>(src) = z;
        *reinterpret_cast<float2*>(src + d) = z;
        *reinterpret_cast<float2*>(src + 2 * d) = z;
      }
      if (kg == 0) {
        const uint32_t xaddr = tc::smem_u32(xslot);
#pragma unroll 1
        for (int q = 1; q < S; ++q) {
#pragma unroll
          for (int i = 0; i < 2; ++i) {
            const float mo = ld_cluster_f32(xaddr + (uint32_t)((NJ * 4 + i) * 32 + lane) * 4u, (uint32_t)q);
            const float lo = ld_cluster_f32(xaddr + (uint32_t)((NJ * 4 + 2 + i) * 32 + lane) * 4u, (uint32_t)q);
            const float m_new = fmaxf(st.m[i], mo);
            const float m_safe = m_new == -CUDART_INF_F ? 0.f : m_new;
            const float aa = ex2(st.m[i] - m_safe), bb = ex2(mo - m_safe);
            st.m[i] = m_new;
            st.l[i] = st.l[i] * aa + lo * bb;
#pragma unroll
            for (int j = 0; j < NJ; ++j) {
              const float o0 = ld_cluster_f32(xaddr + (uint32_t)((j * 4 + 2 * i) * 32 + lane) * 4u, (uint32_t)q);
              const float o1 = ld_cluster_f32(xaddr + (uint32_t)((j * 4 + 2 * i + 1) * 32 + lane) * 4u, (uint32_t)q);
              st.o[j][2 * i] = st.o[j][2 * i] * aa + o0 * bb;
              st.o[j][2 * i + 1] = st.o[j][2 * i + 1] * aa + o1 * bb;
            }
          }
        }
      }
    }
  }
  if (kg == 0 && rank == 0) {
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      const int t = mt * 16 + g + 8 * i;
      if (t < T) {
        const float inv = st.l[i] > 0.f ? 1.f / st.l[i] : 0.f;       // a sequence that failed its cache check gives zeros
        bf16* dst = a.out + (size_t)(r * T + t) * d + h * HD + 2 * c;
#pragma unroll
        for (int j = 0; j < NJ; ++j)
          *reinterpret_cast<uint32_t*>(dst + 8 * j) = pack2(st.o[j][2 * i] * inv, st.o[j][2 * i + 1] * inv);
      }
    }
  }
  if (S > 1) cluster_sync_all();      // no rank leaves while rank 0 may still read its state
}

template <int HD>
int launch_hd(const AttentionRowsArgs& a, cudaStream_t s) {
  using L = Layout<HD>;
  if (ensure_dynamic_smem(reinterpret_cast<const void*>(attention_rows_kernel<HD>), L::kBytes) != cudaSuccess)
    return VVS_ERR_CUDA;
  cudaLaunchConfig_t cfg = {};
  // few (sequence, head) items: split each item's keys over a cluster of 2, 4 or 8 CTAs, as long as
  // the grid still fits the GPU at three CTAs per SM and a rank keeps a dozen key blocks of a full cache
  // (measured: the 7B shape, 64 items of up to 75 blocks, is fastest split four ways, 3.65 against 4.06 ms
  // per step; the XL shape, 40 items of up to 10 blocks, is fastest unsplit)
  const int blocks_max = (a.s_max + L::kKB - 1) / L::kKB;
  int split = 1;
  while (split < 8 && (long long)a.n_heads * a.n_rows * split * 2 <= 3LL * a.n_sms && blocks_max >= 12 * split)
    split *= 2;
  cfg.gridDim = dim3(a.n_heads, a.n_rows, split);
  cfg.blockDim = dim3(kThreads, 1, 1);
  cfg.dynamicSmemBytes = L::kBytes;
  cfg.stream = s;
  cudaLaunchAttribute attr[2];
  int na = 0;
  if (a.pdl) {
    attr[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[na].val.programmaticStreamSerializationAllowed = 1;
    ++na;
  }
  if (split > 1) {
    attr[na].id = cudaLaunchAttributeClusterDimension;
    attr[na].val.clusterDim.x = 1;
    attr[na].val.clusterDim.y = 1;
    attr[na].val.clusterDim.z = (unsigned)split;
    ++na;
  }
  cfg.attrs = attr;
  cfg.numAttrs = na;
  return cudaLaunchKernelEx(&cfg, attention_rows_kernel<HD>, a) == cudaSuccess ? VVS_OK : VVS_ERR_CUDA;
}

}  // namespace

bool attention_rows_applicable(const vvs_model_desc& md, int t_len) {
  return md.dtype == VVS_DTYPE_BF16 && (md.head_dim == 64 || md.head_dim == 128) && t_len >= 1 && t_len <= kMaxT;
}

int launch_attention_rows(const AttentionRowsArgs& a, cudaStream_t s) {
  if (a.hd == 64) return launch_hd<64>(a, s);
  if (a.hd == 128) return launch_hd<128>(a, s);
  return VVS_ERR_SHAPE;
}

}  // namespace vvs
