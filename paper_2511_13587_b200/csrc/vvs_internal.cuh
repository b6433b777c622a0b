// Internal declarations of the verify-step library: context, scratch layout, launchers.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <map>
#include <mutex>
#include <utility>
#include <vector>

#include "vvs.h"

#define VVS_CUDA_OK(expr)                         \
  do {                                            \
    cudaError_t e__ = (expr);                     \
    if (e__ != cudaSuccess) return VVS_ERR_CUDA;  \
  } while (0)

namespace vvs {

// Raises a kernel's dynamic shared-memory limit to at least `bytes` on the CURRENT device.  The
// attribute is per device: the table of what has been set is keyed by (device, kernel), so a
// process that creates contexts on several GPUs configures each of them.
inline cudaError_t ensure_dynamic_smem(const void* kernel, int bytes) {
  static std::mutex mu;
  static std::map<std::pair<int, const void*>, int> done;
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  std::lock_guard<std::mutex> lock(mu);
  int& have = done[std::make_pair(dev, kernel)];
  if (have >= bytes) return cudaSuccess;
  e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e == cudaSuccess) have = bytes;
  return e;
}

// Scratch memory of a context.  Row index m of an activation matrix is r * T + t with
// r = c * B + b (cond sequences first).  "Decision rows" are (b, t) pairs: index b * T + t.
struct Workspace {
  float* x = nullptr;        // [M, d]   fp32 residual stream
  void* xn = nullptr;        // [M, d]   T normalised activations (GEMM input)
  float* qkv = nullptr;      // [M, 3d]  fp32 projections before RoPE
  void* q = nullptr;         // [M, d]   T queries after RoPE
  void* attn = nullptr;      // [M, d]   T attention output
  float* gu = nullptr;       // [M, 2ff] fp32 gate | up
  void* act = nullptr;       // [M, ff]  T silu(gate) * up
  void* hid = nullptr;       // [M, d]   T features when the caller does not ask for them
  float* logits_raw = nullptr;  // [M, V] fp32 per-sequence logits (generic path)
  float* logits = nullptr;      // [B*T, V] fp32 guided logits / temperature (generic path)
  float* part_m = nullptr;   // [n_tiles, B*T] per-tile running max
  float* part_s = nullptr;   // [n_tiles, B*T] per-tile sum of exp(l - max)
  float* stat_m = nullptr;   // [B*T] row max
  float* stat_inv = nullptr; // [B*T] 1 / sum exp(l - max)
  float* l_tok = nullptr;    // [B, K] guided logit of each drafted token
  float* l_nbr = nullptr;    // [B, K, kmax] guided logits of its neighbours (entry 0 unused)
  int32_t* sel_row = nullptr;   // [B] decision row (b*T + t) the next token is sampled from, -1 none
  int32_t* sel_kind = nullptr;  // [B] 0 = residual of draft n, 1 = bonus
  float* p_row = nullptr;    // [B, V] target probabilities of the selected row
  float* logits_small = nullptr; // [min(M, 64), V] guided logits of calls with few decision rows (tensor-core path)
  void* sel_hid = nullptr;   // [n_cfg * B, d] features of the selected rows (tensor-core LM head, row mode)
  double* r_part = nullptr;  // [B, n_chunks] per-chunk residual mass
  double* p_part = nullptr;  // [B, n_chunks] per-chunk target mass (fallback when residual is 0)
  float* rope_inv_freq = nullptr;  // [head_dim/2] angle per unit coordinate of each pair
  // tensor-core path
  int32_t* slot_pos = nullptr;   // [M] cache slot of each block row, -1 if its sequence overflows
  int32_t* seq_order = nullptr;  // [R] sequences by descending fill level (longest attention items first)
  uint32_t* anc_mask = nullptr;  // [M] bit j set: block row j of the same sequence is visible (ancestor or self)
  double* tree_res = nullptr;    // [2][max_rows, V] residuals of the tree walk (ping-pong)
  int32_t* tree_path = nullptr;  // [max_rows, 32] accepted nodes when the caller does not ask for them
  float* rope_cos = nullptr;     // [M, head_dim/2]
  float* rope_sin = nullptr;     // [M, head_dim/2]
  float* sk_scratch = nullptr;   // [M, max(3d, 2ff)] fp32 split-K sums; all zero between kernels
  int* sk_counters = nullptr;    // [passes, tiles] split-K arrival counters; zero between kernels
  float* attn_part_o = nullptr;  // [R*H, chunks, T, hd] un-normalised split-KV outputs
  float* attn_part_ml = nullptr; // [R*H, chunks, T, 2] chunk max / sum
  int* attn_counters = nullptr;  // [R*H] split-KV arrival counters; zero between kernels
  // whole-chain kernel (at most 32 block tokens)
  CUtensorMap* chain_wmaps = nullptr;          // [n_layers][5] weight descriptors, device copy
  float* chain_qkv = nullptr;    // [2][32, 3d] fp32 split-K sums of the QKV projection (by layer parity)
  float* chain_gu = nullptr;     // [2][32, 2ff] fp32 split-K sums of gate | up
  float* chain_ss = nullptr;     // [2 * n_layers][32] sums of squares of the residual rows
  unsigned* chain_sync = nullptr;  // [4] grid-barrier arrivals, epoch base, abort flag
  // streaming chain kernel (at most 32 block tokens)
  // stage inputs in B-fragment order (32 tokens x width bf16 each)
  void* cs_xn1 = nullptr;        // residual * first norm scale
  void* cs_xn2 = nullptr;        // residual * second norm scale
  void* cs_attn = nullptr;       // attention output
  void* cs_act = nullptr;        // silu(gate) * up
  float* cs_ss1 = nullptr;       // [d / 16][32] sums of squares of the residual rows per 16-column tile
  float* cs_ss2 = nullptr;
  unsigned* cs_flags = nullptr;  // [n_layers * 5 + 2] stage arrival counters, embedding counter, abort word
  int32_t* status = nullptr; // device status word
};

struct Layer {
  const void *w_qkv, *w_o, *w_gate, *w_up, *w_down, *norm1, *norm2;
};

// TMA descriptors of one layer's projection matrices (bf16 contexts)
struct LayerMaps {
  CUtensorMap w_qkv, w_o, w_gate, w_up, w_down;
};

}  // namespace vvs

namespace vvs {
// One captured verify step: replayed whenever a call repeats the same arguments.
struct GraphEntry {
  std::vector<unsigned char> key;  // argument and output structs, byte for byte
  cudaGraphExec_t exec = nullptr;
  int launches = 0;
  unsigned long long last_use = 0;
};
}  // namespace vvs

namespace vvs {
// Share of the decoder weights one CTA of the streaming chain kernel owns, the same in every layer:
// contiguous ranges of 16-row tiles of the QKV, output, gate / up (pairs) and down projections,
// its rank in the order attention items are dealt out, and the byte offset of its stream inside a
// layer's packed block.
struct ChainCtaPlan {
  int t0[4];
  int n[4];
  int att_rank;
  int pad;
  unsigned long long off;
};
struct ChainStreamPlan {
  int grid = 0;
  std::vector<ChainCtaPlan> cta;
  unsigned long long layer_bytes = 0;
  int n_prod[5] = {0, 0, 0, 0, 0};   // CTAs with work in each stage (attention: set per call)
};
}  // namespace vvs

struct vvs_ctx {
  vvs_model_desc desc;
  vvs::Workspace ws;
  void* arena = nullptr;
  size_t arena_bytes = 0;
  bool weights_bound = false;
  const void* tok_emb = nullptr;
  const void* norm_f = nullptr;
  const void* w_lm = nullptr;
  vvs::Layer* layers = nullptr;  // host array [n_layers]
  bool tensor_core_path = false;     // bf16 contexts unless VVS_DEBUG_GENERIC is set
  bool use_pdl = true;               // programmatic dependent launch of the tensor-core GEMMs
  bool use_chain_kernels = false;  // debug: the persistent whole-chain kernels for calls of at most 32 tokens
  vvs::LayerMaps* layer_maps = nullptr;  // host array [n_layers]
  std::vector<const __nv_bfloat16*> chain_norms;  // host [n_layers][2] norm-scale pointers
  vvs::ChainStreamPlan cs_plan;        // streaming chain kernel: split of the weights over the CTAs
  void* cs_packed = nullptr;           // device: private re-packed copy of the layer weights
  vvs::ChainCtaPlan* cs_d_plan = nullptr;  // device copy of cs_plan.cta
  CUtensorMap lm_map;
  int n_sms = 148;
  // CUDA-graph replay of vvs_verify (one graph per distinct argument set, small LRU cache)
  bool use_graph = true;
  cudaStream_t capture_stream = nullptr;
  std::vector<vvs::GraphEntry> graphs;
  unsigned long long graph_clock = 0;
  const int32_t* nbr_row_ptr = nullptr;
  const int32_t* nbr_col = nullptr;
  int64_t nbr_nnz = 0;
  int device = 0;
  int launches = 0;
  // optional per-launch event timing (vvs_profile_enable)
  bool profiling = false;
  cudaEvent_t* prof_events = nullptr;  // pairs (start, stop)
  int* prof_class = nullptr;           // class of each recorded pair
  int prof_capacity = 0;               // pairs
  int prof_used = 0;
};

namespace vvs {

constexpr int kSampleChunk = 1024;  // codebook entries per residual-mass chunk

// The one definition of a target probability from a guided logit and its row statistics; every
// kernel that emits or compares probabilities calls it, so decisions and emitted values agree
// bit for bit.
__device__ __forceinline__ float prob_of(float l, float m, float inv) { return expf(l - m) * inv; }

// ---- generic kernels (any storage type), kernels_generic.cu ---------------------------------
template <typename T>
void launch_embed(const T* tok_emb, const int32_t* block, float* x, int n_images, int n_cfg,
                  int t_len, int d, int tok_rows, int32_t* status, cudaStream_t s);
template <typename T>
void launch_rmsnorm(const float* x, const T* scale, T* out, int m, int d, float eps, cudaStream_t s);
// c[m, n] (+)= sum_k a[m, k] * w[n, k]; c fp32 with leading dimension ldc
template <typename T>
void launch_gemm_nt(const T* a, const T* w, float* c, int m, int n, int k, int ldc, bool accumulate,
                    cudaStream_t s);
template <typename T>
void launch_rope_append(float* qkv, const float* inv_freq, T* q, T* kv_k, T* kv_v,
                        const int32_t* cache_len, const vvs_model_desc& md, int layer, int kv_rows,
                        int n_rows, int t_len, int32_t* status, cudaStream_t s, const float* tab_cos = nullptr,
                        const float* tab_sin = nullptr, bool clear_src = false);
template <typename T>
void launch_attention(const T* q, const T* kv_k, const T* kv_v, const int32_t* cache_len, T* out,
                      const vvs_model_desc& md, int layer, int kv_rows, int n_rows, int t_len,
                      cudaStream_t s);
template <typename T>
void launch_silu_mul(float* gu, T* act, int m, int ff, cudaStream_t s, bool clear_src = false, bool pdl = false);
void launch_rmsnorm_rows(const float* x, const __nv_bfloat16* scale, __nv_bfloat16* out, int m, int d, float eps,
                         bool pdl, cudaStream_t s);
void launch_guide(const float* raw, float* logits, int n_images, int n_cfg, int rows_per_seq, int v,
                  float cfg_scale, float inv_temp, cudaStream_t s);
void launch_row_stats(const float* logits, float* part_m, float* part_s, int n_rows, int v,
                      cudaStream_t s);

// ---- tensor-core projection GEMM, gemm_tc.cu ----------------------------------------------------
enum { GEMM_EPI_STORE = 0, GEMM_EPI_ADD = 1, GEMM_EPI_QKV = 2, GEMM_EPI_SWIGLU = 3, GEMM_EPI_ADD2 = 4 };
struct GemmTcPlan {
  int nt, passes, tiles, kb_total, splits, stages, smem_bytes, tmem_cols;
};
struct GemmTcArgs {
  int m, n, k;                 // tokens, weight rows (per matrix), reduction length
  const CUtensorMap* tm_a;     // weights [n, k]
  const CUtensorMap* tm_a2;    // second weight matrix (SWIGLU: up), else null
  const CUtensorMap* tm_b;     // activations [m, k], box rows = plan.nt
  bool pdl;
  float* scratch; int ld_scratch; int* counters; int32_t* status;
  float* out; int ldo;         // STORE / ADD
  int cluster_mode;            // ADD with many tokens: 0 = split-K sums added with reductions in arrival order;
                               // 1 / 2 = the K splits of a tile form a thread-block cluster that adds its partial
                               // tiles in rank order through distributed shared memory and then stores (1) or adds
                               // to (2) `out`, each element by exactly one thread: no atomics, repeatable bits
  __nv_bfloat16* q; __nv_bfloat16* kv_k; __nv_bfloat16* kv_v;  // QKV
  const int32_t* slot_pos; const float* rope_cos; const float* rope_sin;
  int d, n_heads, hd, s_max, layer, kv_rows, t_len;
  __nv_bfloat16* act; int ff;  // SWIGLU
};
int make_tmap_bf16_2d(CUtensorMap* out, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows);
int make_weight_tmap(CUtensorMap* out, const void* w, int rows, int cols);
GemmTcPlan plan_gemm_tc(int m, int n, int k, bool dual, bool allow_split, int n_sms, int split_cap = 32);
int launch_gemm_tc(int epi, const GemmTcPlan& plan, const GemmTcArgs& g, cudaStream_t s);
void launch_rope_table(const int32_t* cache_len, const int32_t* tree_parent, int n_images, int n_forced,
                       const Workspace& ws, const vvs_model_desc& md, int n_rows,
                       int t_len, cudaStream_t s, unsigned* clear_words = nullptr, int n_clear = 0);

// ---- tensor-core attention, attention_tc.cu ----------------------------------------------------------
struct AttentionTcArgs {
  const CUtensorMap* tm_q;   // q [M, d], box {64, 16 or 32}
  const CUtensorMap* tm_k;   // cache viewed as [layers*kv_rows*heads*s_max, hd], box {64, 128}
  const CUtensorMap* tm_v;
  const int32_t* cache_len;
  const uint32_t* anc_mask;  // [M] visible block rows per block row
  __nv_bfloat16* out;
  float* part_o; float* part_ml; int* counters; int32_t* status;
  int d, n_heads, hd, s_max, layer, kv_rows, t_len, n_rows;
  bool pdl;
};
int launch_attention_tc(const AttentionTcArgs& a, cudaStream_t s);

// ---- row-batched attention with fused rotation / cache append, attention_rows.cu ----------------------
struct AttentionRowsArgs {
  float* qkv;                  // [M, 3 d] fp32 split-K sums of the QKV projection; read, then cleared
  __nv_bfloat16* kv_k;         // cache [layers][kv_rows][heads][s_max][hd]; slots fill .. fill + T - 1 are written
  __nv_bfloat16* kv_v;
  const int32_t* cache_len;    // [R]
  const float* rope_cos;       // [M, hd / 2] rotation table of the step
  const float* rope_sin;
  const uint32_t* anc_mask;    // [M] visible block rows per block row
  const int32_t* seq_order;    // [R] the sequence CTA row y works on: longest caches first
  __nv_bfloat16* out;          // [M, d]
  int d, n_heads, hd, s_max, layer, kv_rows, t_len, n_rows, n_sms;
  bool pdl;
};
bool attention_rows_applicable(const vvs_model_desc& md, int t_len);
int launch_attention_rows(const AttentionRowsArgs& a, cudaStream_t s);

// ---- LM head with fused decision epilogue, lmhead_tc.cu -------------------------------------------
struct LmHeadArgs {
  int v, k, bt, n_cfg;           // codebook size, d_model, decision rows, 1 or 2 feature rows per decision row
  const CUtensorMap* tm_a;       // codebook rows of w_lm [v, k]
  const CUtensorMap* tm_b;       // features [n_cfg * bt, k] (cond rows, then uncond rows), box rows = lmhead_box_rows(bt)
  bool pdl;
  int n_sms;                     // SMs of the device (0: 148)
  float cfg_scale, inv_temp;
  float* part_m; float* part_s;  // [n_tiles, bt] softmax partials per 128-code tile
  float* logits_out;             // optional [bt, v] guided logits
  int32_t* status;
  int rows_per_seq, first_row, n_draft_max, vocab_offset, relaxed, nbr_k, kmax, drafts_ld;
  const int32_t* drafts; const int32_t* row_ptr; const int32_t* col;
  float* l_tok; float* l_nbr;
  int row_mode;                  // 1: bt = images, write probabilities of the selected rows to p_row
  const int32_t* sel_row; const float* stat_m; const float* stat_inv; float* p_row;
};
int lmhead_box_rows(int bt);
int launch_lmhead_tc(const LmHeadArgs& a, cudaStream_t s);
void launch_gather_sel_rows(const void* hid, const int32_t* sel_row, void* out, int n_images, int n_cfg, int bt,
                            int d, cudaStream_t s);

// ---- whole-chain persistent kernel, fused_chain.cu ---------------------------------------------
struct FusedChainArgs {
  const vvs_model_desc* md;
  int n_rows, n_images, t_len, kv_rows, n_sms;
  const CUtensorMap* wmaps;             // device
  const __nv_bfloat16* const* norms_host;  // HOST array [n_layers][2] of device pointers
  const __nv_bfloat16* tok_emb;
  const int32_t* block;
  float* x; float* qkv_acc; float* gu_acc; float* ss;
  const int32_t* cache_len;
  __nv_bfloat16* kv_k; __nv_bfloat16* kv_v;
  const CUtensorMap* tm_k;              // host copies of the cache descriptors (box {64, 128})
  const CUtensorMap* tm_v;
  const int32_t* slot_pos; const uint32_t* anc_mask; const float* rope_cos; const float* rope_sin;
  float* part_o; float* part_ml;
  unsigned* sync_words;
  int32_t* status;
};
// Walk of the candidate trees (tree calls of vvs_verify) and the cache compaction after it.
struct TreeParams {
  int n_images, n_cfg, n_forced, n_draft_max, t_len, vocab, vocab_offset;
  const int32_t* parent;      // [B, T]
  const int32_t* drafts;      // embedding-table ids of the draft nodes, row stride drafts_ld
  int drafts_ld;
  const float* probs;         // [B, T, V] target rows of all block rows
  const float* draft_probs;   // [B, K, V]
  const float* uniforms;      // [B, K+1]
  const int32_t* cache_len;
  double* res;                // [2][B, V]
  int relaxed, nbr_k, adjusted;   // relaxed acceptance on the current residual; adjusted-residual flag
  float delta;
  const int32_t* row_ptr; const int32_t* col;
  int32_t* accept_len; int32_t* accept_path; int32_t* next_token; int32_t* new_len; int32_t* n_commit;
  uint8_t* accept_mask; float* margins;
  int32_t* status;
};
void launch_tree_walk(const TreeParams& p, cudaStream_t s);
void launch_tree_commit(void* kv_k, void* kv_v, const int32_t* cache_len, const int32_t* accept_len,
                        const int32_t* accept_path, const vvs_model_desc& md, int kv_rows, int n_images, int n_cfg,
                        int n_forced, int n_draft_max, cudaStream_t s);
bool fused_chain_applicable(const vvs_model_desc& md, int n_rows, int t_len);
size_t fused_chain_smem_bytes(const vvs_model_desc& md, int t_len, int* w_stages);
int launch_fused_chain(const FusedChainArgs& a, cudaStream_t s);

// ---- streaming chain kernel, chain_stream.cu ------------------------------------------------------
struct ChainStreamArgs {
  const vvs_model_desc* md;
  int n_rows, n_images, t_len, kv_rows;
  const ChainStreamPlan* plan;
  const ChainCtaPlan* d_plan;           // device
  const void* packed;                   // device
  const __nv_bfloat16* const* norms_host;  // HOST array [n_layers][2] of device pointers
  const __nv_bfloat16* tok_emb;
  const int32_t* block;
  float* x;
  __nv_bfloat16 *xn1, *xn2, *qbuf, *attn, *act;
  float *ss1, *ss2;
  const int32_t* cache_len;
  __nv_bfloat16* kv_k; __nv_bfloat16* kv_v;
  const CUtensorMap* tm_k;              // host: cache as [rows, head_dim], box {64, chain_stream_kb()}
  const CUtensorMap* tm_v;
  const int32_t* slot_pos; const uint32_t* anc_mask; const float* rope_cos; const float* rope_sin;
  unsigned* flags;                      // zero at launch
  int32_t* status;
};
bool chain_stream_applicable(const vvs_model_desc& md, int n_rows, int t_len);
bool chain_stream_plan(const vvs_model_desc& md, int grid, ChainStreamPlan& out);
size_t chain_stream_packed_bytes(const vvs_model_desc& md, const ChainStreamPlan& plan);
int chain_stream_pack(const vvs_model_desc& md, const ChainStreamPlan& plan, const ChainCtaPlan* d_plan,
                      const Layer* layers, void* packed, cudaStream_t s);
int chain_stream_kb(const vvs_model_desc& md);
size_t chain_stream_flag_words(const vvs_model_desc& md);
int chain_stream_configure();
int launch_chain_stream(const ChainStreamArgs& a, cudaStream_t s);
void launch_bounded_wait_selftest(int32_t* status, int32_t* report, cudaStream_t s);

// ---- decision stage, kernels_decide.cu -----------------------------------------------------
struct DecideParams {
  int n_images, n_cfg, rows_per_seq, first_row, n_draft_max, vocab, vocab_offset;
  int mode, nbr_k, kmax;
  float delta;
  int adjusted;               // relaxed mode: the residual's p is the adjusted target of the rejected draft
  const int32_t* drafts;      // [B, drafts_ld] embedding ids
  int drafts_ld;
  const int32_t* n_draft;     // [B] or null
  const float* draft_probs;   // [B, K, V]
  const float* uniforms;      // [B, K+1]
  const int32_t* row_ptr;
  const int32_t* col;
  const float* direct_probs;  // non-null: the gathered values and the sampled rows are target
                              // probabilities [B*rows_per_seq, V] given by the caller, not logits
  const int32_t* cache_len;   // [R] or null (epilogue entry)
  int n_forced;
  int32_t* accept_len;
  int32_t* next_token;
  int32_t* new_len;
  int32_t* n_commit;
  uint8_t* accept_mask;
  float* margins;
};
void launch_finalize_stats(const Workspace& ws, int n_tiles, int n_rows, cudaStream_t s);
void launch_gather_logits(const float* logits, const Workspace& ws, const DecideParams& p, cudaStream_t s);
void launch_accept(const Workspace& ws, const DecideParams& p, cudaStream_t s);
void launch_probs_from_logits(const float* logits, const Workspace& ws, float* probs, int n_rows,
                              int v, cudaStream_t s);
void launch_select_p_row(const float* logits, const Workspace& ws, int n_images, int v, cudaStream_t s);
void launch_adjust_target(const Workspace& ws, const DecideParams& p, cudaStream_t s);
void launch_residual_mass(const Workspace& ws, const DecideParams& p, cudaStream_t s);
void launch_sample(const Workspace& ws, const DecideParams& p, cudaStream_t s);

// ---- dynamic skip decision, kernels_skip.cu -----------------------------------------------------
int launch_skip_decide(const int32_t* paths, const int32_t* path_len, const float* codebook,
                       const uint8_t* last_verified, int n_images, int n_paths, int max_len, int vocab, int dim,
                       int stride, float alpha, float threshold, uint8_t* decision, float* sim, int32_t* status,
                       cudaStream_t s);

int launch_select_unverified(const int32_t* paths, const int32_t* path_len, const float* uniforms, int n_images,
                             int n_paths, int max_len, int32_t* out_path, int32_t* out_gamma, int32_t* out_tokens,
                             int32_t* status, cudaStream_t s);

// ---- feature cache, kernels_fcache.cu ---------------------------------------------------------
void launch_fcache_reset(const vvs_fcache& fc, cudaStream_t s);
void launch_fcache_store(const vvs_fcache& fc, const void* hidden, int rows_per_seq, int d,
                         int elem_bytes, const int32_t* base_pos, const int32_t* n_store,
                         int32_t* status, cudaStream_t s);
void launch_fcache_fetch(const vvs_fcache& fc, const uint8_t* skip_mask, int n_images,
                         const int32_t* gamma, int gamma_max, int staleness, int d, int elem_bytes,
                         void* out, int32_t* out_pos, int32_t* status, cudaStream_t s);

}  // namespace vvs
