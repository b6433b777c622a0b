// C ABI of the verify-step library: argument checks, scratch layout, launch sequences.
#include <cmath>
#include <cstdlib>
#include <cstring>
#include <new>

#include "vvs_internal.cuh"

using namespace vvs;

namespace {

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline size_t elem_bytes(const vvs_model_desc& d) { return d.dtype == VVS_DTYPE_BF16 ? 2 : 4; }

// Carves the scratch arena; with base == nullptr only the total size is computed.
struct Carver {
  char* base;
  size_t off = 0;
  template <typename P>
  void take(P*& p, size_t bytes) {
    off = (off + 255) & ~size_t(255);
    if (base) p = reinterpret_cast<P*>(base + off);
    off += bytes;
  }
};

size_t layout(const vvs_model_desc& d, Workspace& ws, char* base) {
  Carver c{base};
  const size_t es = elem_bytes(d);
  const size_t M = (size_t)d.max_rows * d.max_block;  // activation rows; also bounds B*T
  const size_t V = d.vocab, dm = d.d_model, ff = d.d_ff;
  const size_t n_tiles = (V + 127) / 128;
  const size_t n_chunks = (V + kSampleChunk - 1) / kSampleChunk;
  c.take(ws.status, 256);
  c.take(ws.rope_inv_freq, (size_t)d.head_dim / 2 * 4);
  if (d.n_layers > 0) {
    c.take(ws.x, M * dm * 4);
    c.take(ws.xn, M * dm * es);
    c.take(ws.qkv, M * 3 * dm * 4);
    c.take(ws.q, M * dm * es);
    c.take(ws.attn, M * dm * es);
    c.take(ws.gu, M * 2 * ff * 4);
    c.take(ws.act, M * ff * es);
    c.take(ws.hid, M * dm * es);
    if (d.dtype == VVS_DTYPE_BF16) {
      const size_t wide = 3 * dm > 2 * ff ? 3 * dm : 2 * ff;
      const size_t tiles = (wide + 127) / 128, passes = (M + 255) / 256;
      c.take(ws.slot_pos, M * 4);
      c.take(ws.seq_order, (size_t)d.max_rows * 4);
      c.take(ws.rope_cos, M * (size_t)(d.head_dim / 2) * 4);
      c.take(ws.rope_sin, M * (size_t)(d.head_dim / 2) * 4);
      c.take(ws.sk_scratch, M * wide * 4);
      c.take(ws.sk_counters, tiles * passes * 4);
      const size_t chunks = ((size_t)d.s_max + 127) / 128, rh = (size_t)d.max_rows * d.n_heads;
      c.take(ws.attn_part_o, rh * chunks * d.max_block * d.head_dim * 4);
      c.take(ws.attn_part_ml, rh * chunks * d.max_block * 2 * 4);
      c.take(ws.attn_counters, rh * 4);
      c.take(ws.chain_wmaps, (size_t)d.n_layers * 5 * sizeof(CUtensorMap));
      c.take(ws.chain_qkv, (size_t)2 * 32 * 3 * dm * 4);
      c.take(ws.chain_gu, (size_t)2 * 32 * 2 * ff * 4);
      c.take(ws.chain_ss, (size_t)2 * d.n_layers * 32 * 4);
      c.take(ws.chain_sync, 256);
      c.take(ws.cs_xn1, (size_t)32 * dm * 2);
      c.take(ws.cs_xn2, (size_t)32 * dm * 2);
      c.take(ws.cs_attn, (size_t)32 * dm * 2);
      c.take(ws.cs_act, (size_t)32 * ff * 2);
      c.take(ws.cs_ss1, (size_t)(dm / 16 + 1) * 32 * 4);
      c.take(ws.cs_ss2, (size_t)(dm / 16 + 1) * 32 * 4);
      c.take(ws.cs_flags, chain_stream_flag_words(d) * 4);
    }
  }
  // full logits exist only on the generic path (float32 contexts, or bf16 ones forced onto it)
  if (d.dtype != VVS_DTYPE_BF16 || std::getenv("VVS_DEBUG_GENERIC")) {
    c.take(ws.logits_raw, M * V * 4);
    c.take(ws.logits, M * V * 4);
  } else {
    c.take(ws.sel_hid, (size_t)d.max_rows * dm * es);

  }
  c.take(ws.part_m, n_tiles * M * 4);
  c.take(ws.part_s, n_tiles * M * 4);
  c.take(ws.stat_m, M * 4);
  c.take(ws.stat_inv, M * 4);
  c.take(ws.l_tok, M * 4);
  c.take(ws.l_nbr, M * (size_t)d.max_nbr_k * 4);
  c.take(ws.sel_row, (size_t)d.max_rows * 4);
  c.take(ws.sel_kind, (size_t)d.max_rows * 4);
  c.take(ws.p_row, (size_t)d.max_rows * V * 4);
  c.take(ws.r_part, (size_t)d.max_rows * n_chunks * 8);
  c.take(ws.p_part, (size_t)d.max_rows * n_chunks * 8);
  if (d.dtype == VVS_DTYPE_BF16 && d.n_layers > 0) c.take(ws.anc_mask, M * 4);
  c.take(ws.tree_res, (size_t)2 * d.max_rows * V * 8);
  c.take(ws.tree_path, (size_t)d.max_rows * 32 * 4);
  if (d.dtype == VVS_DTYPE_BF16 && !std::getenv("VVS_DEBUG_GENERIC")) c.take(ws.logits_small, (M < 64 ? M : 64) * V * 4);
  return (c.off + 255) & ~size_t(255);
}

int check_desc(const vvs_model_desc* d) {
  if (!d) return VVS_ERR_INVALID_ARG;
  if (d->dtype != VVS_DTYPE_FP32 && d->dtype != VVS_DTYPE_BF16) return VVS_ERR_INVALID_ARG;
  if (d->deterministic != 0 && d->deterministic != 1) return VVS_ERR_INVALID_ARG;
  if (d->rope_mode < VVS_ROPE_NONE || d->rope_mode > VVS_ROPE_2D_GRID) return VVS_ERR_INVALID_ARG;
  if (d->n_layers < 0 || d->d_model <= 0 || d->vocab <= 0 || d->vocab_offset < 0) return VVS_ERR_SHAPE;
  if (d->lm_rows < d->vocab_offset + d->vocab) return VVS_ERR_SHAPE;
  if (d->vocab > 65535 * 128) return VVS_ERR_SHAPE;      // the LM head puts one 128-code tile on each grid row
  if (d->d_model % 8) return VVS_ERR_SHAPE;
  if (d->max_rows < 1 || d->max_block < 1 || d->max_block > 32 || d->max_nbr_k < 1) return VVS_ERR_SHAPE;
  if (d->n_layers > 0) {
    if (d->head_dim != 64 && d->head_dim != 128) return VVS_ERR_SHAPE;
    if (d->n_heads <= 0 || d->n_heads * d->head_dim != d->d_model) return VVS_ERR_SHAPE;
    if (d->d_ff <= 0 || d->d_ff % 8) return VVS_ERR_SHAPE;
    if (d->s_max < 1 || d->tok_rows < 1) return VVS_ERR_SHAPE;
    if (d->rope_mode == VVS_ROPE_2D_GRID && (d->rope_grid_w < 1 || d->n_prefix < 0)) return VVS_ERR_SHAPE;
    if (!(d->rms_eps > 0.f) || !(d->rope_base > 1.f)) return VVS_ERR_INVALID_ARG;
  }
  return VVS_OK;
}

// Brackets one kernel launch: counts it and, when profiling, records an event pair around it.
struct Launch {
  vvs_ctx* ctx;
  cudaStream_t s;
  int slot = -1;
  Launch(vvs_ctx* c, int cls, cudaStream_t st) : ctx(c), s(st) {
    if (ctx->profiling && ctx->prof_used < ctx->prof_capacity) {
      slot = ctx->prof_used++;
      ctx->prof_class[slot] = cls;
      cudaEventRecord(ctx->prof_events[2 * slot], s);
    }
  }
  ~Launch() {
    ctx->launches += 1;
    if (slot >= 0) cudaEventRecord(ctx->prof_events[2 * slot + 1], s);
  }
};
#define VVS_LAUNCH(cls, call) do { Launch l__(ctx, cls, s); call; } while (0)

DecideParams decide_params(const vvs_ctx* ctx, int rows_per_seq, int first_row, const int32_t* drafts,
                           int drafts_ld, const vvs_verify_args* a, const vvs_verify_out* o,
                           bool with_cache) {
  const vvs_model_desc& md = ctx->desc;
  DecideParams p{};
  p.n_images = a->n_images; p.n_cfg = a->n_cfg; p.rows_per_seq = rows_per_seq; p.first_row = first_row;
  p.n_draft_max = a->n_draft_max; p.vocab = md.vocab; p.vocab_offset = md.vocab_offset;
  p.mode = a->mode; p.nbr_k = a->mode == VVS_MODE_RELAXED ? a->nbr_k : 1; p.kmax = md.max_nbr_k;
  p.delta = a->delta;
  p.adjusted = (a->mode == VVS_MODE_RELAXED && a->nbr_k > 1 && a->adjusted_residual) ? 1 : 0;
  p.drafts = drafts; p.drafts_ld = drafts_ld; p.n_draft = a->n_draft;
  p.draft_probs = a->draft_probs; p.uniforms = a->uniforms;
  p.row_ptr = ctx->nbr_row_ptr; p.col = ctx->nbr_col;
  p.direct_probs = nullptr;
  p.cache_len = with_cache ? a->cache_len : nullptr; p.n_forced = a->n_forced;
  p.accept_len = o->accept_len; p.next_token = o->next_token;
  p.new_len = with_cache ? o->new_len : nullptr;
  p.n_commit = with_cache ? o->n_commit : nullptr;
  p.accept_mask = o->accept_mask; p.margins = o->margins;
  return p;
}

// LM head over the codebook rows, guidance, softmax statistics, decisions.  Generic path: the
// per-sequence logits and the guided logits live in scratch.
template <typename T>
int run_decisions(vvs_ctx* ctx, const T* hid, int rows_per_seq, int first_row, const int32_t* drafts,
                  int drafts_ld, const vvs_verify_args* a, const vvs_verify_out* o, bool with_cache,
                  cudaStream_t s) {
  const vvs_model_desc& md = ctx->desc;
  Workspace& ws = ctx->ws;
  const int B = a->n_images, C = a->n_cfg, R = B * C;
  const int M = R * rows_per_seq, V = md.vocab, BT = B * rows_per_seq;
  const T* w_lm = static_cast<const T*>(ctx->w_lm) + (size_t)md.vocab_offset * md.d_model;

  DecideParams p = decide_params(ctx, rows_per_seq, first_row, drafts, drafts_ld, a, o, with_cache);


  if (ctx->tensor_core_path) {
    // LM head with guidance, softmax partials and gathers fused into its epilogue
    CUtensorMap tm_hid, tm_sel;
    if (make_tmap_bf16_2d(&tm_hid, hid, (uint64_t)M, (uint64_t)md.d_model, (uint32_t)lmhead_box_rows(BT)) != VVS_OK ||
        make_tmap_bf16_2d(&tm_sel, ws.sel_hid, (uint64_t)R, (uint64_t)md.d_model, (uint32_t)lmhead_box_rows(B)) != VVS_OK)
      return VVS_ERR_CUDA;
    LmHeadArgs la{};
    la.v = V; la.k = md.d_model; la.bt = BT; la.n_cfg = C; la.tm_a = &ctx->lm_map; la.tm_b = &tm_hid;
    la.pdl = ctx->use_pdl; la.n_sms = ctx->n_sms; la.cfg_scale = a->cfg_scale; la.inv_temp = 1.f / a->temperature;
    // few decision rows: the guided logits are written out (under a megabyte at 9 rows) and the
    // sampled row is read back from them; otherwise a second pass over the head recomputes it
    float* lbuf = o->target_probs ? o->target_probs : (BT <= 64 ? ws.logits_small : nullptr);
    la.part_m = ws.part_m; la.part_s = ws.part_s; la.logits_out = lbuf; la.status = ws.status;
    la.rows_per_seq = rows_per_seq; la.first_row = first_row; la.n_draft_max = p.n_draft_max;
    la.vocab_offset = md.vocab_offset; la.relaxed = (p.mode == VVS_MODE_RELAXED && p.nbr_k > 1) ? 1 : 0;
    la.nbr_k = p.nbr_k; la.kmax = p.kmax; la.drafts_ld = drafts_ld; la.drafts = drafts;
    la.row_ptr = p.row_ptr; la.col = p.col; la.l_tok = ws.l_tok; la.l_nbr = ws.l_nbr;
    int rc = VVS_OK;
    VVS_LAUNCH(VVS_PROF_GEMM, rc = launch_lmhead_tc(la, s));
    if (rc != VVS_OK) return rc;
    VVS_LAUNCH(VVS_PROF_OTHER, launch_finalize_stats(ws, (V + 127) / 128, BT, s));
    VVS_LAUNCH(VVS_PROF_OTHER, launch_accept(ws, p, s));
    if (lbuf) {
      VVS_LAUNCH(VVS_PROF_OTHER, launch_select_p_row(lbuf, ws, B, V, s));
      if (o->target_probs)
        VVS_LAUNCH(VVS_PROF_OTHER, launch_probs_from_logits(o->target_probs, ws, o->target_probs, BT, V, s));
      if (p.adjusted) VVS_LAUNCH(VVS_PROF_OTHER, launch_adjust_target(ws, p, s));
      VVS_LAUNCH(VVS_PROF_OTHER, launch_residual_mass(ws, p, s));
      VVS_LAUNCH(VVS_PROF_OTHER, launch_sample(ws, p, s));
      return cudaGetLastError() == cudaSuccess ? VVS_OK : VVS_ERR_CUDA;
    }
    VVS_LAUNCH(VVS_PROF_OTHER, launch_gather_sel_rows(hid, ws.sel_row, ws.sel_hid, B, C, BT, md.d_model, s));
    LmHeadArgs lr{};
    lr.v = V; lr.k = md.d_model; lr.bt = B; lr.n_cfg = C; lr.tm_a = &ctx->lm_map; lr.tm_b = &tm_sel;
    lr.pdl = ctx->use_pdl; lr.n_sms = ctx->n_sms; lr.cfg_scale = a->cfg_scale; lr.inv_temp = 1.f / a->temperature; lr.status = ws.status;
    lr.row_mode = 1; lr.sel_row = ws.sel_row; lr.stat_m = ws.stat_m; lr.stat_inv = ws.stat_inv; lr.p_row = ws.p_row;
    VVS_LAUNCH(VVS_PROF_GEMM, rc = launch_lmhead_tc(lr, s));
    if (rc != VVS_OK) return rc;
    if (p.adjusted) VVS_LAUNCH(VVS_PROF_OTHER, launch_adjust_target(ws, p, s));
    VVS_LAUNCH(VVS_PROF_OTHER, launch_residual_mass(ws, p, s));
    VVS_LAUNCH(VVS_PROF_OTHER, launch_sample(ws, p, s));
    return cudaGetLastError() == cudaSuccess ? VVS_OK : VVS_ERR_CUDA;
  }
  VVS_LAUNCH(VVS_PROF_GEMM, launch_gemm_nt<T>(hid, w_lm, ws.logits_raw, M, V, md.d_model, V, false, s));
  VVS_LAUNCH(VVS_PROF_OTHER, launch_guide(ws.logits_raw, ws.logits, B, C, rows_per_seq, V, a->cfg_scale,
                                          1.f / a->temperature, s));
  VVS_LAUNCH(VVS_PROF_OTHER, launch_row_stats(ws.logits, ws.part_m, ws.part_s, BT, V, s));
  VVS_LAUNCH(VVS_PROF_OTHER, launch_finalize_stats(ws, 1, BT, s));
  if (p.n_draft_max > 0) VVS_LAUNCH(VVS_PROF_OTHER, launch_gather_logits(ws.logits, ws, p, s));
  VVS_LAUNCH(VVS_PROF_OTHER, launch_accept(ws, p, s));
  if (o->target_probs)
    VVS_LAUNCH(VVS_PROF_OTHER, launch_probs_from_logits(ws.logits, ws, o->target_probs, BT, V, s));
  VVS_LAUNCH(VVS_PROF_OTHER, launch_select_p_row(ws.logits, ws, B, V, s));
  if (p.adjusted) VVS_LAUNCH(VVS_PROF_OTHER, launch_adjust_target(ws, p, s));
  VVS_LAUNCH(VVS_PROF_OTHER, launch_residual_mass(ws, p, s));
  VVS_LAUNCH(VVS_PROF_OTHER, launch_sample(ws, p, s));
  return cudaGetLastError() == cudaSuccess ? VVS_OK : VVS_ERR_CUDA;
}

template <typename T>
int run_verify(vvs_ctx* ctx, const vvs_verify_args* a, const vvs_verify_out* o, cudaStream_t s) {
  const vvs_model_desc& md = ctx->desc;
  Workspace& ws = ctx->ws;
  const int B = a->n_images, C = a->n_cfg, R = B * C, Tn = a->n_forced + a->n_draft_max;
  const int M = R * Tn, d = md.d_model, ff = md.d_ff;
  T* kv_k = static_cast<T*>(a->kv_k);
  T* kv_v = static_cast<T*>(a->kv_v);
  T* xn = static_cast<T*>(ws.xn);
  T* q = static_cast<T*>(ws.q);
  T* attn = static_cast<T*>(ws.attn);
  T* act = static_cast<T*>(ws.act);
  T* hid = o->hidden ? static_cast<T*>(o->hidden) : static_cast<T*>(ws.hid);

  VVS_LAUNCH(VVS_PROF_OTHER, launch_embed<T>(static_cast<const T*>(ctx->tok_emb), a->block, ws.x, B, C, Tn,
                                             d, md.tok_rows, ws.status, s));
  for (int l = 0; l < md.n_layers; ++l) {
    const Layer& L = ctx->layers[l];
    VVS_LAUNCH(VVS_PROF_OTHER, launch_rmsnorm<T>(ws.x, static_cast<const T*>(L.norm1), xn, M, d, md.rms_eps, s));
    VVS_LAUNCH(VVS_PROF_GEMM,
               launch_gemm_nt<T>(xn, static_cast<const T*>(L.w_qkv), ws.qkv, M, 3 * d, d, 3 * d, false, s));
    VVS_LAUNCH(VVS_PROF_OTHER, launch_rope_append<T>(ws.qkv, ws.rope_inv_freq, q, kv_k, kv_v, a->cache_len, md,
                                                     l, a->kv_rows, R, Tn, ws.status, s));
    VVS_LAUNCH(VVS_PROF_ATTENTION,
               launch_attention<T>(q, kv_k, kv_v, a->cache_len, attn, md, l, a->kv_rows, R, Tn, s));
    VVS_LAUNCH(VVS_PROF_GEMM, launch_gemm_nt<T>(attn, static_cast<const T*>(L.w_o), ws.x, M, d, d, d, true, s));
    VVS_LAUNCH(VVS_PROF_OTHER, launch_rmsnorm<T>(ws.x, static_cast<const T*>(L.norm2), xn, M, d, md.rms_eps, s));
    VVS_LAUNCH(VVS_PROF_GEMM,
               launch_gemm_nt<T>(xn, static_cast<const T*>(L.w_gate), ws.gu, M, ff, d, 2 * ff, false, s));
    VVS_LAUNCH(VVS_PROF_GEMM,
               launch_gemm_nt<T>(xn, static_cast<const T*>(L.w_up), ws.gu + ff, M, ff, d, 2 * ff, false, s));
    VVS_LAUNCH(VVS_PROF_OTHER, launch_silu_mul<T>(ws.gu, act, M, ff, s));
    VVS_LAUNCH(VVS_PROF_GEMM, launch_gemm_nt<T>(act, static_cast<const T*>(L.w_down), ws.x, M, d, ff, d, true, s));
  }
  VVS_LAUNCH(VVS_PROF_OTHER, launch_rmsnorm<T>(ws.x, static_cast<const T*>(ctx->norm_f), hid, M, d, md.rms_eps, s));
  if (cudaGetLastError() != cudaSuccess) return VVS_ERR_CUDA;
  return run_decisions<T>(ctx, hid, Tn, a->n_forced - 1, a->block + a->n_forced, Tn, a, o, true, s);
}

// Tree calls: LM head with guidance over all block rows, probabilities written out, walk of the
// tree on them, then the K/V of the accepted nodes move up behind the forced rows.
int run_tree_decisions(vvs_ctx* ctx, const __nv_bfloat16* hid, const vvs_verify_args* a, const vvs_verify_out* o,
                       cudaStream_t s) {
  const vvs_model_desc& md = ctx->desc;
  Workspace& ws = ctx->ws;
  const int B = a->n_images, C = a->n_cfg, R = B * C, Tn = a->n_forced + a->n_draft_max;
  const int M = R * Tn, V = md.vocab, BT = B * Tn;
  CUtensorMap tm_hid;
  if (make_tmap_bf16_2d(&tm_hid, hid, (uint64_t)M, (uint64_t)md.d_model, (uint32_t)lmhead_box_rows(BT)) != VVS_OK)
    return VVS_ERR_CUDA;
  LmHeadArgs la{};
  la.v = V; la.k = md.d_model; la.bt = BT; la.n_cfg = C; la.tm_a = &ctx->lm_map; la.tm_b = &tm_hid;
  la.pdl = ctx->use_pdl; la.n_sms = ctx->n_sms; la.cfg_scale = a->cfg_scale; la.inv_temp = 1.f / a->temperature;
  la.part_m = ws.part_m; la.part_s = ws.part_s; la.logits_out = o->target_probs; la.status = ws.status;
  la.rows_per_seq = Tn; la.first_row = a->n_forced - 1; la.n_draft_max = 0;
  la.vocab_offset = md.vocab_offset; la.relaxed = 0; la.nbr_k = 1; la.kmax = md.max_nbr_k; la.drafts_ld = Tn;
  la.drafts = a->block + a->n_forced; la.row_ptr = ctx->nbr_row_ptr; la.col = ctx->nbr_col;
  la.l_tok = ws.l_tok; la.l_nbr = ws.l_nbr;
  int rc = VVS_OK;
  VVS_LAUNCH(VVS_PROF_GEMM, rc = launch_lmhead_tc(la, s));
  if (rc != VVS_OK) return rc;
  VVS_LAUNCH(VVS_PROF_OTHER, launch_finalize_stats(ws, (V + 127) / 128, BT, s));
  VVS_LAUNCH(VVS_PROF_OTHER, launch_probs_from_logits(o->target_probs, ws, o->target_probs, BT, V, s));
  TreeParams tp{};
  tp.n_images = B; tp.n_cfg = C; tp.n_forced = a->n_forced; tp.n_draft_max = a->n_draft_max; tp.t_len = Tn;
  tp.vocab = V; tp.vocab_offset = md.vocab_offset; tp.parent = a->tree_parent; tp.drafts = a->block + a->n_forced;
  tp.drafts_ld = Tn;
  tp.probs = o->target_probs; tp.draft_probs = a->draft_probs; tp.uniforms = a->uniforms; tp.cache_len = a->cache_len;
  tp.res = ws.tree_res; tp.accept_len = o->accept_len;
  tp.relaxed = (a->mode == VVS_MODE_RELAXED && a->nbr_k > 1) ? 1 : 0; tp.nbr_k = a->nbr_k; tp.delta = a->delta;
  tp.adjusted = (tp.relaxed && a->adjusted_residual) ? 1 : 0; tp.row_ptr = ctx->nbr_row_ptr; tp.col = ctx->nbr_col;
  tp.accept_path = o->accept_path ? o->accept_path : ws.tree_path;
  tp.next_token = o->next_token; tp.new_len = o->new_len; tp.n_commit = o->n_commit;
  tp.accept_mask = o->accept_mask; tp.margins = o->margins; tp.status = ws.status;
  VVS_LAUNCH(VVS_PROF_OTHER, launch_tree_walk(tp, s));
  if (a->n_draft_max > 0)
    VVS_LAUNCH(VVS_PROF_OTHER, launch_tree_commit(a->kv_k, a->kv_v, a->cache_len, o->accept_len, tp.accept_path, md,
                                                  a->kv_rows, B, C, a->n_forced, a->n_draft_max, s));
  return cudaGetLastError() == cudaSuccess ? VVS_OK : VVS_ERR_CUDA;
}

// bf16 contexts: projections on the tensor cores (gemm_tc.cu), everything else as above.
int run_verify_tc(vvs_ctx* ctx, const vvs_verify_args* a, const vvs_verify_out* o, cudaStream_t s) {
  using T = __nv_bfloat16;
  const vvs_model_desc& md = ctx->desc;
  Workspace& ws = ctx->ws;
  const int B = a->n_images, C = a->n_cfg, R = B * C, Tn = a->n_forced + a->n_draft_max;
  const int M = R * Tn, d = md.d_model, ff = md.d_ff;
  T* kv_k = static_cast<T*>(a->kv_k);
  T* kv_v = static_cast<T*>(a->kv_v);
  T* xn = static_cast<T*>(ws.xn);
  T* q = static_cast<T*>(ws.q);
  T* attn = static_cast<T*>(ws.attn);
  T* act = static_cast<T*>(ws.act);
  T* hid = o->hidden ? static_cast<T*>(o->hidden) : static_cast<T*>(ws.hid);

  const GemmTcPlan p_qkv = plan_gemm_tc(M, 3 * d, d, false, true, ctx->n_sms, (md.deterministic != 0) ? 8 : 32);
  const GemmTcPlan p_o = plan_gemm_tc(M, d, d, false, true, ctx->n_sms, (md.deterministic != 0) ? 8 : 32);
  const GemmTcPlan p_gu = plan_gemm_tc(M, ff, d, true, true, ctx->n_sms);
  const GemmTcPlan p_g1 = plan_gemm_tc(M, ff, d, false, true, ctx->n_sms, (md.deterministic != 0) ? 8 : 32);   // gate and up as two launches
  // "wide": split-K sums into fp32, rotation / attention per (sequence, head), element-wise gate.  Taken
  // above 64 tokens, and by every call of a fixed-order context that the streaming chain kernel does
  // not serve (the fused-epilogue projections below add their splits in arrival order)
  const bool stream_chain = ctx->use_chain_kernels && md.deterministic && ctx->cs_packed && chain_stream_applicable(md, R, Tn);
  // VVS_DEBUG_CHAIN_KERNELS (read at vvs_create) selects the previous generation, kept for comparison
  // and still parity-tested: for calls of at most 32 tokens a persistent whole-chain kernel -- the
  // streaming one (fixed-order contexts) or the split-K tcgen05 one with grid barriers (arrival-order
  // contexts) -- and for 33-64 tokens in arrival-order contexts the fused-epilogue projections with
  // the split-KV attention kernel.  Measured slower than the per-projection kernels below at both
  // benchmark shapes (XL: 1.31 / 1.77 ms against 1.09 / 1.52; 7B: 5.33 / 6.24 against 3.65 / 4.42).
  const bool legacy = ctx->use_chain_kernels && !md.deterministic;
  const bool fused_chain = legacy && fused_chain_applicable(md, R, Tn);
  const bool wide = !stream_chain && !fused_chain && (M > 64 || !legacy);
  // many tokens in a context that asked for fixed-order sums: the K splits of a projection tile are a
  // thread-block cluster (at most 8 CTAs, the portable size) that adds its partial tiles in rank order
  // through distributed shared memory; otherwise the splits add into L2 in arrival order (faster)
  const bool fixed_order = wide && md.deterministic != 0;
  const int cap = fixed_order ? 8 : 32;
  const int cm_store = fixed_order ? 1 : 0, cm_add = fixed_order ? 2 : 0;
  const GemmTcPlan p_down = plan_gemm_tc(M, d, ff, false, true, ctx->n_sms, cap);
  CUtensorMap tm_xn, tm_attn, tm_act, tm_q, tm_k, tm_v;
  const uint64_t kv_total_rows = (uint64_t)md.n_layers * a->kv_rows * md.n_heads * md.s_max;
  if (make_tmap_bf16_2d(&tm_q, q, (uint64_t)M, (uint64_t)d, Tn <= 16 ? 16u : 32u) != VVS_OK ||
      make_tmap_bf16_2d(&tm_k, kv_k, kv_total_rows, (uint64_t)md.head_dim, 128u) != VVS_OK ||
      make_tmap_bf16_2d(&tm_v, kv_v, kv_total_rows, (uint64_t)md.head_dim, 128u) != VVS_OK)
    return VVS_ERR_CUDA;
  AttentionTcArgs at{};
  at.tm_q = &tm_q; at.tm_k = &tm_k; at.tm_v = &tm_v; at.cache_len = a->cache_len; at.anc_mask = ws.anc_mask;
  at.out = attn;
  at.part_o = ws.attn_part_o; at.part_ml = ws.attn_part_ml; at.counters = ws.attn_counters;
  at.status = ws.status; at.d = d; at.n_heads = md.n_heads; at.hd = md.head_dim; at.s_max = md.s_max;
  at.kv_rows = a->kv_rows; at.t_len = Tn; at.n_rows = R; at.pdl = ctx->use_pdl;
  if (make_tmap_bf16_2d(&tm_xn, xn, (uint64_t)M, (uint64_t)d, (uint32_t)p_qkv.nt) != VVS_OK ||
      make_tmap_bf16_2d(&tm_attn, attn, (uint64_t)M, (uint64_t)d, (uint32_t)p_o.nt) != VVS_OK ||
      make_tmap_bf16_2d(&tm_act, act, (uint64_t)M, (uint64_t)ff, (uint32_t)p_down.nt) != VVS_OK)
    return VVS_ERR_CUDA;

  // gate and up as ONE launch (two weight tiles per stage, two accumulators, sums added side by side)
  // when the pair is small enough to be bound by launch latency rather than by its weight stream:
  // measured at 18 tokens 1.097 -> 1.024 ms per step at the XL shape (17.7 MB per pair) and 3.65 ->
  // 3.82 ms at the 7B shape (180 MB per pair); no gain at 288 tokens (several token passes)
  const bool gu_dual = !fixed_order && p_gu.passes == 1 && (size_t)2 * ff * d * sizeof(T) < ((size_t)64 << 20);
  CUtensorMap tm_xn2;
  if (make_tmap_bf16_2d(&tm_xn2, xn, (uint64_t)M, (uint64_t)d, (uint32_t)p_gu.nt) != VVS_OK) return VVS_ERR_CUDA;
  const bool rows_attention = wide && attention_rows_applicable(md, Tn);
  AttentionRowsArgs ar{};
  ar.qkv = ws.qkv; ar.kv_k = kv_k; ar.kv_v = kv_v; ar.cache_len = a->cache_len; ar.rope_cos = ws.rope_cos;
  ar.rope_sin = ws.rope_sin; ar.anc_mask = ws.anc_mask; ar.seq_order = ws.seq_order; ar.out = attn; ar.d = d; ar.n_heads = md.n_heads;
  ar.hd = md.head_dim; ar.s_max = md.s_max; ar.kv_rows = a->kv_rows; ar.t_len = Tn; ar.n_rows = R; ar.n_sms = ctx->n_sms; ar.pdl = ctx->use_pdl;

  GemmTcArgs base{};
  base.m = M; base.pdl = ctx->use_pdl; base.status = ws.status;
  base.scratch = ws.sk_scratch; base.counters = ws.sk_counters;
  base.q = q; base.kv_k = kv_k; base.kv_v = kv_v; base.slot_pos = ws.slot_pos;
  base.rope_cos = ws.rope_cos; base.rope_sin = ws.rope_sin;
  base.d = d; base.n_heads = md.n_heads; base.hd = md.head_dim; base.s_max = md.s_max;
  base.kv_rows = a->kv_rows; base.t_len = Tn; base.act = act; base.ff = ff;

  int rc = VVS_OK;
  if (stream_chain) {
    // at most 32 tokens: embedding and every decoder layer run as one persistent dataflow kernel
    CUtensorMap ck, cv;
    const uint32_t kb = (uint32_t)chain_stream_kb(md);
    if (make_tmap_bf16_2d(&ck, kv_k, kv_total_rows, (uint64_t)md.head_dim, kb) != VVS_OK ||
        make_tmap_bf16_2d(&cv, kv_v, kv_total_rows, (uint64_t)md.head_dim, kb) != VVS_OK)
      return VVS_ERR_CUDA;
    ChainStreamArgs cs{};
    cs.md = &md; cs.n_rows = R; cs.n_images = B; cs.t_len = Tn; cs.kv_rows = a->kv_rows;
    cs.plan = &ctx->cs_plan; cs.d_plan = ctx->cs_d_plan; cs.packed = ctx->cs_packed;
    cs.norms_host = ctx->chain_norms.data();
    cs.tok_emb = static_cast<const T*>(ctx->tok_emb); cs.block = a->block;
    cs.x = ws.x; cs.xn1 = static_cast<T*>(ws.cs_xn1); cs.xn2 = static_cast<T*>(ws.cs_xn2); cs.qbuf = q;
    cs.attn = static_cast<T*>(ws.cs_attn); cs.act = static_cast<T*>(ws.cs_act);
    cs.ss1 = ws.cs_ss1; cs.ss2 = ws.cs_ss2;
    cs.cache_len = a->cache_len; cs.kv_k = kv_k; cs.kv_v = kv_v; cs.tm_k = &ck; cs.tm_v = &cv;
    cs.slot_pos = ws.slot_pos; cs.anc_mask = ws.anc_mask; cs.rope_cos = ws.rope_cos; cs.rope_sin = ws.rope_sin;
    cs.flags = ws.cs_flags; cs.status = ws.status;
    VVS_LAUNCH(VVS_PROF_OTHER, launch_rope_table(a->cache_len, a->tree_parent, B, a->n_forced, ws, md, R, Tn, s,
                                                 ws.cs_flags, (int)chain_stream_flag_words(md)));
    VVS_LAUNCH(VVS_PROF_CHAIN, rc = launch_chain_stream(cs, s));
    if (rc != VVS_OK) return rc;
    VVS_LAUNCH(VVS_PROF_OTHER, launch_rmsnorm<T>(ws.x, static_cast<const T*>(ctx->norm_f), hid, M, d, md.rms_eps, s));
    if (cudaGetLastError() != cudaSuccess) return VVS_ERR_CUDA;
    if (a->tree_parent) return run_tree_decisions(ctx, hid, a, o, s);
    return run_decisions<T>(ctx, hid, Tn, a->n_forced - 1, a->block + a->n_forced, Tn, a, o, true, s);
  }
  if (fused_chain) {
    // at most 32 tokens: the whole decoder chain runs as one persistent kernel
    FusedChainArgs fc{};
    fc.md = &md; fc.n_rows = R; fc.n_images = B; fc.t_len = Tn; fc.kv_rows = a->kv_rows; fc.n_sms = ctx->n_sms;
    fc.wmaps = ws.chain_wmaps; fc.norms_host = ctx->chain_norms.data();
    fc.tok_emb = static_cast<const T*>(ctx->tok_emb); fc.block = a->block;
    fc.x = ws.x; fc.qkv_acc = ws.chain_qkv; fc.gu_acc = ws.chain_gu; fc.ss = ws.chain_ss;
    fc.cache_len = a->cache_len; fc.kv_k = kv_k; fc.kv_v = kv_v; fc.tm_k = &tm_k; fc.tm_v = &tm_v;
    fc.slot_pos = ws.slot_pos; fc.anc_mask = ws.anc_mask; fc.rope_cos = ws.rope_cos; fc.rope_sin = ws.rope_sin;
    fc.part_o = ws.attn_part_o; fc.part_ml = ws.attn_part_ml; fc.sync_words = ws.chain_sync;
    fc.status = ws.status;
    VVS_LAUNCH(VVS_PROF_OTHER, launch_rope_table(a->cache_len, a->tree_parent, B, a->n_forced, ws, md, R, Tn, s));
    VVS_LAUNCH(VVS_PROF_CHAIN, rc = launch_fused_chain(fc, s));
    if (rc != VVS_OK) return rc;
    VVS_LAUNCH(VVS_PROF_OTHER, launch_rmsnorm<T>(ws.x, static_cast<const T*>(ctx->norm_f), hid, M, d, md.rms_eps, s));
    if (cudaGetLastError() != cudaSuccess) return VVS_ERR_CUDA;
    if (a->tree_parent) return run_tree_decisions(ctx, hid, a, o, s);
    return run_decisions<T>(ctx, hid, Tn, a->n_forced - 1, a->block + a->n_forced, Tn, a, o, true, s);
  }
  VVS_LAUNCH(VVS_PROF_OTHER, launch_embed<T>(static_cast<const T*>(ctx->tok_emb), a->block, ws.x, B, C, Tn,
                                             d, md.tok_rows, ws.status, s));
  VVS_LAUNCH(VVS_PROF_OTHER, launch_rope_table(a->cache_len, a->tree_parent, B, a->n_forced, ws, md, R, Tn, s));
  if (wide) {
    // the split-K sums of the QKV and gate / up projections are added into these buffers; the
    // kernels that consume them clear what they read, so one clearing per call is enough (it also
    // covers a previous call that ended early)
    if (cudaMemsetAsync(ws.qkv, 0, (size_t)M * 3 * d * sizeof(float), s) != cudaSuccess ||
        cudaMemsetAsync(ws.gu, 0, (size_t)M * 2 * ff * sizeof(float), s) != cudaSuccess)
      return VVS_ERR_CUDA;
  }
  for (int l = 0; l < md.n_layers && rc == VVS_OK; ++l) {
    const Layer& L = ctx->layers[l];
    const LayerMaps& W = ctx->layer_maps[l];
    // many rows: the warp-per-row norm, launched as a programmatic dependent of the projection before it
    const bool rows_norm = wide && d % 8 == 0;
    if (rows_norm)
      VVS_LAUNCH(VVS_PROF_OTHER, launch_rmsnorm_rows(ws.x, static_cast<const __nv_bfloat16*>(L.norm1), xn, M, d, md.rms_eps, ctx->use_pdl && l > 0, s));
    else
      VVS_LAUNCH(VVS_PROF_OTHER, launch_rmsnorm<T>(ws.x, static_cast<const T*>(L.norm1), xn, M, d, md.rms_eps, s));
    if (wide) {
      // many tokens: a per-thread epilogue over hundreds of tokens is slower than a plain split-K
      // sum into fp32 followed by one thread per element for rotation, rounding and cache append
      GemmTcArgs g = base;
      g.n = 3 * d; g.k = d; g.tm_a = &W.w_qkv; g.tm_b = &tm_xn; g.out = ws.qkv; g.ldo = 3 * d;
      g.cluster_mode = cm_store;
      VVS_LAUNCH(VVS_PROF_GEMM, rc = launch_gemm_tc(GEMM_EPI_ADD, p_qkv, g, s));
      if (rows_attention) {
        // rotation, rounding, cache append and attention of each (sequence, head) in one kernel
        ar.layer = l;
        if (rc == VVS_OK) VVS_LAUNCH(VVS_PROF_ATTENTION, rc = launch_attention_rows(ar, s));
      } else {
        VVS_LAUNCH(VVS_PROF_OTHER, launch_rope_append<T>(ws.qkv, ws.rope_inv_freq, q, kv_k, kv_v, a->cache_len, md,
                                                         l, a->kv_rows, R, Tn, ws.status, s,
                                                         a->tree_parent ? ws.rope_cos : nullptr,
                                                         a->tree_parent ? ws.rope_sin : nullptr, true));
      }
    } else {
      GemmTcArgs g = base;
      g.n = 3 * d; g.k = d; g.tm_a = &W.w_qkv; g.tm_b = &tm_xn; g.ld_scratch = 3 * d; g.layer = l;
      VVS_LAUNCH(VVS_PROF_GEMM, rc = launch_gemm_tc(GEMM_EPI_QKV, p_qkv, g, s));
    }
    if (rc == VVS_OK && !(wide && rows_attention)) {
      at.layer = l;
      VVS_LAUNCH(VVS_PROF_ATTENTION, rc = launch_attention_tc(at, s));
    }
    if (rc == VVS_OK) {
      GemmTcArgs g = base;
      g.n = d; g.k = d; g.tm_a = &W.w_o; g.tm_b = &tm_attn; g.out = ws.x; g.ldo = d;
      g.cluster_mode = cm_add;
      VVS_LAUNCH(VVS_PROF_GEMM, rc = launch_gemm_tc(GEMM_EPI_ADD, p_o, g, s));
    }
    if (rows_norm)
      VVS_LAUNCH(VVS_PROF_OTHER, launch_rmsnorm_rows(ws.x, static_cast<const __nv_bfloat16*>(L.norm2), xn, M, d, md.rms_eps, ctx->use_pdl, s));
    else
      VVS_LAUNCH(VVS_PROF_OTHER, launch_rmsnorm<T>(ws.x, static_cast<const T*>(L.norm2), xn, M, d, md.rms_eps, s));
    if (rc == VVS_OK && wide && gu_dual) {
      GemmTcArgs g = base;
      g.n = ff; g.k = d; g.tm_a = &W.w_gate; g.tm_a2 = &W.w_up; g.tm_b = &tm_xn2; g.out = ws.gu; g.ldo = 2 * ff;
      VVS_LAUNCH(VVS_PROF_GEMM, rc = launch_gemm_tc(GEMM_EPI_ADD2, p_gu, g, s));
      VVS_LAUNCH(VVS_PROF_OTHER, launch_silu_mul<T>(ws.gu, act, M, ff, s, true, ctx->use_pdl));
    } else if (rc == VVS_OK && wide) {
      GemmTcArgs g = base;
      g.n = ff; g.k = d; g.tm_a = &W.w_gate; g.tm_b = &tm_xn; g.out = ws.gu; g.ldo = 2 * ff;
      g.cluster_mode = cm_store;
      VVS_LAUNCH(VVS_PROF_GEMM, rc = launch_gemm_tc(GEMM_EPI_ADD, p_g1, g, s));
      g.tm_a = &W.w_up; g.out = ws.gu + ff;
      if (rc == VVS_OK) VVS_LAUNCH(VVS_PROF_GEMM, rc = launch_gemm_tc(GEMM_EPI_ADD, p_g1, g, s));
      VVS_LAUNCH(VVS_PROF_OTHER, launch_silu_mul<T>(ws.gu, act, M, ff, s, true, ctx->use_pdl));
    } else if (rc == VVS_OK) {
      GemmTcArgs g = base;
      g.n = ff; g.k = d; g.tm_a = &W.w_gate; g.tm_a2 = &W.w_up; g.tm_b = &tm_xn; g.ld_scratch = 2 * ff;
      VVS_LAUNCH(VVS_PROF_GEMM, rc = launch_gemm_tc(GEMM_EPI_SWIGLU, p_gu, g, s));
    }
    if (rc == VVS_OK) {
      GemmTcArgs g = base;
      g.n = d; g.k = ff; g.tm_a = &W.w_down; g.tm_b = &tm_act; g.out = ws.x; g.ldo = d;
      g.cluster_mode = cm_add;
      VVS_LAUNCH(VVS_PROF_GEMM, rc = launch_gemm_tc(GEMM_EPI_ADD, p_down, g, s));
    }
  }
  if (rc != VVS_OK) return rc;
  if (wide && d % 8 == 0)
    VVS_LAUNCH(VVS_PROF_OTHER, launch_rmsnorm_rows(ws.x, static_cast<const __nv_bfloat16*>(ctx->norm_f), hid, M, d, md.rms_eps, ctx->use_pdl, s));
  else
    VVS_LAUNCH(VVS_PROF_OTHER, launch_rmsnorm<T>(ws.x, static_cast<const T*>(ctx->norm_f), hid, M, d, md.rms_eps, s));
  if (cudaGetLastError() != cudaSuccess) return VVS_ERR_CUDA;
  if (a->tree_parent) return run_tree_decisions(ctx, hid, a, o, s);
  return run_decisions<T>(ctx, hid, Tn, a->n_forced - 1, a->block + a->n_forced, Tn, a, o, true, s);
}

int enqueue_verify(vvs_ctx* ctx, const vvs_verify_args* a, const vvs_verify_out* o, cudaStream_t s) {
  if (ctx->tensor_core_path) return run_verify_tc(ctx, a, o, s);
  return ctx->desc.dtype == VVS_DTYPE_BF16 ? run_verify<__nv_bfloat16>(ctx, a, o, s)
                                           : run_verify<float>(ctx, a, o, s);
}

// The step is ~150-270 small kernels; launching them one by one costs more host time than the
// GPU needs to run them.  Each distinct argument set is therefore captured once into a CUDA graph
// (on a private stream, so the caller may use the legacy default stream) and replayed afterwards.
int verify_via_graph(vvs_ctx* ctx, const vvs_verify_args* a, const vvs_verify_out* o, cudaStream_t s) {
  // the key is built field by field into zeroed storage: padding bytes of the caller's structs
  // must not make two equal calls look different
  vvs_verify_args ka;
  std::memset(&ka, 0, sizeof(ka));
  ka.n_images = a->n_images; ka.n_cfg = a->n_cfg; ka.n_forced = a->n_forced; ka.n_draft_max = a->n_draft_max;
  ka.block = a->block; ka.n_draft = a->n_draft; ka.kv_k = a->kv_k; ka.kv_v = a->kv_v; ka.kv_rows = a->kv_rows;
  ka.cache_len = a->cache_len;   // cache_len_host: host-side validation only, not part of the device work
  ka.draft_probs = a->draft_probs; ka.uniforms = a->uniforms; ka.cfg_scale = a->cfg_scale;
  ka.temperature = a->temperature; ka.mode = a->mode; ka.nbr_k = a->nbr_k; ka.delta = a->delta;
  ka.tree_parent = a->tree_parent; ka.adjusted_residual = a->adjusted_residual;
  std::vector<unsigned char> key(sizeof(ka) + sizeof(*o));
  std::memcpy(key.data(), &ka, sizeof(ka));
  std::memcpy(key.data() + sizeof(ka), o, sizeof(*o));   // nine pointers, no padding
  ++ctx->graph_clock;
  for (auto& g : ctx->graphs) {
    if (g.key == key) {
      g.last_use = ctx->graph_clock;
      ctx->launches = g.launches;
      return cudaGraphLaunch(g.exec, s) == cudaSuccess ? VVS_OK : VVS_ERR_CUDA;
    }
  }
  cudaGraph_t graph = nullptr;
  if (cudaStreamBeginCapture(ctx->capture_stream, cudaStreamCaptureModeThreadLocal) != cudaSuccess) {
    cudaGetLastError();
    ctx->use_graph = false;
    ctx->launches = 0;
    return enqueue_verify(ctx, a, o, s);
  }
  ctx->launches = 0;
  const int rc = enqueue_verify(ctx, a, o, ctx->capture_stream);
  const cudaError_t e = cudaStreamEndCapture(ctx->capture_stream, &graph);
  cudaGraphExec_t exec = nullptr;
  if (rc != VVS_OK || e != cudaSuccess || !graph ||
      cudaGraphInstantiate(&exec, graph, 0) != cudaSuccess) {
    cudaGetLastError();
    if (graph) cudaGraphDestroy(graph);
    ctx->use_graph = false;  // capture is not available here: fall back to plain launches
    ctx->launches = 0;
    return enqueue_verify(ctx, a, o, s);
  }
  cudaGraphDestroy(graph);
  if (ctx->graphs.size() >= 64) {  // evict the least recently used entry
    size_t victim = 0;
    for (size_t i = 1; i < ctx->graphs.size(); ++i)
      if (ctx->graphs[i].last_use < ctx->graphs[victim].last_use) victim = i;
    cudaGraphExecDestroy(ctx->graphs[victim].exec);
    ctx->graphs.erase(ctx->graphs.begin() + victim);
  }
  GraphEntry ge;
  ge.key = std::move(key);
  ge.exec = exec;
  ge.launches = ctx->launches;
  ge.last_use = ctx->graph_clock;
  ctx->graphs.push_back(std::move(ge));
  return cudaGraphLaunch(exec, s) == cudaSuccess ? VVS_OK : VVS_ERR_CUDA;
}

int check_decision_args(const vvs_ctx* ctx, const vvs_verify_args* a, const vvs_verify_out* o,
                        int rows_per_seq) {
  const vvs_model_desc& md = ctx->desc;
  if (!a || !o) return VVS_ERR_INVALID_ARG;
  if (!ctx->weights_bound) return VVS_ERR_NOT_BOUND;
  if (a->n_images < 1 || (a->n_cfg != 1 && a->n_cfg != 2) || a->n_draft_max < 0) return VVS_ERR_SHAPE;
  if (a->n_images * a->n_cfg > md.max_rows || rows_per_seq > md.max_block || rows_per_seq < 1)
    return VVS_ERR_SHAPE;
  if (!a->uniforms || !o->accept_len || !o->next_token) return VVS_ERR_INVALID_ARG;
  if (a->n_draft_max > 0 && !a->draft_probs) return VVS_ERR_INVALID_ARG;
  if (!(a->temperature > 0.f) || !std::isfinite(a->temperature) || !std::isfinite(a->cfg_scale))
    return VVS_ERR_INVALID_ARG;
  if (a->mode != VVS_MODE_STRICT && a->mode != VVS_MODE_RELAXED) return VVS_ERR_INVALID_ARG;
  if (a->adjusted_residual != 0 && a->adjusted_residual != 1) return VVS_ERR_INVALID_ARG;
  if (a->mode == VVS_MODE_RELAXED) {
    if (a->nbr_k < 1 || a->nbr_k > md.max_nbr_k) return VVS_ERR_SHAPE;
    if (!(a->delta >= 0.f)) return VVS_ERR_INVALID_ARG;  // also rejects NaN
    if (a->nbr_k > 1 && (!ctx->nbr_row_ptr || !ctx->nbr_col)) return VVS_ERR_NOT_BOUND;
  }
  if (!aligned16(a->draft_probs) || !aligned16(o->target_probs)) return VVS_ERR_ALIGN;
  return VVS_OK;
}

}  // namespace

extern "C" {

int vvs_workspace_bytes(const vvs_model_desc* desc, size_t* out_bytes) {
  int rc = check_desc(desc);
  if (rc != VVS_OK) return rc;
  if (!out_bytes) return VVS_ERR_INVALID_ARG;
  Workspace tmp;
  *out_bytes = layout(*desc, tmp, nullptr);
  return VVS_OK;
}

int vvs_create(const vvs_model_desc* desc, vvs_ctx** out) {
  if (out) *out = nullptr;
  int rc = check_desc(desc);
  if (rc != VVS_OK) return rc;
  if (!out) return VVS_ERR_INVALID_ARG;
  vvs_ctx* ctx = new (std::nothrow) vvs_ctx();
  if (!ctx) return VVS_ERR_NOMEM;
  ctx->desc = *desc;
  if (cudaGetDevice(&ctx->device) != cudaSuccess) { delete ctx; return VVS_ERR_CUDA; }
  Workspace tmp;
  ctx->arena_bytes = layout(*desc, tmp, nullptr);
  if (cudaMalloc(&ctx->arena, ctx->arena_bytes) != cudaSuccess) {
    cudaGetLastError();
    delete ctx;
    return VVS_ERR_NOMEM;
  }
  layout(*desc, ctx->ws, static_cast<char*>(ctx->arena));
  if (cudaMemset(ctx->arena, 0, ctx->arena_bytes) != cudaSuccess) { vvs_destroy(ctx); return VVS_ERR_CUDA; }
  // rotation angle per unit coordinate of each consecutive pair
  const int half = desc->head_dim / 2;
  if (half > 0) {
    float* f = static_cast<float*>(std::malloc(sizeof(float) * half));
    if (!f) { vvs_destroy(ctx); return VVS_ERR_NOMEM; }
    for (int i = 0; i < half; ++i) {
      if (desc->rope_mode == VVS_ROPE_2D_GRID) {
        int j = i % (half / 2);
        f[i] = (float)std::pow((double)desc->rope_base, -2.0 * j / (double)half);
      } else {
        f[i] = (float)std::pow((double)desc->rope_base, -2.0 * i / (double)desc->head_dim);
      }
    }
    cudaError_t e = cudaMemcpy(ctx->ws.rope_inv_freq, f, sizeof(float) * half, cudaMemcpyHostToDevice);
    std::free(f);
    if (e != cudaSuccess) { vvs_destroy(ctx); return VVS_ERR_CUDA; }
  }
  if (desc->n_layers > 0) {
    ctx->layers = new (std::nothrow) Layer[desc->n_layers]();
    ctx->layer_maps = new (std::nothrow) LayerMaps[desc->n_layers]();
    if (!ctx->layers || !ctx->layer_maps) { vvs_destroy(ctx); return VVS_ERR_NOMEM; }
  }
  // Debug switches only: VVS_DEBUG_GENERIC runs bf16 contexts on the generic kernels,
  // VVS_DEBUG_NO_PDL launches the tensor-core GEMMs without programmatic dependent launch,
  // VVS_DEBUG_NO_CHAIN runs small calls through the per-projection kernels too.
  ctx->tensor_core_path = desc->dtype == VVS_DTYPE_BF16 && !std::getenv("VVS_DEBUG_GENERIC");
  ctx->use_pdl = !std::getenv("VVS_DEBUG_NO_PDL");
  ctx->use_graph = !std::getenv("VVS_DEBUG_NO_GRAPH");
  ctx->use_chain_kernels = std::getenv("VVS_DEBUG_CHAIN_KERNELS") != nullptr;
  if (cudaStreamCreateWithFlags(&ctx->capture_stream, cudaStreamNonBlocking) != cudaSuccess) {
    cudaGetLastError();
    ctx->capture_stream = nullptr;
    ctx->use_graph = false;
  }
  if (cudaDeviceGetAttribute(&ctx->n_sms, cudaDevAttrMultiProcessorCount, ctx->device) != cudaSuccess ||
      ctx->n_sms < 1)
    ctx->n_sms = 148;
  if (ctx->tensor_core_path && desc->n_layers > 0 && chain_stream_configure() != VVS_OK) {
    cudaGetLastError();
    ctx->use_chain_kernels = false;
  }
  *out = ctx;
  return VVS_OK;
}

static void drop_graphs(vvs_ctx* ctx) {
  for (auto& g : ctx->graphs)
    if (g.exec) cudaGraphExecDestroy(g.exec);
  ctx->graphs.clear();
}

int vvs_destroy(vvs_ctx* ctx) {
  if (!ctx) return VVS_ERR_INVALID_ARG;
  vvs_profile_enable(ctx, 0);
  drop_graphs(ctx);
  if (ctx->capture_stream) cudaStreamDestroy(ctx->capture_stream);
  if (ctx->arena) cudaFree(ctx->arena);
  if (ctx->cs_packed) cudaFree(ctx->cs_packed);
  if (ctx->cs_d_plan) cudaFree(ctx->cs_d_plan);
  delete[] ctx->layers;
  delete[] ctx->layer_maps;
  delete ctx;
  return VVS_OK;
}

int vvs_bind_weights(vvs_ctx* ctx, const vvs_weights* w) {
  if (!ctx || !w) return VVS_ERR_INVALID_ARG;
  const int n = ctx->desc.n_layers;
  if (!w->w_lm) return VVS_ERR_INVALID_ARG;
  if (!aligned16(w->w_lm)) return VVS_ERR_ALIGN;
  if (n > 0) {
    if (!w->tok_emb || !w->norm_f || !w->layers) return VVS_ERR_INVALID_ARG;
    if (!aligned16(w->tok_emb) || !aligned16(w->norm_f)) return VVS_ERR_ALIGN;
    for (int l = 0; l < n; ++l) {
      const vvs_layer_weights& s = w->layers[l];
      const void* ptrs[7] = {s.w_qkv, s.w_o, s.w_gate, s.w_up, s.w_down, s.norm1, s.norm2};
      for (const void* p : ptrs) {
        if (!p) return VVS_ERR_INVALID_ARG;
        if (!aligned16(p)) return VVS_ERR_ALIGN;
      }
    }
    for (int l = 0; l < n; ++l) {
      const vvs_layer_weights& s = w->layers[l];
      ctx->layers[l] = Layer{s.w_qkv, s.w_o, s.w_gate, s.w_up, s.w_down, s.norm1, s.norm2};
    }
  }
  if (ctx->tensor_core_path) {
    const vvs_model_desc& md = ctx->desc;
    const int d = md.d_model, ff = md.d_ff;
    int rc = VVS_OK;
    for (int l = 0; l < n && rc == VVS_OK; ++l) {
      const vvs_layer_weights& s = w->layers[l];
      LayerMaps& m = ctx->layer_maps[l];
      rc = make_weight_tmap(&m.w_qkv, s.w_qkv, 3 * d, d);
      if (rc == VVS_OK) rc = make_weight_tmap(&m.w_o, s.w_o, d, d);
      if (rc == VVS_OK) rc = make_weight_tmap(&m.w_gate, s.w_gate, ff, d);
      if (rc == VVS_OK) rc = make_weight_tmap(&m.w_up, s.w_up, ff, d);
      if (rc == VVS_OK) rc = make_weight_tmap(&m.w_down, s.w_down, d, ff);
    }
    if (rc == VVS_OK)
      rc = make_weight_tmap(&ctx->lm_map,
                            static_cast<const __nv_bfloat16*>(w->w_lm) + (size_t)md.vocab_offset * d,
                            md.vocab, d);
    if (rc != VVS_OK) return rc;
    if (n > 0) {
      // device copies for the whole-chain kernel, which walks all layers inside one launch
      static_assert(sizeof(LayerMaps) == 5 * sizeof(CUtensorMap), "LayerMaps is five descriptors");
      ctx->chain_norms.resize(2 * (size_t)n);
      for (int l = 0; l < n; ++l) {
        ctx->chain_norms[2 * l] = static_cast<const __nv_bfloat16*>(w->layers[l].norm1);
        ctx->chain_norms[2 * l + 1] = static_cast<const __nv_bfloat16*>(w->layers[l].norm2);
      }
      if (cudaMemcpy(ctx->ws.chain_wmaps, ctx->layer_maps, (size_t)n * sizeof(LayerMaps),
                     cudaMemcpyHostToDevice) != cudaSuccess)
        return VVS_ERR_CUDA;
      // private copy of the layer weights in the streaming order of the chain kernel
      if (ctx->cs_packed) { cudaFree(ctx->cs_packed); ctx->cs_packed = nullptr; }
      if (ctx->cs_d_plan) { cudaFree(ctx->cs_d_plan); ctx->cs_d_plan = nullptr; }
      if (ctx->use_chain_kernels && md.deterministic && chain_stream_applicable(md, 1, 1) &&
          chain_stream_plan(md, ctx->n_sms, ctx->cs_plan)) {
        const size_t pbytes = chain_stream_packed_bytes(md, ctx->cs_plan);
        const size_t plbytes = ctx->cs_plan.cta.size() * sizeof(ChainCtaPlan);
        if (cudaMalloc(&ctx->cs_packed, pbytes) != cudaSuccess ||
            cudaMalloc(reinterpret_cast<void**>(&ctx->cs_d_plan), plbytes) != cudaSuccess) {
          cudaGetLastError();
          if (ctx->cs_packed) { cudaFree(ctx->cs_packed); ctx->cs_packed = nullptr; }
          return VVS_ERR_NOMEM;
        }
        if (cudaMemcpy(ctx->cs_d_plan, ctx->cs_plan.cta.data(), plbytes, cudaMemcpyHostToDevice) != cudaSuccess)
          return VVS_ERR_CUDA;
        rc = chain_stream_pack(md, ctx->cs_plan, ctx->cs_d_plan, ctx->layers, ctx->cs_packed, nullptr);
        if (rc != VVS_OK || cudaDeviceSynchronize() != cudaSuccess) return VVS_ERR_CUDA;
      }
    }
  }
  drop_graphs(ctx);  // captured steps hold the old pointers
  ctx->tok_emb = w->tok_emb;
  ctx->norm_f = w->norm_f;
  ctx->w_lm = w->w_lm;
  ctx->weights_bound = true;
  return VVS_OK;
}

int vvs_bind_neighbors(vvs_ctx* ctx, const int32_t* row_ptr, const int32_t* col, int64_t nnz) {
  if (!ctx || !row_ptr || !col || nnz < 0) return VVS_ERR_INVALID_ARG;
  if (!aligned16(row_ptr) || !aligned16(col)) return VVS_ERR_ALIGN;
  drop_graphs(ctx);
  ctx->nbr_row_ptr = row_ptr;
  ctx->nbr_col = col;
  ctx->nbr_nnz = nnz;
  return VVS_OK;
}

int vvs_verify(vvs_ctx* ctx, const vvs_verify_args* a, const vvs_verify_out* o, void* stream) {
  if (!ctx) return VVS_ERR_INVALID_ARG;
  const vvs_model_desc& md = ctx->desc;
  if (md.n_layers < 1) return VVS_ERR_SHAPE;
  if (!a || !o) return VVS_ERR_INVALID_ARG;
  if (a->n_forced < 1) return VVS_ERR_SHAPE;
  const int Tn = a->n_forced + a->n_draft_max;
  int rc = check_decision_args(ctx, a, o, Tn);
  if (rc != VVS_OK) return rc;
  const int R = a->n_images * a->n_cfg;
  if (!a->block || !a->kv_k || !a->kv_v || !a->cache_len || !o->new_len) return VVS_ERR_INVALID_ARG;
  if (a->kv_rows < R) return VVS_ERR_SHAPE;
  if (a->tree_parent) {
    if (a->n_draft || !o->target_probs) return VVS_ERR_INVALID_ARG;
    if (!ctx->tensor_core_path) return VVS_ERR_SHAPE;     // Tn <= 32 = max_block holds for every call
  } else if (o->accept_path) {
    return VVS_ERR_INVALID_ARG;
  }
  if (!aligned16(a->kv_k) || !aligned16(a->kv_v) || !aligned16(o->hidden)) return VVS_ERR_ALIGN;
  if (a->cache_len_host) {
    for (int r = 0; r < R; ++r)
      if (a->cache_len_host[r] < 0 || a->cache_len_host[r] + Tn > md.s_max) return VVS_ERR_CAPACITY;
  }
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
  if (ctx->use_graph && !ctx->profiling &&
      cudaStreamIsCapturing(s, &cap) == cudaSuccess && cap == cudaStreamCaptureStatusNone)
    return verify_via_graph(ctx, a, o, s);
  ctx->launches = 0;
  return enqueue_verify(ctx, a, o, s);
}

int vvs_epilogue(vvs_ctx* ctx, const void* hidden, int32_t n_rows_per_seq, int32_t first_row,
                 const int32_t* drafts, const vvs_verify_args* a, const vvs_verify_out* o,
                 void* stream) {
  if (!ctx || !hidden) return VVS_ERR_INVALID_ARG;
  int rc = check_decision_args(ctx, a, o, n_rows_per_seq);
  if (rc != VVS_OK) return rc;
  if (first_row < 0 || first_row + a->n_draft_max > n_rows_per_seq) return VVS_ERR_SHAPE;
  if (a->n_draft_max > 0 && !drafts) return VVS_ERR_INVALID_ARG;
  if (o->new_len || o->hidden || a->tree_parent || o->accept_path) return VVS_ERR_INVALID_ARG;
  if (!aligned16(hidden)) return VVS_ERR_ALIGN;
  ctx->launches = 0;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (ctx->desc.dtype == VVS_DTYPE_BF16)
    return run_decisions<__nv_bfloat16>(ctx, static_cast<const __nv_bfloat16*>(hidden), n_rows_per_seq,
                                        first_row, drafts, a->n_draft_max, a, o, false, s);
  return run_decisions<float>(ctx, static_cast<const float*>(hidden), n_rows_per_seq, first_row, drafts,
                              a->n_draft_max, a, o, false, s);
}

int vvs_decide(vvs_ctx* ctx, const float* target_probs, int32_t n_rows_per_seq, int32_t first_row,
               const int32_t* drafts, const vvs_verify_args* a, const vvs_verify_out* o, void* stream) {
  if (!ctx || !target_probs || !a || !o) return VVS_ERR_INVALID_ARG;
  if (a->n_cfg != 1) return VVS_ERR_SHAPE;  // probabilities are already guided
  const bool was_bound = ctx->weights_bound;
  ctx->weights_bound = true;                // no weights are read on this path
  int rc = check_decision_args(ctx, a, o, n_rows_per_seq);
  ctx->weights_bound = was_bound;
  if (rc != VVS_OK) return rc;
  if (first_row < 0 || first_row + a->n_draft_max > n_rows_per_seq) return VVS_ERR_SHAPE;
  if (a->n_draft_max > 0 && !drafts) return VVS_ERR_INVALID_ARG;
  if (o->new_len || o->hidden || o->n_commit || o->target_probs) return VVS_ERR_INVALID_ARG;
  if (!a->tree_parent && o->accept_path) return VVS_ERR_INVALID_ARG;
  if (!aligned16(target_probs)) return VVS_ERR_ALIGN;
  ctx->launches = 0;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  Workspace& ws = ctx->ws;
  if (a->tree_parent) {
    // the tree walk on the caller's rows: block rows 0 .. first_row are the forced chain
    if (a->n_draft || !ws.tree_res) return VVS_ERR_INVALID_ARG;
    if (first_row + 1 + a->n_draft_max != n_rows_per_seq) return VVS_ERR_SHAPE;
    TreeParams tp{};
    tp.n_images = a->n_images; tp.n_cfg = 1; tp.n_forced = first_row + 1; tp.n_draft_max = a->n_draft_max;
    tp.t_len = n_rows_per_seq; tp.vocab = ctx->desc.vocab; tp.vocab_offset = ctx->desc.vocab_offset;
    tp.parent = a->tree_parent; tp.drafts = drafts; tp.drafts_ld = a->n_draft_max; tp.probs = target_probs;
    tp.draft_probs = a->draft_probs; tp.uniforms = a->uniforms; tp.res = ws.tree_res;
    tp.relaxed = (a->mode == VVS_MODE_RELAXED && a->nbr_k > 1) ? 1 : 0; tp.nbr_k = a->nbr_k; tp.delta = a->delta;
    tp.adjusted = (tp.relaxed && a->adjusted_residual) ? 1 : 0; tp.row_ptr = ctx->nbr_row_ptr; tp.col = ctx->nbr_col;
    tp.accept_len = o->accept_len; tp.accept_path = o->accept_path ? o->accept_path : ws.tree_path;
    tp.next_token = o->next_token; tp.accept_mask = o->accept_mask; tp.margins = o->margins; tp.status = ws.status;
    VVS_LAUNCH(VVS_PROF_OTHER, launch_tree_walk(tp, s));
    return cudaGetLastError() == cudaSuccess ? VVS_OK : VVS_ERR_CUDA;
  }
  DecideParams p = decide_params(ctx, n_rows_per_seq, first_row, drafts, a->n_draft_max, a, o, false);
  p.direct_probs = target_probs;
  if (p.n_draft_max > 0) VVS_LAUNCH(VVS_PROF_OTHER, launch_gather_logits(target_probs, ws, p, s));
  VVS_LAUNCH(VVS_PROF_OTHER, launch_accept(ws, p, s));
  if (p.adjusted) VVS_LAUNCH(VVS_PROF_OTHER, launch_adjust_target(ws, p, s));   // copies the row, then adjusts it
  VVS_LAUNCH(VVS_PROF_OTHER, launch_residual_mass(ws, p, s));
  VVS_LAUNCH(VVS_PROF_OTHER, launch_sample(ws, p, s));
  return cudaGetLastError() == cudaSuccess ? VVS_OK : VVS_ERR_CUDA;
}

static int check_fcache(const vvs_ctx* ctx, const vvs_fcache* fc) {
  if (!ctx || !fc) return VVS_ERR_INVALID_ARG;
  if (!fc->feat || !fc->fpos || !fc->newest) return VVS_ERR_INVALID_ARG;
  if (fc->n_rows < 1 || fc->cap < 1) return VVS_ERR_SHAPE;
  if (!aligned16(fc->feat)) return VVS_ERR_ALIGN;
  return VVS_OK;
}

int vvs_feature_cache_reset(vvs_ctx* ctx, const vvs_fcache* fc, void* stream) {
  int rc = check_fcache(ctx, fc);
  if (rc != VVS_OK) return rc;
  launch_fcache_reset(*fc, static_cast<cudaStream_t>(stream));
  return cudaGetLastError() == cudaSuccess ? VVS_OK : VVS_ERR_CUDA;
}

int vvs_feature_cache_store(vvs_ctx* ctx, const vvs_fcache* fc, const void* hidden,
                            int32_t n_rows_per_seq, const int32_t* base_pos, const int32_t* n_store,
                            void* stream) {
  int rc = check_fcache(ctx, fc);
  if (rc != VVS_OK) return rc;
  if (!hidden || !base_pos || !n_store) return VVS_ERR_INVALID_ARG;
  if (n_rows_per_seq < 1) return VVS_ERR_SHAPE;
  if (!aligned16(hidden)) return VVS_ERR_ALIGN;
  launch_fcache_store(*fc, hidden, n_rows_per_seq, ctx->desc.d_model, (int)elem_bytes(ctx->desc),
                      base_pos, n_store, ctx->ws.status, static_cast<cudaStream_t>(stream));
  return cudaGetLastError() == cudaSuccess ? VVS_OK : VVS_ERR_CUDA;
}

int vvs_feature_cache_fetch(vvs_ctx* ctx, const vvs_fcache* fc, const uint8_t* skip_mask,
                            int32_t n_images, const int32_t* gamma, int32_t gamma_max,
                            int32_t staleness, void* out, int32_t* out_pos, void* stream) {
  int rc = check_fcache(ctx, fc);
  if (rc != VVS_OK) return rc;
  if (!skip_mask || !gamma || !out || !out_pos) return VVS_ERR_INVALID_ARG;
  if (n_images < 1 || fc->n_rows % n_images != 0 || gamma_max < 1 || staleness < 0) return VVS_ERR_SHAPE;
  if (!aligned16(out)) return VVS_ERR_ALIGN;
  launch_fcache_fetch(*fc, skip_mask, n_images, gamma, gamma_max, staleness, ctx->desc.d_model,
                      (int)elem_bytes(ctx->desc), out, out_pos, ctx->ws.status,
                      static_cast<cudaStream_t>(stream));
  return cudaGetLastError() == cudaSuccess ? VVS_OK : VVS_ERR_CUDA;
}

int vvs_skip_decide(vvs_ctx* ctx, const int32_t* paths, const int32_t* path_len, int32_t n_images,
                    int32_t n_paths, int32_t max_len, const float* codebook, int32_t vocab, int32_t dim,
                    const uint8_t* last_verified, int32_t stride, float alpha, float threshold,
                    uint8_t* decision, float* similarity, void* stream) {
  if (!ctx || !paths || !codebook || !decision || !similarity) return VVS_ERR_INVALID_ARG;
  if (n_images < 1 || n_paths < 1 || max_len < 1 || vocab < 1 || dim < 1 || stride < 1) return VVS_ERR_SHAPE;
  if (!(alpha > 0.f) || !std::isfinite(alpha) || std::isnan(threshold)) return VVS_ERR_INVALID_ARG;
  return launch_skip_decide(paths, path_len, codebook, last_verified, n_images, n_paths, max_len, vocab, dim,
                            stride, alpha, threshold, decision, similarity, ctx->ws.status,
                            static_cast<cudaStream_t>(stream));
}

int vvs_select_unverified(vvs_ctx* ctx, const int32_t* paths, const int32_t* path_len, int32_t n_images,
                          int32_t n_paths, int32_t max_len, const float* uniforms, int32_t* out_path,
                          int32_t* out_gamma, int32_t* out_tokens, void* stream) {
  if (!ctx || !paths || !uniforms || !out_path || !out_gamma || !out_tokens) return VVS_ERR_INVALID_ARG;
  if (n_images < 1 || n_paths < 1 || max_len < 1) return VVS_ERR_SHAPE;
  return launch_select_unverified(paths, path_len, uniforms, n_images, n_paths, max_len, out_path, out_gamma,
                                  out_tokens, ctx->ws.status, static_cast<cudaStream_t>(stream));
}

int vvs_device_status(vvs_ctx* ctx, void* stream, int32_t* out_bits) {
  if (!ctx || !out_bits) return VVS_ERR_INVALID_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  int32_t bits = 0;
  VVS_CUDA_OK(cudaMemcpyAsync(&bits, ctx->ws.status, sizeof(bits), cudaMemcpyDeviceToHost, s));
  VVS_CUDA_OK(cudaMemsetAsync(ctx->ws.status, 0, sizeof(bits), s));
  VVS_CUDA_OK(cudaStreamSynchronize(s));
  *out_bits = bits;
  if ((bits & VVS_DEV_TIMEOUT) && ctx->ws.chain_sync) {
    // a grid barrier of the whole-chain kernel gave up: its arrival counter is no longer a
    // multiple of the grid size, start again from zero
    VVS_CUDA_OK(cudaMemsetAsync(ctx->ws.chain_sync, 0, 16, s));
    VVS_CUDA_OK(cudaStreamSynchronize(s));
  }
  if (bits & VVS_DEV_TIMEOUT) return VVS_ERR_DEVICE_TIMEOUT;
  if (bits & (VVS_DEV_BAD_TOKEN | VVS_DEV_CACHE_OVERFLOW | VVS_DEV_BAD_NEIGHBOUR | VVS_DEV_BAD_ARG))
    return VVS_ERR_DEVICE_BOUNDS;
  return VVS_OK;
}

int vvs_selftest_bounded_wait(vvs_ctx* ctx, void* stream, int32_t* gave_up) {
  if (!ctx || !gave_up) return VVS_ERR_INVALID_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  // two report words at the end of the status line (the status word itself is the first)
  int32_t* report = ctx->ws.status + 16;
  VVS_CUDA_OK(cudaMemsetAsync(report, 0, 2 * sizeof(int32_t), s));
  launch_bounded_wait_selftest(ctx->ws.status, report, s);
  int32_t host[2] = {0, 0};
  VVS_CUDA_OK(cudaMemcpyAsync(host, report, sizeof(host), cudaMemcpyDeviceToHost, s));
  VVS_CUDA_OK(cudaStreamSynchronize(s));
  gave_up[0] = host[0] == 0 ? 1 : 0;
  gave_up[1] = host[1] != 0 ? 1 : 0;
  return cudaGetLastError() == cudaSuccess ? VVS_OK : VVS_ERR_CUDA;
}

int vvs_last_launch_count(const vvs_ctx* ctx) { return ctx ? ctx->launches : 0; }

int vvs_profile_enable(vvs_ctx* ctx, int on) {
  if (!ctx) return VVS_ERR_INVALID_ARG;
  if (!on) {
    for (int i = 0; i < 2 * ctx->prof_capacity; ++i) cudaEventDestroy(ctx->prof_events[i]);
    delete[] ctx->prof_events;
    delete[] ctx->prof_class;
    ctx->prof_events = nullptr;
    ctx->prof_class = nullptr;
    ctx->prof_capacity = ctx->prof_used = 0;
    ctx->profiling = false;
    return VVS_OK;
  }
  if (ctx->profiling) return VVS_OK;
  const int cap = 16384;
  ctx->prof_events = new (std::nothrow) cudaEvent_t[2 * cap];
  ctx->prof_class = new (std::nothrow) int[cap];
  if (!ctx->prof_events || !ctx->prof_class) return VVS_ERR_NOMEM;
  for (int i = 0; i < 2 * cap; ++i) {
    if (cudaEventCreate(&ctx->prof_events[i]) != cudaSuccess) {
      ctx->prof_capacity = i / 2;
      vvs_profile_enable(ctx, 0);
      return VVS_ERR_CUDA;
    }
  }
  ctx->prof_capacity = cap;
  ctx->prof_used = 0;
  ctx->profiling = true;
  return VVS_OK;
}

int vvs_profile_read(vvs_ctx* ctx, void* stream, float* ms, int32_t* launches) {
  if (!ctx || !ms || !launches) return VVS_ERR_INVALID_ARG;
  VVS_CUDA_OK(cudaStreamSynchronize(static_cast<cudaStream_t>(stream)));
  for (int i = 0; i < ctx->prof_used; ++i) {
    float t = 0.f;
    VVS_CUDA_OK(cudaEventElapsedTime(&t, ctx->prof_events[2 * i], ctx->prof_events[2 * i + 1]));
    ms[ctx->prof_class[i]] += t;
    launches[ctx->prof_class[i]] += 1;
  }
  ctx->prof_used = 0;
  return VVS_OK;
}

const char* vvs_strerror(int status) {
  switch (status) {
    case VVS_OK: return "ok";
    case VVS_ERR_INVALID_ARG: return "invalid argument";
    case VVS_ERR_SHAPE: return "shape outside the model description or its limits";
    case VVS_ERR_ALIGN: return "device pointer not 16-byte aligned";
    case VVS_ERR_CAPACITY: return "KV cache capacity exceeded";
    case VVS_ERR_NOT_BOUND: return "weights or neighbour table not bound";
    case VVS_ERR_CUDA: return "CUDA runtime error";
    case VVS_ERR_DEVICE_TIMEOUT: return "bounded device-side wait ran out";
    case VVS_ERR_DEVICE_BOUNDS: return "device-side index check failed";
    case VVS_ERR_NOMEM: return "out of memory";
    default: return "unknown status";
  }
}

}  // extern "C"
