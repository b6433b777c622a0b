/*
 * vvs.h -- C ABI of the B200 (sm_100a) target-model verification step of VVS speculative
 * decoding for visual autoregressive models.
 *
 * One call of vvs_verify is lines 9-10 of the paper's Algorithm 2 ("VVS with Partial
 * Verification Skipping"): the target model M_T scores the candidate block in one parallel
 * pass against its KV cache (Sec. 2, "Speculative Decoding"), and Verify() applies the
 * sequential acceptance test, stops at the first rejection and resamples (Sec. 2).
 * vvs_feature_cache_store / _fetch are UpdateCache() (Alg. 2 line 11) and Retrieve()
 * (Alg. 2 line 5) of the token-level feature cache (Sec. 4.3).
 *
 * Naming: p = TARGET distribution, q = DRAFT distribution (the paper's Sec. 2 uses the
 * opposite letters).
 *
 * General rules
 *   - Every function returns VVS_OK (0) or a negative vvs_status.  Host-side argument errors
 *     are returned before anything is launched.  No exceptions.  Process-wide state is limited
 *     to per-device kernel attributes set once and the scratch array of vvs_decide_noalloc.
 *   - "device" pointers are CUDA device memory of the context's GPU, owned by the caller,
 *     16-byte aligned unless stated otherwise.  "host" pointers are ordinary host memory.
 *     The library never frees caller memory and keeps no reference to host arrays after a
 *     call returns (the per-layer pointer table is copied).
 *   - All work is enqueued on the CUDA stream passed to the call (a cudaStream_t cast to
 *     void*; NULL = the default stream) and is asynchronous.  A context holds scratch memory
 *     used by every call on it: calls on one context must be stream-ordered, one context per
 *     concurrently used stream.
 *   - Conditions only the GPU can see (token id out of range, cache overflow computed from
 *     device-resident lengths, a bounded wait that ran out) set bits in a device status word,
 *     read with vvs_device_status; the offending access is skipped, never executed.
 *   - Storage type T is float for VVS_DTYPE_FP32 contexts and bfloat16 for VVS_DTYPE_BF16.
 *     Accumulation, softmax and normalisation statistics are float32; decisions (acceptance
 *     ratios, pooled masses, the sampling CDF) accumulate in float64.
 */
#ifndef VVS_H_
#define VVS_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum vvs_status {
  VVS_OK = 0,
  VVS_ERR_INVALID_ARG = -1,    /* NULL where a pointer is required, bad enum, bad scalar */
  VVS_ERR_SHAPE = -2,          /* sizes inconsistent with the model description / limits */
  VVS_ERR_ALIGN = -3,          /* a device pointer is not 16-byte aligned */
  VVS_ERR_CAPACITY = -4,       /* cache fill + block length exceeds s_max */
  VVS_ERR_NOT_BOUND = -5,      /* weights (or the neighbour table, in relaxed mode) not bound */
  VVS_ERR_CUDA = -6,           /* a CUDA runtime call failed */
  VVS_ERR_DEVICE_TIMEOUT = -7, /* a bounded device-side wait gave up */
  VVS_ERR_DEVICE_BOUNDS = -8,  /* a device-side index check failed; the access was skipped */
  VVS_ERR_NOMEM = -9           /* workspace allocation failed */
} vvs_status;

enum { VVS_DTYPE_FP32 = 0, VVS_DTYPE_BF16 = 1 };
enum { VVS_ROPE_NONE = 0, VVS_ROPE_1D = 1, VVS_ROPE_2D_GRID = 2 };
enum { VVS_MODE_STRICT = 0, VVS_MODE_RELAXED = 1 };

/* Bits of the device status word (vvs_device_status). */
enum {
  VVS_DEV_BAD_TOKEN = 1,      /* block token outside the embedding table / draft outside codebook */
  VVS_DEV_CACHE_OVERFLOW = 2, /* cache_len[r] + T > s_max, or cache_len < 0: row skipped */
  VVS_DEV_BAD_NEIGHBOUR = 4,  /* CSR column outside [0, V) or row_ptr not monotone */
  VVS_DEV_TIMEOUT = 8,        /* a bounded wait on a barrier ran out */
  VVS_DEV_FCACHE_MISS = 16,   /* feature-cache fetch asked for a position not in the ring */
  VVS_DEV_BAD_ARG = 32        /* n_draft / gamma / n_store outside its documented range */
};

typedef struct vvs_ctx vvs_ctx;

/* Decoder-only transformer of the target model.  The paper treats M_T as given (LlamaGen-XL,
 * Lumina-mGPT); the architecture is the one those models share: pre-norm RMSNorm with a
 * learned scale, rotary position embedding, multi-head attention scaled by 1/sqrt(head_dim),
 * SwiGLU MLP, no biases, untied output head.  d_model must equal n_heads * head_dim. */
typedef struct vvs_model_desc {
  int32_t n_layers;
  int32_t d_model;
  int32_t n_heads;
  int32_t head_dim;      /* 64 or 128 */
  int32_t d_ff;          /* SwiGLU inner width */
  int32_t vocab;         /* V: size of the image codebook = number of logits per position;
                            at most 65535 * 128 (VVS_ERR_SHAPE beyond) */
  int32_t vocab_offset;  /* first row of the image codebook inside w_lm and the id space */
  int32_t lm_rows;       /* rows of w_lm (>= vocab_offset + vocab) */
  int32_t tok_rows;      /* rows of tok_emb */
  int32_t s_max;         /* KV-cache capacity (positions) per sequence */
  int32_t rope_mode;     /* VVS_ROPE_*; pairs are (2i, 2i+1); 1D: angle = pos * base^(-2i/hd);
                            2D_GRID: positions < n_prefix unrotated, image token n sits at grid
                            (n / rope_grid_w, n % rope_grid_w); pairs of the first head half
                            rotate by row, of the second half by column, with
                            angle = coord * base^(-2j/(hd/2)), j the pair index in its half */
  int32_t rope_grid_w;
  int32_t n_prefix;
  int32_t dtype;         /* VVS_DTYPE_*: type of weights, KV cache, hidden states */
  int32_t max_rows;      /* largest R = n_images * n_cfg a call may use */
  int32_t max_block;     /* largest T = n_forced + n_draft_max a call may use (<= 32) */
  int32_t max_nbr_k;     /* largest neighbour count k in relaxed mode (>= 1) */
  float rms_eps;
  float rope_base;
  int32_t deterministic; /* bf16 contexts:
                            1 = every sum of the decoder is taken in a fixed order, so the same call
                                gives the same bits every time (target_probs, hidden, the appended
                                K / V rows and hence next_token): the K splits of a projection tile
                                form a thread-block cluster that adds its partial tiles in rank order
                                through distributed shared memory, each output written by one thread;
                            0 = split-K partial sums are added in L2 in arrival order: faster (a
                                quarter to a third per step; measured numbers in the repository's
                                notes), the last bits of the logits differ from run to run, and a
                                residual sample over many nearly equally likely codes need not repeat.
                            float32 contexts are always repeatable. */
} vvs_model_desc;

/* Per-layer weights, device, type T.  Projection matrices are [out_features, in_features]
 * row-major: w_qkv [3*d_model, d_model] (q rows, then k rows, then v rows; head h owns rows
 * h*head_dim..), w_o [d_model, d_model], w_gate and w_up [d_ff, d_model],
 * w_down [d_model, d_ff], norm1 / norm2 [d_model]. */
typedef struct vvs_layer_weights {
  const void* w_qkv;
  const void* w_o;
  const void* w_gate;
  const void* w_up;
  const void* w_down;
  const void* norm1;
  const void* norm2;
} vvs_layer_weights;

typedef struct vvs_weights {
  const void* tok_emb;             /* device T [tok_rows, d_model] */
  const void* norm_f;              /* device T [d_model] */
  const void* w_lm;                /* device T [lm_rows, d_model]; only rows
                                      vocab_offset .. vocab_offset+vocab-1 are read */
  const vvs_layer_weights* layers; /* HOST array [n_layers] of device pointers */
} vvs_weights;

/* Create a context on the current CUDA device and allocate its scratch memory (sized from
 * max_rows, max_block, max_nbr_k; see vvs_workspace_bytes).  *out is NULL on failure. */
int vvs_create(const vvs_model_desc* desc, vvs_ctx** out);
int vvs_destroy(vvs_ctx* ctx);
/* Scratch bytes vvs_create will allocate for this description (host computation only). */
int vvs_workspace_bytes(const vvs_model_desc* desc, size_t* out_bytes);

/* Bind caller-owned weights.  Checks non-NULL and 16-byte alignment (VVS_ERR_ALIGN).  Nothing is
 * copied: the weights must stay valid and unchanged while the context uses them.  (Only under the
 * debug switch VVS_DEBUG_CHAIN_KERNELS, read by vvs_create, a fixed-order context also builds a
 * re-packed device copy of the layer weights here for its streaming whole-chain kernel.) */
int vvs_bind_weights(vvs_ctx* ctx, const vvs_weights* w);

/* Bind the latent-space neighbour table used by relaxed acceptance (Sec. 2, LANTERN rule):
 * CSR over codebook indices, device int32.  row_ptr [vocab+1]; the neighbours of code x are
 * col[row_ptr[x] .. row_ptr[x+1]) in ascending latent distance with x ITSELF FIRST (entry 0 is
 * taken to be x and is not read).  nnz = row_ptr[vocab]. */
int vvs_bind_neighbors(vvs_ctx* ctx, const int32_t* row_ptr, const int32_t* col, int64_t nnz);

/* Inputs of one verification step.  B = n_images, C = n_cfg, R = B*C sequences ordered
 * [cond_0 .. cond_{B-1}, uncond_0 .. uncond_{B-1}], F = n_forced >= 1, K = n_draft_max,
 * T = F + K block rows per sequence. */
typedef struct vvs_verify_args {
  int32_t n_images;
  int32_t n_cfg;          /* 1: no guidance; 2: logits l = l_u + cfg_scale * (l_c - l_u) */
  int32_t n_forced;       /* committed tokens whose K/V is not cached yet (the last accepted
                             token; with post verification, Sec. 4.1, also the unverified ones) */
  int32_t n_draft_max;
  const int32_t* block;   /* device [B, T] embedding-table ids: F forced tokens, then K drafts.
                             Drafts must lie in [vocab_offset, vocab_offset + vocab). cond and
                             uncond sequences of an image carry the same block */
  const int32_t* n_draft; /* device [B], drafts actually proposed per image (0..K); NULL = K */
  void* kv_k;             /* device T [n_layers][kv_rows][n_heads][s_max][head_dim], keys after */
  void* kv_v;             /*   RoPE / values.  Slots cache_len[r] .. cache_len[r]+T-1 of every
                               layer are WRITTEN by the call (Sec. 4.1: restores KV entries) */
  int32_t kv_rows;        /* sequence dimension of the cache allocation (>= R) */
  const int32_t* cache_len;      /* device [R] fill level L_r (positions already cached) */
  const int32_t* cache_len_host; /* optional HOST copy [R]: enables the VVS_ERR_CAPACITY check
                                    before launch; NULL = checked on the device only */
  const float* draft_probs; /* device [B, K, V] drafter distributions q_i over the codebook */
  const float* uniforms;    /* device [B, K+1] in (0,1): column i < K judges draft i, column K
                               drives the single residual / bonus sample */
  float cfg_scale;
  float temperature;        /* logits are divided by it before the softmax (paper: 1.0) */
  int32_t mode;             /* VVS_MODE_* */
  int32_t nbr_k;            /* relaxed: use the first nbr_k entries of each CSR row */
  float delta;              /* relaxed: pooled neighbour mass (excluding p(x)) stays <= delta;
                               INFINITY = pool all nbr_k neighbours */
  const int32_t* tree_parent; /* NULL: the K drafts are a chain.  Otherwise device [B, T]: parent block
                               row of every block row of a candidate TREE (the drafter of the paper
                               proposes a token tree, Sec. 5): -1 for row 0, t - 1 for the forced rows
                               t < F, and for draft node t >= F any row in [F - 1, t).  Row t then
                               attends the cache and its ancestors only and sits at position
                               cache_len + depth(t); draft_probs[b, i] is the drafter's distribution
                               at the PARENT of node F + i (siblings carry the same row) and the
                               children of a node are taken to be independent draws from it.
                               Verification walks the tree from row F - 1: the children of the current
                               node are tried in index order, child x passes iff
                               u < min(1, p_res(x) / q(x)), a rejection replaces p_res by
                               norm(max(0, p_res - q)); when no child is left the next token is drawn
                               from p_res (from the node's own target row if it is a leaf).  In
                               relaxed mode the numerator of a child's ratio is the pooled mass of
                               the child and its neighbours in the CURRENT p_res (the chain's relaxed
                               rule with p_res in the place of p; the paper prints no tree rule).
                               Tree calls need a bf16 context, n_draft == NULL and
                               out->target_probs (the walk reads whole target rows). */
  int32_t adjusted_residual; /* relaxed mode only, 0 (default) or 1.  0: after a rejection the next
                               token is drawn from norm(max(0, p - q)) with the plain target row p.
                               1: from norm(max(0, p~ - q)), p~ the adjusted target of the rejected
                               draft x - the pooled mass of the accepted set A sits on x, the other
                               members of A carry none, all other codes keep their probability (the
                               distribution under which the relaxed test is the plain speculative
                               test; Sec. 2 cites the relaxed rule without printing its residual).
                               Ignored in strict mode; must be 0 or 1. */
} vvs_verify_args;

/* Outputs, device memory allocated by the caller.  Optional ones may be NULL and are then
 * never computed or written. */
typedef struct vvs_verify_out {
  int32_t* accept_len;  /* [B] number of accepted drafts (accepted-prefix length) */
  int32_t* next_token;  /* [B] embedding-table id sampled from norm(max(0, p - q)) at the first
                           rejected position, or from the bonus row p_{T-1} if all accepted */
  int32_t* new_len;     /* [R] cache_len + F + accept_len: fill level after the step */
  int32_t* n_commit;    /* optional [R] F + accept_len: block rows whose K/V and features are now
                           committed (the n_store argument of vvs_feature_cache_store) */
  uint8_t* accept_mask; /* optional [B, K] */
  float* target_probs;  /* optional [B, T, V] float32 target distributions after guidance */
  void* hidden;         /* optional T [R, T, d_model] features (final-norm output) */
  int32_t* accept_path; /* optional [B, K] (tree calls): block rows of the accepted nodes, root side
                           first, then -1.  After a tree call the K/V of the accepted nodes have been
                           moved to slots cache_len + F .. cache_len + F + accept_len - 1, so the
                           cache is contiguous again; `hidden` stays in block-row order */
  float* margins;       /* optional [B, K+1]: |u_i - ratio_i| for judged drafts (INFINITY for
                           drafts not judged) and, in column K, the distance of the sample
                           point to the nearest CDF bin edge as a fraction of the total mass */
} vvs_verify_out;

/* The verification step.  The first call with a given set of argument and output pointers captures
 * the step into a CUDA graph (a few milliseconds of host time, graph memory allocated by the
 * runtime); later calls with the same pointers replay it, so a decode loop should reuse its
 * buffers (up to 64 distinct argument sets are kept).  A call made while `stream` is itself being
 * captured is enqueued directly.
 * Steps: embedding gather; n_layers x { RMSNorm, QKV projection,
 * RoPE, KV append, block-vs-cache attention causal inside the block, output projection,
 * RMSNorm, SwiGLU MLP }; final RMSNorm (= features); LM head over the codebook rows; guidance;
 * softmax; strict min(1, p/q) or relaxed min(1, P_A/q) acceptance with the accepted-prefix
 * rule; residual / bonus sample.  Rows of the block whose acceptance fails leave garbage K/V
 * beyond new_len, overwritten by the next call. */
int vvs_verify(vvs_ctx* ctx, const vvs_verify_args* args, const vvs_verify_out* out, void* stream);

/* The decision part alone on given features: hidden is device T [R, n_rows_per_seq, d_model];
 * draft i is judged against row first_row + i, the bonus row is first_row + K (if
 * n_rows_per_seq <= first_row + K there is no bonus row and next_token = -1 when all drafts
 * pass).  `drafts` is device int32 [B, K] embedding-table ids.  kv_*, cache_len, block and
 * n_forced of `args` are ignored; out->new_len and out->hidden must be NULL. */
int vvs_epilogue(vvs_ctx* ctx, const void* hidden, int32_t n_rows_per_seq, int32_t first_row,
                 const int32_t* drafts, const vvs_verify_args* args, const vvs_verify_out* out,
                 void* stream);

/* Verify(logits_t, C_t) alone (Alg. 2 line 10; Sec. 2): acceptance test, accepted prefix and
 * residual / bonus sample on target probabilities the caller already holds (guidance and
 * softmax already applied).  target_probs is device float32 [B, n_rows_per_seq, V]; rows,
 * first_row and drafts as in vvs_epilogue.  args->n_cfg must be 1; cfg_scale and temperature are
 * ignored; out->new_len, n_commit, hidden and target_probs must be NULL.  Needs no weights.
 * With args->tree_parent (device [B, n_rows_per_seq], as in vvs_verify with n_forced =
 * first_row + 1 and first_row + 1 + K == n_rows_per_seq) the K drafts are the nodes of a
 * candidate tree and the walk of vvs_verify's tree calls runs on the given rows;
 * out->accept_path may then be given.  No cache is touched. */
int vvs_decide(vvs_ctx* ctx, const float* target_probs, int32_t n_rows_per_seq, int32_t first_row,
               const int32_t* drafts, const vvs_verify_args* args, const vvs_verify_out* out,
               void* stream);

/* (No counterpart in the paper: this entry point exists for deployment reasons only.)
 * vvs_decide without a context and without any allocation.  Some callers may not call
 * cudaMalloc at all: code that runs inside a serving process whose allocator reserved the whole
 * GPU at start-up, a plugin whose host forbids allocations, or a latency-critical loop that
 * cannot afford the device-wide synchronisation an allocation implies.  For them the scratch of
 * the decision kernels lives in one fixed array in device memory that is part of the library
 * image: about 325 KB held on every GPU that loads the library, until the process exits.  The
 * function calls no cudaMalloc / cudaFree and no allocating library routine.
 *
 * Capacity (larger sizes return VVS_ERR_SHAPE): n_images <= 64, n_draft_max <= 16,
 * nbr_k <= 64, vocab <= 65536.
 *
 * Chains only: args->tree_parent and out->accept_path must be NULL, and args->adjusted_residual
 * must be 0 (it needs a writable copy of the sampled row): VVS_ERR_INVALID_ARG otherwise.
 *
 * Arguments are those of vvs_decide, with what a context would carry passed explicitly: vocab,
 * vocab_offset, and the CSR neighbour table (device int32, may be NULL in strict mode).
 * status_bits: optional device int32 the VVS_DEV_* bits are OR-ed into (caller clears it);
 * NULL = a private word inside the scratch array, cleared by each call and not readable.
 *
 * The first call on each device looks up the array's device address (cudaGetSymbolAddress, with
 * that device current) and caches it; make that first call outside any stream capture.  All
 * calls on a device share the one array, which still holds the previous call's values (each
 * call rewrites what it reads): two calls whose kernels may overlap on the GPU (different
 * streams without ordering, or several host threads) race on it and must be serialised. */
#define VVS_NOALLOC_MAX_IMAGES 64
#define VVS_NOALLOC_MAX_DRAFTS 16
#define VVS_NOALLOC_MAX_NBR_K 64
#define VVS_NOALLOC_MAX_VOCAB 65536
int vvs_decide_noalloc(const float* target_probs, int32_t vocab, int32_t vocab_offset,
                       int32_t n_rows_per_seq, int32_t first_row, const int32_t* drafts,
                       const int32_t* nbr_row_ptr, const int32_t* nbr_col,
                       const vvs_verify_args* args, const vvs_verify_out* out,
                       int32_t* status_bits, void* stream);

/* Token-level feature cache (Sec. 4.3): per sequence a ring of `cap` slots holding the most
 * recent features, addressed by absolute position (slot = pos mod cap).  All arrays are
 * device memory owned by the caller; vvs_feature_cache_reset marks every slot empty. */
typedef struct vvs_fcache {
  void* feat;       /* T [n_rows, cap, d_model] */
  int32_t* fpos;    /* [n_rows, cap] position held by each slot, -1 = empty */
  int32_t* newest;  /* [n_rows] newest position ever stored, -1 = none */
  int32_t n_rows;
  int32_t cap;      /* the paper keeps n = max accepted length = 5 features per sequence */
} vvs_fcache;

int vvs_feature_cache_reset(vvs_ctx* ctx, const vvs_fcache* fc, void* stream);

/* UpdateCache(h_t): for each sequence r, copy hidden[r, t, :] for t < n_store[r] into the slot
 * of position base_pos[r] + t, tag the slot, raise newest[r].  hidden is device
 * T [n_rows, n_rows_per_seq, d_model]; base_pos, n_store device int32 [n_rows]
 * (0 <= n_store[r] <= min(n_rows_per_seq, cap)).  Storing a position again overwrites it (how
 * post verification writes refreshed features back, Sec. 4.1). */
int vvs_feature_cache_store(vvs_ctx* ctx, const vvs_fcache* fc, const void* hidden,
                            int32_t n_rows_per_seq, const int32_t* base_pos,
                            const int32_t* n_store, void* stream);

/* Retrieve(C, a): for sequences of images with skip_mask[b] != 0 (device uint8 [n_images],
 * row r belongs to image r mod n_images), gather the gamma[r] most recent features ending
 * `staleness` positions before the newest one, oldest first, into out[r, j, :] (device
 * T [n_rows, gamma_max, d_model]) and their positions into out_pos[r, j] (device int32
 * [n_rows, gamma_max]).  A position that is not in the ring gives out_pos = -1, a zero row and
 * the VVS_DEV_FCACHE_MISS status bit.  Rows of unmasked images and entries j >= gamma[r] are
 * not touched. */
int vvs_feature_cache_fetch(vvs_ctx* ctx, const vvs_fcache* fc, const uint8_t* skip_mask,
                            int32_t n_images, const int32_t* gamma, int32_t gamma_max,
                            int32_t staleness, void* out, int32_t* out_pos, void* stream);

/* Dynamic verification skipping (Sec. 4.4 "Fine-grained Skipped Step Scheduling", Eq. 2,
 * Algorithm 1): for every image, decide whether the next step may bypass target verification.
 *   paths          device int32 [n_images, n_paths, max_len] candidate token paths of the draft
 *                  tree as codebook indices (0 .. vocab-1); path i of an image has path_len[i] tokens
 *   path_len       device int32 [n_images, n_paths], or NULL = every path has max_len tokens
 *   codebook       device float32 [vocab, dim] latent embeddings E of the VQ codebook
 *   last_verified  device uint8 [n_images] (V_last), or NULL = every image's last step was verified
 * Alg. 1: an image whose last step was not verified never skips (decision 0, similarity 0).
 * Otherwise the paths are down-sampled (every stride-th path, the paper uses 2), and
 * S_bar = sum_l w_l S^(l), w_l = alpha^l / sum_k alpha^k (Eq. 2), is compared with the threshold:
 * decision[b] = 1 (skip) iff S_bar >= threshold; similarity[b] = S_bar.  Where the paper is silent:
 * S^(l) is the mean cosine similarity over all unordered pairs of kept paths of the embeddings of
 * their tokens at depth l; the depth is the shortest kept path; a zero embedding has cosine 0; a
 * single kept path gives S_bar = 1, depth 0 gives 0.  Limits (VVS_ERR_SHAPE beyond): 64 kept
 * paths, max_len 16.  A token outside the codebook sets VVS_DEV_BAD_TOKEN and counts as cosine 0.
 * Sums are taken in float64 in a fixed order: the same inputs give the same bits. */
int vvs_skip_decide(vvs_ctx* ctx, const int32_t* paths, const int32_t* path_len, int32_t n_images,
                    int32_t n_paths, int32_t max_len, const float* codebook, int32_t vocab, int32_t dim,
                    const uint8_t* last_verified, int32_t stride, float alpha, float threshold,
                    uint8_t* decision, float* similarity, void* stream);

/* Unverified token selection with truncation (Sec. 4.2, Eq. 3; "UniformSample" in Algorithm 2): the
 * tokens a verification-free step accepts.  For every image one candidate path is drawn uniformly,
 * index floor(uniforms[b] * n_paths) with uniforms device float32 [n_images] in (0, 1), and cut to
 * its first gamma = min(L_s, floor(L_bar)) tokens, L_s its own length and L_bar the mean length of
 * all n_paths paths of the image.  paths / path_len as in vvs_skip_decide (path_len NULL = max_len).
 * Outputs (device int32): out_path [n_images] the drawn index, out_gamma [n_images],
 * out_tokens [n_images, max_len] the kept tokens followed by -1.  A length outside 0..max_len is
 * clamped and sets VVS_DEV_BAD_ARG. */
int vvs_select_unverified(vvs_ctx* ctx, const int32_t* paths, const int32_t* path_len, int32_t n_images,
                          int32_t n_paths, int32_t max_len, const float* uniforms, int32_t* out_path,
                          int32_t* out_gamma, int32_t* out_tokens, void* stream);

/* Synchronise `stream`, copy the device status word to *out_bits (VVS_DEV_* bits) and clear
 * it.  Returns VVS_ERR_DEVICE_TIMEOUT / VVS_ERR_DEVICE_BOUNDS if such a bit was set. */
int vvs_device_status(vvs_ctx* ctx, void* stream, int32_t* out_bits);

/* Self-test of the failure path of the library's bounded device-side waits (no counterpart in the
 * paper).  Launches one tiny kernel in which a thread waits, through the same helpers the tensor-core
 * kernels and the streaming chain kernel use but with a limit of a few hundred polls, on barriers
 * nobody ever arrives on.  Each wait must give up and return: gave_up[0] / gave_up[1] (host int32[2])
 * are set to 1 for the two helpers, the VVS_DEV_TIMEOUT bit is left in the device status word (so
 * the next vvs_device_status returns VVS_ERR_DEVICE_TIMEOUT and clears it), and the context stays
 * usable.  Synchronises `stream`.  Nothing in it can hang: the waits are the bounded ones. */
int vvs_selftest_bounded_wait(vvs_ctx* ctx, void* stream, int32_t* gave_up);

/* Number of kernels the last vvs_verify / vvs_epilogue call on this context launched. */
int vvs_last_launch_count(const vvs_ctx* ctx);

/* Per-kernel-class device timing for roofline reports.  While enabled, every launch of
 * vvs_verify / vvs_epilogue is bracketed by CUDA events on the call's stream (this costs time:
 * never enable it around a headline measurement).  Classes: 0 = projection / LM-head GEMMs,
 * 1 = attention, 2 = everything else, 3 = the whole-chain kernel (embedding and every decoder
 * layer in one launch; used by calls of at most 32 block tokens, which then have no class-0 / 1
 * launches except the LM head).  vvs_profile_read synchronises the stream, ADDS the milliseconds
 * and launch counts recorded since the last read to ms[4] / launches[4] (host arrays) and forgets
 * them.  Events are created by vvs_profile_enable, not on the verify path. */
enum { VVS_PROF_GEMM = 0, VVS_PROF_ATTENTION = 1, VVS_PROF_OTHER = 2, VVS_PROF_CHAIN = 3, VVS_PROF_CLASSES = 4 };
int vvs_profile_enable(vvs_ctx* ctx, int on);
int vvs_profile_read(vvs_ctx* ctx, void* stream, float* ms, int32_t* launches);

const char* vvs_strerror(int status);

#ifdef __cplusplus
}
#endif
#endif /* VVS_H_ */
