// vvs_decide_noalloc: the decision stage (acceptance test, accepted prefix, residual / bonus
// sample) for callers that must not allocate device memory.  Same kernels as vvs_decide; the only
// difference is where their scratch lives: in the fixed device array below instead of a context's
// cudaMalloc'ed arena.
#include <mutex>

#include "vvs_internal.cuh"

using namespace vvs;

namespace {

constexpr int kMaxImages = VVS_NOALLOC_MAX_IMAGES;
constexpr int kMaxDrafts = VVS_NOALLOC_MAX_DRAFTS;
constexpr int kMaxNbrK = VVS_NOALLOC_MAX_NBR_K;
constexpr int kMaxVocab = VVS_NOALLOC_MAX_VOCAB;
constexpr int kMaxChunks = (kMaxVocab + kSampleChunk - 1) / kSampleChunk;

// Byte offsets inside the scratch array (each a multiple of 256).
constexpr size_t kOffStatus = 0;
constexpr size_t kOffSelRow = 256;
constexpr size_t kOffSelKind = kOffSelRow + 256;
constexpr size_t kOffLTok = kOffSelKind + 256;
constexpr size_t kOffLNbr = kOffLTok + sizeof(float) * kMaxImages * kMaxDrafts;
constexpr size_t kOffRPart = kOffLNbr + sizeof(float) * kMaxImages * kMaxDrafts * kMaxNbrK;
constexpr size_t kOffPPart = kOffRPart + sizeof(double) * kMaxImages * kMaxChunks;
constexpr size_t kScratchBytes = kOffPPart + sizeof(double) * kMaxImages * kMaxChunks;
static_assert(sizeof(int32_t) * kMaxImages <= 256, "selection arrays must fit their 256-byte slots");
static_assert(kScratchBytes <= 400 * 1024, "keep the resident scratch modest");

// Resident on every GPU that loads this library, from load until the process exits (~325 KB).
// In host code this name is only a stand-in for the symbol, not a device address: the address
// the kernels get comes from cudaGetSymbolAddress below.
static __device__ __align__(256) unsigned char g_noalloc_scratch[kScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
unsigned char* g_scratch_addr[kMaxDevices] = {};  // device address of the array, per device ordinal

// Once per device, with that device current: resolve the device address of the scratch array.
int scratch_for_current_device(unsigned char** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return VVS_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_mu);
  if (!g_scratch_addr[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || !p) {
      cudaGetLastError();
      return VVS_ERR_CUDA;
    }
    g_scratch_addr[dev] = static_cast<unsigned char*>(p);
  }
  *out = g_scratch_addr[dev];
  return VVS_OK;
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace

extern "C" int vvs_decide_noalloc(const float* target_probs, int32_t vocab, int32_t vocab_offset,
                                  int32_t n_rows_per_seq, int32_t first_row, const int32_t* drafts,
                                  const int32_t* nbr_row_ptr, const int32_t* nbr_col,
                                  const vvs_verify_args* a, const vvs_verify_out* o,
                                  int32_t* status_bits, void* stream) {
  if (!target_probs || !a || !o) return VVS_ERR_INVALID_ARG;
  if (!a->uniforms || !o->accept_len || !o->next_token) return VVS_ERR_INVALID_ARG;
  if (a->n_cfg != 1 || a->n_images < 1 || a->n_draft_max < 0 || n_rows_per_seq < 1) return VVS_ERR_SHAPE;
  // fixed capacity of the resident scratch
  if (a->n_images > kMaxImages || a->n_draft_max > kMaxDrafts || vocab < 1 || vocab > kMaxVocab)
    return VVS_ERR_SHAPE;
  if (vocab_offset < 0 || first_row < 0 || first_row + a->n_draft_max > n_rows_per_seq) return VVS_ERR_SHAPE;
  if (a->n_draft_max > 0 && (!drafts || !a->draft_probs)) return VVS_ERR_INVALID_ARG;
  if (a->mode != VVS_MODE_STRICT && a->mode != VVS_MODE_RELAXED) return VVS_ERR_INVALID_ARG;
  if (a->mode == VVS_MODE_RELAXED) {
    if (a->nbr_k < 1 || a->nbr_k > kMaxNbrK) return VVS_ERR_SHAPE;
    if (!(a->delta >= 0.f)) return VVS_ERR_INVALID_ARG;
    if (a->nbr_k > 1 && (!nbr_row_ptr || !nbr_col)) return VVS_ERR_NOT_BOUND;
  }
  if (o->new_len || o->n_commit || o->hidden || o->target_probs) return VVS_ERR_INVALID_ARG;
  // chains only: a candidate tree would need the walk's float64 scratch rows, which this array has not
  if (a->tree_parent || o->accept_path) return VVS_ERR_INVALID_ARG;
  if (a->adjusted_residual != 0) return VVS_ERR_INVALID_ARG;   // needs a writable copy of the sampled row
  if (!aligned16(target_probs) || !aligned16(a->draft_probs)) return VVS_ERR_ALIGN;

  unsigned char* base = nullptr;
  int rc = scratch_for_current_device(&base);
  if (rc != VVS_OK) return rc;
  cudaStream_t s = static_cast<cudaStream_t>(stream);

  Workspace ws;  // only the members the decision kernels touch
  ws.status = status_bits ? status_bits : reinterpret_cast<int32_t*>(base + kOffStatus);
  ws.sel_row = reinterpret_cast<int32_t*>(base + kOffSelRow);
  ws.sel_kind = reinterpret_cast<int32_t*>(base + kOffSelKind);
  ws.l_tok = reinterpret_cast<float*>(base + kOffLTok);
  ws.l_nbr = reinterpret_cast<float*>(base + kOffLNbr);
  ws.r_part = reinterpret_cast<double*>(base + kOffRPart);
  ws.p_part = reinterpret_cast<double*>(base + kOffPPart);
  // The array keeps the previous call's contents.  Every slot read below is written earlier in
  // this same call, except the private status word, which must start at zero.
  if (!status_bits && cudaMemsetAsync(base + kOffStatus, 0, 256, s) != cudaSuccess) return VVS_ERR_CUDA;

  DecideParams p{};
  p.n_images = a->n_images; p.n_cfg = 1; p.rows_per_seq = n_rows_per_seq; p.first_row = first_row;
  p.n_draft_max = a->n_draft_max; p.vocab = vocab; p.vocab_offset = vocab_offset;
  p.mode = a->mode; p.nbr_k = a->mode == VVS_MODE_RELAXED ? a->nbr_k : 1; p.kmax = kMaxNbrK;
  p.delta = a->delta;
  p.drafts = drafts; p.drafts_ld = a->n_draft_max; p.n_draft = a->n_draft;
  p.draft_probs = a->draft_probs; p.uniforms = a->uniforms;
  p.row_ptr = nbr_row_ptr; p.col = nbr_col;
  p.direct_probs = target_probs;
  p.n_forced = 1;
  p.accept_len = o->accept_len; p.next_token = o->next_token;
  p.accept_mask = o->accept_mask; p.margins = o->margins;

  if (p.n_draft_max > 0) launch_gather_logits(target_probs, ws, p, s);
  launch_accept(ws, p, s);
  launch_residual_mass(ws, p, s);
  launch_sample(ws, p, s);
  return cudaGetLastError() == cudaSuccess ? VVS_OK : VVS_ERR_CUDA;
}
