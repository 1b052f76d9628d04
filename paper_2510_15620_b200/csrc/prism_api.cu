// Host side of the C ABI: handle, workspaces, the layer-major request driver with chunked execution
// (Sec. 4.3) and overlapped layer streaming (Sec. 4.2), probe -> route -> compact after the
// designated layers (Sec. 4.1), final top-K.  All arithmetic of the method runs in the kernels.
#include <algorithm>
#include <cstdio>
#include <cstring>
#include <iterator>
#include <new>
#include <string>
#include <vector>

#include "../../include/prism.h"
#include "common.cuh"

using namespace prism;

static_assert(sizeof(prism_probe_record) == sizeof(ProbeRecordDev), "probe record layouts must match");
static_assert(PRISM_MAX_CLUSTERS == kMaxClusters && PRISM_MAX_CANDIDATES == kMaxCandidates, "limits must match");

namespace {

struct LayerDev {  // device pointers of one layer's tensors (resident, or inside a streaming slot)
  const void *g_attn, *w_qkv, *g_q, *g_k, *w_o, *g_ffn, *w_gate, *w_up, *w_down;
};

struct LayerMaps {  // TMA descriptors of the B operands
  TmaDesc qkv, o, gate, up, down;
};

struct EncVec {  // fp32 copies of one encoder block's vectors
  const float *b_qkv, *b_o, *ln1_g, *ln1_b, *b_ffn1, *b_ffn2, *ln2_g, *ln2_b;
};

}  // namespace

struct prism_handle {
  prism_model_cfg cfg{};
  std::vector<prism_layer_weights> layers;  // caller's pointers (device, or pinned host when streamed)
  const void *embed = nullptr, *g_final = nullptr, *score_head = nullptr;
  // encoder stack (cfg.arch == PRISM_ARCH_ENCODER)
  bool enc = false;
  std::vector<prism_encoder_layer_weights> enc_layers;
  std::vector<EncVec> enc_vec;
  const void *pos_embed = nullptr, *head_dense_w = nullptr;
  float* probe_scratch = nullptr;  // [2, max_candidates, D]
  void* qkv_prefix = nullptr;      // q/k/v rows of a shared query prefix, kept for the later chunks of a layer
  // W4 weights (cfg.weight_format == PRISM_WFMT_W4): the layer about to run is rebuilt as bf16 here
  bool w4 = false;
  void* wq[5] = {nullptr, nullptr, nullptr, nullptr, nullptr};  // w_qkv, w_o, w_gate, w_up, w_down
  LayerMaps maps_w4{};
  const float *type_f = nullptr, *emb_g = nullptr, *emb_b = nullptr, *head_db = nullptr, *head_ow = nullptr, *head_ob = nullptr;
  int esz = 4;
  int chunk_tokens = 0;
  bool tc = false;  // tensor-core GEMM path
  bool pair = false;  // ... on CTA pairs (the default) rather than single CTAs
  bool flip = true;   // consecutive kernels of a layer walk the rows in opposite directions (L2 reuse)
  bool last_rev = false;  // direction of the kernel launched last
  int fa = 0;       // attention path: 0 SIMT, 1 tcgen05, 2 warp-level MMA

  std::vector<void*> dev_allocs;
  std::vector<void*> host_allocs;
  int64_t workspace_bytes = 0;
  int64_t launches = 0;
  std::string err;

  float* x[2] = {nullptr, nullptr};
  int *tokens = nullptr, *pos = nullptr, *cu[2] = {nullptr, nullptr}, *seq2orig[2] = {nullptr, nullptr};
  int* old_of_new = nullptr;
  void *a_norm = nullptr, *qkv = nullptr, *attn = nullptr, *hbuf = nullptr;
  float *scores = nullptr, *res_score = nullptr, *w_diff = nullptr, *rope_cos = nullptr, *rope_sin = nullptr, *rope_fused = nullptr;
  int *res_idx = nullptr, *errword = nullptr;
  RouteState* state = nullptr;
  ProbeRecordDev* recs = nullptr;
  float* trace_scores = nullptr;
  int* trace_ids = nullptr;
  unsigned char* owned_dev = nullptr;  // candidate-sharded runs: which candidates this rank runs

  // Dynamic offloading of the hidden states (Sec. 4.3): x[0], x[1] are pinned host memory, the layers run on one
  // of three device chunk buffers; chunk c is fetched on in_stream, computed on the request's stream and written
  // back on out_stream.
  bool offload = false;
  float* xc[3] = {nullptr, nullptr, nullptr};
  cudaStream_t in_stream = nullptr, out_stream = nullptr;
  cudaEvent_t ev_in[3] = {nullptr, nullptr, nullptr}, ev_done[3] = {nullptr, nullptr, nullptr},
              ev_slot_out[3] = {nullptr, nullptr, nullptr}, ev_main = nullptr;
  std::vector<cudaEvent_t> ev_chunk_out;  // per chunk index: its last write-back

  // Embedding table caching (Sec. 4.4): `embed` is the pinned host table, the device holds cache_rows rows.
  int cache_rows = 0;
  unsigned char* cache_dev = nullptr;  // [cache_rows, D] in the table's element type
  int* tok2slot_dev = nullptr;         // [vocab]: row of a token in the cache (valid for the tokens of the request)
  int* pairs_dev = nullptr;            // (token, slot) of the rows to fetch
  int* h_tokens = nullptr;             // pinned: the request's token ids
  int* h_pairs = nullptr;              // pinned
  std::vector<int> slot_of_tok, tok_of_slot;
  std::vector<uint64_t> slot_stamp;    // request number of the slot's last use (0 = never)
  std::vector<uint64_t> tok_seen;      // request number in which the token was last looked up
  uint64_t request_no = 0;
  int64_t cache_hits = 0, cache_misses = 0, cache_evictions = 0;
  void* route_scratch = nullptr;
  int *in_query = nullptr, *in_cand = nullptr, *in_off = nullptr, *out_idx = nullptr;
  float* out_score = nullptr;

  // pinned host mirrors
  int* h_cu = nullptr;       // offsets of the live batch
  int* h_cu_next = nullptr;  // offsets after the pending prune decision
  int* h_off = nullptr;
  RouteState* h_state = nullptr;
  int* h_err = nullptr;

  // streaming
  unsigned char* slot[2] = {nullptr, nullptr};
  size_t slot_bytes = 0;
  size_t off_g_attn = 0, off_qkv = 0, off_gq = 0, off_gk = 0, off_o = 0, off_g_ffn = 0, off_gate = 0, off_up = 0,
         off_down = 0;
  cudaStream_t copy_stream = nullptr;
  cudaEvent_t ev_copied[2] = {nullptr, nullptr}, ev_freed[2] = {nullptr, nullptr};

  // optional per-kernel timing (prism_profile): event pairs around every launch of a request
  bool prof_on = false;
  struct ProfEntry { int cat; double work; cudaEvent_t a, b; };
  std::vector<ProfEntry> prof_pending;
  std::vector<cudaEvent_t> prof_pool;
  prism_kernel_stat prof_acc[PRISM_N_KERNEL_CLASSES] = {};

  // TMA descriptors
  TmaDesc map_a_norm{}, map_attn{}, map_hbuf{};
  std::vector<LayerMaps> maps;  // per layer (resident) or per slot (streamed)
};

namespace {

int fail(prism_handle* h, int code, const std::string& msg) {
  if (h) h->err = msg;
  return code;
}

int cuda_fail(prism_handle* h, cudaError_t e, const char* what) {
  return fail(h, e == cudaErrorMemoryAllocation ? PRISM_ERR_NOMEM : PRISM_ERR_CUDA,
              std::string(what) + ": " + cudaGetErrorString(e));
}

#define PRISM_CUDA(h, call)                                    \
  do {                                                         \
    cudaError_t e__ = (call);                                  \
    if (e__ != cudaSuccess) return cuda_fail((h), e__, #call); \
  } while (0)

#define PRISM_LAUNCH(h, call)                                  \
  do {                                                         \
    cudaError_t e__ = (call);                                  \
    (h)->launches++;                                           \
    if (e__ != cudaSuccess) return cuda_fail((h), e__, #call); \
  } while (0)

cudaEvent_t prof_event(prism_handle* h) {
  if (!h->prof_pool.empty()) {
    cudaEvent_t e = h->prof_pool.back();
    h->prof_pool.pop_back();
    return e;
  }
  cudaEvent_t e = nullptr;
  cudaEventCreate(&e);
  return e;
}

// A launch that is attributed to kernel class `cat` with `work` algorithmic flops or bytes.
#define PRISM_LAUNCH_P(h, st, cat, work, call)                                   \
  do {                                                                           \
    cudaEvent_t ea__ = nullptr, eb__ = nullptr;                                  \
    if ((h)->prof_on) {                                                          \
      ea__ = prof_event(h);                                                      \
      eb__ = prof_event(h);                                                      \
      cudaEventRecord(ea__, (st));                                               \
    }                                                                            \
    cudaError_t e__ = (call);                                                    \
    (h)->launches++;                                                             \
    if ((h)->prof_on) {                                                          \
      cudaEventRecord(eb__, (st));                                               \
      (h)->prof_pending.push_back(prism_handle::ProfEntry{(cat), (double)(work), ea__, eb__}); \
    }                                                                            \
    if (e__ != cudaSuccess) return cuda_fail((h), e__, #call);                   \
  } while (0)

void prof_collect(prism_handle* h) {
  for (auto& p : h->prof_pending) {
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, p.a, p.b) == cudaSuccess) {
      h->prof_acc[p.cat].ms += ms;
      h->prof_acc[p.cat].work += p.work;
      h->prof_acc[p.cat].launches += 1;
    }
    h->prof_pool.push_back(p.a);
    h->prof_pool.push_back(p.b);
  }
  h->prof_pending.clear();
}

template <typename T>
cudaError_t dev_alloc(prism_handle* h, T** p, size_t count) {
  size_t bytes = std::max<size_t>(count * sizeof(T), 256);
  void* q = nullptr;
  cudaError_t e = cudaMalloc(&q, bytes);
  if (e != cudaSuccess) return e;
  h->dev_allocs.push_back(q);
  h->workspace_bytes += (int64_t)bytes;
  *p = reinterpret_cast<T*>(q);
  return cudaSuccess;
}

template <typename T>
cudaError_t host_alloc(prism_handle* h, T** p, size_t count) {
  void* q = nullptr;
  cudaError_t e = cudaMallocHost(&q, std::max<size_t>(count * sizeof(T), 64));
  if (e != cudaSuccess) return e;
  h->host_allocs.push_back(q);
  *p = reinterpret_cast<T*>(q);
  return cudaSuccess;
}

size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// Bytes of per-token chunk intermediates: normed input, qkv, attention output, SwiGLU output.
size_t per_token_bytes(const prism_model_cfg& c, int esz) {
  const size_t nqkv = (size_t)(c.n_q_heads + 2 * c.n_kv_heads) * c.head_dim;
  return ((size_t)c.hidden + nqkv + (size_t)c.n_q_heads * c.head_dim + (size_t)c.ffn) * esz;
}

// Bytes of an [n, k] layer matrix as the caller stores it (and as it crosses the host link when streamed).
size_t matrix_bytes(const prism_handle* h, size_t n, size_t k) {
  return h->w4 ? w4_blob_bytes(n, k, (size_t)h->cfg.quant_group) : n * k * (size_t)h->esz;
}

LayerDev layer_in_slot(const prism_handle* h, int s) {
  const unsigned char* b = h->slot[s];
  if (h->enc)  // the four matrices; the vectors were widened to fp32 device copies at creation
    return LayerDev{nullptr, b + h->off_qkv, nullptr, nullptr, b + h->off_o, nullptr, b + h->off_gate, b + h->off_gate,
                    b + h->off_down};
  LayerDev d;
  d.g_attn = b + h->off_g_attn;
  d.w_qkv = b + h->off_qkv;
  d.g_q = b + h->off_gq;
  d.g_k = b + h->off_gk;
  d.w_o = b + h->off_o;
  d.g_ffn = b + h->off_g_ffn;
  d.w_gate = b + h->off_gate;
  d.w_up = b + h->off_up;
  d.w_down = b + h->off_down;
  return d;
}

LayerDev layer_resident(const prism_handle* h, int l) {
  if (h->enc) {  // the two FFN maps take the places of gate and down
    const prism_encoder_layer_weights& e = h->enc_layers[l];
    return LayerDev{nullptr, e.w_qkv, nullptr, nullptr, e.w_o, nullptr, e.w_ffn1, e.w_ffn1, e.w_ffn2};
  }
  const prism_layer_weights& w = h->layers[l];
  return LayerDev{w.g_attn, w.w_qkv, w.g_q, w.g_k, w.w_o, w.g_ffn, w.w_gate, w.w_up, w.w_down};
}

cudaError_t build_maps(const prism_handle* h, const LayerDev& d, LayerMaps* m) {
  const prism_model_cfg& c = h->cfg;
  const uint64_t nqkv = (uint64_t)(c.n_q_heads + 2 * c.n_kv_heads) * c.head_dim;
  const uint64_t hd = (uint64_t)c.n_q_heads * c.head_dim;
  cudaError_t e;
  if ((e = make_tma_2d_bf16(&m->qkv, d.w_qkv, nqkv, c.hidden, 128, 64))) return e;
  if ((e = make_tma_2d_bf16(&m->o, d.w_o, c.hidden, hd, 128, 64))) return e;
  if ((e = make_tma_2d_bf16(&m->gate, d.w_gate, c.ffn, c.hidden, 128, 64))) return e;
  if ((e = make_tma_2d_bf16(&m->up, d.w_up, c.ffn, c.hidden, 128, 64))) return e;
  if ((e = make_tma_2d_bf16(&m->down, d.w_down, c.hidden, c.ffn, 128, 64))) return e;
  return cudaSuccess;
}

// Enqueue the host->device copy of layer l into slot s on the copy stream.
int enqueue_layer_copy(prism_handle* h, int l, int s) {
  const prism_model_cfg& c = h->cfg;
  const size_t e = h->esz, d = c.hidden, dh = c.head_dim;
  const size_t nqkv = (size_t)(c.n_q_heads + 2 * c.n_kv_heads) * dh, hd = (size_t)c.n_q_heads * dh;
  unsigned char* b = h->slot[s];
  cudaStream_t cs = h->copy_stream;
  if (h->enc) {
    const prism_encoder_layer_weights& w = h->enc_layers[l];
    PRISM_CUDA(h, cudaMemcpyAsync(b + h->off_qkv, w.w_qkv, matrix_bytes(h, nqkv, d), cudaMemcpyHostToDevice, cs));
    PRISM_CUDA(h, cudaMemcpyAsync(b + h->off_o, w.w_o, matrix_bytes(h, d, hd), cudaMemcpyHostToDevice, cs));
    PRISM_CUDA(h, cudaMemcpyAsync(b + h->off_gate, w.w_ffn1, matrix_bytes(h, c.ffn, d), cudaMemcpyHostToDevice, cs));
    PRISM_CUDA(h, cudaMemcpyAsync(b + h->off_down, w.w_ffn2, matrix_bytes(h, d, c.ffn), cudaMemcpyHostToDevice, cs));
    PRISM_CUDA(h, cudaEventRecord(h->ev_copied[s], cs));
    return PRISM_OK;
  }
  const prism_layer_weights& w = h->layers[l];
  PRISM_CUDA(h, cudaMemcpyAsync(b + h->off_g_attn, w.g_attn, d * e, cudaMemcpyHostToDevice, cs));
  PRISM_CUDA(h, cudaMemcpyAsync(b + h->off_qkv, w.w_qkv, matrix_bytes(h, nqkv, d), cudaMemcpyHostToDevice, cs));
  if (c.qk_norm) {
    PRISM_CUDA(h, cudaMemcpyAsync(b + h->off_gq, w.g_q, dh * e, cudaMemcpyHostToDevice, cs));
    PRISM_CUDA(h, cudaMemcpyAsync(b + h->off_gk, w.g_k, dh * e, cudaMemcpyHostToDevice, cs));
  }
  PRISM_CUDA(h, cudaMemcpyAsync(b + h->off_o, w.w_o, matrix_bytes(h, d, hd), cudaMemcpyHostToDevice, cs));
  PRISM_CUDA(h, cudaMemcpyAsync(b + h->off_g_ffn, w.g_ffn, d * e, cudaMemcpyHostToDevice, cs));
  PRISM_CUDA(h, cudaMemcpyAsync(b + h->off_gate, w.w_gate, matrix_bytes(h, c.ffn, d), cudaMemcpyHostToDevice, cs));
  PRISM_CUDA(h, cudaMemcpyAsync(b + h->off_up, w.w_up, matrix_bytes(h, c.ffn, d), cudaMemcpyHostToDevice, cs));
  PRISM_CUDA(h, cudaMemcpyAsync(b + h->off_down, w.w_down, matrix_bytes(h, d, c.ffn), cudaMemcpyHostToDevice, cs));
  PRISM_CUDA(h, cudaEventRecord(h->ev_copied[s], cs));
  return PRISM_OK;
}

int validate_cfg(const prism_model_cfg& c, std::string* why) {
  auto bad = [&](const char* m) { *why = m; return PRISM_ERR_INVALID_ARG; };
  if (c.n_layers < 1 || c.n_layers > PRISM_MAX_LAYERS) return bad("n_layers out of range");
  if (c.hidden < 4 || c.n_q_heads < 1 || c.n_kv_heads < 1 || c.head_dim < 2 || c.ffn < 1 || c.vocab < 2)
    return bad("non-positive model dimension");
  if (c.n_q_heads % c.n_kv_heads) return bad("n_q_heads must be a multiple of n_kv_heads");
  if (c.dtype != PRISM_FP32 && c.dtype != PRISM_BF16) return bad("dtype must be PRISM_FP32 or PRISM_BF16");
  if (c.max_seq_len < 1 || c.max_candidates < 1 || c.max_total_tokens < 1) return bad("maxima must be positive");
  if (c.max_candidates > PRISM_MAX_CANDIDATES) return bad("max_candidates exceeds PRISM_MAX_CANDIDATES");
  if (c.activation_budget_bytes < 0) return bad("negative activation budget");
  if (c.weight_residency != PRISM_WEIGHTS_DEVICE && c.weight_residency != PRISM_WEIGHTS_HOST_STREAMED)
    return bad("unknown weight_residency");
  if (!(c.rope_theta > 0.f) || !(c.rms_eps >= 0.f)) return bad("rope_theta must be > 0 and rms_eps >= 0");
  if (c.embed_cache_rows < 0) return bad("negative embed_cache_rows");
  if (c.hidden_offload != 0 && c.hidden_offload != 1) return bad("hidden_offload must be 0 or 1");
  if (c.hidden_offload && c.activation_budget_bytes <= 0) return bad("hidden_offload needs an activation budget");
  if (c.shared_prefix != PRISM_PREFIX_AUTO && c.shared_prefix != PRISM_PREFIX_OFF) return bad("shared_prefix must be 0 or 1");
  if (c.arch != PRISM_ARCH_DECODER && c.arch != PRISM_ARCH_ENCODER) return bad("unknown arch");
  if (c.weight_format != PRISM_WFMT_PLAIN && c.weight_format != PRISM_WFMT_W4) return bad("unknown weight_format");
  if (c.weight_format == PRISM_WFMT_W4) {
    if (c.quant_group != 32 && c.quant_group != 64 && c.quant_group != 128) return bad("quant_group must be 32, 64 or 128");
    if (c.dtype != PRISM_BF16) { *why = "W4 weights need bf16"; return PRISM_ERR_UNSUPPORTED; }
    if (c.hidden % c.quant_group || c.ffn % c.quant_group || (c.n_q_heads * c.head_dim) % c.quant_group)
      return bad("quant_group must divide hidden, ffn and n_q_heads * head_dim");
  }
  auto unsup = [&](const char* m) { *why = m; return PRISM_ERR_UNSUPPORTED; };
  const bool enc = c.arch == PRISM_ARCH_ENCODER;
  if (enc) {
    if (c.qk_norm) return bad("the encoder stack has no QK-norm");
    if (c.pos_offset < 0 || c.max_positions < 1 || (long long)c.max_seq_len + c.pos_offset > c.max_positions)
      return bad("max_seq_len + pos_offset exceeds max_positions");
    if (c.gemm_impl != PRISM_IMPL_AUTO && c.gemm_impl != PRISM_IMPL_SIMT) return unsup("encoder GEMMs: AUTO or SIMT");
    if (c.attention_impl == PRISM_IMPL_MMA) return unsup("encoder attention: AUTO, SOLO or SIMT");
  }
  if (c.head_dim % 2 || c.head_dim > 256) return unsup("head_dim must be even and <= 256");
  if (c.hidden % 4 || c.hidden > 8192) return unsup("hidden must be a multiple of 4 and <= 8192");
  if (c.dtype == PRISM_BF16) {
    if (c.hidden % 8 || c.ffn % 8 || c.head_dim % 8) return unsup("bf16 mode needs hidden, ffn, head_dim multiples of 8");
    if (!enc && c.gemm_impl != PRISM_IMPL_SIMT && (c.ffn % 128)) return unsup("tensor-core SwiGLU needs ffn multiple of 128");
    if (c.attention_impl != PRISM_IMPL_SIMT && c.head_dim != 128 && !(enc && c.head_dim == 64))
      return unsup("tensor-core attention needs head_dim 128 (encoder stack: 128 or 64)");
  }
  return PRISM_OK;
}

}  // namespace

extern "C" {

const char* prism_status_str(int s) {
  switch (s) {
    case PRISM_OK: return "PRISM_OK";
    case PRISM_ERR_INVALID_ARG: return "PRISM_ERR_INVALID_ARG";
    case PRISM_ERR_SHAPE_LIMIT: return "PRISM_ERR_SHAPE_LIMIT";
    case PRISM_ERR_BAD_INPUT: return "PRISM_ERR_BAD_INPUT";
    case PRISM_ERR_BUDGET: return "PRISM_ERR_BUDGET";
    case PRISM_ERR_CUDA: return "PRISM_ERR_CUDA";
    case PRISM_ERR_TIMEOUT: return "PRISM_ERR_TIMEOUT";
    case PRISM_ERR_NOMEM: return "PRISM_ERR_NOMEM";
    case PRISM_ERR_UNSUPPORTED: return "PRISM_ERR_UNSUPPORTED";
    default: return "PRISM_ERR_UNKNOWN";
  }
}

const char* prism_last_error(const prism_handle* h) { return h ? h->err.c_str() : ""; }

int64_t prism_launch_count(const prism_handle* h) { return h ? h->launches : 0; }

int prism_embed_cache_stats(const prism_handle* h, int64_t* hits, int64_t* misses, int64_t* evictions) {
  if (!h) return PRISM_ERR_INVALID_ARG;
  if (hits) *hits = h->cache_hits;
  if (misses) *misses = h->cache_misses;
  if (evictions) *evictions = h->cache_evictions;
  return PRISM_OK;
}

int prism_profile(prism_handle* h, int enable) {
  if (!h) return PRISM_ERR_INVALID_ARG;
  h->prof_on = enable != 0;
  return PRISM_OK;
}

int prism_profile_read(prism_handle* h, prism_kernel_stat* out, int reset) {
  if (!h || !out) return PRISM_ERR_INVALID_ARG;
  for (int i = 0; i < PRISM_N_KERNEL_CLASSES; ++i) {
    out[i] = h->prof_acc[i];
    if (reset) h->prof_acc[i] = prism_kernel_stat{};
  }
  return PRISM_OK;
}

void prism_destroy(prism_handle* h) {
  if (!h) return;
  cudaDeviceSynchronize();
  for (void* p : h->dev_allocs) cudaFree(p);
  for (void* p : h->host_allocs) cudaFreeHost(p);
  for (int s = 0; s < 2; ++s) {
    if (h->ev_copied[s]) cudaEventDestroy(h->ev_copied[s]);
    if (h->ev_freed[s]) cudaEventDestroy(h->ev_freed[s]);
  }
  if (h->copy_stream) cudaStreamDestroy(h->copy_stream);
  if (h->in_stream) cudaStreamDestroy(h->in_stream);
  if (h->out_stream) cudaStreamDestroy(h->out_stream);
  for (int i = 0; i < 3; ++i) {
    if (h->ev_in[i]) cudaEventDestroy(h->ev_in[i]);
    if (h->ev_done[i]) cudaEventDestroy(h->ev_done[i]);
    if (h->ev_slot_out[i]) cudaEventDestroy(h->ev_slot_out[i]);
  }
  if (h->ev_main) cudaEventDestroy(h->ev_main);
  for (cudaEvent_t e : h->ev_chunk_out) cudaEventDestroy(e);
  for (auto& p : h->prof_pending) { cudaEventDestroy(p.a); cudaEventDestroy(p.b); }
  for (cudaEvent_t e : h->prof_pool) cudaEventDestroy(e);
  delete h;
}

static int create_impl(prism_handle* h, const prism_model_cfg* cfg, const prism_weights* w,
                       const prism_encoder_weights* ew) {
  const prism_model_cfg& c = *cfg;
  h->cfg = c;
  h->enc = ew != nullptr;
  h->w4 = c.weight_format == PRISM_WFMT_W4;
  h->esz = c.dtype == PRISM_BF16 ? 2 : 4;
  h->tc = c.dtype == PRISM_BF16 && (c.gemm_impl == PRISM_IMPL_AUTO || c.gemm_impl == PRISM_IMPL_SOLO);
  h->pair = c.gemm_impl == PRISM_IMPL_AUTO;
  // 0: CUDA cores, 1: tcgen05 one query head per CTA, 2: mma.sync, 3: tcgen05 two query heads per CTA: pairs that
  // share a K / V head (even group sizes; head_dim 128 or 64) or, at head_dim 64, pairs of heads with a K / V head each
  const int group_sz = c.n_q_heads / c.n_kv_heads;
  const bool two_heads = (group_sz & 1) == 0 ? (c.head_dim == 128 || c.head_dim == 64)
                                             : (group_sz == 1 && c.head_dim == 64 && (c.n_q_heads & 1) == 0);
  h->fa = c.dtype != PRISM_BF16 ? 0
          : c.attention_impl == PRISM_IMPL_AUTO ? (two_heads ? 3 : 1)
          : c.attention_impl == PRISM_IMPL_SOLO ? 1
          : c.attention_impl == PRISM_IMPL_MMA  ? 2 : 0;
  const bool streamed = c.weight_residency == PRISM_WEIGHTS_HOST_STREAMED;
  if (h->enc) {
    const void* glob[] = {ew->embed, ew->pos_embed, ew->type_embed, ew->emb_ln_g, ew->emb_ln_b, ew->head_dense_w,
                          ew->head_dense_b, ew->head_out_w, ew->head_out_b, ew->layers};
    for (const void* p : glob)
      if (!p) return fail(h, PRISM_ERR_INVALID_ARG, "null weight pointer");
    if ((reinterpret_cast<uintptr_t>(ew->embed) & 15) || (reinterpret_cast<uintptr_t>(ew->pos_embed) & 15) ||
        (reinterpret_cast<uintptr_t>(ew->head_dense_w) & 15))
      return fail(h, PRISM_ERR_INVALID_ARG, "embedding tables and head matrix must be 16-byte aligned");
    h->embed = ew->embed;
    h->pos_embed = ew->pos_embed;
    h->head_dense_w = ew->head_dense_w;
    h->enc_layers.assign(ew->layers, ew->layers + c.n_layers);
    for (const prism_encoder_layer_weights& lw : h->enc_layers) {
      const void* mats[] = {lw.w_qkv, lw.w_o, lw.w_ffn1, lw.w_ffn2};
      for (const void* p : mats)
        if (!p || (reinterpret_cast<uintptr_t>(p) & 15)) return fail(h, PRISM_ERR_INVALID_ARG, "layer tensor null or not 16-byte aligned");
      const void* vecs[] = {lw.b_qkv, lw.b_o, lw.ln1_g, lw.ln1_b, lw.b_ffn1, lw.b_ffn2, lw.ln2_g, lw.ln2_b};
      for (const void* p : vecs)
        if (!p) return fail(h, PRISM_ERR_INVALID_ARG, "layer vector null");
    }
  } else {
  if (!w->embed || !w->g_final || !w->score_head || !w->layers) return fail(h, PRISM_ERR_INVALID_ARG, "null weight pointer");
  h->embed = w->embed;
  h->g_final = w->g_final;
  h->score_head = w->score_head;
  h->layers.assign(w->layers, w->layers + c.n_layers);
  }
  for (int l = 0; l < c.n_layers && !h->enc; ++l) {
    const prism_layer_weights& lw = h->layers[l];
    const void* req[] = {lw.g_attn, lw.w_qkv, lw.w_o, lw.g_ffn, lw.w_gate, lw.w_up, lw.w_down};
    for (const void* p : req)
      if (!p || (reinterpret_cast<uintptr_t>(p) & 15)) return fail(h, PRISM_ERR_INVALID_ARG, "layer tensor null or not 16-byte aligned");
    if (c.qk_norm && (!lw.g_q || !lw.g_k)) return fail(h, PRISM_ERR_INVALID_ARG, "qk_norm set but g_q/g_k null");
  }

  const size_t D = c.hidden, T = c.max_total_tokens, N = c.max_candidates;
  const size_t nqkv = (size_t)(c.n_q_heads + 2 * c.n_kv_heads) * c.head_dim, hd = (size_t)c.n_q_heads * c.head_dim;
  // Chunked execution: hidden states of all sequences (both ping-pong buffers) + one chunk's
  // intermediates must fit the activation budget.
  const size_t hidden_bytes = 2 * T * D * sizeof(float);
  const size_t ptb = per_token_bytes(c, h->esz);
  size_t chunk = T;
  h->offload = c.hidden_offload != 0;
  if (h->offload) {
    // three chunks of hidden states and one chunk of intermediates on the device
    const size_t per_row = 3 * D * sizeof(float) + ptb;
    chunk = std::min(T, (size_t)c.activation_budget_bytes / per_row);
    if (chunk < (size_t)c.max_seq_len)
      return fail(h, PRISM_ERR_BUDGET, "activation budget cannot hold three chunks of one max_seq_len sequence");
  } else if (c.activation_budget_bytes > 0) {
    const size_t budget = (size_t)c.activation_budget_bytes;
    if (budget <= hidden_bytes || (budget - hidden_bytes) / ptb < (size_t)c.max_seq_len)
      return fail(h, PRISM_ERR_BUDGET, "activation budget cannot hold the hidden states plus one max_seq_len sequence");
    chunk = std::min(T, (budget - hidden_bytes) / ptb);
  }
  h->chunk_tokens = (int)chunk;

  if (h->offload) {
    PRISM_CUDA(h, host_alloc(h, &h->x[0], T * D));
    PRISM_CUDA(h, host_alloc(h, &h->x[1], T * D));
    for (int i = 0; i < 3; ++i) {
      PRISM_CUDA(h, dev_alloc(h, &h->xc[i], chunk * D));
      PRISM_CUDA(h, cudaEventCreateWithFlags(&h->ev_in[i], cudaEventDisableTiming));
      PRISM_CUDA(h, cudaEventCreateWithFlags(&h->ev_done[i], cudaEventDisableTiming));
      PRISM_CUDA(h, cudaEventCreateWithFlags(&h->ev_slot_out[i], cudaEventDisableTiming));
    }
    PRISM_CUDA(h, cudaEventCreateWithFlags(&h->ev_main, cudaEventDisableTiming));
    PRISM_CUDA(h, cudaStreamCreateWithFlags(&h->in_stream, cudaStreamNonBlocking));
    PRISM_CUDA(h, cudaStreamCreateWithFlags(&h->out_stream, cudaStreamNonBlocking));
  } else {
    PRISM_CUDA(h, dev_alloc(h, &h->x[0], T * D));
    PRISM_CUDA(h, dev_alloc(h, &h->x[1], T * D));
  }
  PRISM_CUDA(h, dev_alloc(h, &h->tokens, T));
  PRISM_CUDA(h, dev_alloc(h, &h->pos, T));
  for (int i = 0; i < 2; ++i) {
    PRISM_CUDA(h, dev_alloc(h, &h->cu[i], N + 1));
    PRISM_CUDA(h, dev_alloc(h, &h->seq2orig[i], N));
  }
  PRISM_CUDA(h, dev_alloc(h, &h->old_of_new, N));
  PRISM_CUDA(h, dev_alloc(h, (unsigned char**)&h->a_norm, chunk * D * h->esz));
  PRISM_CUDA(h, dev_alloc(h, (unsigned char**)&h->qkv, chunk * nqkv * h->esz));
  PRISM_CUDA(h, dev_alloc(h, (unsigned char**)&h->attn, chunk * hd * h->esz));
  PRISM_CUDA(h, dev_alloc(h, (unsigned char**)&h->hbuf, chunk * (size_t)c.ffn * h->esz));
  PRISM_CUDA(h, dev_alloc(h, (unsigned char**)&h->qkv_prefix, 128 * nqkv * h->esz));
  PRISM_CUDA(h, dev_alloc(h, &h->scores, N));
  PRISM_CUDA(h, dev_alloc(h, &h->res_idx, N));
  PRISM_CUDA(h, dev_alloc(h, &h->res_score, N));
  PRISM_CUDA(h, dev_alloc(h, &h->w_diff, D));
  PRISM_CUDA(h, dev_alloc(h, &h->rope_cos, (size_t)c.max_seq_len * (c.head_dim / 2)));
  PRISM_CUDA(h, dev_alloc(h, &h->rope_sin, (size_t)c.max_seq_len * (c.head_dim / 2)));
  if (c.head_dim == 128) PRISM_CUDA(h, dev_alloc(h, &h->rope_fused, (size_t)c.max_seq_len * 128));
  PRISM_CUDA(h, dev_alloc(h, &h->errword, 1));
  PRISM_CUDA(h, dev_alloc(h, &h->state, 1));
  PRISM_CUDA(h, dev_alloc(h, &h->recs, (size_t)c.n_layers));
  PRISM_CUDA(h, dev_alloc(h, &h->trace_scores, (size_t)c.n_layers * N));
  PRISM_CUDA(h, dev_alloc(h, &h->trace_ids, (size_t)c.n_layers * N));
  PRISM_CUDA(h, dev_alloc(h, &h->owned_dev, N));
  if (c.embed_cache_rows > 0) {
    if ((reinterpret_cast<uintptr_t>(h->embed) & 15) || (D * h->esz) % 16)
      return fail(h, PRISM_ERR_INVALID_ARG, "the host embedding table must be 16-byte aligned with rows of a multiple of 16 bytes");
    cudaPointerAttributes pa{};
    if (cudaPointerGetAttributes(&pa, h->embed) != cudaSuccess || pa.type != cudaMemoryTypeHost) {
      cudaGetLastError();
      return fail(h, PRISM_ERR_INVALID_ARG, "embed_cache_rows > 0 needs the embedding table in pinned host memory");
    }
    h->cache_rows = std::min(c.embed_cache_rows, c.vocab);
    const size_t C = (size_t)h->cache_rows, ntok = T + (size_t)c.max_seq_len;
    PRISM_CUDA(h, dev_alloc(h, &h->cache_dev, C * D * h->esz));
    PRISM_CUDA(h, dev_alloc(h, &h->tok2slot_dev, (size_t)c.vocab));
    PRISM_CUDA(h, dev_alloc(h, &h->pairs_dev, 2 * C));
    PRISM_CUDA(h, host_alloc(h, &h->h_tokens, ntok));
    PRISM_CUDA(h, host_alloc(h, &h->h_pairs, 2 * C));
    PRISM_CUDA(h, cudaMemset(h->tok2slot_dev, 0, (size_t)c.vocab * sizeof(int)));
    h->slot_of_tok.assign((size_t)c.vocab, -1);
    h->tok_of_slot.assign(C, -1);
    h->slot_stamp.assign(C, 0);
    h->tok_seen.assign((size_t)c.vocab, 0);
  }
  PRISM_CUDA(h, dev_alloc(h, (unsigned char**)&h->route_scratch, route_scratch_bytes((int)N)));
  PRISM_CUDA(h, dev_alloc(h, &h->in_query, (size_t)c.max_seq_len));
  PRISM_CUDA(h, dev_alloc(h, &h->in_cand, T));
  PRISM_CUDA(h, dev_alloc(h, &h->in_off, N + 1));
  PRISM_CUDA(h, dev_alloc(h, &h->out_idx, N));
  PRISM_CUDA(h, dev_alloc(h, &h->out_score, N));
  PRISM_CUDA(h, host_alloc(h, &h->h_cu, N + 1));
  PRISM_CUDA(h, host_alloc(h, &h->h_cu_next, N + 1));
  PRISM_CUDA(h, host_alloc(h, &h->h_off, N + 1));
  PRISM_CUDA(h, host_alloc(h, &h->h_state, 1));
  PRISM_CUDA(h, host_alloc(h, &h->h_err, 1));
  PRISM_CUDA(h, cudaMemset(h->errword, 0, sizeof(int)));

  if (streamed) {
    const size_t e = h->esz, dh = c.head_dim;
    size_t off = 0;
    auto place_b = [&](size_t* o, size_t bytes) { *o = off; off = align_up(off + bytes, 256); };
    auto place = [&](size_t* o, size_t elems) { place_b(o, elems * e); };
    if (!h->enc) place(&h->off_g_attn, D);
    place_b(&h->off_qkv, matrix_bytes(h, nqkv, D));
    if (!h->enc) place(&h->off_gq, dh);
    if (!h->enc) place(&h->off_gk, dh);
    place_b(&h->off_o, matrix_bytes(h, D, hd));
    if (!h->enc) place(&h->off_g_ffn, D);
    place_b(&h->off_gate, matrix_bytes(h, c.ffn, D));
    if (!h->enc) place_b(&h->off_up, matrix_bytes(h, c.ffn, D));
    place_b(&h->off_down, matrix_bytes(h, D, c.ffn));
    h->slot_bytes = off;
    for (int s = 0; s < 2; ++s) PRISM_CUDA(h, dev_alloc(h, &h->slot[s], off));
    PRISM_CUDA(h, cudaStreamCreateWithFlags(&h->copy_stream, cudaStreamNonBlocking));
    for (int s = 0; s < 2; ++s) {
      PRISM_CUDA(h, cudaEventCreateWithFlags(&h->ev_copied[s], cudaEventDisableTiming));
      PRISM_CUDA(h, cudaEventCreateWithFlags(&h->ev_freed[s], cudaEventDisableTiming));
    }
  }

  if (h->w4) {
    const size_t F = (size_t)c.ffn, elems[5] = {nqkv * D, D * hd, F * D, F * D, D * F};
    for (int i = 0; i < 5; ++i) PRISM_CUDA(h, dev_alloc(h, (unsigned char**)&h->wq[i], elems[i] * 2));
  }
  if (h->tc) {
    PRISM_CUDA(h, make_tma_2d_bf16(&h->map_a_norm, h->a_norm, chunk, D, 128, 64));
    PRISM_CUDA(h, make_tma_2d_bf16(&h->map_attn, h->attn, chunk, hd, 128, 64));
    PRISM_CUDA(h, make_tma_2d_bf16(&h->map_hbuf, h->hbuf, chunk, c.ffn, 128, 64));
    if (h->w4) {
      // the GEMMs always read the bf16 scratch: one set of weight maps
      const LayerDev d{nullptr, h->wq[0], nullptr, nullptr, h->wq[1], nullptr, h->wq[2], h->wq[3], h->wq[4]};
      PRISM_CUDA(h, build_maps(h, d, &h->maps_w4));
    } else if (streamed) {
      h->maps.resize(2);
      for (int s = 0; s < 2; ++s) PRISM_CUDA(h, build_maps(h, layer_in_slot(h, s), &h->maps[s]));
    } else {
      h->maps.resize(c.n_layers);
      for (int l = 0; l < c.n_layers; ++l) PRISM_CUDA(h, build_maps(h, layer_resident(h, l), &h->maps[l]));
    }
  }

  if (h->enc) {
    // fp32 copies of every vector (biases, LayerNorm gain and shift, head vectors): one buffer, 16-byte aligned slices
    const size_t F = (size_t)c.ffn;
    const size_t per_layer = align_up(nqkv, 4) + 6 * align_up(D, 4) + align_up(F, 4);
    const size_t glob = 5 * align_up(D, 4) + 4;
    float* buf = nullptr;
    PRISM_CUDA(h, dev_alloc(h, &buf, per_layer * c.n_layers + glob));
    float* cur = buf;
    auto widen = [&](const void* src, size_t n, const float** dst) -> cudaError_t {
      *dst = cur;
      cudaError_t e = launch_to_f32(src, c.dtype, (int)n, cur, 0);
      cur += align_up(n, 4);
      return e;
    };
    PRISM_CUDA(h, widen(ew->type_embed, D, &h->type_f));
    PRISM_CUDA(h, widen(ew->emb_ln_g, D, &h->emb_g));
    PRISM_CUDA(h, widen(ew->emb_ln_b, D, &h->emb_b));
    PRISM_CUDA(h, widen(ew->head_dense_b, D, &h->head_db));
    PRISM_CUDA(h, widen(ew->head_out_w, D, &h->head_ow));
    PRISM_CUDA(h, widen(ew->head_out_b, 1, &h->head_ob));
    PRISM_CUDA(h, dev_alloc(h, &h->probe_scratch, 2 * N * D));
    h->enc_vec.resize(c.n_layers);
    for (int l = 0; l < c.n_layers; ++l) {
      const prism_encoder_layer_weights& lw = h->enc_layers[l];
      EncVec& v = h->enc_vec[l];
      PRISM_CUDA(h, widen(lw.b_qkv, nqkv, &v.b_qkv));
      PRISM_CUDA(h, widen(lw.b_o, D, &v.b_o));
      PRISM_CUDA(h, widen(lw.ln1_g, D, &v.ln1_g));
      PRISM_CUDA(h, widen(lw.ln1_b, D, &v.ln1_b));
      PRISM_CUDA(h, widen(lw.b_ffn1, F, &v.b_ffn1));
      PRISM_CUDA(h, widen(lw.b_ffn2, D, &v.b_ffn2));
      PRISM_CUDA(h, widen(lw.ln2_g, D, &v.ln2_g));
      PRISM_CUDA(h, widen(lw.ln2_b, D, &v.ln2_b));
    }
  } else {
    PRISM_LAUNCH(h, launch_rope_table(h->rope_cos, h->rope_sin, c.max_seq_len, c.head_dim, c.rope_theta, 0));
    if (h->rope_fused) PRISM_LAUNCH(h, launch_rope_table_fused(h->rope_fused, c.max_seq_len, c.rope_theta, 0));
    PRISM_LAUNCH(h, launch_score_diff(h->score_head, c.dtype, c.hidden, h->w_diff, 0));
  }
  PRISM_CUDA(h, cudaDeviceSynchronize());
  return PRISM_OK;
}

static int create_any(const prism_model_cfg* cfg, const prism_weights* w, const prism_encoder_weights* ew,
                      prism_handle** out);

int prism_create(const prism_model_cfg* cfg, const prism_weights* w, prism_handle** out) {
  if (out) *out = nullptr;
  if (!cfg || !w || !out || cfg->arch != PRISM_ARCH_DECODER) return PRISM_ERR_INVALID_ARG;
  return create_any(cfg, w, nullptr, out);
}

int prism_create_encoder(const prism_model_cfg* cfg, const prism_encoder_weights* w, prism_handle** out) {
  if (out) *out = nullptr;
  if (!cfg || !w || !out || cfg->arch != PRISM_ARCH_ENCODER) return PRISM_ERR_INVALID_ARG;
  return create_any(cfg, nullptr, w, out);
}

static int create_any(const prism_model_cfg* cfg, const prism_weights* w, const prism_encoder_weights* ew,
                      prism_handle** out) {
  std::string why;
  int rc = validate_cfg(*cfg, &why);
  if (rc != PRISM_OK) return rc;
  prism_handle* h = new (std::nothrow) prism_handle();
  if (!h) return PRISM_ERR_NOMEM;
  rc = create_impl(h, cfg, w, ew);
  if (rc != PRISM_OK) {
    prism_destroy(h);
    return rc;
  }
  *out = h;
  return PRISM_OK;
}

}  // extern "C"

namespace {

int validate_schedule(const prism_handle* h, const prism_prune_schedule* s, int k_eff, std::string* why) {
  auto bad = [&](const char* m) { *why = m; return PRISM_ERR_INVALID_ARG; };
  if (!s) return PRISM_OK;
  if (s->mode != PRISM_PRUNE_NONE && s->mode != PRISM_PRUNE_FIXED_KEEP && s->mode != PRISM_PRUNE_CLUSTER)
    return bad("unknown prune mode");
  if (s->mode == PRISM_PRUNE_NONE) return PRISM_OK;
  if (s->n_probes < 0 || (s->n_probes > 0 && !s->probe_layers)) return bad("probe_layers missing");
  int prev = 0;
  for (int j = 0; j < s->n_probes; ++j) {
    const int l = s->probe_layers[j];
    if (l <= prev || l >= h->cfg.n_layers) return bad("probe_layers must be strictly increasing in [1, n_layers)");
    prev = l;
  }
  if (s->mode == PRISM_PRUNE_FIXED_KEEP) {
    if (s->n_probes > 0 && !s->keep_counts) return bad("keep_counts missing");
    for (int j = 0; j < s->n_probes; ++j)
      if (s->keep_counts[j] < k_eff || s->keep_counts[j] < 1) return bad("keep_counts must be >= K");
  } else {
    const int k = s->n_clusters == 0 ? 3 : s->n_clusters;
    if (k < 2 || k > PRISM_MAX_CLUSTERS) return bad("n_clusters must be in [2, PRISM_MAX_CLUSTERS]");
    if (s->std_ddof != 0 && s->std_ddof != 1) return bad("std_ddof must be 0 or 1");
    if (s->cv_threshold != s->cv_threshold) return bad("cv_threshold is NaN");
  }
  return PRISM_OK;
}

// The direction the next kernel takes the rows in: opposite to its predecessor's, so that it starts on what
// was written last and is still in L2 (the layer's tensors are larger than L2 at full batch).  Kernels
// without a direction argument count as forward.
bool next_dir(prism_handle* h, bool supported) {
  const bool rev = supported && h->flip && !h->last_rev;
  h->last_rev = rev;
  return rev;
}

cudaError_t gemm_tc_any(prism_handle* h, const TmaDesc& a, const TmaDesc& b0, const TmaDesc& b1, void* out, float* resid,
                        int m, int n, int k, int epi, const QkvRopeArgs* qa, cudaStream_t st, const float* bias = nullptr) {
  const bool rev = next_dir(h, h->pair);
  return h->pair ? launch_gemm_tc2(a, b0, b1, out, resid, m, n, k, epi, qa, h->errword, st, rev, bias)
                 : launch_gemm_tc(a, b0, b1, out, resid, m, n, k, epi, qa, h->errword, st);
}

// One decoder block over rows [r0, r0+rows) (sequences [s0, s1)) of the live batch.
// x is the whole batch's hidden-state matrix, or (x_is_chunk) the buffer holding just this chunk's rows.
// prefix > 0: rows [0, prefix) of the batch are the query shared by all sequences, cu holds the sequences' own rows,
// max_len counts prefix + own rows; the chunk that starts at row 0 contains the prefix rows.
// chunk_of_many: 0 = the batch is one chunk; 1 = first of several chunks (it holds the prefix rows: their q/k/v are
// saved for the others); 2 = a later chunk (attention reads the saved prefix rows and writes none).
int run_layer_chunk(prism_handle* h, const LayerDev& W, const LayerMaps* maps, float* x, const int* cu_dev, int s0, int s1,
                    int r0, int rows, int max_len, cudaStream_t st, bool x_is_chunk = false, int prefix = 0,
                    int chunk_of_many = 0) {
  const prism_model_cfg& c = h->cfg;
  const int D = c.hidden, dh = c.head_dim;
  const int nqkv = (c.n_q_heads + 2 * c.n_kv_heads) * dh, hd = c.n_q_heads * dh;
  float* xr = x_is_chunk ? x : x + (size_t)r0 * D;
  const double esz = h->esz, R = rows;
  const double norm_bytes = R * D * (4.0 + esz);
  double attn_flops = 0.0;
  for (int s = s0; s < s1; ++s) {
    const double L = h->h_cu[s + 1] - h->h_cu[s] + prefix;
    attn_flops += (c.causal ? 2.0 : 4.0) * L * L * c.n_q_heads * dh;
  }
  PRISM_LAUNCH_P(h, st, PRISM_K_RMSNORM, norm_bytes, launch_rmsnorm(xr, W.g_attn, c.dtype, rows, D, c.rms_eps, h->a_norm, st, next_dir(h, true)));
  const bool fused_rope = h->tc && dh == 128;  // QK-norm + RoPE inside the QKV GEMM's epilogue
  if (fused_rope) {
    QkvRopeArgs qa{h->pos + r0, h->rope_fused, (const __nv_bfloat16*)W.g_q, (const __nv_bfloat16*)W.g_k,
                   c.n_q_heads, c.n_kv_heads, c.qk_norm, c.rms_eps};
    PRISM_LAUNCH_P(h, st, PRISM_K_GEMM_QKV, 2.0 * R * nqkv * D,
                   gemm_tc_any(h, h->map_a_norm, maps->qkv, maps->qkv, h->qkv, nullptr, rows, nqkv, D, kEpiQkvRope, &qa, st));
  } else if (h->tc)
    PRISM_LAUNCH_P(h, st, PRISM_K_GEMM_QKV, 2.0 * R * nqkv * D,
                   gemm_tc_any(h, h->map_a_norm, maps->qkv, maps->qkv, h->qkv, nullptr, rows, nqkv, D, kEpiStore, nullptr, st));
  else
    PRISM_LAUNCH_P(h, st, PRISM_K_GEMM_QKV, 2.0 * R * nqkv * D,
                   launch_gemm_simt(h->a_norm, W.w_qkv, nullptr, h->qkv, nullptr, rows, nqkv, D, c.dtype, kEpiStore, st));
  if (!fused_rope)
  PRISM_LAUNCH_P(h, st, PRISM_K_ROPE, 2.0 * R * (c.n_q_heads + c.n_kv_heads) * dh * esz,
                 launch_qknorm_rope(h->qkv, c.dtype, h->pos + r0, rows, c.n_q_heads, c.n_kv_heads, dh, c.qk_norm, W.g_q, W.g_k,
                                    c.rms_eps, h->rope_cos, h->rope_sin, st));
  if (h->fa != 3) next_dir(h, false);  // the other attention kernels walk forward
  if (prefix && chunk_of_many == 1)
    PRISM_CUDA(h, cudaMemcpyAsync(h->qkv_prefix, h->qkv, (size_t)prefix * nqkv * h->esz, cudaMemcpyDeviceToDevice, st));
  if (h->fa == 3)
    PRISM_LAUNCH_P(h, st, PRISM_K_ATTENTION, attn_flops,
                   launch_attention_tc2(h->qkv, h->attn, cu_dev, s0, s1 - s0, r0, rows, max_len, c.n_q_heads, c.n_kv_heads, c.causal,
                                        h->errword, st, next_dir(h, true), prefix,
                                        (prefix && chunk_of_many) ? h->qkv_prefix : nullptr, chunk_of_many != 2, dh));
  else if (h->fa == 1)
    PRISM_LAUNCH_P(h, st, PRISM_K_ATTENTION, attn_flops,
                   launch_attention_tc(h->qkv, h->attn, cu_dev, s0, s1 - s0, r0, rows, max_len, c.n_q_heads, c.n_kv_heads, c.causal,
                                       h->errword, st));
  else if (h->fa == 2)
    PRISM_LAUNCH_P(h, st, PRISM_K_ATTENTION, attn_flops,
                   launch_attention_mma(h->qkv, h->attn, cu_dev, s0, s1 - s0, r0, max_len, c.n_q_heads, c.n_kv_heads, c.causal, st));
  else
    PRISM_LAUNCH_P(h, st, PRISM_K_ATTENTION, attn_flops,
                   launch_attention_simt(h->qkv, h->attn, cu_dev, s0, s1 - s0, r0, max_len, c.n_q_heads, c.n_kv_heads, dh,
                                         c.causal, c.dtype, st));
  if (h->tc)
    PRISM_LAUNCH_P(h, st, PRISM_K_GEMM_O, 2.0 * R * D * hd,
                   gemm_tc_any(h, h->map_attn, maps->o, maps->o, nullptr, xr, rows, D, hd, kEpiResidual, nullptr, st));
  else
    PRISM_LAUNCH_P(h, st, PRISM_K_GEMM_O, 2.0 * R * D * hd,
                   launch_gemm_simt(h->attn, W.w_o, nullptr, nullptr, xr, rows, D, hd, c.dtype, kEpiResidual, st));
  PRISM_LAUNCH_P(h, st, PRISM_K_RMSNORM, norm_bytes, launch_rmsnorm(xr, W.g_ffn, c.dtype, rows, D, c.rms_eps, h->a_norm, st, next_dir(h, true)));
  if (h->tc)
    PRISM_LAUNCH_P(h, st, PRISM_K_GEMM_GATEUP, 4.0 * R * c.ffn * D,
                   gemm_tc_any(h, h->map_a_norm, maps->gate, maps->up, h->hbuf, nullptr, rows, c.ffn, D, kEpiSwiGLU, nullptr, st));
  else
    PRISM_LAUNCH_P(h, st, PRISM_K_GEMM_GATEUP, 4.0 * R * c.ffn * D,
                   launch_gemm_simt(h->a_norm, W.w_gate, W.w_up, h->hbuf, nullptr, rows, c.ffn, D, c.dtype, kEpiSwiGLU, st));
  if (h->tc)
    PRISM_LAUNCH_P(h, st, PRISM_K_GEMM_DOWN, 2.0 * R * D * c.ffn,
                   gemm_tc_any(h, h->map_hbuf, maps->down, maps->down, nullptr, xr, rows, D, c.ffn, kEpiResidual, nullptr, st));
  else
    PRISM_LAUNCH_P(h, st, PRISM_K_GEMM_DOWN, 2.0 * R * D * c.ffn,
                   launch_gemm_simt(h->hbuf, W.w_down, nullptr, nullptr, xr, rows, D, c.ffn, c.dtype, kEpiResidual, st));
  return PRISM_OK;
}

// One post-norm encoder block over the same rows.  The block starts with the LayerNorm its predecessor left
// pending (the embedding LayerNorm for block 0, else LN2 of block l - 1), so that, as in the decoder path, a
// chunk's normed GEMM input is produced right before it is consumed; LN2 of the last executed block is applied by
// the probe to the one row it reads.
int run_layer_chunk_encoder(prism_handle* h, int l, const LayerDev& W, const LayerMaps* maps, float* x, const int* cu_dev,
                            int s0, int s1, int r0, int rows, int max_len, cudaStream_t st, bool x_is_chunk = false) {
  const prism_model_cfg& c = h->cfg;
  const int D = c.hidden, dh = c.head_dim, F = c.ffn;
  const int nqkv = (c.n_q_heads + 2 * c.n_kv_heads) * dh, hd = c.n_q_heads * dh;
  float* xr = x_is_chunk ? x : x + (size_t)r0 * D;
  const EncVec& V = h->enc_vec[l];
  const float* g0 = l == 0 ? h->emb_g : h->enc_vec[l - 1].ln2_g;
  const float* b0 = l == 0 ? h->emb_b : h->enc_vec[l - 1].ln2_b;
  const double R = rows, norm_bytes = R * D * (8.0 + h->esz);
  double attn_flops = 0.0;
  for (int s = s0; s < s1; ++s) {
    const double L = h->h_cu[s + 1] - h->h_cu[s];
    attn_flops += (c.causal ? 2.0 : 4.0) * L * L * c.n_q_heads * dh;
  }
  PRISM_LAUNCH_P(h, st, PRISM_K_RMSNORM, norm_bytes, launch_layernorm(xr, g0, b0, c.dtype, rows, D, c.rms_eps, h->a_norm, st, next_dir(h, true)));
  if (h->tc)
    PRISM_LAUNCH_P(h, st, PRISM_K_GEMM_QKV, 2.0 * R * nqkv * D,
                   gemm_tc_any(h, h->map_a_norm, maps->qkv, maps->qkv, h->qkv, nullptr, rows, nqkv, D, kEpiStoreBias, nullptr, st, V.b_qkv));
  else
    PRISM_LAUNCH_P(h, st, PRISM_K_GEMM_QKV, 2.0 * R * nqkv * D,
                   launch_gemm_simt(h->a_norm, W.w_qkv, nullptr, h->qkv, nullptr, rows, nqkv, D, c.dtype, kEpiStoreBias, st, V.b_qkv));
  next_dir(h, false);
  if (h->fa == 3)
    PRISM_LAUNCH_P(h, st, PRISM_K_ATTENTION, attn_flops,
                   launch_attention_tc2(h->qkv, h->attn, cu_dev, s0, s1 - s0, r0, rows, max_len, c.n_q_heads, c.n_kv_heads, c.causal,
                                        h->errword, st, false, 0, nullptr, true, dh));
  else if (h->fa == 1)
    PRISM_LAUNCH_P(h, st, PRISM_K_ATTENTION, attn_flops,
                   launch_attention_tc(h->qkv, h->attn, cu_dev, s0, s1 - s0, r0, rows, max_len, c.n_q_heads, c.n_kv_heads, c.causal,
                                       h->errword, st, dh));
  else
    PRISM_LAUNCH_P(h, st, PRISM_K_ATTENTION, attn_flops,
                   launch_attention_simt(h->qkv, h->attn, cu_dev, s0, s1 - s0, r0, max_len, c.n_q_heads, c.n_kv_heads, dh,
                                         c.causal, c.dtype, st));
  if (h->tc)
    PRISM_LAUNCH_P(h, st, PRISM_K_GEMM_O, 2.0 * R * D * hd,
                   gemm_tc_any(h, h->map_attn, maps->o, maps->o, nullptr, xr, rows, D, hd, kEpiResidualBias, nullptr, st, V.b_o));
  else
    PRISM_LAUNCH_P(h, st, PRISM_K_GEMM_O, 2.0 * R * D * hd,
                   launch_gemm_simt(h->attn, W.w_o, nullptr, nullptr, xr, rows, D, hd, c.dtype, kEpiResidualBias, st, V.b_o));
  PRISM_LAUNCH_P(h, st, PRISM_K_RMSNORM, norm_bytes, launch_layernorm(xr, V.ln1_g, V.ln1_b, c.dtype, rows, D, c.rms_eps, h->a_norm, st, next_dir(h, true)));
  if (h->tc)
    PRISM_LAUNCH_P(h, st, PRISM_K_GEMM_GATEUP, 2.0 * R * F * D,
                   gemm_tc_any(h, h->map_a_norm, maps->gate, maps->gate, h->hbuf, nullptr, rows, F, D, kEpiGeluBias, nullptr, st, V.b_ffn1));
  else
    PRISM_LAUNCH_P(h, st, PRISM_K_GEMM_GATEUP, 2.0 * R * F * D,
                   launch_gemm_simt(h->a_norm, W.w_gate, nullptr, h->hbuf, nullptr, rows, F, D, c.dtype, kEpiGeluBias, st, V.b_ffn1));
  if (h->tc)
    PRISM_LAUNCH_P(h, st, PRISM_K_GEMM_DOWN, 2.0 * R * D * F,
                   gemm_tc_any(h, h->map_hbuf, maps->down, maps->down, nullptr, xr, rows, D, F, kEpiResidualBias, nullptr, st, V.b_ffn2));
  else
    PRISM_LAUNCH_P(h, st, PRISM_K_GEMM_DOWN, 2.0 * R * D * F,
                   launch_gemm_simt(h->hbuf, W.w_down, nullptr, nullptr, xr, rows, D, F, c.dtype, kEpiResidualBias, st, V.b_ffn2));
  return PRISM_OK;
}

// Embedding table caching (Sec. 4.4).  The request's token ids come to the host; every distinct token either has a
// row in the device cache (hit) or gets one: a free row first, else the row whose last use lies furthest back
// among those this request does not use.  The missing rows are then read from the pinned host table by one kernel.
// Token ids outside the vocabulary are skipped here; the pack kernel reports them.
int cache_prepare(prism_handle* h, const int* query, int lq, const int* cand, int n_cand, cudaStream_t st) {
  const prism_model_cfg& c = h->cfg;
  if (n_cand < 0 || (long long)n_cand + lq > (long long)c.max_total_tokens + c.max_seq_len)
    return fail(h, PRISM_ERR_SHAPE_LIMIT, "token total exceeds max_total_tokens");
  if (lq > 0) PRISM_CUDA(h, cudaMemcpyAsync(h->h_tokens, query, (size_t)lq * sizeof(int), cudaMemcpyDeviceToHost, st));
  if (n_cand > 0)
    PRISM_CUDA(h, cudaMemcpyAsync(h->h_tokens + lq, cand, (size_t)n_cand * sizeof(int), cudaMemcpyDeviceToHost, st));
  PRISM_CUDA(h, cudaStreamSynchronize(st));
  const uint64_t now = ++h->request_no;
  std::vector<int> missing, hit_slots;
  int64_t distinct = 0;
  for (int i = 0; i < lq + n_cand; ++i) {
    const int t = h->h_tokens[i];
    if (t < 0 || t >= c.vocab || h->tok_seen[t] == now) continue;
    h->tok_seen[t] = now;
    ++distinct;
    const int s = h->slot_of_tok[t];
    if (s >= 0) hit_slots.push_back(s);
    else missing.push_back(t);
  }
  if (distinct > h->cache_rows) {
    // a refused request leaves the cache as it found it: no row has been stamped yet, so the order in which rows
    // will be evicted is unchanged; the marks and the request number are taken back
    for (int i = 0; i < lq + n_cand; ++i) {
      const int t = h->h_tokens[i];
      if (t >= 0 && t < c.vocab) h->tok_seen[t] = 0;
    }
    --h->request_no;
    return fail(h, PRISM_ERR_SHAPE_LIMIT, "the request has more distinct tokens than the embedding cache has rows");
  }
  for (int s : hit_slots) h->slot_stamp[s] = now;
  h->cache_hits += distinct - (int64_t)missing.size();
  h->cache_misses += (int64_t)missing.size();
  if (missing.empty()) return PRISM_OK;
  // rows this request does not use, least recently used first (never-used rows have stamp 0)
  std::vector<int> victims;
  victims.reserve((size_t)h->cache_rows);
  for (int s = 0; s < h->cache_rows; ++s)
    if (h->slot_stamp[s] != now) victims.push_back(s);
  const size_t need = missing.size();
  std::partial_sort(victims.begin(), victims.begin() + (std::ptrdiff_t)need, victims.end(), [&](int a, int b) {
    return h->slot_stamp[a] != h->slot_stamp[b] ? h->slot_stamp[a] < h->slot_stamp[b] : a < b;
  });
  for (size_t i = 0; i < need; ++i) {
    const int t = missing[i], s = victims[i];
    if (h->tok_of_slot[s] >= 0) {
      h->slot_of_tok[h->tok_of_slot[s]] = -1;
      ++h->cache_evictions;
    }
    h->tok_of_slot[s] = t;
    h->slot_of_tok[t] = s;
    h->slot_stamp[s] = now;
    h->h_pairs[2 * i] = t;
    h->h_pairs[2 * i + 1] = s;
  }
  PRISM_CUDA(h, cudaMemcpyAsync(h->pairs_dev, h->h_pairs, 2 * need * sizeof(int), cudaMemcpyHostToDevice, st));
  PRISM_LAUNCH(h, launch_cache_fill(h->embed, h->cache_dev, h->pairs_dev, (int)need, c.hidden * (int)h->esz, h->tok2slot_dev, st));
  // the pinned pair list is reused by the next request: this one's copy must have left it
  PRISM_CUDA(h, cudaStreamSynchronize(st));
  return PRISM_OK;
}

// Candidate-sharded runs (Shard non-null): this rank packs only the candidates it owns (the others are sequences
// of length zero), probes write 0 for them, and before every prune decision `reduce` sums the score vector over
// the ranks, after which every rank evaluates the same rule on the same numbers.
struct Shard {
  const uint8_t* owned;  // host, N bytes
  float* exchange;       // device, N floats
  prism_exchange_fn reduce;
  void* ctx;
};

int select_impl(prism_handle* h, const int32_t* query, int32_t lq, const int32_t* cand, const int32_t* off, int32_t N,
                int32_t K, const prism_prune_schedule* sched, int32_t* topk_idx, float* topk_scores, int32_t* n_out,
                prism_trace* trace, cudaStream_t st, const Shard* shard = nullptr) {
  const prism_model_cfg& c = h->cfg;
  h->err.clear();
  if (trace) {
    trace->n_records = 0;
    trace->layers_run = 0;
    trace->n_chunks_max = 0;
    trace->workspace_bytes = h->workspace_bytes;
    trace->shared_prefix_rows = 0;
  }
  const int k_eff = std::min(K, N);
  std::string why;
  int rc = validate_schedule(h, sched, k_eff, &why);
  if (rc != PRISM_OK) return fail(h, rc, why);
  if (N > c.max_candidates) return fail(h, PRISM_ERR_SHAPE_LIMIT, "N exceeds max_candidates");
  if (N == 0) {
    *n_out = 0;
    return PRISM_OK;
  }
  const bool streamed = c.weight_residency == PRISM_WEIGHTS_HOST_STREAMED;
  const int mode = sched ? sched->mode : PRISM_PRUNE_NONE;
  const int n_probes = mode == PRISM_PRUNE_NONE ? 0 : sched->n_probes;

  // Offsets to the host: launch geometry, limits and chunk planning need them.
  PRISM_CUDA(h, cudaMemcpyAsync(h->h_off, off, (size_t)(N + 1) * sizeof(int), cudaMemcpyDeviceToHost, st));
  PRISM_CUDA(h, cudaStreamSynchronize(st));
  if (h->h_off[0] != 0) return fail(h, PRISM_ERR_BAD_INPUT, "cand_offsets[0] != 0");
  long long total = 0;
  h->h_cu[0] = 0;
  for (int i = 0; i < N; ++i)
    if (h->h_off[i + 1] < h->h_off[i]) return fail(h, PRISM_ERR_BAD_INPUT, "cand_offsets not monotone");
  if (h->h_off[N] > 0 && !cand) return fail(h, PRISM_ERR_INVALID_ARG, "cand_tokens is null but cand_offsets[N] > 0");
  // Shared query prefix: under causal attention the query's rows are the same in every sequence, so they are
  // stored and computed once in front of the documents (rows [0, lq)); cu then holds document rows only.
  long long own_docs = 0;  // document tokens of the candidates this rank runs
  for (int i = 0; i < N; ++i)
    if (!shard || shard->owned[i]) own_docs += (long long)h->h_off[i + 1] - h->h_off[i];
  (void)own_docs;
  const int prefix = (c.shared_prefix == PRISM_PREFIX_AUTO && !h->enc && h->fa == 3 && c.causal && N >= 2 &&
                      lq >= 8 && lq <= 120 && (lq & 7) == 0)
                         ? lq
                         : 0;
  if (prefix) {
    total = lq;
    h->h_cu[0] = lq;
    if (trace) trace->shared_prefix_rows = prefix;
  }
  for (int i = 0; i < N; ++i) {
    if (shard && !shard->owned[i]) {  // another rank's candidate: no rows here
      h->h_cu[i + 1] = (int)total;
      continue;
    }
    const long long dl = (long long)h->h_off[i + 1] - h->h_off[i];
    if (dl + lq > c.max_seq_len) return fail(h, PRISM_ERR_SHAPE_LIMIT, "a sequence exceeds max_seq_len");
    if (dl + lq > h->chunk_tokens) return fail(h, PRISM_ERR_BUDGET, "a sequence exceeds the chunk the activation budget allows");
    if (dl + lq < 1) return fail(h, PRISM_ERR_INVALID_ARG, "empty sequence (query_len = 0 and an empty document)");
    total += prefix ? dl : dl + lq;
    if (total > c.max_total_tokens) return fail(h, PRISM_ERR_SHAPE_LIMIT, "token total exceeds max_total_tokens");
    h->h_cu[i + 1] = (int)total;
  }

  RouteState init{};
  init.n_active = N;
  init.n_tokens = (int)total;
  init.k_rem = k_eff;
  *h->h_state = init;
  PRISM_CUDA(h, cudaMemcpyAsync(h->state, h->h_state, sizeof(RouteState), cudaMemcpyHostToDevice, st));
  PRISM_CUDA(h, cudaMemsetAsync(h->errword, 0, sizeof(int), st));

  if (h->cache_rows > 0 && (rc = cache_prepare(h, query, lq, cand, h->h_off[N], st)) != PRISM_OK) return rc;

  int cur = 0;  // ping-pong index of x / cu / seq2orig
  const unsigned char* owned_dev = nullptr;
  if (shard) {
    PRISM_CUDA(h, cudaMemcpyAsync(h->owned_dev, shard->owned, (size_t)N, cudaMemcpyHostToDevice, st));
    owned_dev = h->owned_dev;
  }
  PRISM_LAUNCH_P(h, st, PRISM_K_PACK, 8.0 * N,
                 launch_pack_offsets(off, N, lq, h->cu[cur], h->seq2orig[cur], h->errword, st, owned_dev, prefix > 0));
  PRISM_LAUNCH_P(h, st, PRISM_K_PACK, 12.0 * total,
                 launch_pack_tokens(query, lq, cand, off, h->cu[cur], N, (int)total, c.vocab, h->tokens, h->pos, h->errword, st,
                                    prefix > 0));
  if (h->enc)
    PRISM_LAUNCH_P(h, st, PRISM_K_EMBED, (double)total * c.hidden * (4.0 + 2.0 * h->esz),
                   launch_embed_encoder(h->cache_rows > 0 ? h->cache_dev : h->embed, h->pos_embed, h->type_f, c.dtype, h->tokens,
                                        h->pos, c.pos_offset, (int)total, c.hidden, h->x[cur], st,
                                        h->cache_rows > 0 ? h->tok2slot_dev : nullptr));
  else
  PRISM_LAUNCH_P(h, st, PRISM_K_EMBED, (double)total * c.hidden * (4.0 + h->esz),
                 launch_embed(h->cache_rows > 0 ? h->cache_dev : h->embed, c.dtype, h->tokens, (int)total, c.hidden, h->x[cur], st,
                              h->cache_rows > 0 ? h->tok2slot_dev : nullptr));

  if (streamed) {
    // The previous request drained both streams before returning, so both slots are free.
    for (int l = 0; l < std::min(2, c.n_layers); ++l)
      if ((rc = enqueue_layer_copy(h, l, l)) != PRISM_OK) return rc;
  }

  int n = N, T = (int)total, n_rec = 0, probe_j = 0, layers_run = 0, chunks_max = 0;
  int n_mine = N;  // live candidates this rank runs
  if (shard) {
    n_mine = 0;
    for (int i = 0; i < N; ++i) n_mine += shard->owned[i] ? 1 : 0;
  }
  bool done = false;
  // hidden-state offload bookkeeping
  bool main_dirty = true, slot_used[3] = {false, false, false};
  int chunk_out_valid = 0;  // chunk indices below this have a write-back event from the previous layer
  int last_out = -1;        // chunk index of the latest write-back enqueued on out_stream
  if (h->offload) {
    // a failed request may have left copies in flight
    PRISM_CUDA(h, cudaStreamSynchronize(h->in_stream));
    PRISM_CUDA(h, cudaStreamSynchronize(h->out_stream));
  }
  for (int l = 0; l < c.n_layers && !done; ++l) {
    const int s = l & 1;
    LayerDev W = streamed ? layer_in_slot(h, s) : layer_resident(h, l);
    const LayerMaps* maps = !h->tc ? nullptr : h->w4 ? &h->maps_w4 : &h->maps[streamed ? s : l];
    if (streamed) {
      PRISM_CUDA(h, cudaStreamWaitEvent(st, h->ev_copied[s], 0));
      pdl_skip_next();
    }
    if (h->w4) {
      // rebuild the layer's five matrices as bf16; the stream orders this after the previous layer's last GEMM
      const int D = c.hidden, F = c.ffn, nq = (c.n_q_heads + 2 * c.n_kv_heads) * c.head_dim, hd = c.n_q_heads * c.head_dim;
      // decoder: qkv, o, gate, up, down; encoder: qkv, o, ffn1, ffn2 (the last into the "down" scratch)
      const int nm = h->enc ? 4 : 5;
      const void* src[5] = {W.w_qkv, W.w_o, W.w_gate, h->enc ? W.w_down : W.w_up, W.w_down};
      void* dst[5] = {h->wq[0], h->wq[1], h->wq[2], h->enc ? h->wq[4] : h->wq[3], h->wq[4]};
      const int rows[5] = {nq, D, F, h->enc ? D : F, D}, cols[5] = {D, hd, D, h->enc ? F : D, F};
      double bytes = 0.0;  // 4 bits in, 16 bits out per weight, plus one scale and zero point per group
      for (int i = 0; i < nm; ++i) bytes += (double)rows[i] * cols[i] * (2.5 + 3.0 / c.quant_group);
      PRISM_LAUNCH_P(h, st, PRISM_K_DEQUANT, bytes, launch_dequant_w4_batch(src, rows, cols, dst, nm, c.quant_group, st));
      W.w_qkv = h->wq[0];
      W.w_o = h->wq[1];
      W.w_gate = h->wq[2];
      W.w_up = h->enc ? h->wq[2] : h->wq[3];
      W.w_down = h->wq[4];
    }
    // chunks on sequence boundaries: the longest prefix of the remaining sequences that fits
    int s0 = 0, chunks = 0;
    const bool many = prefix && h->h_cu[n] > h->chunk_tokens;  // a shared prefix over several chunks
    while (s0 < n) {
      // with a shared prefix the first chunk starts at row 0 and holds the prefix rows as well
      const int base = (prefix && s0 == 0) ? 0 : h->h_cu[s0];
      int s1 = s0 + 1, max_len = h->h_cu[s1] - h->h_cu[s0];
      while (s1 < n && h->h_cu[s1 + 1] - base <= h->chunk_tokens) {
        max_len = std::max(max_len, h->h_cu[s1 + 1] - h->h_cu[s1]);
        ++s1;
      }
      const int r0 = base, rows = h->h_cu[s1] - r0;
      const int of_many = !many ? 0 : s0 == 0 ? 1 : 2;
      if (prefix && !h->offload) {
        if ((rc = run_layer_chunk(h, W, maps, h->x[cur], h->cu[cur], s0, s1, r0, rows, prefix + max_len, st, false, prefix,
                                  of_many)) != PRISM_OK)
          return rc;
      } else if (h->enc && !h->offload) {
        if ((rc = run_layer_chunk_encoder(h, l, W, maps, h->x[cur], h->cu[cur], s0, s1, r0, rows, max_len, st)) != PRISM_OK) return rc;
      } else if (!h->offload) {
        if ((rc = run_layer_chunk(h, W, maps, h->x[cur], h->cu[cur], s0, s1, r0, rows, max_len, st)) != PRISM_OK) return rc;
      } else if (rows > 0) {
        // Chunk `chunks` goes through device buffer chunks % 3: fetched on in_stream once the buffer's previous
        // occupant has been written back and this chunk's rows on the host are final (its own write-back of the
        // previous layer, or the request stream's embedding / compaction), computed here, written back on
        // out_stream.  The host enqueues chunk after chunk, so the fetch of chunk c + 1 and the write-back of
        // chunk c - 1 run under the computation of chunk c: at most three chunks are on the device.
        const int slot = chunks % 3;
        const size_t bytes = (size_t)rows * c.hidden * sizeof(float);
        float* hx = h->x[cur] + (size_t)r0 * c.hidden;
        while ((size_t)chunks >= h->ev_chunk_out.size()) {
          cudaEvent_t e = nullptr;
          PRISM_CUDA(h, cudaEventCreateWithFlags(&e, cudaEventDisableTiming));
          h->ev_chunk_out.push_back(e);
        }
        if (main_dirty) {  // the request stream wrote the host copy (embedding, compaction) since the last fetch
          PRISM_CUDA(h, cudaEventRecord(h->ev_main, st));
          main_dirty = false;
          chunk_out_valid = 0;
        }
        PRISM_CUDA(h, cudaStreamWaitEvent(h->in_stream, h->ev_main, 0));
        if (slot_used[slot]) PRISM_CUDA(h, cudaStreamWaitEvent(h->in_stream, h->ev_slot_out[slot], 0));
        if (chunks < chunk_out_valid) PRISM_CUDA(h, cudaStreamWaitEvent(h->in_stream, h->ev_chunk_out[chunks], 0));
        PRISM_CUDA(h, cudaMemcpyAsync(h->xc[slot], hx, bytes, cudaMemcpyHostToDevice, h->in_stream));
        PRISM_CUDA(h, cudaEventRecord(h->ev_in[slot], h->in_stream));
        PRISM_CUDA(h, cudaStreamWaitEvent(st, h->ev_in[slot], 0));
        pdl_skip_next();
        rc = h->enc ? run_layer_chunk_encoder(h, l, W, maps, h->xc[slot], h->cu[cur], s0, s1, r0, rows, max_len, st, true)
                    : run_layer_chunk(h, W, maps, h->xc[slot], h->cu[cur], s0, s1, r0, rows, prefix + max_len, st, true, prefix,
                                      of_many);
        if (rc != PRISM_OK) return rc;
        PRISM_CUDA(h, cudaEventRecord(h->ev_done[slot], st));
        PRISM_CUDA(h, cudaStreamWaitEvent(h->out_stream, h->ev_done[slot], 0));
        PRISM_CUDA(h, cudaMemcpyAsync(hx, h->xc[slot], bytes, cudaMemcpyDeviceToHost, h->out_stream));
        PRISM_CUDA(h, cudaEventRecord(h->ev_slot_out[slot], h->out_stream));
        PRISM_CUDA(h, cudaEventRecord(h->ev_chunk_out[chunks], h->out_stream));
        slot_used[slot] = true;
        last_out = chunks;
      }
      s0 = s1;
      ++chunks;
    }
    if (h->offload) chunk_out_valid = chunks;  // the next layer's chunk c waits for this layer's write-back of chunk c
    chunks_max = std::max(chunks_max, chunks);
    if (trace && trace->tokens_per_layer) trace->tokens_per_layer[l] = prefix ? T - prefix + n_mine * prefix : T;
    layers_run = l + 1;
    if (streamed) {
      PRISM_CUDA(h, cudaEventRecord(h->ev_freed[s], st));
    }

    const bool is_final = (layers_run == c.n_layers);
    const bool is_probe = probe_j < n_probes && sched->probe_layers[probe_j] == layers_run;
    if (h->offload && (is_final || is_probe) && last_out >= 0) {
      // probe and compaction read the host copy on the request's stream: every write-back must have landed
      // (out_stream is in order, so its latest event covers them all)
      PRISM_CUDA(h, cudaStreamWaitEvent(st, h->ev_chunk_out[last_out], 0));
      pdl_skip_next();
      main_dirty = true;  // whatever the request stream does to the host copy now must precede later fetches
    }
    if (is_final || is_probe) {
      RouteParams p{};
      p.mode = mode;
      p.keep_count = (mode == PRISM_PRUNE_FIXED_KEEP && is_probe) ? sched->keep_counts[probe_j] : 0;
      p.cv_threshold = sched ? sched->cv_threshold : 0.0;
      p.n_clusters = (sched && sched->n_clusters) ? sched->n_clusters : 3;
      p.ddof = sched ? sched->std_ddof : 0;
      p.select_winners = sched ? sched->select_winners : 1;
      p.is_final = is_final ? 1 : 0;
      p.layer = layers_run;
      p.prefix = prefix;
      p.owned = (prefix && shard) ? h->owned_dev : nullptr;
      const int nxt = cur ^ 1;
      float* score_buf = shard ? shard->exchange : h->scores;
      if (h->enc) {
        const EncVec& V = h->enc_vec[layers_run - 1];  // the last executed block's LN2 is still pending
        PRISM_LAUNCH_P(h, st, PRISM_K_PROBE, (double)n * c.hidden * (4.0 + (double)c.hidden * h->esz),
                       launch_probe_encoder(h->x[cur], h->cu[cur], n, c.hidden, V.ln2_g, V.ln2_b, c.rms_eps, h->head_dense_w,
                                            c.dtype, h->head_db, h->head_ow, h->head_ob, score_buf, h->probe_scratch, st));
        h->launches += 2;  // the probe is three kernels
      } else
      PRISM_LAUNCH_P(h, st, PRISM_K_PROBE, 4.0 * n * c.hidden,
                     launch_probe(h->x[cur], h->cu[cur], n, c.hidden, h->g_final, c.dtype, h->w_diff, c.rms_eps, score_buf, st, prefix,
                                  (prefix && shard) ? h->owned_dev : nullptr, h->seq2orig[cur]));
      if (shard && shard->reduce(shard->ctx, n, st) != 0) return fail(h, PRISM_ERR_CUDA, "the score exchange callback failed");
      PRISM_LAUNCH_P(h, st, PRISM_K_ROUTE, 8.0 * n, launch_route(score_buf, h->cu[cur], h->seq2orig[cur], n, p, h->cu[nxt], h->seq2orig[nxt], h->old_of_new,
                                   h->state, h->res_idx, h->res_score, h->recs + n_rec,
                                   h->trace_scores + (size_t)n_rec * c.max_candidates,
                                   h->trace_ids + (size_t)n_rec * c.max_candidates, h->route_scratch, st));
      ++n_rec;
      if (is_probe) ++probe_j;
      PRISM_CUDA(h, cudaMemcpyAsync(h->h_state, h->state, sizeof(RouteState), cudaMemcpyDeviceToHost, st));
      PRISM_CUDA(h, cudaMemcpyAsync(h->h_err, h->errword, sizeof(int), cudaMemcpyDeviceToHost, st));
      if (!is_final)
        PRISM_CUDA(h, cudaMemcpyAsync(h->h_cu_next, h->cu[nxt], (size_t)(n + 1) * sizeof(int), cudaMemcpyDeviceToHost, st));
      PRISM_CUDA(h, cudaStreamSynchronize(st));  // the one host round trip per scored layer
      if (*h->h_err & kErrTimeout) return fail(h, PRISM_ERR_TIMEOUT, "a bounded device-side wait expired");
      if (*h->h_err & (kErrBadToken | kErrBadOffsets)) return fail(h, PRISM_ERR_BAD_INPUT, "token id outside [0, vocab) or bad offsets");
      const RouteState stt = *h->h_state;
      done = stt.done != 0;
      if (!done && stt.n_active < n) {
        // survivors move to the other buffer, order kept; offsets and positions follow
        std::swap(h->h_cu, h->h_cu_next);
        PRISM_LAUNCH_P(h, st, PRISM_K_COMPACT, 8.0 * stt.n_tokens * c.hidden,
                       launch_compact_rows(h->x[cur], h->x[nxt], h->cu[cur], h->cu[nxt], h->old_of_new, stt.n_active,
                                           stt.n_tokens, c.hidden, st, prefix));
        PRISM_LAUNCH_P(h, st, PRISM_K_PACK, 4.0 * stt.n_tokens, launch_positions(h->cu[nxt], stt.n_active, stt.n_tokens, h->pos, st, prefix));
        cur = nxt;
        n = stt.n_active;
        T = stt.n_tokens;
        n_mine = stt.pad0;
      }
    }
    if (streamed && !done && l + 2 < c.n_layers) {
      PRISM_CUDA(h, cudaStreamWaitEvent(h->copy_stream, h->ev_freed[s], 0));
      if ((rc = enqueue_layer_copy(h, l + 2, s)) != PRISM_OK) return rc;
    }
  }

  PRISM_CUDA(h, cudaMemcpyAsync(topk_idx, h->res_idx, (size_t)k_eff * sizeof(int), cudaMemcpyDeviceToDevice, st));
  PRISM_CUDA(h, cudaMemcpyAsync(topk_scores, h->res_score, (size_t)k_eff * sizeof(float), cudaMemcpyDeviceToDevice, st));
  if (trace) {
    const int take = std::min(n_rec, trace->capacity);
    if (take > 0 && trace->records)
      PRISM_CUDA(h, cudaMemcpyAsync(trace->records, h->recs, (size_t)take * sizeof(prism_probe_record), cudaMemcpyDeviceToHost, st));
    for (int r = 0; r < take; ++r) {
      if (trace->scores)
        PRISM_CUDA(h, cudaMemcpyAsync(trace->scores + (size_t)r * N, h->trace_scores + (size_t)r * c.max_candidates,
                                      (size_t)N * sizeof(float), cudaMemcpyDeviceToHost, st));
      if (trace->ids)
        PRISM_CUDA(h, cudaMemcpyAsync(trace->ids + (size_t)r * N, h->trace_ids + (size_t)r * c.max_candidates,
                                      (size_t)N * sizeof(int), cudaMemcpyDeviceToHost, st));
    }
    trace->n_records = take;
    trace->layers_run = layers_run;
    trace->n_chunks_max = chunks_max;
  }
  PRISM_CUDA(h, cudaStreamSynchronize(st));
  if (streamed) PRISM_CUDA(h, cudaStreamSynchronize(h->copy_stream));
  if (h->prof_on) prof_collect(h);
  if (h->h_state->n_result != k_eff) return fail(h, PRISM_ERR_CUDA, "internal: result count mismatch");
  *n_out = k_eff;
  return PRISM_OK;
}

int check_args(prism_handle* h, const void* q, int lq, const void* cand, const void* off, int N, int K, const void* oi,
               const void* os, const void* n_out) {
  if (!h) return PRISM_ERR_INVALID_ARG;
  if (!n_out) return fail(h, PRISM_ERR_INVALID_ARG, "n_out is null");
  if (N < 0 || K < 1 || lq < 0) return fail(h, PRISM_ERR_INVALID_ARG, "N < 0, K < 1 or query_len < 0");
  if (!off || !oi || !os || (lq > 0 && !q)) return fail(h, PRISM_ERR_INVALID_ARG, "null pointer argument");
  if (lq > h->cfg.max_seq_len) return fail(h, PRISM_ERR_SHAPE_LIMIT, "query_len exceeds max_seq_len");
  (void)cand;  // may be null when every document is empty: checked once the offsets are on the host
  return PRISM_OK;
}

}  // namespace

extern "C" {

int prism_select(prism_handle* h, const int32_t* query_tokens, int32_t query_len, const int32_t* cand_tokens,
                 const int32_t* cand_offsets, int32_t N, int32_t K, const prism_prune_schedule* sched, int32_t* topk_idx,
                 float* topk_scores, int32_t* n_out, prism_trace* trace, void* cuda_stream) {
  int rc = check_args(h, query_tokens, query_len, cand_tokens, cand_offsets, N, K, topk_idx, topk_scores, n_out);
  if (rc != PRISM_OK) return rc;
  *n_out = 0;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  rc = select_impl(h, query_tokens, query_len, cand_tokens, cand_offsets, N, K, sched, topk_idx, topk_scores, n_out, trace, st);
  if (rc != PRISM_OK) {
    *n_out = 0;
    cudaStreamSynchronize(st);
    if (h->copy_stream) cudaStreamSynchronize(h->copy_stream);
  }
  return rc;
}

int prism_select_calibrated(prism_handle* h, const int32_t* query_tokens, int32_t query_len, const int32_t* cand_tokens,
                            const int32_t* cand_offsets, int32_t N, int32_t K, const prism_prune_schedule* sched,
                            prism_calibrator* cal, int32_t* topk_idx, float* topk_scores, int32_t* n_out, prism_trace* trace,
                            void* cuda_stream) {
  int rc = check_args(h, query_tokens, query_len, cand_tokens, cand_offsets, N, K, topk_idx, topk_scores, n_out);
  if (rc != PRISM_OK) return rc;
  *n_out = 0;
  if (!cal || !sched || sched->mode != PRISM_PRUNE_CLUSTER) return fail(h, PRISM_ERR_INVALID_ARG, "calibration needs a CLUSTER schedule and a calibrator");
  if (!(cal->raise_factor > 1.0) || !(cal->lower_factor > 0.0 && cal->lower_factor < 1.0) || cal->sample_every < 1 ||
      cal->window < 1 || !(cal->min_threshold <= cal->max_threshold) || !(cal->threshold == cal->threshold) ||
      !(cal->target_precision >= 0.0 && cal->target_precision <= 1.0))
    return fail(h, PRISM_ERR_INVALID_ARG, "malformed calibrator");
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  prism_prune_schedule s = *sched;
  s.cv_threshold = cal->threshold;
  rc = select_impl(h, query_tokens, query_len, cand_tokens, cand_offsets, N, K, &s, topk_idx, topk_scores, n_out, trace, st);
  if (rc != PRISM_OK) {
    *n_out = 0;
    cudaStreamSynchronize(st);
    if (h->copy_stream) cudaStreamSynchronize(h->copy_stream);
    return rc;
  }
  const bool sample = (cal->n_requests % cal->sample_every) == 0;
  cal->n_requests++;
  const int k_eff = *n_out;
  if (!sample || k_eff == 0) return PRISM_OK;
  // ground truth: the same request without pruning, into the handle's own output buffers
  std::vector<int> pruned(k_eff), full(k_eff);
  PRISM_CUDA(h, cudaMemcpyAsync(pruned.data(), topk_idx, (size_t)k_eff * sizeof(int), cudaMemcpyDeviceToHost, st));
  PRISM_CUDA(h, cudaStreamSynchronize(st));
  prism_prune_schedule none{};
  none.mode = PRISM_PRUNE_NONE;
  int n_full = 0;
  rc = select_impl(h, query_tokens, query_len, cand_tokens, cand_offsets, N, K, &none, h->out_idx, h->out_score, &n_full, nullptr, st);
  if (rc != PRISM_OK) return rc;
  PRISM_CUDA(h, cudaMemcpyAsync(full.data(), h->out_idx, (size_t)k_eff * sizeof(int), cudaMemcpyDeviceToHost, st));
  PRISM_CUDA(h, cudaStreamSynchronize(st));
  std::sort(pruned.begin(), pruned.end());
  std::sort(full.begin(), full.end());
  std::vector<int> both;
  std::set_intersection(pruned.begin(), pruned.end(), full.begin(), full.end(), std::back_inserter(both));
  const double precision = (double)both.size() / (double)k_eff;
  cal->last_precision = precision;
  cal->precision_sum += precision;
  cal->n_sampled++;
  if (++cal->n_in_window >= cal->window) {
    const double mean = cal->precision_sum / (double)cal->n_in_window;
    cal->last_window_precision = mean;
    double t = cal->threshold * (mean < cal->target_precision ? cal->raise_factor : cal->lower_factor);
    t = std::min(cal->max_threshold, std::max(cal->min_threshold, t));
    cal->threshold = t;
    cal->n_in_window = 0;
    cal->precision_sum = 0.0;
    cal->n_adjustments++;
  }
  return PRISM_OK;
}

int prism_select_sharded(prism_handle* h, const int32_t* query_tokens, int32_t query_len, const int32_t* cand_tokens,
                         const int32_t* cand_offsets, int32_t N, int32_t K, const prism_prune_schedule* sched,
                         const uint8_t* owned, float* exchange, prism_exchange_fn reduce, void* ctx, int32_t* topk_idx,
                         float* topk_scores, int32_t* n_out, prism_trace* trace, void* cuda_stream) {
  int rc = check_args(h, query_tokens, query_len, cand_tokens, cand_offsets, N, K, topk_idx, topk_scores, n_out);
  if (rc != PRISM_OK) return rc;
  *n_out = 0;
  if (!owned || !exchange || !reduce) return fail(h, PRISM_ERR_INVALID_ARG, "owned, exchange or reduce is null");
  if (N > h->cfg.max_candidates) return fail(h, PRISM_ERR_SHAPE_LIMIT, "N exceeds max_candidates");
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  const Shard shard{owned, exchange, reduce, ctx};
  rc = select_impl(h, query_tokens, query_len, cand_tokens, cand_offsets, N, K, sched, topk_idx, topk_scores, n_out, trace, st,
                   &shard);
  if (rc != PRISM_OK) {
    *n_out = 0;
    cudaStreamSynchronize(st);
    if (h->copy_stream) cudaStreamSynchronize(h->copy_stream);
  }
  return rc;
}

int prism_select_host(prism_handle* h, const int32_t* query_tokens, int32_t query_len, const int32_t* cand_tokens,
                      const int32_t* cand_offsets, int32_t N, int32_t K, const prism_prune_schedule* sched,
                      int32_t* topk_idx, float* topk_scores, int32_t* n_out, prism_trace* trace, void* cuda_stream) {
  int rc = check_args(h, query_tokens, query_len, cand_tokens, cand_offsets, N, K, topk_idx, topk_scores, n_out);
  if (rc != PRISM_OK) return rc;
  *n_out = 0;
  if (N > h->cfg.max_candidates) return fail(h, PRISM_ERR_SHAPE_LIMIT, "N exceeds max_candidates");
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  const long long n_cand = N > 0 ? cand_offsets[N] : 0;  // host buffer: readable here
  if (n_cand < 0) return fail(h, PRISM_ERR_BAD_INPUT, "cand_offsets[N] negative");
  if (n_cand > h->cfg.max_total_tokens) return fail(h, PRISM_ERR_SHAPE_LIMIT, "token total exceeds max_total_tokens");
  if (n_cand > 0 && !cand_tokens) return fail(h, PRISM_ERR_INVALID_ARG, "cand_tokens is null");
  if (query_len > 0)
    PRISM_CUDA(h, cudaMemcpyAsync(h->in_query, query_tokens, (size_t)query_len * sizeof(int), cudaMemcpyHostToDevice, st));
  if (n_cand > 0)
    PRISM_CUDA(h, cudaMemcpyAsync(h->in_cand, cand_tokens, (size_t)n_cand * sizeof(int), cudaMemcpyHostToDevice, st));
  PRISM_CUDA(h, cudaMemcpyAsync(h->in_off, cand_offsets, (size_t)(N + 1) * sizeof(int), cudaMemcpyHostToDevice, st));
  rc = select_impl(h, h->in_query, query_len, h->in_cand, h->in_off, N, K, sched, h->out_idx, h->out_score, n_out, trace, st);
  if (rc == PRISM_OK && *n_out > 0) {
    cudaError_t e = cudaMemcpyAsync(topk_idx, h->out_idx, (size_t)*n_out * sizeof(int), cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(topk_scores, h->out_score, (size_t)*n_out * sizeof(float), cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) rc = cuda_fail(h, e, "copy of the result to the host");
  }
  if (rc != PRISM_OK) {
    *n_out = 0;
    cudaStreamSynchronize(st);
    if (h->copy_stream) cudaStreamSynchronize(h->copy_stream);
  }
  return rc;
}

}  // extern "C"
