// Shared declarations of the PRISM CUDA path (internal; the public surface is include/*.h).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

namespace prism {

constexpr int kMaxCandidates = 4096;
constexpr int kMaxClusters = 8;

// Device error word bits (written by kernels instead of trapping).
constexpr int kErrBadToken = 1;    // token id outside [0, vocab)
constexpr int kErrBadOffsets = 2;  // non-monotone candidate offsets
constexpr int kErrTimeout = 4;     // a bounded mbarrier wait gave up
constexpr int kErrInternal = 8;

// Epilogues of the projection GEMMs (C = A[M,K] * B[N,K]^T).
enum Epilogue : int {
  kEpiStore = 0,     // out[M,N] = acc                               (QKV projection)
  kEpiResidual = 1,  // x[M,N] += acc, x fp32 residual stream        (O-proj, down-proj)
  kEpiSwiGLU = 2,    // out[M,N] = silu(acc_gate) * acc_up           (gate/up projection)
  kEpiQkvRope = 3,   // QKV projection with QK-norm + rotary embedding applied to the q and k heads
  // encoder stack: every linear map has a bias (fp32 vector of n entries)
  kEpiStoreBias = 4,     // out[M,N] = acc + bias                        (QKV projection)
  kEpiGeluBias = 5,      // out[M,N] = gelu(acc + bias), gelu(x) = x Phi(x)   (first FFN map)
  kEpiResidualBias = 6,  // x[M,N] += acc + bias                         (O-proj, second FFN map)
};

// Inputs of the fused QK-norm + RoPE epilogue (head_dim 128; rotary table rows of 64 floats).
struct QkvRopeArgs {
  const int* pos;        // [m] position of each row inside its sequence
  const float* tab;      // [max_pos, 2, 64]: for half h, cos(32h + 0..31) then sin(32h + 0..31) of pos * theta^(-i/64)
  const __nv_bfloat16* g_q;  // [128] (used when qk_norm)
  const __nv_bfloat16* g_k;  // [128]
  int hq, hkv, qk_norm;
  float eps;
};

struct RouteParams {
  int mode;  // PRISM_PRUNE_*
  int keep_count;
  double cv_threshold;
  int n_clusters;
  int ddof;
  int select_winners;
  int is_final;  // 1: last layer, append the best k_rem and stop
  int layer;
  int prefix;    // shared query prefix: rows in front of the batch that belong to every sequence (0 = none)
  const unsigned char* owned;  // candidate-sharded run with a prefix: which original candidates this rank runs (else null)
};

// Request state that lives on the device and is mirrored to the host after every scored layer.
struct RouteState {
  int n_active;
  int n_tokens;
  int k_rem;
  int n_result;
  int done;
  int err;
  int pad0;  // written by the routing kernel: survivors that this rank runs (all of them unless candidate-sharded)
  int pad1;
};

struct ProbeRecordDev {  // layout mirrors prism_probe_record
  int layer, n_active_before, fired, n_selected, n_dropped, n_deferred, k_rem_after, n_cuts;
  int cuts[kMaxClusters];
  int tokens_before;
  int pad;
  double cv;
};

// Bytes of global scratch the routing kernel needs for n candidates.
constexpr size_t route_scratch_bytes(int n) {
  return ((size_t)n + 1) * sizeof(double) * 4            // P1, P2, D[2]
         + ((size_t)n + 1) * sizeof(int) * kMaxClusters  // argmin table
         + ((size_t)n + 1) * sizeof(int) * 2             // valid flags, sorted positions
         + 256;
}

// Arguments of the one-step routing entry points that the kernel itself cannot defend against: an unknown
// mode, a FIXED_KEEP count below 1 (the survivor count would go negative and the new offsets would be written in
// front of the caller's buffer) or a ddof other than 0 / 1.
inline bool route_args_ok(int n, int mode, int keep_count, int n_clusters, int ddof, int max_n) {
  if (n < 0 || n > max_n) return false;
  if (mode != 0 && mode != 1 && mode != 2) return false;
  if (mode == 1 && keep_count < 1) return false;
  if (n_clusters < 2 || n_clusters > kMaxClusters) return false;
  return ddof == 0 || ddof == 1;
}

// Raise a kernel's dynamic shared-memory limit once per device (the attribute is per device; `done` is a
// bit mask over device ordinals, so concurrent callers at worst set it twice).
template <typename Kernel>
inline cudaError_t ensure_dynamic_smem(Kernel kernel, int bytes, std::atomic<unsigned long long>& done) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  const unsigned long long bit = 1ull << (dev & 63);
  if (done.load(std::memory_order_acquire) & bit) return cudaSuccess;
  e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e != cudaSuccess) return e;
  done.fetch_or(bit, std::memory_order_release);
  return cudaSuccess;
}

// Opaque 128-byte TMA tensor map (mirrors CUtensorMap so that headers need not include cuda.h).
struct alignas(64) TmaDesc {
  unsigned char bytes[128];
};

// Programmatic dependent launch: a kernel that starts with pdl_sync() may be launched with
// cudaLaunchAttributeProgrammaticStreamSerialization.  Its blocks are then scheduled as soon as every block of the
// kernel before it in the stream has started (that kernel's own pdl_sync() releases them), run their set-up
// (barrier initialisation, tensor-memory allocation), and wait at this point until the predecessor has completed and
// its writes are visible.  Nothing before the call may touch memory another kernel writes.
#ifdef __CUDACC__
__device__ __forceinline__ void pdl_sync() {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
}
#endif
// Whether a launcher sets the attribute for a kernel over `rows` rows: it pays where kernels are short (the
// launch and set-up it hides are a few microseconds), and measured neutral to slightly negative on full batches, so it
// is used up to 16 Ki rows.  PRISM_NO_PDL in the environment turns it off altogether.
bool pdl_enabled();
// After a cross-stream dependency was enqueued (cudaStreamWaitEvent), the next launch of this thread goes out
// without the attribute, so that nothing of it can be scheduled ahead of that dependency.
void pdl_skip_next();
inline bool pdl_for(long long rows) {
  const bool on = pdl_enabled();  // consumes a pending pdl_skip_next()
  return on && rows <= 16384;
}

// ---- launchers (each returns the CUDA error of the launch; none synchronises) -----------------
// owned (nullable, device, n bytes): candidates with owned[i] == 0 get length zero (candidate-sharded runs).
cudaError_t launch_pack_offsets(const int* cand_offsets, int n, int query_len, int* cu, int* seq2orig,
                                int* err, cudaStream_t st, const unsigned char* owned = nullptr, bool shared_prefix = false);
cudaError_t launch_pack_tokens(const int* query, int query_len, const int* cand_tokens,
                               const int* cand_offsets, const int* cu, int n, int total, int vocab,
                               int* tokens, int* pos, int* err, cudaStream_t st, bool shared_prefix = false);
// Shared query prefix (prefix = query_len > 0 below): the query's rows are stored once in front of the batch,
// cu[i] is the first DOCUMENT row of sequence i, and a sequence is the prefix rows followed by its own rows.
cudaError_t launch_positions(const int* cu, int n, int total, int* pos, cudaStream_t st, int prefix = 0);
cudaError_t launch_embed(const void* table, int dtype, const int* tokens, int total, int d, float* x,
                         cudaStream_t st, const int* tok2slot = nullptr);
// Sec. 4.4 embedding table caching: rows of the pinned host table into rows of the device cache.
cudaError_t launch_cache_fill(const void* host_table, void* cache, const int* pairs, int n_rows, int row_bytes,
                              int* tok2slot, cudaStream_t st);
cudaError_t launch_rmsnorm(const float* x, const void* gain, int dtype, int rows, int d, float eps,
                           void* out, cudaStream_t st, bool reverse = false);
cudaError_t launch_rope_table(float* cos_t, float* sin_t, int max_pos, int head_dim, float theta,
                              cudaStream_t st);
cudaError_t launch_rope_table_fused(float* tab, int max_pos, float theta, cudaStream_t st);
cudaError_t launch_qknorm_rope(void* qkv, int dtype, const int* pos, int rows, int n_q_heads,
                               int n_kv_heads, int head_dim, int qk_norm, const void* g_q,
                               const void* g_k, float eps, const float* cos_t, const float* sin_t,
                               cudaStream_t st);
cudaError_t launch_probe(const float* x, const int* cu, int n, int d, const void* g_final, int dtype,
                         const float* w_diff, float eps, float* scores, cudaStream_t st, int prefix = 0,
                         const unsigned char* owned = nullptr, const int* seq2orig = nullptr);
// ---- encoder stack (post-norm blocks with LayerNorm, learned positions, first-token classification head) ----
// x[t,:] = table[tokens[t],:] + pos_table[pos[t] + pos_offset,:] + type_row (fp32 sum; the embedding LayerNorm is
// the first norm of the first block)
cudaError_t launch_embed_encoder(const void* table, const void* pos_table, const float* type_row, int dtype,
                                 const int* tokens, const int* pos, int pos_offset, int total, int d, float* x,
                                 cudaStream_t st, const int* tok2slot = nullptr);
// In place: x[r,:] = (x[r,:] - mean) / sqrt(var + eps) * gain + shift (fp32), and the same values in element type
// `dtype` to out (the next GEMM's input).
cudaError_t launch_layernorm(float* x, const float* gain, const float* shift, int dtype, int rows, int d, float eps,
                             void* out, cudaStream_t st, bool reverse = false);
// Score of sequence i from its FIRST row: LayerNorm (gain, shift) of the row, then
// out_w . tanh(dense_w y + dense_b) + out_b.  dense_w [d, d] has element type `dtype`, the vectors are fp32.
// scratch: 2 * n * d floats.  Three launches.
cudaError_t launch_probe_encoder(const float* x, const int* cu, int n, int d, const float* gain, const float* shift,
                                 float eps, const void* dense_w, int dtype, const float* dense_b, const float* out_w,
                                 const float* out_b, float* scores, float* scratch, cudaStream_t st);
// W4 weights: bytes of the packed blob of an [n, k] matrix, and the offsets of its scale and zero-point sections.
inline size_t w4_align16(size_t v) { return (v + 15) / 16 * 16; }
inline size_t w4_scales_offset(size_t n, size_t k) { return w4_align16(n * k / 2); }
inline size_t w4_zeros_offset(size_t n, size_t k, size_t group) { return w4_align16(w4_scales_offset(n, k) + 2 * n * (k / group)); }
inline size_t w4_blob_bytes(size_t n, size_t k, size_t group) { return w4_align16(w4_zeros_offset(n, k, group) + n * (k / group)); }
// out[n, k] bf16 = scale * (code - zero) per group of `group` input channels
cudaError_t launch_dequant_w4(const void* blob, int n, int k, int group, void* out, cudaStream_t st);
// the same for up to five matrices in one launch (a layer)
cudaError_t launch_dequant_w4_batch(const void* const* blobs, const int* n, const int* k, void* const* outs, int count,
                                    int group, cudaStream_t st);
// n values of element type `dtype` widened to fp32
cudaError_t launch_to_f32(const void* src, int dtype, int n, float* dst, cudaStream_t st);
cudaError_t launch_score_diff(const void* score_head, int dtype, int d, float* w_diff, cudaStream_t st);
cudaError_t launch_compact_rows(const float* x_old, float* x_new, const int* cu_old, const int* cu_new,
                                const int* old_of_new, int n_new, int total_new, int d, cudaStream_t st, int prefix = 0);

cudaError_t launch_gemm_simt(const void* a, const void* b, const void* b2, void* out, float* resid, int m,
                             int n, int k, int dtype, int epilogue, cudaStream_t st, const float* bias = nullptr);
cudaError_t launch_attention_simt(const void* qkv, void* out, const int* cu, int seq0, int nseq, int row0,
                                  int max_len, int n_q_heads, int n_kv_heads, int head_dim, int causal,
                                  int dtype, cudaStream_t st);

// Tensor-core path (bf16).  make_tma_2d_bf16 describes a row-major [rows, cols] bf16 matrix that is
// fetched in boxes of box_rows x 64 columns with the 128-byte swizzle the MMA descriptors expect.
cudaError_t make_tma_2d_bf16(TmaDesc* out, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows,
                             uint32_t box_cols);
// Store-side maps of the GEMM epilogues: fp32 [rows, cols] in 32x32 boxes (128-byte swizzle) and bf16
// [rows, cols] in 32x32 boxes (64-byte swizzle).
cudaError_t make_tma_2d_f32_box32(TmaDesc* out, const void* base, uint64_t rows, uint64_t cols);
cudaError_t make_tma_2d_bf16_box32_sw64(TmaDesc* out, const void* base, uint64_t rows, uint64_t cols);
int gemm_tc_sm_count();
// b0/b1 describe the first and second 128 weight rows of a tile: the same matrix for plain
// projections, the gate and the up matrix for kEpiSwiGLU.
cudaError_t launch_gemm_tc(const TmaDesc& a, const TmaDesc& b0, const TmaDesc& b1, void* out, float* resid, int m,
                           int n, int k, int epilogue, const QkvRopeArgs* qa, int* err, cudaStream_t st);
// The same GEMM on CTA pairs (tcgen05 cta_group::2, 256x256 tiles per cluster of two CTAs).
cudaError_t launch_gemm_tc2(const TmaDesc& a, const TmaDesc& b0, const TmaDesc& b1, void* out, float* resid, int m,
                            int n, int k, int epilogue, const QkvRopeArgs* qa, int* err, cudaStream_t st, bool reverse = false,
                            const float* bias = nullptr);
// head_dim 128 or 64
cudaError_t launch_attention_tc(const void* qkv, void* out, const int* cu, int seq0, int nseq, int row0, int rows,
                                int max_len, int n_q_heads, int n_kv_heads, int causal, int* err, cudaStream_t st,
                                int head_dim = 128);
// Two query heads of a key/value group per CTA, persistent (needs an even group size n_q_heads / n_kv_heads).
cudaError_t launch_attention_tc2(const void* qkv, void* out, const int* cu, int seq0, int nseq, int row0, int rows,
                                int max_len, int n_q_heads, int n_kv_heads, int causal, int* err, cudaStream_t st, bool reverse = false, int prefix = 0,
                                const void* qkv_prefix = nullptr, bool write_prefix = true, int head_dim = 128);
cudaError_t launch_attention_mma(const void* qkv, void* out, const int* cu, int seq0, int nseq, int row0,
                                 int max_len, int n_q_heads, int n_kv_heads, int causal, cudaStream_t st);

cudaError_t launch_route(const float* scores, const int* cu_old, const int* seq2orig_old, int n,
                         const RouteParams& p, int* cu_new, int* seq2orig_new, int* old_of_new,
                         RouteState* state, int* res_idx, float* res_score, ProbeRecordDev* rec,
                         float* trace_scores, int* trace_ids, void* scratch, cudaStream_t st);

}  // namespace prism
