/*
 * prism_ops.h -- the individual steps of the PRISM hot path as C entry points.
 *
 * prism_select (prism.h) chains these steps; they are exported one by one so that every kernel can be
 * checked against the CPU oracle and timed in isolation.  All pointers are DEVICE pointers unless
 * marked host; every call only enqueues work on `stream` (a cudaStream_t, NULL = default stream)
 * and returns a prism_status; nothing is copied to the host and nothing synchronises, except where a
 * call says it allocates temporary device scratch (cudaMalloc/cudaFree synchronise implicitly).
 * `dtype` is PRISM_FP32 or PRISM_BF16 and names the element type of weights and activations; the
 * residual stream x and all scores are float.  The caller owns every buffer.
 */
#ifndef PRISM_OPS_H_
#define PRISM_OPS_H_

#include "prism.h"

#ifdef __cplusplus
extern "C" {
#endif

/* Packing (Sec. 4.5 "consolidate all candidates into one monolithic batch", padding-free):
 * cu[N+1] = exclusive scan of (query_len + doc_len_i); seq2orig[i] = i; tokens[total] = query in front
 * of every document; pos[t] = position of row t inside its sequence.  err_word (int, zeroed by the
 * caller) receives bit 1 for a token id outside [0, vocab) and bit 2 for bad offsets.
 * `total` = sum of all sequence lengths (the caller knows the offsets). */
PRISM_API int prism_op_pack(const int32_t* query, int32_t query_len, const int32_t* cand_tokens, const int32_t* cand_offsets,
                  int32_t N, int32_t total, int32_t vocab, int32_t* tokens, int32_t* pos, int32_t* cu,
                  int32_t* seq2orig, int32_t* err_word, void* stream);

/* Embedding lookup into the fp32 residual stream: x[t,:] = table[tokens[t],:]. */
PRISM_API int prism_op_embed(const void* table, int32_t dtype, const int32_t* tokens, int32_t total, int32_t d, float* x,
                   void* stream);

/* RMSNorm: out[r,:] = x[r,:] / sqrt(mean(x[r,:]^2) + eps) * gain; out has element type `dtype`. */
PRISM_API int prism_op_rmsnorm(const float* x, const void* gain, int32_t dtype, int32_t rows, int32_t d, float eps, void* out,
                     void* stream);

/* Optional per-head RMSNorm over head_dim (gains g_q / g_k), then the rotary embedding with half-split
 * pairing (j, j + head_dim/2) and angle pos * theta^(-2j/head_dim); in place on the q and k heads of
 * qkv [rows, (Hq+2Hkv)*head_dim].  Allocates and frees a temporary rotary table of max_pos rows. */
PRISM_API int prism_op_qknorm_rope(void* qkv, int32_t dtype, const int32_t* pos, int32_t rows, int32_t n_q_heads,
                         int32_t n_kv_heads, int32_t head_dim, int32_t qk_norm, const void* g_q, const void* g_k,
                         float eps, float theta, int32_t max_pos, void* stream);

/* Projection GEMM C = A[m,k] * B[n,k]^T with a fused epilogue:
 *   epilogue 0: out[m,n] = C                      (dtype elements)
 *   epilogue 1: resid[m,n] += C                   (float residual stream; out unused)
 *   epilogue 2: out[m,n] = silu(A*B^T) * (A*B2^T) (SwiGLU; B = gate rows, B2 = up rows)
 * impl PRISM_IMPL_AUTO uses the tcgen05 tensor-core kernel on CTA pairs in bf16 mode (k, n multiples of 8;
 * n a multiple of 128 for epilogue 2; out and resid 16-byte aligned: they are written through TMA),
 * PRISM_IMPL_SOLO the single-CTA tcgen05 kernel, PRISM_IMPL_SIMT the CUDA-core kernel.  The tensor-core
 * kernels report an expired bounded wait in err_word bit 4 (nullable for SIMT). */
PRISM_API int prism_op_gemm(const void* a, const void* b, const void* b2, void* out, float* resid, int32_t m, int32_t n,
                  int32_t k, int32_t dtype, int32_t epilogue, int32_t impl, int32_t* err_word, void* stream);

/* The QKV projection with QK-norm and the rotary embedding fused into its epilogue (tensor-core path,
 * bf16, head_dim 128): out[m, (Hq+2Hkv)*128] = rope(qknorm(a[m,k] * w_qkv^T)) on the q and k heads, plain
 * projection on the v heads.  Equals prism_op_gemm(epilogue 0) followed by prism_op_qknorm_rope, except
 * that norm and rotation act on the fp32 accumulator (one rounding to bf16 instead of two).
 * The first call for a (device, theta, max_pos) builds a rotary table of max_pos rows (cudaMalloc) and
 * keeps it until the process exits or the parameters change; later calls only enqueue the kernel. */
PRISM_API int prism_op_gemm_qkv_rope(const void* a, const void* w_qkv, void* out, int32_t m, int32_t k,
                                     int32_t n_q_heads, int32_t n_kv_heads, int32_t qk_norm, const void* g_q,
                                     const void* g_k, float eps, const int32_t* pos, float theta, int32_t max_pos,
                                     int32_t* err_word, void* stream);

/* Attention over packed sequences: for sequence s (rows cu[s]..cu[s+1]) and query head h (kv head
 * h / (Hq/Hkv)): out = softmax(q k^T / sqrt(head_dim) [+ causal mask]) v.  qkv [total, (Hq+2Hkv)*dh],
 * out [total, Hq*dh].  total = cu[n_seq] rows; max_len >= the longest sequence.  impl: PRISM_IMPL_AUTO =
 * tcgen05 kernel (bf16; two query heads per CTA when Hq/Hkv is even (head_dim 128 or 64: the pair shares its KV
 * head) or when Hq = Hkv is even at head_dim 64 (a KV head per query head); else one head per CTA; reports an
 * expired bounded wait in err_word bit 4), PRISM_IMPL_SOLO = the one-head tcgen05
 * kernel, PRISM_IMPL_MMA = warp-level MMA kernel (bf16, head_dim 128), PRISM_IMPL_SIMT = CUDA cores. */
PRISM_API int prism_op_attention(const void* qkv, void* out, const int32_t* cu, int32_t n_seq, int32_t total,
                                 int32_t max_len, int32_t n_q_heads, int32_t n_kv_heads, int32_t head_dim,
                                 int32_t causal, int32_t dtype, int32_t impl, int32_t* err_word, void* stream);

/* ---- encoder stack (the encoder-only reranker of Sec. 6.1, Table 1; see PRISM_ARCH_ENCODER in prism.h) ---- */

/* Linear map with a bias: C = A[m,k] B[n,k]^T + bias[n] (bias fp32, device, 16-byte aligned).
 * epilogue 0: out[m,n] = C in element type `dtype`; 1: resid[m,n] += C (fp32); 2: out = gelu(C), gelu(x) = x Phi(x).
 * impl: PRISM_IMPL_AUTO = the tcgen05 kernel on CTA pairs (bf16; n and k multiples of 8; err_word as for
 * prism_op_gemm), PRISM_IMPL_SIMT = CUDA cores (fp32 or bf16). */
PRISM_API int prism_op_gemm_bias(const void* a, const void* b, const float* bias, void* out, float* resid, int32_t m, int32_t n,
                       int32_t k, int32_t dtype, int32_t epilogue, int32_t impl, int32_t* err_word, void* stream);

/* LayerNorm over rows of d (multiple of 4, <= 8192) fp32 values, IN PLACE: x = (x - mean) / sqrt(var + eps) * gain +
 * shift (biased variance; gain and shift fp32), and the same values in element type `dtype` to out[rows, d]. */
PRISM_API int prism_op_layernorm(float* x, const float* gain, const float* shift, int32_t dtype, int32_t rows, int32_t d, float eps,
                       void* out, void* stream);

/* Encoder input embedding: x[t,:] = table[tokens[t],:] + pos_table[pos[t] + pos_offset,:] + type_row (fp32 sum;
 * tables of element type `dtype`, type_row fp32).  The embedding LayerNorm is a separate prism_op_layernorm. */
PRISM_API int prism_op_embed_encoder(const void* table, const void* pos_table, const float* type_row, int32_t dtype,
                           const int32_t* tokens, const int32_t* pos, int32_t pos_offset, int32_t total, int32_t d, float* x,
                           void* stream);

/* Encoder score probe: for each sequence, LayerNorm (gain, shift, eps) of its FIRST row, then
 * out_w . tanh(dense_w y + dense_b) + out_b[0].  dense_w [d, d] in element type `dtype`, all vectors fp32.
 * A sequence without rows scores 0.  d a multiple of 4.  Allocates and frees a temporary scratch of 2 n d floats. */
PRISM_API int prism_op_probe_encoder(const float* x, const int32_t* cu, int32_t n, int32_t d, const float* gain, const float* shift,
                           float eps, const void* dense_w, int32_t dtype, const float* dense_b, const float* out_w,
                           const float* out_b, float* scores, void* stream);

/* W4 -> bf16 (PRISM_WFMT_W4 in prism.h gives the packed layout): out[n, k] bf16 from the packed blob of an [n, k]
 * matrix with `group` input channels per scale / zero point (group a multiple of 32, k a multiple of group; blob and
 * out device pointers, 16-byte aligned). */
PRISM_API int prism_op_dequant_w4(const void* blob, int32_t n, int32_t k, int32_t group, void* out, void* stream);

/* Score probe (Sec. 4.1: the model's classifier on an intermediate hidden state): for each sequence,
 * final RMSNorm of its last row, then logit(score_head row 0) - logit(score_head row 1).
 * Allocates and frees a temporary [d] float vector. */
PRISM_API int prism_op_probe(const float* x, const int32_t* cu, int32_t n, int32_t d, const void* g_final,
                   const void* score_head, int32_t dtype, float eps, float* scores, void* stream);

/* One pruning decision (Sec. 4.1): rank, CV, clustering, routing, survivor offsets.
 *   in : scores[n], cu_old[n+1], seq2orig_old[n]; state[8] = {n_active, n_tokens, k_rem, n_result,
 *        done, err, 0, 0} (only k_rem and n_result are read); sched fields as in prism_prune_schedule
 *        (keep_count applies to FIXED_KEEP); is_final = 1 scores the last layer; layer is recorded.
 *   out: cu_new[n_new+1], seq2orig_new[n_new], old_of_new[n_new] (old batch position of each
 *        survivor), state (updated), res_idx/res_score (leavers appended at n_result), rec (one
 *        prism_probe_record in device memory, nullable).
 * n <= PRISM_MAX_CANDIDATES.  Allocates and frees temporary device scratch. */
PRISM_API int prism_op_route(const float* scores, const int32_t* cu_old, const int32_t* seq2orig_old, int32_t n, int32_t mode,
                   int32_t keep_count, double cv_threshold, int32_t n_clusters, int32_t std_ddof,
                   int32_t select_winners, int32_t is_final, int32_t layer, int32_t* cu_new, int32_t* seq2orig_new,
                   int32_t* old_of_new, int32_t* state, int32_t* res_idx, float* res_score, prism_probe_record* rec,
                   void* stream);

/* The same pruning decision as prism_op_route for callers that cannot allocate device memory.  (The
 * paper has no counterpart: this is a property of the library, not of the method.)
 *
 * Who needs it: a host program whose own memory pool has already claimed the whole GPU, so that a
 * cudaMalloc made on its behalf fails; or a serving loop that must not stall, because cudaMalloc and
 * cudaFree wait for the device to go idle.  prism_op_route allocates and frees its clustering scratch
 * on every call; this entry point calls no cudaMalloc, cudaFree or any other allocating routine.  Its
 * scratch is an array of about 74 KB built into the library image, which every GPU that loads the
 * library keeps until the process ends.
 *
 * Limits and rules:
 *   - n <= PRISM_ROUTE_STATIC_MAX_CANDIDATES; a larger n returns PRISM_ERR_SHAPE_LIMIT and nothing runs.
 *   - The first call on each device looks up the array's address on that device (the device must be
 *     current).  Make that first call outside any stream capture.
 *   - All calls share the one array, and it keeps what the previous call left there.  The kernel
 *     writes every scratch word before it reads it, so nothing has to be cleared between calls; but
 *     two calls that overlap on the GPU (different streams, no ordering between them) race on it.
 *     Calls on one stream are safe.
 *   - Arguments, outputs and the result are exactly those of prism_op_route; the call only enqueues
 *     the kernel on `stream` and does not synchronise. */
#define PRISM_ROUTE_STATIC_MAX_CANDIDATES 1024
PRISM_API int prism_op_route_static(const float* scores, const int32_t* cu_old, const int32_t* seq2orig_old,
                                    int32_t n, int32_t mode, int32_t keep_count, double cv_threshold,
                                    int32_t n_clusters, int32_t std_ddof, int32_t select_winners,
                                    int32_t is_final, int32_t layer, int32_t* cu_new, int32_t* seq2orig_new,
                                    int32_t* old_of_new, int32_t* state, int32_t* res_idx, float* res_score,
                                    prism_probe_record* rec, void* stream);

/* Survivor gather (Fig. 4: only the deferred candidates are retained): row t of the new batch, owned
 * by new sequence s, is copied from x_old[cu_old[old_of_new[s]] + (t - cu_new[s])]. */
PRISM_API int prism_op_compact(const float* x_old, float* x_new, const int32_t* cu_old, const int32_t* cu_new,
                     const int32_t* old_of_new, int32_t n_new, int32_t total_new, int32_t d, void* stream);

/* Self-test of the bounded device-side wait that every tensor-core kernel uses (PRISM_ERR_TIMEOUT path):
 * one thread waits on a barrier that nothing arrives at, gives up after limit_cycles (1 .. 2e9 SM clock
 * cycles), sets bit 4 of err_word (device int32, zeroed by the caller) and the kernel returns.  Nothing
 * hangs or faults; the device stays usable. */
PRISM_API int prism_op_wait_selftest(uint64_t limit_cycles, int32_t* err_word, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* PRISM_OPS_H_ */
