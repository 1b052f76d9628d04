// C entry points for the individual steps (include/prism_ops.h): thin wrappers over the launchers
// that prism_select chains.
#include "../../include/prism_ops.h"
#include "common.cuh"

using namespace prism;

namespace {
int st_of(cudaError_t e) {
  if (e == cudaSuccess) return PRISM_OK;
  return e == cudaErrorMemoryAllocation ? PRISM_ERR_NOMEM : (e == cudaErrorInvalidValue ? PRISM_ERR_INVALID_ARG : PRISM_ERR_CUDA);
}
cudaStream_t S(void* s) { return reinterpret_cast<cudaStream_t>(s); }
}  // namespace

extern "C" {

int prism_op_pack(const int32_t* query, int32_t query_len, const int32_t* cand_tokens, const int32_t* cand_offsets,
                  int32_t N, int32_t total, int32_t vocab, int32_t* tokens, int32_t* pos, int32_t* cu,
                  int32_t* seq2orig, int32_t* err_word, void* stream) {
  if (N < 0 || N > kMaxCandidates || query_len < 0 || total < 0 || !cand_offsets || !cu || !seq2orig || !err_word)
    return PRISM_ERR_INVALID_ARG;
  cudaError_t e = launch_pack_offsets(cand_offsets, N, query_len, cu, seq2orig, err_word, S(stream));
  if (e == cudaSuccess)
    e = launch_pack_tokens(query, query_len, cand_tokens, cand_offsets, cu, N, total, vocab, tokens, pos, err_word, S(stream));
  return st_of(e);
}

int prism_op_embed(const void* table, int32_t dtype, const int32_t* tokens, int32_t total, int32_t d, float* x,
                   void* stream) {
  if (!table || !tokens || !x || d % 8) return PRISM_ERR_INVALID_ARG;
  return st_of(launch_embed(table, dtype, tokens, total, d, x, S(stream)));
}

int prism_op_rmsnorm(const float* x, const void* gain, int32_t dtype, int32_t rows, int32_t d, float eps, void* out,
                     void* stream) {
  if (!x || !gain || !out || d % 4) return PRISM_ERR_INVALID_ARG;
  return st_of(launch_rmsnorm(x, gain, dtype, rows, d, eps, out, S(stream)));
}

int prism_op_qknorm_rope(void* qkv, int32_t dtype, const int32_t* pos, int32_t rows, int32_t n_q_heads,
                         int32_t n_kv_heads, int32_t head_dim, int32_t qk_norm, const void* g_q, const void* g_k,
                         float eps, float theta, int32_t max_pos, void* stream) {
  if (!qkv || !pos || head_dim % 2 || head_dim > 256 || max_pos < 1) return PRISM_ERR_INVALID_ARG;
  float* tab = nullptr;
  const size_t half = head_dim / 2;
  cudaError_t e = cudaMalloc(&tab, 2 * (size_t)max_pos * half * sizeof(float));
  if (e != cudaSuccess) return st_of(e);
  e = launch_rope_table(tab, tab + (size_t)max_pos * half, max_pos, head_dim, theta, S(stream));
  if (e == cudaSuccess)
    e = launch_qknorm_rope(qkv, dtype, pos, rows, n_q_heads, n_kv_heads, head_dim, qk_norm, g_q, g_k, eps, tab,
                           tab + (size_t)max_pos * half, S(stream));
  cudaStreamSynchronize(S(stream));
  cudaFree(tab);
  return st_of(e);
}

int prism_op_gemm(const void* a, const void* b, const void* b2, void* out, float* resid, int32_t m, int32_t n,
                  int32_t k, int32_t dtype, int32_t epilogue, int32_t impl, int32_t* err_word, void* stream) {
  if (!a || !b || m < 0 || n < 1 || k < 1 || epilogue < 0 || epilogue > 2) return PRISM_ERR_INVALID_ARG;
  if (epilogue == kEpiSwiGLU && !b2) return PRISM_ERR_INVALID_ARG;
  if (epilogue == kEpiResidual ? !resid : !out) return PRISM_ERR_INVALID_ARG;
  if (dtype == PRISM_BF16 && (impl == PRISM_IMPL_AUTO || impl == PRISM_IMPL_SOLO)) {
    if (!err_word || (k % 8) || (n % 8) || (epilogue == kEpiSwiGLU && n % 128)) return PRISM_ERR_UNSUPPORTED;
    TmaDesc ma, mb0, mb1;
    cudaError_t e = make_tma_2d_bf16(&ma, a, (uint64_t)m, (uint64_t)k, 128, 64);
    if (e == cudaSuccess) e = make_tma_2d_bf16(&mb0, b, (uint64_t)n, (uint64_t)k, 128, 64);
    if (e == cudaSuccess) e = make_tma_2d_bf16(&mb1, epilogue == kEpiSwiGLU ? b2 : b, (uint64_t)n, (uint64_t)k, 128, 64);
    if (e == cudaSuccess)
      e = impl == PRISM_IMPL_AUTO ? launch_gemm_tc2(ma, mb0, mb1, out, resid, m, n, k, epilogue, nullptr, err_word, S(stream))
                                  : launch_gemm_tc(ma, mb0, mb1, out, resid, m, n, k, epilogue, nullptr, err_word, S(stream));
    return st_of(e);
  }
  return st_of(launch_gemm_simt(a, b, b2, out, resid, m, n, k, dtype, epilogue, S(stream)));
}

int prism_op_dequant_w4(const void* blob, int32_t n, int32_t k, int32_t group, void* out, void* stream) {
  if (!blob || !out || n < 0 || k < 32 || group < 32 || (k % group) || (group % 32)) return PRISM_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(blob) & 15) || (reinterpret_cast<uintptr_t>(out) & 15)) return PRISM_ERR_INVALID_ARG;
  return st_of(launch_dequant_w4(blob, n, k, group, out, S(stream)));
}

int prism_op_gemm_bias(const void* a, const void* b, const float* bias, void* out, float* resid, int32_t m, int32_t n,
                       int32_t k, int32_t dtype, int32_t epilogue, int32_t impl, int32_t* err_word, void* stream) {
  if (!a || !b || !bias || m < 0 || n < 1 || k < 1 || epilogue < 0 || epilogue > 2) return PRISM_ERR_INVALID_ARG;
  if (epilogue == 1 ? !resid : !out) return PRISM_ERR_INVALID_ARG;
  const int epi = epilogue == 0 ? kEpiStoreBias : epilogue == 1 ? kEpiResidualBias : kEpiGeluBias;
  if (dtype == PRISM_BF16 && impl == PRISM_IMPL_AUTO) {
    if (!err_word || (k % 8) || (n % 8)) return PRISM_ERR_UNSUPPORTED;
    TmaDesc ma, mb;
    cudaError_t e = make_tma_2d_bf16(&ma, a, (uint64_t)m, (uint64_t)k, 128, 64);
    if (e == cudaSuccess) e = make_tma_2d_bf16(&mb, b, (uint64_t)n, (uint64_t)k, 128, 64);
    if (e == cudaSuccess) e = launch_gemm_tc2(ma, mb, mb, out, resid, m, n, k, epi, nullptr, err_word, S(stream), false, bias);
    return st_of(e);
  }
  if (impl != PRISM_IMPL_SIMT && dtype == PRISM_BF16) return PRISM_ERR_UNSUPPORTED;
  return st_of(launch_gemm_simt(a, b, nullptr, out, resid, m, n, k, dtype, epi, S(stream), bias));
}

int prism_op_layernorm(float* x, const float* gain, const float* shift, int32_t dtype, int32_t rows, int32_t d, float eps,
                       void* out, void* stream) {
  if (!x || !gain || !shift || !out || rows < 0 || d < 4 || (d % 4) || d > 8192) return PRISM_ERR_INVALID_ARG;
  return st_of(launch_layernorm(x, gain, shift, dtype, rows, d, eps, out, S(stream)));
}

int prism_op_embed_encoder(const void* table, const void* pos_table, const float* type_row, int32_t dtype,
                           const int32_t* tokens, const int32_t* pos, int32_t pos_offset, int32_t total, int32_t d, float* x,
                           void* stream) {
  if (!table || !pos_table || !type_row || !tokens || !pos || !x || total < 0 || (d % 4) || pos_offset < 0)
    return PRISM_ERR_INVALID_ARG;
  if (dtype == PRISM_BF16 && (d % 8)) return PRISM_ERR_INVALID_ARG;
  return st_of(launch_embed_encoder(table, pos_table, type_row, dtype, tokens, pos, pos_offset, total, d, x, S(stream)));
}

int prism_op_probe_encoder(const float* x, const int32_t* cu, int32_t n, int32_t d, const float* gain, const float* shift,
                           float eps, const void* dense_w, int32_t dtype, const float* dense_b, const float* out_w,
                           const float* out_b, float* scores, void* stream) {
  if (!x || !cu || !gain || !shift || !dense_w || !dense_b || !out_w || !out_b || !scores || n < 0 || d < 1 || d > 8192)
    return PRISM_ERR_INVALID_ARG;
  if (n == 0) return PRISM_OK;
  if (d % 4) return PRISM_ERR_INVALID_ARG;
  float* scratch = nullptr;
  cudaError_t e = cudaMalloc(&scratch, 2 * (size_t)n * d * sizeof(float));
  if (e != cudaSuccess) return st_of(e);
  e = launch_probe_encoder(x, cu, n, d, gain, shift, eps, dense_w, dtype, dense_b, out_w, out_b, scores, scratch, S(stream));
  cudaStreamSynchronize(S(stream));
  cudaFree(scratch);
  return st_of(e);
}

int prism_op_gemm_qkv_rope(const void* a, const void* w_qkv, void* out, int32_t m, int32_t k, int32_t n_q_heads,
                           int32_t n_kv_heads, int32_t qk_norm, const void* g_q, const void* g_k, float eps,
                           const int32_t* pos, float theta, int32_t max_pos, int32_t* err_word, void* stream) {
  if (!a || !w_qkv || !out || !pos || !err_word || m < 0 || k < 1 || (k % 8) || max_pos < 1) return PRISM_ERR_INVALID_ARG;
  if (qk_norm && (!g_q || !g_k)) return PRISM_ERR_INVALID_ARG;
  const int n = (n_q_heads + 2 * n_kv_heads) * 128;
  // The rotary table is built once per (device, theta, max_pos) and kept until the process exits.
  static float* tab = nullptr;
  static int tab_dev = -1, tab_pos = 0;
  static float tab_theta = 0.f;
  int dev = 0;
  cudaGetDevice(&dev);
  cudaError_t e = cudaSuccess;
  if (!tab || tab_dev != dev || tab_pos != max_pos || tab_theta != theta) {
    if (tab) {
      cudaDeviceSynchronize();
      cudaFree(tab);
      tab = nullptr;
    }
    e = cudaMalloc(&tab, (size_t)max_pos * 128 * sizeof(float));
    if (e != cudaSuccess) return st_of(e);
    e = launch_rope_table_fused(tab, max_pos, theta, S(stream));
    if (e == cudaSuccess) e = cudaStreamSynchronize(S(stream));
    tab_dev = dev;
    tab_pos = max_pos;
    tab_theta = theta;
  }
  TmaDesc ma, mb;
  if (e == cudaSuccess) e = make_tma_2d_bf16(&ma, a, (uint64_t)m, (uint64_t)k, 128, 64);
  if (e == cudaSuccess) e = make_tma_2d_bf16(&mb, w_qkv, (uint64_t)n, (uint64_t)k, 128, 64);
  QkvRopeArgs qa{pos, tab, (const __nv_bfloat16*)g_q, (const __nv_bfloat16*)g_k, n_q_heads, n_kv_heads, qk_norm, eps};
  if (e == cudaSuccess) e = launch_gemm_tc2(ma, mb, mb, out, nullptr, m, n, k, kEpiQkvRope, &qa, err_word, S(stream));
  return st_of(e);
}

int prism_op_attention(const void* qkv, void* out, const int32_t* cu, int32_t n_seq, int32_t total, int32_t max_len,
                       int32_t n_q_heads, int32_t n_kv_heads, int32_t head_dim, int32_t causal, int32_t dtype,
                       int32_t impl, int32_t* err_word, void* stream) {
  if (!qkv || !out || !cu || n_seq < 0 || total < 0 || n_kv_heads < 1 || n_q_heads % n_kv_heads) return PRISM_ERR_INVALID_ARG;
  if (dtype == PRISM_BF16 && impl != PRISM_IMPL_SIMT) {
    if (head_dim != 128 && !(head_dim == 64 && impl != PRISM_IMPL_MMA)) return PRISM_ERR_UNSUPPORTED;
    if (impl == PRISM_IMPL_AUTO || impl == PRISM_IMPL_SOLO) {
      if (!err_word) return PRISM_ERR_INVALID_ARG;
      const int group = n_q_heads / n_kv_heads;
      const bool two_heads = (group & 1) == 0 ? true : (group == 1 && head_dim == 64 && (n_q_heads & 1) == 0);
      if (impl == PRISM_IMPL_AUTO && two_heads)
        return st_of(launch_attention_tc2(qkv, out, cu, 0, n_seq, 0, total, max_len, n_q_heads, n_kv_heads, causal,
                                          err_word, S(stream), false, 0, nullptr, true, head_dim));
      return st_of(launch_attention_tc(qkv, out, cu, 0, n_seq, 0, total, max_len, n_q_heads, n_kv_heads, causal, err_word,
                                       S(stream), head_dim));
    }
    return st_of(launch_attention_mma(qkv, out, cu, 0, n_seq, 0, max_len, n_q_heads, n_kv_heads, causal, S(stream)));
  }
  if (head_dim > 256) return PRISM_ERR_UNSUPPORTED;
  return st_of(launch_attention_simt(qkv, out, cu, 0, n_seq, 0, max_len, n_q_heads, n_kv_heads, head_dim, causal, dtype,
                                     S(stream)));
}

int prism_op_probe(const float* x, const int32_t* cu, int32_t n, int32_t d, const void* g_final,
                   const void* score_head, int32_t dtype, float eps, float* scores, void* stream) {
  if (!x || !cu || !g_final || !score_head || !scores || d % 4) return PRISM_ERR_INVALID_ARG;
  float* wd = nullptr;
  cudaError_t e = cudaMalloc(&wd, (size_t)d * sizeof(float));
  if (e != cudaSuccess) return st_of(e);
  e = launch_score_diff(score_head, dtype, d, wd, S(stream));
  if (e == cudaSuccess) e = launch_probe(x, cu, n, d, g_final, dtype, wd, eps, scores, S(stream));
  cudaStreamSynchronize(S(stream));
  cudaFree(wd);
  return st_of(e);
}

int prism_op_route(const float* scores, const int32_t* cu_old, const int32_t* seq2orig_old, int32_t n, int32_t mode,
                   int32_t keep_count, double cv_threshold, int32_t n_clusters, int32_t std_ddof,
                   int32_t select_winners, int32_t is_final, int32_t layer, int32_t* cu_new, int32_t* seq2orig_new,
                   int32_t* old_of_new, int32_t* state, int32_t* res_idx, float* res_score, prism_probe_record* rec,
                   void* stream) {
  if (!scores || !cu_old || !seq2orig_old || !cu_new || !seq2orig_new || !old_of_new || !state || !res_idx || !res_score)
    return PRISM_ERR_INVALID_ARG;
  if (!route_args_ok(n, mode, keep_count, n_clusters, std_ddof, kMaxCandidates)) return PRISM_ERR_INVALID_ARG;
  void* scratch = nullptr;
  cudaError_t e = cudaMalloc(&scratch, route_scratch_bytes(n));
  if (e != cudaSuccess) return st_of(e);
  RouteParams p{};
  p.mode = mode;
  p.keep_count = keep_count;
  p.cv_threshold = cv_threshold;
  p.n_clusters = n_clusters;
  p.ddof = std_ddof;
  p.select_winners = select_winners;
  p.is_final = is_final;
  p.layer = layer;
  e = launch_route(scores, cu_old, seq2orig_old, n, p, cu_new, seq2orig_new, old_of_new,
                   reinterpret_cast<RouteState*>(state), res_idx, res_score, reinterpret_cast<ProbeRecordDev*>(rec),
                   nullptr, nullptr, scratch, S(stream));
  cudaStreamSynchronize(S(stream));
  cudaFree(scratch);
  return st_of(e);
}

int prism_op_compact(const float* x_old, float* x_new, const int32_t* cu_old, const int32_t* cu_new,
                     const int32_t* old_of_new, int32_t n_new, int32_t total_new, int32_t d, void* stream) {
  if (!x_old || !x_new || !cu_old || !cu_new || !old_of_new || d % 4) return PRISM_ERR_INVALID_ARG;
  return st_of(launch_compact_rows(x_old, x_new, cu_old, cu_new, old_of_new, n_new, total_new, d, S(stream)));
}

}  // extern "C"
