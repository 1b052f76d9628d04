// CUDA-core (SIMT) GEMM and attention.  These are the production path of the fp32 mode (the tiny
// configuration whose tolerance, 1e-4, rules out reduced-precision tensor-core inputs) and the
// validation path of the bf16 mode (same bf16 inputs, fp32 accumulation, no tensor cores).
#include "common.cuh"

namespace prism {

namespace {

__device__ __forceinline__ float ldf(const float* p) { return *p; }
__device__ __forceinline__ float ldf(const __nv_bfloat16* p) { return __bfloat162float(*p); }
__device__ __forceinline__ void stf(float* p, float v) { *p = v; }
__device__ __forceinline__ void stf(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }

// C[M,N] = A[M,K] * B[N,K]^T, 64x64 tile, 16x16 threads, 4x4 per thread, K step 16.
// kEpiSwiGLU computes two products (B = gate rows, B2 = up rows) and writes silu(g)*u.
template <typename T, int kEpi>
__global__ void __launch_bounds__(256) k_gemm_simt(const T* __restrict__ a, const T* __restrict__ b,
                                                   const T* __restrict__ b2, T* __restrict__ out,
                                                   float* __restrict__ resid, int m, int n, int k,
                                                   const float* __restrict__ bias) {
  constexpr int BM = 64, BN = 64, BK = 16;
  __shared__ float sa[BK][BM + 1];
  __shared__ float sb[BK][BN + 1];
  __shared__ float sb2[kEpi == kEpiSwiGLU ? BK : 1][BN + 1];
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
  float acc[4][4] = {}, acc2[4][4] = {};
  for (int k0 = 0; k0 < k; k0 += BK) {
    for (int e = threadIdx.x; e < BM * BK; e += 256) {
      const int r = e / BK, c = e % BK;
      const int gm = m0 + r, gn = n0 + r, gk = k0 + c;
      sa[c][r] = (gm < m && gk < k) ? ldf(a + (size_t)gm * k + gk) : 0.f;
      sb[c][r] = (gn < n && gk < k) ? ldf(b + (size_t)gn * k + gk) : 0.f;
      if constexpr (kEpi == kEpiSwiGLU) sb2[c][r] = (gn < n && gk < k) ? ldf(b2 + (size_t)gn * k + gk) : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < BK; ++kk) {
      float av[4], bv[4], cv[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        av[i] = sa[kk][ty * 4 + i];
        bv[i] = sb[kk][tx * 4 + i];
        if constexpr (kEpi == kEpiSwiGLU) cv[i] = sb2[kk][tx * 4 + i];
      }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
          if constexpr (kEpi == kEpiSwiGLU) acc2[i][j] = fmaf(av[i], cv[j], acc2[i][j]);
        }
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int gm = m0 + ty * 4 + i;
    if (gm >= m) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int gn = n0 + tx * 4 + j;
      if (gn >= n) continue;
      const size_t o = (size_t)gm * n + gn;
      if constexpr (kEpi == kEpiStore) stf(out + o, acc[i][j]);
      if constexpr (kEpi == kEpiResidual) resid[o] += acc[i][j];
      if constexpr (kEpi == kEpiSwiGLU) {
        const float g = acc[i][j];
        stf(out + o, g / (1.f + expf(-g)) * acc2[i][j]);
      }
      if constexpr (kEpi == kEpiStoreBias) stf(out + o, acc[i][j] + bias[gn]);
      if constexpr (kEpi == kEpiGeluBias) {
        const float y = acc[i][j] + bias[gn];
        stf(out + o, 0.5f * y * (1.f + erff(y * 0.70710678118654752f)));
      }
      if constexpr (kEpi == kEpiResidualBias) resid[o] += acc[i][j] + bias[gn];
    }
  }
}

// Attention, one warp per (query row, head).  Lanes split head_dim; keys are visited in order with
// an online softmax.  dh <= 256.
template <typename T>
__global__ void __launch_bounds__(128) k_attention_simt(const T* __restrict__ qkv, T* __restrict__ out,
                                                        const int* __restrict__ cu, int seq0, int row0, int hq,
                                                        int hkv, int dh, int causal) {
  const int s = seq0 + blockIdx.z;
  const int beg = cu[s], len = cu[s + 1] - beg;
  const int t = blockIdx.x * 4 + (threadIdx.x >> 5);
  if (t >= len) return;
  const int h = blockIdx.y, kvh = h / (hq / hkv), lane = threadIdx.x & 31;
  const size_t ld = (size_t)(hq + 2 * hkv) * dh;
  const T* base = qkv + (size_t)(beg - row0) * ld;
  const T* q = base + (size_t)t * ld + (size_t)h * dh;
  const int per = (dh + 31) / 32;  // <= 8
  float qv[8], o[8];
  for (int i = 0; i < per; ++i) {
    const int c = lane + 32 * i;
    qv[i] = c < dh ? ldf(q + c) : 0.f;
    o[i] = 0.f;
  }
  const float scale = rsqrtf((float)dh);
  float mx = -INFINITY, den = 0.f;
  const int last = causal ? t : len - 1;
  for (int u = 0; u <= last; ++u) {
    const T* kr = base + (size_t)u * ld + (size_t)(hq + kvh) * dh;
    const T* vr = base + (size_t)u * ld + (size_t)(hq + hkv + kvh) * dh;
    float d = 0.f;
    for (int i = 0; i < per; ++i) {
      const int c = lane + 32 * i;
      if (c < dh) d += qv[i] * ldf(kr + c);
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) d += __shfl_xor_sync(0xffffffffu, d, off);
    d *= scale;
    const float nm = fmaxf(mx, d);
    const float corr = expf(mx - nm), p = expf(d - nm);
    den = den * corr + p;
    for (int i = 0; i < per; ++i) {
      const int c = lane + 32 * i;
      if (c < dh) o[i] = o[i] * corr + p * ldf(vr + c);
    }
    mx = nm;
  }
  T* orow = out + (size_t)(beg - row0 + t) * ((size_t)hq * dh) + (size_t)h * dh;
  for (int i = 0; i < per; ++i) {
    const int c = lane + 32 * i;
    if (c < dh) stf(orow + c, o[i] / den);
  }
}

}  // namespace

cudaError_t launch_gemm_simt(const void* a, const void* b, const void* b2, void* out, float* resid, int m,
                             int n, int k, int dtype, int epilogue, cudaStream_t st, const float* bias) {
  if (m <= 0 || n <= 0) return cudaSuccess;
  if (epilogue >= kEpiStoreBias && !bias) return cudaErrorInvalidValue;
  dim3 grid((n + 63) / 64, (m + 63) / 64);
#define PRISM_SIMT(T, E) \
  k_gemm_simt<T, E><<<grid, 256, 0, st>>>((const T*)a, (const T*)b, (const T*)b2, (T*)out, resid, m, n, k, bias)
  if (dtype == 1) {
    if (epilogue == kEpiStore) PRISM_SIMT(__nv_bfloat16, kEpiStore);
    else if (epilogue == kEpiResidual) PRISM_SIMT(__nv_bfloat16, kEpiResidual);
    else if (epilogue == kEpiStoreBias) PRISM_SIMT(__nv_bfloat16, kEpiStoreBias);
    else if (epilogue == kEpiGeluBias) PRISM_SIMT(__nv_bfloat16, kEpiGeluBias);
    else if (epilogue == kEpiResidualBias) PRISM_SIMT(__nv_bfloat16, kEpiResidualBias);
    else PRISM_SIMT(__nv_bfloat16, kEpiSwiGLU);
  } else {
    if (epilogue == kEpiStore) PRISM_SIMT(float, kEpiStore);
    else if (epilogue == kEpiResidual) PRISM_SIMT(float, kEpiResidual);
    else if (epilogue == kEpiStoreBias) PRISM_SIMT(float, kEpiStoreBias);
    else if (epilogue == kEpiGeluBias) PRISM_SIMT(float, kEpiGeluBias);
    else if (epilogue == kEpiResidualBias) PRISM_SIMT(float, kEpiResidualBias);
    else PRISM_SIMT(float, kEpiSwiGLU);
  }
#undef PRISM_SIMT
  return cudaGetLastError();
}

cudaError_t launch_attention_simt(const void* qkv, void* out, const int* cu, int seq0, int nseq, int row0,
                                  int max_len, int n_q_heads, int n_kv_heads, int head_dim, int causal,
                                  int dtype, cudaStream_t st) {
  if (nseq <= 0 || max_len <= 0) return cudaSuccess;
  dim3 grid((max_len + 3) / 4, n_q_heads, nseq);
  if (dtype == 1)
    k_attention_simt<__nv_bfloat16><<<grid, 128, 0, st>>>((const __nv_bfloat16*)qkv, (__nv_bfloat16*)out, cu,
                                                          seq0, row0, n_q_heads, n_kv_heads, head_dim, causal);
  else
    k_attention_simt<float><<<grid, 128, 0, st>>>((const float*)qkv, (float*)out, cu, seq0, row0, n_q_heads,
                                                  n_kv_heads, head_dim, causal);
  return cudaGetLastError();
}

}  // namespace prism
