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

// C[M,N] = A[M,K] * B[N,K]^T, TM x TM tile (64 or 32), 4x4 outputs per thread, K step 16.  The next K step's
// operands are fetched into registers while the current one is multiplied.  Every output element is one fmaf chain
// over k = 0, 1, 2, ... whatever the tile size, so a row's result depends neither on the tile size nor on where
// the row sits in the batch.
// kEpiSwiGLU computes two products (B = gate rows, B2 = up rows) and writes silu(g)*u.
template <typename T, int kEpi, int TM>
__global__ void __launch_bounds__(TM * TM / 16) k_gemm_simt(const T* __restrict__ a, const T* __restrict__ b,
                                                            const T* __restrict__ b2, T* __restrict__ out,
                                                            float* __restrict__ resid, int m, int n, int k,
                                                            const float* __restrict__ bias) {
  constexpr int BM = TM, BN = TM, BK = 16, NT = TM * TM / 16, TX = TM / 4, PER = BM * BK / NT;
  constexpr bool kTwo = kEpi == kEpiSwiGLU;
  __shared__ float sa[BK][BM + 1];
  __shared__ float sb[BK][BN + 1];
  __shared__ float sb2[kTwo ? BK : 1][BN + 1];
  pdl_sync();
  const int tx = threadIdx.x % TX, ty = threadIdx.x / TX;
  const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
  float acc[4][4] = {}, acc2[4][4] = {};
  float ra[PER], rb[PER], rc[PER];
  auto fetch = [&](int k0) {
#pragma unroll
    for (int i = 0; i < PER; ++i) {
      const int e = threadIdx.x + i * NT;
      const int r = e / BK, c = e % BK;
      const int gm = m0 + r, gn = n0 + r, gk = k0 + c;
      ra[i] = (gm < m && gk < k) ? ldf(a + (size_t)gm * k + gk) : 0.f;
      rb[i] = (gn < n && gk < k) ? ldf(b + (size_t)gn * k + gk) : 0.f;
      if constexpr (kTwo) rc[i] = (gn < n && gk < k) ? ldf(b2 + (size_t)gn * k + gk) : 0.f;
    }
  };
  fetch(0);
  for (int k0 = 0; k0 < k; k0 += BK) {
#pragma unroll
    for (int i = 0; i < PER; ++i) {
      const int e = threadIdx.x + i * NT;
      const int r = e / BK, c = e % BK;
      sa[c][r] = ra[i];
      sb[c][r] = rb[i];
      if constexpr (kTwo) sb2[c][r] = rc[i];
    }
    __syncthreads();
    if (k0 + BK < k) fetch(k0 + BK);
#pragma unroll
    for (int kk = 0; kk < BK; ++kk) {
      float av[4], bv[4], cv[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        av[i] = sa[kk][ty * 4 + i];
        bv[i] = sb[kk][tx * 4 + i];
        if constexpr (kTwo) cv[i] = sb2[kk][tx * 4 + i];
      }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
          if constexpr (kTwo) acc2[i][j] = fmaf(av[i], cv[j], acc2[i][j]);
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

// Attention, one warp per (query row, head).  Keys are visited 32 at a time with an online softmax: every lane
// forms the score of one key (the query row sits in shared memory), the chunk's maximum and sum come from warp
// shuffles, and the lanes then split head_dim to add the chunk's probability-weighted value rows.  dh <= 256.
template <typename T>
__global__ void __launch_bounds__(128) k_attention_simt(const T* __restrict__ qkv, T* __restrict__ out,
                                                        const int* __restrict__ cu, int seq0, int row0, int hq,
                                                        int hkv, int dh, int causal) {
  pdl_sync();
  __shared__ __align__(16) float sq[4][256];
  const int s = seq0 + blockIdx.z;
  const int beg = cu[s], len = cu[s + 1] - beg;
  const int w = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int t = blockIdx.x * 4 + w;
  if (t >= len) return;  // whole warps leave; the others synchronise among their own lanes only
  const int h = blockIdx.y, kvh = h / (hq / hkv);
  const size_t ld = (size_t)(hq + 2 * hkv) * dh;
  const T* base = qkv + (size_t)(beg - row0) * ld;
  const T* q = base + (size_t)t * ld + (size_t)h * dh;
  for (int c = lane; c < dh; c += 32) sq[w][c] = ldf(q + c);
  __syncwarp();
  const int per = (dh + 31) / 32;  // <= 8
  float o[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) o[i] = 0.f;
  const float scale = rsqrtf((float)dh);
  float mx = -INFINITY, den = 0.f;
  const int last = causal ? t : len - 1;
  const size_t koff = (size_t)(hq + kvh) * dh, voff = (size_t)(hq + hkv + kvh) * dh;
  for (int u0 = 0; u0 <= last; u0 += 32) {
    const int u = u0 + lane;
    float d = -INFINITY;
    if (u <= last) {
      const T* kr = base + (size_t)u * ld + koff;
      float acc = 0.f;
      if constexpr (sizeof(T) == 4) {
        // 16-byte loads where every key row starts on a 16-byte boundary (row pitch and head offsets are then
        // multiples of 16 bytes too)
        if ((dh & 3) == 0 && (reinterpret_cast<uintptr_t>(qkv) & 15) == 0) {
          const float4* k4 = reinterpret_cast<const float4*>(kr);
          const float4* q4 = reinterpret_cast<const float4*>(sq[w]);
          for (int c = 0; c < (dh >> 2); ++c) {
            const float4 kv = k4[c], qv = q4[c];
            acc = fmaf(qv.x, kv.x, acc);
            acc = fmaf(qv.y, kv.y, acc);
            acc = fmaf(qv.z, kv.z, acc);
            acc = fmaf(qv.w, kv.w, acc);
          }
        } else {
          for (int c = 0; c < dh; ++c) acc = fmaf(sq[w][c], ldf(kr + c), acc);
        }
      } else {
        for (int c = 0; c < dh; ++c) acc = fmaf(sq[w][c], ldf(kr + c), acc);
      }
      d = acc * scale;
    }
    float cm = d;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) cm = fmaxf(cm, __shfl_xor_sync(0xffffffffu, cm, off));
    const float nm = fmaxf(mx, cm);      // finite: lane 0's key of every chunk is visible
    const float corr = expf(mx - nm);    // 0 for the first chunk
    const float p = u <= last ? expf(d - nm) : 0.f;
    float ps = p;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) ps += __shfl_xor_sync(0xffffffffu, ps, off);
    den = den * corr + ps;
#pragma unroll
    for (int i = 0; i < 8; ++i) o[i] *= corr;
    const int nv = min(32, last - u0 + 1);
    for (int uu = 0; uu < nv; ++uu) {
      const float pu = __shfl_sync(0xffffffffu, p, uu);
      const T* vr = base + (size_t)(u0 + uu) * ld + voff;
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const int c = lane + 32 * i;
        if (i < per && c < dh) o[i] = fmaf(pu, ldf(vr + c), o[i]);
      }
    }
    mx = nm;
  }
  T* orow = out + (size_t)(beg - row0 + t) * ((size_t)hq * dh) + (size_t)h * dh;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int c = lane + 32 * i;
    if (i < per && c < dh) stf(orow + c, o[i] / den);
  }
}

}  // namespace

namespace {
template <typename K, typename... Args>
cudaError_t launch_pdl(K kernel, dim3 grid, int threads, cudaStream_t st, long long rows, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = dim3(threads);
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl_for(rows) ? 1 : 0;
  if (cudaError_t e = cudaLaunchKernelEx(&cfg, kernel, args...)) return e;
  return cudaGetLastError();
}
}  // namespace

cudaError_t launch_gemm_simt(const void* a, const void* b, const void* b2, void* out, float* resid, int m,
                             int n, int k, int dtype, int epilogue, cudaStream_t st, const float* bias) {
  if (m <= 0 || n <= 0) return cudaSuccess;
  if (epilogue >= kEpiStoreBias && !bias) return cudaErrorInvalidValue;
  // 64 x 64 tiles where they fill the machine twice over, else 32 x 32 (four times the blocks); same results
  const long long big = (long long)((n + 63) / 64) * ((m + 63) / 64);
  const bool small = big < 2ll * gemm_tc_sm_count();
  const dim3 grid = small ? dim3((n + 31) / 32, (m + 31) / 32) : dim3((n + 63) / 64, (m + 63) / 64);
#define PRISM_SIMT(T, E)                                                                                              \
  return small ? launch_pdl(k_gemm_simt<T, E, 32>, grid, 64, st, m, (const T*)a, (const T*)b, (const T*)b2, (T*)out, \
                            resid, m, n, k, bias)                                                                     \
               : launch_pdl(k_gemm_simt<T, E, 64>, grid, 256, st, m, (const T*)a, (const T*)b, (const T*)b2, (T*)out, \
                            resid, m, n, k, bias)
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
}

cudaError_t launch_attention_simt(const void* qkv, void* out, const int* cu, int seq0, int nseq, int row0,
                                  int max_len, int n_q_heads, int n_kv_heads, int head_dim, int causal,
                                  int dtype, cudaStream_t st) {
  if (nseq <= 0 || max_len <= 0) return cudaSuccess;
  dim3 grid((max_len + 3) / 4, n_q_heads, nseq);
  const long long rows = (long long)max_len * nseq;
  if (dtype == 1)
    return launch_pdl(k_attention_simt<__nv_bfloat16>, grid, 128, st, rows, (const __nv_bfloat16*)qkv, (__nv_bfloat16*)out,
                      cu, seq0, row0, n_q_heads, n_kv_heads, head_dim, causal);
  return launch_pdl(k_attention_simt<float>, grid, 128, st, rows, (const float*)qkv, (float*)out, cu, seq0, row0,
                    n_q_heads, n_kv_heads, head_dim, causal);
}

}  // namespace prism
