// S5: varlen flash attention over packed sequences, bf16, head_dim 128, GQA, causal or
// bidirectional.  One CTA = 64 query rows of one (sequence, head); 4 warps x 16 rows.
// K/V tiles of 64 keys stream through a double-buffered cp.async pipeline; QK^T and PV run on
// warp-level bf16 MMA with fp32 accumulation; softmax is online in fp32 (exp2 with folded scale).
#include "common.cuh"

namespace prism {

namespace {

constexpr int kBM = 64, kBN = 64, kDh = 128;
constexpr int kTileBytes = kBN * kDh * 2;  // 16 KB
constexpr int kAttnSmem = kTileBytes * 5;  // Q + 2 x (K, V)

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

// Byte offset of element (row, col) in a [64][128] bf16 tile whose 16-byte chunks are XOR-swizzled.
__device__ __forceinline__ uint32_t tile_off(int row, int col) {
  return (uint32_t)(row * 256 + ((((col >> 3) ^ (row & 7)) & 15) << 4) + ((col & 7) << 1));
}

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, bool valid) {
  const int sz = valid ? 16 : 0;  // size 0 -> the 16 destination bytes are zero-filled
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(sz) : "memory");
}
__device__ __forceinline__ void cp_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

__device__ __forceinline__ void ldsm4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldsm4t(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void mma16816(float* d, const uint32_t* a, uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack2(float a, float b) {
  __nv_bfloat162 v = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&v);
}

// Copy `rows_valid` rows (of 64) x 128 columns of bf16 into a swizzled tile; missing rows become zero.
__device__ __forceinline__ void load_tile(uint32_t tile, const __nv_bfloat16* src, size_t ld, int rows_valid) {
  for (int e = threadIdx.x; e < 64 * 16; e += 128) {
    const int r = e >> 4, ch = e & 15;
    const bool ok = r < rows_valid;
    const __nv_bfloat16* p = src + (ok ? (size_t)r * ld + ch * 8 : 0);
    cp_async16(tile + r * 256 + ((ch ^ (r & 7)) << 4), p, ok);
  }
}

__global__ void __launch_bounds__(128) k_attention_mma(const __nv_bfloat16* __restrict__ qkv,
                                                       __nv_bfloat16* __restrict__ out, const int* __restrict__ cu,
                                                       int seq0, int row0, int hq, int hkv, int causal,
                                                       float scale_log2) {
  extern __shared__ __align__(128) unsigned char smem[];
  const int s = seq0 + blockIdx.z;
  const int beg = cu[s], len = cu[s + 1] - beg;
  const int qb = (int)gridDim.x - 1 - (int)blockIdx.x;  // heaviest (latest) query blocks first
  if (qb * kBM >= len) return;
  const int h = blockIdx.y, kvh = h / (hq / hkv);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  const size_t ld = (size_t)(hq + 2 * hkv) * kDh;
  const __nv_bfloat16* base = qkv + (size_t)(beg - row0) * ld;
  const __nv_bfloat16* qsrc = base + (size_t)(qb * kBM) * ld + (size_t)h * kDh;
  const __nv_bfloat16* ksrc = base + (size_t)(hq + kvh) * kDh;
  const __nv_bfloat16* vsrc = base + (size_t)(hq + hkv + kvh) * kDh;

  const uint32_t sq = smem_u32(smem), sk = sq + kTileBytes, sv = sk + 2 * kTileBytes;
  const int n_blocks = causal ? qb + 1 : (len + kBN - 1) / kBN;

  load_tile(sq, qsrc, ld, min(kBM, len - qb * kBM));
  load_tile(sk, ksrc, ld, min(kBN, len));
  load_tile(sv, vsrc, ld, min(kBN, len));
  cp_commit();

  uint32_t qf[8][4];
  float o[16][4];
#pragma unroll
  for (int i = 0; i < 16; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
  float mx0 = -INFINITY, mx1 = -INFINITY, l0 = 0.f, l1 = 0.f;
  const int qrow0 = qb * kBM + warp * 16 + g, qrow1 = qrow0 + 8;

  for (int j = 0; j < n_blocks; ++j) {
    const int buf = j & 1;
    if (j + 1 < n_blocks) {  // prefetch the next K/V tile into the other buffer
      const int k0 = (j + 1) * kBN;
      load_tile(sk + (buf ^ 1) * kTileBytes, ksrc + (size_t)k0 * ld, ld, min(kBN, len - k0));
      load_tile(sv + (buf ^ 1) * kTileBytes, vsrc + (size_t)k0 * ld, ld, min(kBN, len - k0));
      cp_commit();
      cp_wait<1>();
    } else {
      cp_wait<0>();
    }
    __syncthreads();
    if (j == 0) {
#pragma unroll
      for (int ks = 0; ks < 8; ++ks) {
        const int r = warp * 16 + (lane & 7) + ((lane >> 3) & 1) * 8, c = ks * 16 + (lane >> 4) * 8;
        ldsm4(sq + tile_off(r, c), qf[ks][0], qf[ks][1], qf[ks][2], qf[ks][3]);
      }
    }
    const uint32_t kt = sk + buf * kTileBytes, vt = sv + buf * kTileBytes;

    // ---- S = Q K^T ------------------------------------------------------------------------
    float sc[8][4];
#pragma unroll
    for (int i = 0; i < 8; ++i) sc[i][0] = sc[i][1] = sc[i][2] = sc[i][3] = 0.f;
#pragma unroll
    for (int ks = 0; ks < 8; ++ks) {
#pragma unroll
      for (int np = 0; np < 4; ++np) {  // pairs of 8-key tiles
        const int r = np * 16 + (lane & 7) + (lane >> 4) * 8, c = ks * 16 + ((lane >> 3) & 1) * 8;
        uint32_t b0, b1, b2, b3;
        ldsm4(kt + tile_off(r, c), b0, b1, b2, b3);
        mma16816(sc[2 * np], qf[ks], b0, b1);
        mma16816(sc[2 * np + 1], qf[ks], b2, b3);
      }
    }
    // ---- mask ------------------------------------------------------------------------------
    const int key0 = j * kBN;
    const bool need_mask = (causal && j == qb) || (key0 + kBN > len);
    if (need_mask) {
#pragma unroll
      for (int i = 0; i < 8; ++i) {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int key = key0 + i * 8 + 2 * t + (e & 1);
          const int qr = (e < 2) ? qrow0 : qrow1;
          if (key >= len || (causal && key > qr)) sc[i][e] = -INFINITY;
        }
      }
    }
    // ---- online softmax --------------------------------------------------------------------
    float m0 = mx0, m1 = mx1;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      m0 = fmaxf(m0, fmaxf(sc[i][0], sc[i][1]));
      m1 = fmaxf(m1, fmaxf(sc[i][2], sc[i][3]));
    }
    m0 = fmaxf(m0, __shfl_xor_sync(0xffffffffu, m0, 1));
    m0 = fmaxf(m0, __shfl_xor_sync(0xffffffffu, m0, 2));
    m1 = fmaxf(m1, __shfl_xor_sync(0xffffffffu, m1, 1));
    m1 = fmaxf(m1, __shfl_xor_sync(0xffffffffu, m1, 2));
    // rows past the sequence end see only masked keys in bidirectional mode: keep them finite
    const float ms0 = (m0 == -INFINITY) ? 0.f : m0 * scale_log2;
    const float ms1 = (m1 == -INFINITY) ? 0.f : m1 * scale_log2;
    const float c0 = exp2f(mx0 * scale_log2 - ms0), c1 = exp2f(mx1 * scale_log2 - ms1);
    mx0 = m0;
    mx1 = m1;
    float rs0 = 0.f, rs1 = 0.f;
    uint32_t pf[4][4];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const float p0 = exp2f(sc[i][0] * scale_log2 - ms0), p1 = exp2f(sc[i][1] * scale_log2 - ms0);
      const float p2 = exp2f(sc[i][2] * scale_log2 - ms1), p3 = exp2f(sc[i][3] * scale_log2 - ms1);
      rs0 += p0 + p1;
      rs1 += p2 + p3;
      pf[i >> 1][(i & 1) * 2 + 0] = pack2(p0, p1);
      pf[i >> 1][(i & 1) * 2 + 1] = pack2(p2, p3);
    }
    l0 = l0 * c0 + rs0;
    l1 = l1 * c1 + rs1;
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      o[i][0] *= c0; o[i][1] *= c0; o[i][2] *= c1; o[i][3] *= c1;
    }
    // ---- O += P V ----------------------------------------------------------------------------
#pragma unroll
    for (int kk = 0; kk < 4; ++kk) {    // 16 keys per step
#pragma unroll
      for (int np = 0; np < 8; ++np) {  // pairs of 8-wide head_dim tiles
        const int r = kk * 16 + (lane & 7) + ((lane >> 3) & 1) * 8, c = np * 16 + (lane >> 4) * 8;
        uint32_t b0, b1, b2, b3;
        ldsm4t(vt + tile_off(r, c), b0, b1, b2, b3);
        mma16816(o[2 * np], pf[kk], b0, b1);
        mma16816(o[2 * np + 1], pf[kk], b2, b3);
      }
    }
    __syncthreads();  // the buffer just read is the prefetch target of the next iteration
  }

  l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
  l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
  l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
  l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
  const float i0 = 1.f / l0, i1 = 1.f / l1;
  const size_t ldo = (size_t)hq * kDh;
  __nv_bfloat16* obase = out + (size_t)(beg - row0) * ldo + (size_t)h * kDh;
#pragma unroll
  for (int i = 0; i < 16; ++i) {
    const int col = i * 8 + 2 * t;
    if (qrow0 < len) *reinterpret_cast<uint32_t*>(obase + (size_t)qrow0 * ldo + col) = pack2(o[i][0] * i0, o[i][1] * i0);
    if (qrow1 < len) *reinterpret_cast<uint32_t*>(obase + (size_t)qrow1 * ldo + col) = pack2(o[i][2] * i1, o[i][3] * i1);
  }
}

}  // namespace

cudaError_t launch_attention_mma(const void* qkv, void* out, const int* cu, int seq0, int nseq, int row0,
                                 int max_len, int n_q_heads, int n_kv_heads, int causal, cudaStream_t st) {
  if (nseq <= 0 || max_len <= 0) return cudaSuccess;
  static std::atomic<unsigned long long> smem_set{0};
  if (cudaError_t e = ensure_dynamic_smem(k_attention_mma, kAttnSmem, smem_set)) return e;
  dim3 grid((max_len + kBM - 1) / kBM, n_q_heads, nseq);
  const float scale_log2 = 1.4426950408889634f / sqrtf((float)kDh);
  k_attention_mma<<<grid, 128, kAttnSmem, st>>>((const __nv_bfloat16*)qkv, (__nv_bfloat16*)out, cu, seq0, row0,
                                                n_q_heads, n_kv_heads, causal, scale_log2);
  return cudaGetLastError();
}

}  // namespace prism
