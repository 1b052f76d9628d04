// HBM-bound kernels of the PRISM hot path: packing, embedding gather, RMSNorm, QK-norm + rotary
// embedding, the score probe and the survivor row gather.  All accesses are 16-byte vectorised
// and coalesced along the hidden dimension; reductions are fp32.
#include <cstdlib>

#include "common.cuh"

namespace prism {

namespace {

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Sum over the block; every thread gets the result.  red must hold 32 floats.
__device__ __forceinline__ float block_sum(float v, float* red) {
  v = warp_sum(v);
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
  __syncthreads();
  if (lane == 0) red[w] = v;
  __syncthreads();
  float t = (lane < nw) ? red[lane] : 0.f;
  t = warp_sum(t);
  return t;
}

__device__ __forceinline__ float to_f(float v) { return v; }
__device__ __forceinline__ float to_f(__nv_bfloat16 v) { return __bfloat162float(v); }
__device__ __forceinline__ void from_f(float& o, float v) { o = v; }
__device__ __forceinline__ void from_f(__nv_bfloat16& o, float v) { o = __float2bfloat16_rn(v); }

// upper_bound(cu[0..n], t) - 1: the sequence that owns packed row t.
__device__ __forceinline__ int seq_of_row(const int* __restrict__ cu, int n, int t) {
  int lo = 0, hi = n;  // invariant: cu[lo] <= t < cu[hi]
  while (hi - lo > 1) {
    int mid = (lo + hi) >> 1;
    if (cu[mid] <= t) lo = mid; else hi = mid;
  }
  return lo;
}

// ------------------------------------------------------------------------------------------------
// S0 pack: cu = exclusive scan of (query_len + doc_len_i), seq2orig = identity.  One block.  With an ownership
// mask (candidate-sharded runs) the candidates of other ranks become sequences of length zero: they keep their
// place in every per-sequence array and take no rows.
// With a shared query prefix (shared = 1) the query's lq rows are stored once, in front of the batch, and
// sequence i keeps only its document rows: cu[i] = lq + sum of the document lengths before i.
__global__ void __launch_bounds__(1024) k_pack_offsets(const int* __restrict__ off, int n, int lq,
                                                       const unsigned char* __restrict__ owned, int shared,
                                                       int* __restrict__ cu, int* __restrict__ seq2orig,
                                                       int* __restrict__ err) {
  __shared__ int warp_tot[32];
  __shared__ int carry;
  if (threadIdx.x == 0) {
    carry = 0;
    if (n > 0 && off[0] != 0) atomicOr(err, kErrBadOffsets);
  }
  __syncthreads();
  for (int base = 0; base < n; base += blockDim.x) {
    int i = base + threadIdx.x;
    int len = 0;
    if (i < n) {
      int dl = off[i + 1] - off[i];
      if (dl < 0) { atomicOr(err, kErrBadOffsets); dl = 0; }
      len = (owned && !owned[i]) ? 0 : (shared ? dl : lq + dl);
      seq2orig[i] = i;
    }
    int v = len;
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      int u = __shfl_up_sync(0xffffffffu, v, o);
      if (lane >= o) v += u;
    }
    if (lane == 31) warp_tot[w] = v;
    __syncthreads();
    if (w == 0) {
      int t = warp_tot[lane];
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        int u = __shfl_up_sync(0xffffffffu, t, o);
        if (lane >= o) t += u;
      }
      warp_tot[lane] = t;
    }
    __syncthreads();
    int excl = carry + (w ? warp_tot[w - 1] : 0) + v - len + (shared ? lq : 0);
    if (i < n) cu[i] = excl;
    __syncthreads();
    if (threadIdx.x == blockDim.x - 1) carry += warp_tot[31];
    __syncthreads();
  }
  if (threadIdx.x == 0) cu[n] = carry + (shared ? lq : 0);
}

// Packed token ids (query in front of every document) and per-token positions.
__global__ void k_pack_tokens(const int* __restrict__ query, int lq, const int* __restrict__ cand,
                              const int* __restrict__ off, const int* __restrict__ cu, int n, int total,
                              int vocab, int shared, int* __restrict__ tokens, int* __restrict__ pos,
                              int* __restrict__ err) {
  for (int t = blockIdx.x * blockDim.x + threadIdx.x; t < total; t += gridDim.x * blockDim.x) {
    int tok, p;
    if (shared && t < lq) {  // the shared query prefix
      p = t;
      tok = query[t];
    } else {
      int s = seq_of_row(cu, n, t);
      p = t - cu[s] + (shared ? lq : 0);  // position inside the sequence query || document
      tok = (p < lq) ? query[p] : cand[off[s] + (p - lq)];
    }
    if (tok < 0 || tok >= vocab) { atomicOr(err, kErrBadToken); tok = 0; }
    tokens[t] = tok;
    pos[t] = p;
  }
}

__global__ void k_positions(const int* __restrict__ cu, int n, int total, int prefix, int* __restrict__ pos) {
  pdl_sync();
  for (int t = blockIdx.x * blockDim.x + threadIdx.x; t < total; t += gridDim.x * blockDim.x) {
    if (t < prefix) {
      pos[t] = t;
    } else {
      int s = seq_of_row(cu, n, t);
      pos[t] = t - cu[s] + prefix;
    }
  }
}

// ------------------------------------------------------------------------------------------------
// S1 embedding gather into the fp32 residual stream.  One block per token row.
// With a row cache (Sec. 4.4) `table` is the cache and tok2slot maps a token id to its row there.
template <typename WT>
__global__ void __launch_bounds__(128) k_embed(const WT* __restrict__ table, const int* __restrict__ tokens,
                                               const int* __restrict__ tok2slot, int d, float* __restrict__ x) {
  const int t = blockIdx.x;
  const int tok = tokens[t];
  const WT* src = table + (size_t)(tok2slot ? tok2slot[tok] : tok) * d;
  float* dst = x + (size_t)t * d;
  if constexpr (sizeof(WT) == 2) {
    for (int c = threadIdx.x * 8; c < d; c += blockDim.x * 8) {
      uint4 raw = *reinterpret_cast<const uint4*>(src + c);
      const __nv_bfloat16* b = reinterpret_cast<const __nv_bfloat16*>(&raw);
      float4 lo = make_float4(to_f(b[0]), to_f(b[1]), to_f(b[2]), to_f(b[3]));
      float4 hi = make_float4(to_f(b[4]), to_f(b[5]), to_f(b[6]), to_f(b[7]));
      *reinterpret_cast<float4*>(dst + c) = lo;
      *reinterpret_cast<float4*>(dst + c + 4) = hi;
    }
  } else {
    for (int c = threadIdx.x * 4; c < d; c += blockDim.x * 4)
      *reinterpret_cast<float4*>(dst + c) = *reinterpret_cast<const float4*>(src + c);
  }
}

// ------------------------------------------------------------------------------------------------
// S2/S7 RMSNorm: y = x * rsqrt(mean(x^2) + eps) * g.  One block per row; the row stays in registers.
template <typename OT, int kVec>
__global__ void __launch_bounds__(256) k_rmsnorm(const float* __restrict__ x, const OT* __restrict__ gain, int d,
                                                 float eps, OT* __restrict__ out, int reverse) {
  __shared__ float red[32];
  const size_t row = reverse ? gridDim.x - 1 - blockIdx.x : blockIdx.x;  // last rows first: see launch_rmsnorm
  const float4* xr = reinterpret_cast<const float4*>(x + row * d);
  const int nv = d >> 2;
  float4 v[kVec];
  float ss = 0.f;
#pragma unroll
  for (int i = 0; i < kVec; ++i) {
    int c = threadIdx.x + i * 256;
    if (c < nv) {
      v[i] = xr[c];
      ss += v[i].x * v[i].x + v[i].y * v[i].y + v[i].z * v[i].z + v[i].w * v[i].w;
    }
  }
  ss = block_sum(ss, red);
  const float r = 1.0f / sqrtf(ss / (float)d + eps);
  OT* orow = out + row * d;
#pragma unroll
  for (int i = 0; i < kVec; ++i) {
    int c = threadIdx.x + i * 256;
    if (c < nv) {
      const OT* g = gain + 4 * c;
      float o0 = v[i].x * r * to_f(g[0]), o1 = v[i].y * r * to_f(g[1]);
      float o2 = v[i].z * r * to_f(g[2]), o3 = v[i].w * r * to_f(g[3]);
      if constexpr (sizeof(OT) == 2) {
        __nv_bfloat162 a = __floats2bfloat162_rn(o0, o1), b = __floats2bfloat162_rn(o2, o3);
        uint2 pk = make_uint2(*reinterpret_cast<uint32_t*>(&a), *reinterpret_cast<uint32_t*>(&b));
        *reinterpret_cast<uint2*>(orow + 4 * c) = pk;
      } else {
        *reinterpret_cast<float4*>(orow + 4 * c) = make_float4(o0, o1, o2, o3);
      }
    }
  }
}

// The same norm with one WARP per row (8 rows per block): every lane keeps kPer float4 of the row in
// flight, which hides HBM latency better than one block per row when the row is only a few KB.
template <typename OT, int kPer>
__global__ void __launch_bounds__(256) k_rmsnorm_warp(const float* __restrict__ x, const OT* __restrict__ gain,
                                                      int rows, int d, float eps, OT* __restrict__ out, int reverse) {
  pdl_sync();
  const int lane = threadIdx.x & 31;
  const long long blk = reverse ? (long long)gridDim.x - 1 - blockIdx.x : blockIdx.x;
  const long long row = blk * 8 + (threadIdx.x >> 5);
  if (row >= rows) return;
  const float4* xr = reinterpret_cast<const float4*>(x + (size_t)row * d);
  const int nv = d >> 2;
  float4 v[kPer];
  float ss = 0.f;
#pragma unroll
  for (int i = 0; i < kPer; ++i) {
    const int c = lane + i * 32;
    if (c < nv) v[i] = xr[c];
  }
#pragma unroll
  for (int i = 0; i < kPer; ++i) {
    const int c = lane + i * 32;
    if (c < nv) ss += v[i].x * v[i].x + v[i].y * v[i].y + v[i].z * v[i].z + v[i].w * v[i].w;
  }
  ss = warp_sum(ss);
  const float r = 1.0f / sqrtf(ss / (float)d + eps);
  OT* orow = out + (size_t)row * d;
#pragma unroll
  for (int i = 0; i < kPer; ++i) {
    const int c = lane + i * 32;
    if (c < nv) {
      const OT* g = gain + 4 * c;
      float o0 = v[i].x * r * to_f(g[0]), o1 = v[i].y * r * to_f(g[1]);
      float o2 = v[i].z * r * to_f(g[2]), o3 = v[i].w * r * to_f(g[3]);
      if constexpr (sizeof(OT) == 2) {
        __nv_bfloat162 a = __floats2bfloat162_rn(o0, o1), b = __floats2bfloat162_rn(o2, o3);
        uint2 pk = make_uint2(*reinterpret_cast<uint32_t*>(&a), *reinterpret_cast<uint32_t*>(&b));
        *reinterpret_cast<uint2*>(orow + 4 * c) = pk;
      } else {
        *reinterpret_cast<float4*>(orow + 4 * c) = make_float4(o0, o1, o2, o3);
      }
    }
  }
}


// ------------------------------------------------------------------------------------------------
// Encoder stack (post-norm blocks; Sec. 6.1 evaluates an encoder-only reranker next to the decoders).
// Input embedding: token row + learned position row (position p reads row p + pos_offset) + the token-type row,
// summed in fp32.  The LayerNorm that follows is the first norm of the first block.  One block per token row.
template <typename WT>
__global__ void __launch_bounds__(128) k_embed_encoder(const WT* __restrict__ table, const WT* __restrict__ pos_table,
                                                       const float* __restrict__ type_row, const int* __restrict__ tokens,
                                                       const int* __restrict__ tok2slot, const int* __restrict__ pos,
                                                       int pos_offset, int d, float* __restrict__ x) {
  const int t = blockIdx.x;
  const int tok = tokens[t];
  const WT* a = table + (size_t)(tok2slot ? tok2slot[tok] : tok) * d;  // with a row cache, `table` is the cache
  const WT* b = pos_table + (size_t)(pos[t] + pos_offset) * d;
  float* dst = x + (size_t)t * d;
  for (int c = threadIdx.x * 4; c < d; c += blockDim.x * 4) {
    const float4 ty = *reinterpret_cast<const float4*>(type_row + c);
    float4 o;
    if constexpr (sizeof(WT) == 2) {
      const uint2 ra = *reinterpret_cast<const uint2*>(a + c), rb = *reinterpret_cast<const uint2*>(b + c);
      const __nv_bfloat16* pa = reinterpret_cast<const __nv_bfloat16*>(&ra);
      const __nv_bfloat16* pb = reinterpret_cast<const __nv_bfloat16*>(&rb);
      o = make_float4(to_f(pa[0]) + to_f(pb[0]) + ty.x, to_f(pa[1]) + to_f(pb[1]) + ty.y,
                      to_f(pa[2]) + to_f(pb[2]) + ty.z, to_f(pa[3]) + to_f(pb[3]) + ty.w);
    } else {
      const float4 fa = *reinterpret_cast<const float4*>(a + c), fb = *reinterpret_cast<const float4*>(b + c);
      o = make_float4(fa.x + fb.x + ty.x, fa.y + fb.y + ty.y, fa.z + fb.z + ty.z, fa.w + fb.w + ty.w);
    }
    *reinterpret_cast<float4*>(dst + c) = o;
  }
}

// LayerNorm in place on the fp32 residual stream, plus a copy in the GEMM input type:
// y = (x - mean) / sqrt(var + eps) * g + b, biased variance, two passes over the row held in registers.
// kWarp: one warp per row (8 rows per block, lanes keep kPer float4), else one block of 256 threads per row.
template <typename OT, int kPer, bool kWarp>
__global__ void __launch_bounds__(256) k_layernorm(float* __restrict__ x, const float* __restrict__ gain,
                                                   const float* __restrict__ shift, int rows, int d, float eps,
                                                   OT* __restrict__ out, int reverse) {
  pdl_sync();
  __shared__ float red[32];
  const int lane = kWarp ? (threadIdx.x & 31) : threadIdx.x;
  constexpr int kStride = kWarp ? 32 : 256;
  const long long blk = reverse ? (long long)gridDim.x - 1 - blockIdx.x : blockIdx.x;
  const long long row = kWarp ? blk * 8 + (threadIdx.x >> 5) : blk;
  if (kWarp && row >= rows) return;
  float4* xr = reinterpret_cast<float4*>(x + (size_t)row * d);
  const int nv = d >> 2;
  float4 v[kPer];
  float sum = 0.f;
#pragma unroll
  for (int i = 0; i < kPer; ++i) {
    const int c = lane + i * kStride;
    if (c < nv) v[i] = xr[c];
  }
#pragma unroll
  for (int i = 0; i < kPer; ++i) {
    const int c = lane + i * kStride;
    if (c < nv) sum += (v[i].x + v[i].y) + (v[i].z + v[i].w);
  }
  sum = kWarp ? warp_sum(sum) : block_sum(sum, red);
  const float mean = sum / (float)d;
  float sq = 0.f;
#pragma unroll
  for (int i = 0; i < kPer; ++i) {
    const int c = lane + i * kStride;
    if (c < nv) {
      v[i].x -= mean; v[i].y -= mean; v[i].z -= mean; v[i].w -= mean;
      sq += v[i].x * v[i].x + v[i].y * v[i].y + v[i].z * v[i].z + v[i].w * v[i].w;
    }
  }
  sq = kWarp ? warp_sum(sq) : block_sum(sq, red);
  const float r = 1.0f / sqrtf(sq / (float)d + eps);
  OT* orow = out + (size_t)row * d;
#pragma unroll
  for (int i = 0; i < kPer; ++i) {
    const int c = lane + i * kStride;
    if (c < nv) {
      const float4 g = *reinterpret_cast<const float4*>(gain + 4 * c), b = *reinterpret_cast<const float4*>(shift + 4 * c);
      const float4 o = make_float4(v[i].x * r * g.x + b.x, v[i].y * r * g.y + b.y, v[i].z * r * g.z + b.z,
                                   v[i].w * r * g.w + b.w);
      xr[c] = o;
      if constexpr (sizeof(OT) == 2) {
        __nv_bfloat162 lo = __floats2bfloat162_rn(o.x, o.y), hi = __floats2bfloat162_rn(o.z, o.w);
        *reinterpret_cast<uint2*>(orow + 4 * c) = make_uint2(*reinterpret_cast<uint32_t*>(&lo), *reinterpret_cast<uint32_t*>(&hi));
      } else {
        *reinterpret_cast<float4*>(orow + 4 * c) = o;
      }
    }
  }
}

// Score probe of the encoder stack (Sec. 4.1: the model's own classifier on an intermediate hidden state): the
// FIRST row of sequence i goes through the pending LayerNorm of the block it leaves, then
// score = out_w . tanh(dense_w y + dense_b) + out_b.  Three small kernels over a scratch of 2 n d floats, every
// sum in a fixed order (the scores are the same bit for bit whatever the chunking or the launch geometry):
//   norm   one block per sequence: y[i,:] = LayerNorm(first row)
//   units  one WARP per output unit j of the dense map: its weight row stays in registers while the warp walks
//          the sequences, t[i,j] = out_w[j] * tanh(w_j . y[i,:] + dense_b[j])
//   sum    one block per sequence: score[i] = sum_j t[i,j] + out_b
__global__ void __launch_bounds__(256) k_probe_enc_norm(const float* __restrict__ x, const int* __restrict__ cu, int d,
                                                        const float* __restrict__ gain, const float* __restrict__ shift,
                                                        float eps, float* __restrict__ y) {
  __shared__ float red[32];
  const int i = blockIdx.x;
  float* yr = y + (size_t)i * d;
  if (cu[i + 1] == cu[i]) {  // a sequence without rows (another rank's candidate)
    for (int c = threadIdx.x; c < d; c += 256) yr[c] = 0.f;
    return;
  }
  const float* row = x + (size_t)cu[i] * d;
  float sum = 0.f;
  for (int c = threadIdx.x; c < d; c += 256) sum += row[c];
  const float mean = block_sum(sum, red) / (float)d;
  float sq = 0.f;
  for (int c = threadIdx.x; c < d; c += 256) {
    const float t = row[c] - mean;
    sq += t * t;
  }
  const float r = 1.0f / sqrtf(block_sum(sq, red) / (float)d + eps);
  for (int c = threadIdx.x; c < d; c += 256) yr[c] = (row[c] - mean) * r * gain[c] + shift[c];
}

// kPer > 0: d = 128 * kPer and the unit's weight row sits in registers (4 * kPer floats per lane);
// kPer = 0: any d that is a multiple of 4, the row is re-read (from L1) for every sequence.
template <typename WT, int kPer>
__global__ void __launch_bounds__(256) k_probe_enc_units(const float* __restrict__ y, int n, int d,
                                                         const WT* __restrict__ dense_w, const float* __restrict__ dense_b,
                                                         const float* __restrict__ out_w, float* __restrict__ t) {
  const int lane = threadIdx.x & 31;
  const int j = blockIdx.x * 8 + (threadIdx.x >> 5);
  if (j >= d) return;
  const WT* wr = dense_w + (size_t)j * d;
  const float bj = dense_b[j], oj = out_w[j];
  auto load4 = [&](int c) {  // weights c .. c + 3 of the row as floats
    if constexpr (sizeof(WT) == 2) {
      const uint2 raw = *reinterpret_cast<const uint2*>(wr + c);
      const __nv_bfloat16* b = reinterpret_cast<const __nv_bfloat16*>(&raw);
      return make_float4(to_f(b[0]), to_f(b[1]), to_f(b[2]), to_f(b[3]));
    } else {
      return *reinterpret_cast<const float4*>(wr + c);
    }
  };
  float4 w[kPer > 0 ? kPer : 1];
  if constexpr (kPer > 0) {
#pragma unroll
    for (int q = 0; q < kPer; ++q) w[q] = load4((lane + 32 * q) * 4);
  }
  for (int i = 0; i < n; ++i) {
    const float4* yr = reinterpret_cast<const float4*>(y + (size_t)i * d);
    float dot = 0.f;
    if constexpr (kPer > 0) {
#pragma unroll
      for (int q = 0; q < kPer; ++q) {
        const float4 v = yr[lane + 32 * q];
        dot = fmaf(w[q].x, v.x, fmaf(w[q].y, v.y, fmaf(w[q].z, v.z, fmaf(w[q].w, v.w, dot))));
      }
    } else {
      for (int c = lane; c < (d >> 2); c += 32) {
        const float4 v = yr[c], ww = load4(c * 4);
        dot = fmaf(ww.x, v.x, fmaf(ww.y, v.y, fmaf(ww.z, v.z, fmaf(ww.w, v.w, dot))));
      }
    }
    dot = warp_sum(dot);
    if (lane == 0) t[(size_t)i * d + j] = oj * tanhf(dot + bj);
  }
}

__global__ void __launch_bounds__(256) k_probe_enc_sum(const float* __restrict__ t, const int* __restrict__ cu, int d,
                                                       const float* __restrict__ out_b, float* __restrict__ scores) {
  __shared__ float red[32];
  const int i = blockIdx.x;
  if (cu[i + 1] == cu[i]) {
    if (threadIdx.x == 0) scores[i] = 0.f;
    return;
  }
  const float* tr = t + (size_t)i * d;
  float s = 0.f;
  for (int c = threadIdx.x; c < d; c += 256) s += tr[c];
  s = block_sum(s, red);
  if (threadIdx.x == 0) scores[i] = s + out_b[0];
}

// W4A16 (Sec. 6.1, the quantised arm): rebuild a packed [n, k] matrix as bf16.  One thread per 8 consecutive
// input channels of a row: 4 code bytes in, 16 bytes out; value = bf16(float(scale) * (code - zero)), the product
// being exact in fp32.  HBM-bound: 0.53 bytes read and 2 written per weight.
// Up to five matrices (one layer) per launch: blockIdx.y selects the matrix, the blocks of a matrix stride over its
// 32-weight pieces (16 code bytes in, 64 bytes out, one scale and zero point: groups are multiples of 32 channels
// and rows of 32 weights, so a piece never straddles a group); two independent pieces per thread in flight.
struct W4Batch {
  const unsigned char* blob[5];
  __nv_bfloat16* out[5];
  int n[5], k[5];
  int count, group;
};

__global__ void __launch_bounds__(256) k_dequant_w4(const W4Batch b) {
  const int mi = blockIdx.y;
  const int k = b.k[mi], group = b.group;
  const unsigned k32 = (unsigned)k >> 5, ng = (unsigned)(k / group), g32 = (unsigned)group >> 5;
  const size_t n = (size_t)b.n[mi];
  const unsigned n_pc = (unsigned)(n * k32);  // < 2^31 for every supported shape (checked by the launcher)
  const unsigned char* codes = b.blob[mi];
  const size_t off_s = (n * k / 2 + 15) / 16 * 16, off_z = (off_s + 2 * n * ng + 15) / 16 * 16;
  const __nv_bfloat16* scales = reinterpret_cast<const __nv_bfloat16*>(codes + off_s);
  const unsigned char* zeros = codes + off_z;
  const uint4* code_words = reinterpret_cast<const uint4*>(codes);  // piece p = 16-byte word p (rows are k/2 bytes)
  uint4* out = reinterpret_cast<uint4*>(b.out[mi]);                 // piece p = 16-byte words 4p .. 4p+3 of the output
  constexpr int kU = 2;
  const unsigned stride = gridDim.x * 256u;
  for (unsigned base = blockIdx.x * 256u + threadIdx.x; base < n_pc; base += stride * kU) {
    uint4 c[kU];
    float sc[kU];
    int z[kU];
#pragma unroll
    for (int u = 0; u < kU; ++u) {
      const unsigned p = base + u * stride;
      if (p < n_pc) {
        const unsigned row = p / k32, g = row * ng + (p - row * k32) / g32;
        c[u] = __ldg(code_words + p);
        sc[u] = __bfloat162float(scales[g]);
        z[u] = zeros[g];
      }
    }
#pragma unroll
    for (int u = 0; u < kU; ++u) {
      const unsigned p = base + u * stride;
      if (p < n_pc) {
        const uint32_t w[4] = {c[u].x, c[u].y, c[u].z, c[u].w};
#pragma unroll
        for (int q = 0; q < 4; ++q) {  // 4 code bytes = 8 weights = one 16-byte store
          uint32_t pk[4];
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const int lo = (int)((w[q] >> (8 * e)) & 15u) - z[u], hi = (int)((w[q] >> (8 * e + 4)) & 15u) - z[u];  // even k, odd k
            const __nv_bfloat162 v = __floats2bfloat162_rn(sc[u] * (float)lo, sc[u] * (float)hi);
            pk[e] = *reinterpret_cast<const uint32_t*>(&v);
          }
          out[(size_t)p * 4 + q] = make_uint4(pk[0], pk[1], pk[2], pk[3]);
        }
      }
    }
  }
}

template <typename WT>
__global__ void k_to_f32(const WT* __restrict__ src, int n, float* __restrict__ dst) {
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gridDim.x * blockDim.x) dst[i] = to_f(src[i]);
}

// ------------------------------------------------------------------------------------------------
// Rotary table in fp64, stored fp32: cos/sin(pos * theta^(-2j/dh)), j < dh/2.
__global__ void k_rope_table(float* __restrict__ cos_t, float* __restrict__ sin_t, int max_pos, int half,
                             double theta) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= max_pos * half) return;
  int p = i / half, j = i % half;
  double inv = pow(theta, -(double)j / (double)half);
  double a = (double)p * inv;
  cos_t[i] = (float)cos(a);
  sin_t[i] = (float)sin(a);
}

// The same angles for head_dim 128, laid out for the fused QKV epilogue: [pos][half][cos 32 | sin 32].
__global__ void k_rope_table_fused(float* __restrict__ tab, int max_pos, double theta) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= max_pos * 64) return;
  int p = i / 64, f = i % 64;  // f = frequency index 0..63
  double a = (double)p * pow(theta, -(double)f / 64.0);
  float* row = tab + (size_t)p * 128 + (f / 32) * 64;
  row[f % 32] = (float)cos(a);
  row[32 + f % 32] = (float)sin(a);
}

// S4 optional per-head RMSNorm over dh, then rotation of pairs (j, j + dh/2).  In place on the q and
// k heads of the packed qkv rows.  One warp per (row, head).
template <typename T>
__global__ void __launch_bounds__(256) k_qknorm_rope(T* __restrict__ qkv, const int* __restrict__ pos, int rows,
                                                     int hq, int hkv, int dh, int qk_norm,
                                                     const T* __restrict__ g_q, const T* __restrict__ g_k,
                                                     float eps, const float* __restrict__ cos_t,
                                                     const float* __restrict__ sin_t) {
  const int heads = hq + hkv;
  const long long wid = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  if (wid >= (long long)rows * heads) return;
  const int row = (int)(wid / heads), h = (int)(wid % heads);
  const int half = dh >> 1;
  T* u = qkv + (size_t)row * (size_t)((hq + 2 * hkv) * dh) + (size_t)h * dh;
  const T* g = (h < hq) ? g_q : g_k;
  float a[4], b[4];  // dh <= 256 -> at most 4 pairs per lane
  float ss = 0.f;
  int cnt = 0;
  for (int j = lane; j < half; j += 32, ++cnt) {
    a[cnt] = to_f(u[j]);
    b[cnt] = to_f(u[j + half]);
    ss += a[cnt] * a[cnt] + b[cnt] * b[cnt];
  }
  float r = 1.f;
  if (qk_norm) {
    ss = warp_sum(ss);
    r = 1.0f / sqrtf(ss / (float)dh + eps);
  }
  const float* ct = cos_t + (size_t)pos[row] * half;
  const float* st = sin_t + (size_t)pos[row] * half;
  cnt = 0;
  for (int j = lane; j < half; j += 32, ++cnt) {
    float x0 = a[cnt], x1 = b[cnt];
    if (qk_norm) {
      x0 = x0 * r * to_f(g[j]);
      x1 = x1 * r * to_f(g[j + half]);
    }
    const float c = ct[j], s = st[j];
    from_f(u[j], x0 * c - x1 * s);
    from_f(u[j + half], x1 * c + x0 * s);
  }
}

// ------------------------------------------------------------------------------------------------
// S10 score probe: final RMSNorm of each sequence's last row, dotted with (w_yes - w_no).
template <typename WT>
__global__ void __launch_bounds__(256) k_probe(const float* __restrict__ x, const int* __restrict__ cu, int d,
                                               const WT* __restrict__ g_final, const float* __restrict__ w_diff,
                                               float eps, int prefix, const unsigned char* __restrict__ owned,
                                               const int* __restrict__ seq2orig, float* __restrict__ scores) {
  pdl_sync();
  __shared__ float red[32];
  const int i = blockIdx.x;
  int last = cu[i + 1] - 1;
  if (cu[i + 1] == cu[i]) {
    // a sequence without rows: another rank's candidate (its score comes from there), or, with a shared query
    // prefix, this rank's candidate with an empty document, which ends with the query
    if (prefix == 0 || (owned && !owned[seq2orig[i]])) {
      if (threadIdx.x == 0) scores[i] = 0.f;
      return;
    }
    last = prefix - 1;
  }
  const float* row = x + (size_t)last * d;
  float ss = 0.f, dot = 0.f;
  for (int c = threadIdx.x * 4; c < d; c += blockDim.x * 4) {
    float4 v = *reinterpret_cast<const float4*>(row + c);
    float4 w = *reinterpret_cast<const float4*>(w_diff + c);
    ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
    dot += v.x * to_f(g_final[c]) * w.x + v.y * to_f(g_final[c + 1]) * w.y +
           v.z * to_f(g_final[c + 2]) * w.z + v.w * to_f(g_final[c + 3]) * w.w;
  }
  ss = block_sum(ss, red);
  dot = block_sum(dot, red);
  if (threadIdx.x == 0) scores[i] = dot / sqrtf(ss / (float)d + eps);
}

template <typename WT>
__global__ void k_score_diff(const WT* __restrict__ head, int d, float* __restrict__ w_diff) {
  int c = blockIdx.x * blockDim.x + threadIdx.x;
  if (c < d) w_diff[c] = to_f(head[c]) - to_f(head[d + c]);
}

// ------------------------------------------------------------------------------------------------
// S12 survivor gather: rows of the kept sequences move to their new packed position, order kept.
__global__ void __launch_bounds__(256) k_compact_rows(const float* __restrict__ x_old, float* __restrict__ x_new,
                                                      const int* __restrict__ cu_old,
                                                      const int* __restrict__ cu_new,
                                                      const int* __restrict__ old_of_new, int n_new,
                                                      int total_new, int d, int prefix) {
  pdl_sync();
  const int nv = d >> 2;
  for (int t = blockIdx.x; t < total_new; t += gridDim.x) {
    int src = t;  // rows of a shared query prefix stay where they are
    if (t >= prefix) {
      const int s = seq_of_row(cu_new, n_new, t);
      src = cu_old[old_of_new[s]] + (t - cu_new[s]);
    }
    const float4* a = reinterpret_cast<const float4*>(x_old + (size_t)src * d);
    float4* b = reinterpret_cast<float4*>(x_new + (size_t)t * d);
    for (int c = threadIdx.x; c < nv; c += 4 * 256) {
      float4 r0 = a[c], r1, r2, r3;
      const bool h1 = c + 256 < nv, h2 = c + 512 < nv, h3 = c + 768 < nv;
      if (h1) r1 = a[c + 256];
      if (h2) r2 = a[c + 512];
      if (h3) r3 = a[c + 768];
      b[c] = r0;
      if (h1) b[c + 256] = r1;
      if (h2) b[c + 512] = r2;
      if (h3) b[c + 768] = r3;
    }
  }
}

}  // namespace

namespace {
thread_local bool t_pdl_skip = false;
}

void pdl_skip_next() { t_pdl_skip = true; }

bool pdl_enabled() {
  static const bool on = std::getenv("PRISM_NO_PDL") == nullptr;
  if (t_pdl_skip) {
    t_pdl_skip = false;
    return false;
  }
  return on;
}

namespace {

// Launch with the programmatic-dependent-launch attribute (the kernel starts with pdl_sync()).
template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kernel)(KArgs...), unsigned grid, unsigned block, cudaStream_t st, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(block);
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl_enabled() ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

inline int grid_for(long long work, int block, int cap = 148 * 16) {
  long long g = (work + block - 1) / block;
  if (g < 1) g = 1;
  if (g > cap) g = cap;
  return (int)g;
}

}  // namespace

cudaError_t launch_pack_offsets(const int* cand_offsets, int n, int query_len, int* cu, int* seq2orig,
                                int* err, cudaStream_t st, const unsigned char* owned, bool shared_prefix) {
  k_pack_offsets<<<1, 1024, 0, st>>>(cand_offsets, n, query_len, owned, shared_prefix ? 1 : 0, cu, seq2orig, err);
  return cudaGetLastError();
}

cudaError_t launch_pack_tokens(const int* query, int query_len, const int* cand_tokens,
                               const int* cand_offsets, const int* cu, int n, int total, int vocab,
                               int* tokens, int* pos, int* err, cudaStream_t st, bool shared_prefix) {
  if (total <= 0) return cudaSuccess;
  k_pack_tokens<<<grid_for(total, 256), 256, 0, st>>>(query, query_len, cand_tokens, cand_offsets, cu, n,
                                                      total, vocab, shared_prefix ? 1 : 0, tokens, pos, err);
  return cudaGetLastError();
}

cudaError_t launch_positions(const int* cu, int n, int total, int* pos, cudaStream_t st, int prefix) {
  if (total <= 0) return cudaSuccess;
  return launch_pdl(k_positions, (unsigned)grid_for(total, 256), 256, st, cu, n, total, prefix, pos);
}

cudaError_t launch_embed(const void* table, int dtype, const int* tokens, int total, int d, float* x,
                         cudaStream_t st, const int* tok2slot) {
  if (total <= 0) return cudaSuccess;
  if (dtype == 1)
    k_embed<__nv_bfloat16><<<total, 128, 0, st>>>((const __nv_bfloat16*)table, tokens, tok2slot, d, x);
  else
    k_embed<float><<<total, 128, 0, st>>>((const float*)table, tokens, tok2slot, d, x);
  return cudaGetLastError();
}

// Embedding-row cache fill: row pairs[2i] of the host table (pinned, read over the host link) goes to cache row
// pairs[2i+1], and the token's entry in tok2slot follows.  One block per row, 16-byte pieces.
__global__ void __launch_bounds__(128) k_cache_fill(const unsigned char* __restrict__ host_table,
                                                    unsigned char* __restrict__ cache, const int* __restrict__ pairs,
                                                    int row_bytes, int* __restrict__ tok2slot) {
  const int tok = pairs[2 * blockIdx.x], slot = pairs[2 * blockIdx.x + 1];
  const uint4* src = reinterpret_cast<const uint4*>(host_table + (size_t)tok * row_bytes);
  uint4* dst = reinterpret_cast<uint4*>(cache + (size_t)slot * row_bytes);
  for (int c = threadIdx.x; c < row_bytes / 16; c += blockDim.x) dst[c] = src[c];
  if (threadIdx.x == 0) tok2slot[tok] = slot;
}

cudaError_t launch_cache_fill(const void* host_table, void* cache, const int* pairs, int n_rows, int row_bytes,
                              int* tok2slot, cudaStream_t st) {
  if (n_rows <= 0) return cudaSuccess;
  if (row_bytes % 16) return cudaErrorInvalidValue;
  k_cache_fill<<<n_rows, 128, 0, st>>>((const unsigned char*)host_table, (unsigned char*)cache, pairs, row_bytes, tok2slot);
  return cudaGetLastError();
}

// reverse: blocks take the rows from the end of the matrix backwards.  The driver alternates the direction
// from one kernel of a layer to the next, so that a kernel starts on the rows its predecessor wrote last,
// which are the ones still in L2 when the tensors are larger than L2.
cudaError_t launch_rmsnorm(const float* x, const void* gain, int dtype, int rows, int d, float eps,
                           void* out, cudaStream_t st, bool reverse) {
  if (rows <= 0) return cudaSuccess;
  const int nv = d >> 2;
  if (nv > 8 * 256) return cudaErrorInvalidValue;
  if (nv <= 16 * 32) {  // rows of up to 8 KB: one warp per row
    const unsigned grid = (unsigned)((rows + 7) / 8);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(256);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl_for(rows) ? 1 : 0;
    const int rev = reverse ? 1 : 0;
#define PRISM_NORMW(OT, V)                                                                                                \
  do {                                                                                                                    \
    cudaError_t le = cudaLaunchKernelEx(&cfg, k_rmsnorm_warp<OT, V>, x, (const OT*)gain, rows, d, eps, (OT*)out, rev);      \
    if (le != cudaSuccess) return le;                                                                                     \
  } while (0)
    if (dtype == 1) {
      if (nv <= 128) PRISM_NORMW(__nv_bfloat16, 4);
      else if (nv <= 256) PRISM_NORMW(__nv_bfloat16, 8);
      else PRISM_NORMW(__nv_bfloat16, 16);
    } else {
      if (nv <= 128) PRISM_NORMW(float, 4);
      else if (nv <= 256) PRISM_NORMW(float, 8);
      else PRISM_NORMW(float, 16);
    }
#undef PRISM_NORMW
    return cudaGetLastError();
  }
#define PRISM_NORM(OT, V) \
  k_rmsnorm<OT, V><<<rows, 256, 0, st>>>(x, (const OT*)gain, d, eps, (OT*)out, reverse ? 1 : 0)
  if (dtype == 1) {
    if (nv <= 256) PRISM_NORM(__nv_bfloat16, 1);
    else if (nv <= 512) PRISM_NORM(__nv_bfloat16, 2);
    else if (nv <= 1024) PRISM_NORM(__nv_bfloat16, 4);
    else PRISM_NORM(__nv_bfloat16, 8);
  } else {
    if (nv <= 256) PRISM_NORM(float, 1);
    else if (nv <= 512) PRISM_NORM(float, 2);
    else if (nv <= 1024) PRISM_NORM(float, 4);
    else PRISM_NORM(float, 8);
  }
#undef PRISM_NORM
  return cudaGetLastError();
}


cudaError_t launch_embed_encoder(const void* table, const void* pos_table, const float* type_row, int dtype,
                                 const int* tokens, const int* pos, int pos_offset, int total, int d, float* x,
                                 cudaStream_t st, const int* tok2slot) {
  if (total <= 0) return cudaSuccess;
  if (d % 4) return cudaErrorInvalidValue;
  if (dtype == 1)
    k_embed_encoder<__nv_bfloat16><<<total, 128, 0, st>>>((const __nv_bfloat16*)table, (const __nv_bfloat16*)pos_table,
                                                          type_row, tokens, tok2slot, pos, pos_offset, d, x);
  else
    k_embed_encoder<float><<<total, 128, 0, st>>>((const float*)table, (const float*)pos_table, type_row, tokens, tok2slot,
                                                  pos, pos_offset, d, x);
  return cudaGetLastError();
}

cudaError_t launch_layernorm(float* x, const float* gain, const float* shift, int dtype, int rows, int d, float eps,
                             void* out, cudaStream_t st, bool reverse) {
  if (rows <= 0) return cudaSuccess;
  const int nv = d >> 2;
  if ((d & 3) || nv > 8 * 256) return cudaErrorInvalidValue;
  const int rev = reverse ? 1 : 0;
  cudaLaunchConfig_t cfg = {};
  cfg.blockDim = dim3(256);
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl_for(rows) ? 1 : 0;
#define PRISM_LN(OT, P, W, G)                                                                                        \
  do {                                                                                                               \
    cfg.gridDim = dim3((unsigned)(G));                                                                                \
    cudaError_t le = cudaLaunchKernelEx(&cfg, k_layernorm<OT, P, W>, x, gain, shift, rows, d, eps, (OT*)out, rev);     \
    if (le != cudaSuccess) return le;                                                                                \
  } while (0)
  if (nv <= 16 * 32) {  // rows of up to 8 KB: one warp per row
    const unsigned grid = (unsigned)((rows + 7) / 8);
    if (dtype == 1) {
      if (nv <= 128) PRISM_LN(__nv_bfloat16, 4, true, grid);
      else if (nv <= 256) PRISM_LN(__nv_bfloat16, 8, true, grid);
      else PRISM_LN(__nv_bfloat16, 16, true, grid);
    } else {
      if (nv <= 128) PRISM_LN(float, 4, true, grid);
      else if (nv <= 256) PRISM_LN(float, 8, true, grid);
      else PRISM_LN(float, 16, true, grid);
    }
  } else {
    if (dtype == 1) {
      if (nv <= 1024) PRISM_LN(__nv_bfloat16, 4, false, rows);
      else PRISM_LN(__nv_bfloat16, 8, false, rows);
    } else {
      if (nv <= 1024) PRISM_LN(float, 4, false, rows);
      else PRISM_LN(float, 8, false, rows);
    }
  }
#undef PRISM_LN
  return cudaGetLastError();
}

cudaError_t launch_probe_encoder(const float* x, const int* cu, int n, int d, const float* gain, const float* shift,
                                 float eps, const void* dense_w, int dtype, const float* dense_b, const float* out_w,
                                 const float* out_b, float* scores, float* scratch, cudaStream_t st) {
  if (n <= 0) return cudaSuccess;
  if (d & 3) return cudaErrorInvalidValue;
  float *y = scratch, *t = scratch + (size_t)n * d;
  k_probe_enc_norm<<<n, 256, 0, st>>>(x, cu, d, gain, shift, eps, y);
  const int grid = (d + 7) / 8;
#define PRISM_UNITS(WT, P) k_probe_enc_units<WT, P><<<grid, 256, 0, st>>>(y, n, d, (const WT*)dense_w, dense_b, out_w, t)
  if (dtype == 1) {
    if (d == 1024) PRISM_UNITS(__nv_bfloat16, 8);
    else if (d == 768) PRISM_UNITS(__nv_bfloat16, 6);
    else if (d == 2048) PRISM_UNITS(__nv_bfloat16, 16);
    else PRISM_UNITS(__nv_bfloat16, 0);
  } else {
    if (d == 1024) PRISM_UNITS(float, 8);
    else PRISM_UNITS(float, 0);
  }
#undef PRISM_UNITS
  k_probe_enc_sum<<<n, 256, 0, st>>>(t, cu, d, out_b, scores);
  return cudaGetLastError();
}

cudaError_t launch_dequant_w4_batch(const void* const* blobs, const int* n, const int* k, void* const* outs, int count,
                                    int group, cudaStream_t st) {
  if (count < 1 || count > 5 || group <= 0 || (group & 31)) return cudaErrorInvalidValue;
  W4Batch b{};
  b.count = count;
  b.group = group;
  long long most = 0;
  for (int i = 0; i < count; ++i) {
    const long long oct = (long long)n[i] * (k[i] >> 5);
    if (n[i] <= 0 || k[i] <= 0 || (k[i] % group) || oct >= (1ll << 31)) return cudaErrorInvalidValue;
    b.blob[i] = static_cast<const unsigned char*>(blobs[i]);
    b.out[i] = static_cast<__nv_bfloat16*>(outs[i]);
    b.n[i] = n[i];
    b.k[i] = k[i];
    most = oct > most ? oct : most;
  }
  // blocks per matrix: enough for the largest one at two pieces per thread, at most 8 per SM and matrix
  const int gx = grid_for((most + 1) / 2, 256, 148 * 8);
  k_dequant_w4<<<dim3(gx, count), 256, 0, st>>>(b);
  return cudaGetLastError();
}

cudaError_t launch_dequant_w4(const void* blob, int n, int k, int group, void* out, cudaStream_t st) {
  if (n <= 0 || k <= 0) return cudaSuccess;
  return launch_dequant_w4_batch(&blob, &n, &k, &out, 1, group, st);
}

cudaError_t launch_to_f32(const void* src, int dtype, int n, float* dst, cudaStream_t st) {
  if (n <= 0) return cudaSuccess;
  const int grid = grid_for(n, 256);
  if (dtype == 1) k_to_f32<__nv_bfloat16><<<grid, 256, 0, st>>>((const __nv_bfloat16*)src, n, dst);
  else k_to_f32<float><<<grid, 256, 0, st>>>((const float*)src, n, dst);
  return cudaGetLastError();
}

cudaError_t launch_rope_table(float* cos_t, float* sin_t, int max_pos, int head_dim, float theta,
                              cudaStream_t st) {
  const int half = head_dim / 2;
  const long long n = (long long)max_pos * half;
  if (n <= 0) return cudaSuccess;
  k_rope_table<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(cos_t, sin_t, max_pos, half, (double)theta);
  return cudaGetLastError();
}

cudaError_t launch_rope_table_fused(float* tab, int max_pos, float theta, cudaStream_t st) {
  const long long n = (long long)max_pos * 64;
  if (n <= 0) return cudaSuccess;
  k_rope_table_fused<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(tab, max_pos, (double)theta);
  return cudaGetLastError();
}

cudaError_t launch_qknorm_rope(void* qkv, int dtype, const int* pos, int rows, int n_q_heads,
                               int n_kv_heads, int head_dim, int qk_norm, const void* g_q,
                               const void* g_k, float eps, const float* cos_t, const float* sin_t,
                               cudaStream_t st) {
  if (rows <= 0) return cudaSuccess;
  const long long warps = (long long)rows * (n_q_heads + n_kv_heads);
  const unsigned grid = (unsigned)((warps + 7) / 8);
  if (dtype == 1)
    k_qknorm_rope<__nv_bfloat16><<<grid, 256, 0, st>>>((__nv_bfloat16*)qkv, pos, rows, n_q_heads, n_kv_heads,
                                                       head_dim, qk_norm, (const __nv_bfloat16*)g_q,
                                                       (const __nv_bfloat16*)g_k, eps, cos_t, sin_t);
  else
    k_qknorm_rope<float><<<grid, 256, 0, st>>>((float*)qkv, pos, rows, n_q_heads, n_kv_heads, head_dim,
                                               qk_norm, (const float*)g_q, (const float*)g_k, eps, cos_t,
                                               sin_t);
  return cudaGetLastError();
}

cudaError_t launch_probe(const float* x, const int* cu, int n, int d, const void* g_final, int dtype,
                         const float* w_diff, float eps, float* scores, cudaStream_t st, int prefix,
                         const unsigned char* owned, const int* seq2orig) {
  if (n <= 0) return cudaSuccess;
  if (owned && !seq2orig) return cudaErrorInvalidValue;
  if (dtype == 1)
    return launch_pdl(k_probe<__nv_bfloat16>, (unsigned)n, 256, st, x, cu, d, (const __nv_bfloat16*)g_final, w_diff, eps, prefix,
                      owned, seq2orig, scores);
  return launch_pdl(k_probe<float>, (unsigned)n, 256, st, x, cu, d, (const float*)g_final, w_diff, eps, prefix, owned, seq2orig,
                    scores);
}

cudaError_t launch_score_diff(const void* score_head, int dtype, int d, float* w_diff, cudaStream_t st) {
  if (dtype == 1)
    k_score_diff<__nv_bfloat16><<<(d + 255) / 256, 256, 0, st>>>((const __nv_bfloat16*)score_head, d, w_diff);
  else
    k_score_diff<float><<<(d + 255) / 256, 256, 0, st>>>((const float*)score_head, d, w_diff);
  return cudaGetLastError();
}

cudaError_t launch_compact_rows(const float* x_old, float* x_new, const int* cu_old, const int* cu_new,
                                const int* old_of_new, int n_new, int total_new, int d, cudaStream_t st, int prefix) {
  if (total_new <= 0) return cudaSuccess;
  int grid = total_new < 148 * 8 ? total_new : 148 * 8;
  return launch_pdl(k_compact_rows, (unsigned)grid, 256, st, x_old, x_new, cu_old, cu_new, old_of_new, n_new, total_new, d, prefix);
}

}  // namespace prism
