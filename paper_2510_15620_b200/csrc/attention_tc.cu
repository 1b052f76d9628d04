// S5 on the 5th-generation tensor cores: varlen flash attention over packed sequences, bf16,
// head_dim 128 (the decoder rerankers) or 64 (the encoder stack), GQA, causal or bidirectional.  One query head per CTA: this kernel serves odd group sizes
// Hq/Hkv and PRISM_IMPL_SOLO; even group sizes take the two-heads-per-CTA kernel of attention_tc2.cu.
//
// One CTA = 128 query rows of one (sequence, head); two CTAs fit on an SM.  Warp-specialised:
//   warp 0      TMA producer: Q once, then K_j tiles (64 keys) into a 3-deep ring and V_j tiles into a
//               2-deep ring; a K slot is released as soon as its Q K^T has run, a V slot after P V
//   warp 1      score issuer: S_j = Q K_j^T (tcgen05.mma M128 N64 K16 x 8) into one of two TMEM buffers
//   warp 10     output issuer: O += P_j V_j (M128 N128 K16 x 4; P read from TENSOR MEMORY, V as an
//               MN-major shared-memory operand) into TMEM.  Two issuing threads, so that the next
//               scores never queue behind the wait for the current probabilities.
//   warps 2..9  softmax: two threads per query row (warps w and w+4 share a 32-row TMEM lane quarter and
//               take 32 of the 64 key columns each); read S_j from TMEM, exchange the row maximum,
//               exponentiate against a running reference maximum and store P_j as packed bf16 back
//               into the first 32 columns of the S_j buffer (tcgen05.st); O stays in TMEM and is
//               rescaled (TMEM read-modify-write) only when a row's maximum outgrows the reference by
//               more than 2^8.
// S_{j+1} and S_{j+2}... are issued as soon as their K tile has landed and their TMEM buffer is free (the
// output issuer releases buffer j&1 with a commit after P_j V_j), so the tensor core computes the next
// scores while the softmax warps work.  Every mbarrier wait is bounded; on expiry the kernel records kErrTimeout, all
// roles drain to the common exit and the tensor memory is freed.  Every TMA load is a plain per-CTA load.
#include "tc_common.cuh"

namespace prism {

namespace {

using namespace tc;

constexpr int BM = 128, BN = 64;
constexpr int NK = 3, NV = 2;                 // ring depths
constexpr int kXchBytes = 2 * 128 * 2;        // per-row exchange of the block maximum (bf16) between the two threads of a row
// Tiles for head_dim DH (sizes for DH = 128; half of it for 64): Q 32 KB as DH/64 [128 x 64] swizzled sub-tiles,
// K and V 16 KB each as DH/64 [64 x 64] sub-tiles; 112 KB in all.
// No alignment slack: two CTAs per SM only fit if nothing is wasted.  The kernel checks that its
// shared window starts on a 1024-byte boundary (the swizzled tiles need it) and reports if not.
__host__ __device__ constexpr int tile_bytes_of(int dh) { return BM * dh * 2 + NK * BN * dh * 2 + NV * BN * dh * 2; }
__host__ __device__ constexpr int smem_bytes_of(int dh) { return tile_bytes_of(dh) + 256 + kXchBytes; }
static_assert(2 * (smem_bytes_of(128) + 1024) <= 233472, "two CTAs per SM must fit in 228 KB of shared memory");
constexpr int kThreads = 352;                 // TMA warp, score-MMA warp, 8 softmax warps, output-MMA warp
constexpr int kTmemCols = 256;                // S: 2 x 64, O: up to 128

__device__ __forceinline__ float ex2(float x) {  // 2^x on the special-function unit; -inf -> 0
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
template <int DH>
__global__ void __launch_bounds__(kThreads, 2)
k_attention_tc(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_kv,
               __nv_bfloat16* __restrict__ out, const int* __restrict__ cu, int seq0, int row0, int hq, int hkv,
               int causal, float scale_log2, int* __restrict__ err) {
  constexpr int NS = DH / 64;  // 64-column sub-tiles per head
  constexpr int kQBytes = BM * DH * 2, kKBytes = BN * DH * 2, kVBytes = BN * DH * 2;
  constexpr int kTileBytes = tile_bytes_of(DH);
  extern __shared__ unsigned char smem_raw[];
  pdl_sync();  // the offsets below are another kernel's output
  const int s = seq0 + blockIdx.z;
  const int beg = cu[s] - row0, len = cu[s + 1] - cu[s];
  const int qb = (int)gridDim.x - 1 - (int)blockIdx.x;  // heaviest query blocks first
  if (qb * BM >= len) return;
  const int h = blockIdx.y, kvh = h / (hq / hkv);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  const uint32_t base = smem_u32(smem_raw);
  unsigned char* gen = smem_raw;
  const uint32_t s_q = base, s_k = base + kQBytes, s_v = s_k + NK * kKBytes;
  uint64_t* bars = reinterpret_cast<uint64_t*>(gen + kTileBytes);
  // q, k_full[3], k_empty[3], v_full[2], v_empty[2], s_full[2], s_empty[2], p_full, o_full
  const uint32_t b_q = smem_u32(bars), b_k_full = smem_u32(bars + 1), b_k_empty = smem_u32(bars + 4);
  const uint32_t b_v_full = smem_u32(bars + 7), b_v_empty = smem_u32(bars + 9);
  const uint32_t b_s_full = smem_u32(bars + 11), b_s_empty = smem_u32(bars + 13);
  const uint32_t b_p_full = smem_u32(bars + 15), b_o_full = smem_u32(bars + 16);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 17);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  __nv_bfloat16* xch = reinterpret_cast<__nv_bfloat16*>(gen + kTileBytes + 256);  // [2][128]
  float* xch_l = reinterpret_cast<float*>(gen);  // [2][128] over the Q tile, used once all MMAs are done
  if (base & 1023u) {  // cannot run correctly: say so instead of computing garbage
    if (threadIdx.x == 0) atomicOr(err, kErrInternal);
    return;
  }

  const int kv_end = causal ? min(len, (qb + 1) * BM) : len;
  const int n_blocks = (kv_end + BN - 1) / BN;

  if (threadIdx.x == 0) {
    mbar_init(b_q, 1);
    for (int i = 0; i < NK; ++i) {
      mbar_init(b_k_full + 8 * i, 1);
      mbar_init(b_k_empty + 8 * i, 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(b_v_full + 8 * i, 1);
      mbar_init(b_v_empty + 8 * i, 1);
      mbar_init(b_s_full + 8 * i, 1);
      mbar_init(b_s_empty + 8 * i, 1);  // released by a commit of the output issuer
    }
    mbar_init(b_p_full, 8);
    mbar_init(b_o_full, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(kTmemCols));
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::);
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  const uint32_t t_s = tmem, t_o = tmem + 2 * BN;  // columns [0,128): S buffers (P_j aliases the first 32 of S_j), [128,256): O

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      mbar_expect_tx(b_q, kQBytes);
#pragma unroll
      for (int x = 0; x < NS; ++x) tma_load_2d(s_q + x * (kQBytes / NS), &map_q, h * DH + 64 * x, beg + qb * BM, b_q);
      const int kcol = (hq + kvh) * DH, vcol = (hq + hkv + kvh) * DH;
      // K runs one block ahead of V: step t issues K_t, then V_{t-1}.
      for (int t = 0; t <= n_blocks; ++t) {
        if (t < n_blocks) {
          const int st = t % NK, u = t / NK;
          if (!mbar_wait(b_k_empty + 8 * st, (u & 1) ^ 1, err, abort_flag)) break;
          const uint32_t sk = s_k + st * kKBytes;
          mbar_expect_tx(b_k_full + 8 * st, kKBytes);
#pragma unroll
          for (int x = 0; x < NS; ++x)
            tma_load_2d(sk + x * (kKBytes / NS), &map_kv, kcol + 64 * x, beg + t * BN, b_k_full + 8 * st);
        }
        if (t >= 1) {
          const int j = t - 1, st = j & 1, u = j >> 1;
          if (!mbar_wait(b_v_empty + 8 * st, (u & 1) ^ 1, err, abort_flag)) break;
          const uint32_t sv = s_v + st * kVBytes;
          mbar_expect_tx(b_v_full + 8 * st, kVBytes);
#pragma unroll
          for (int x = 0; x < NS; ++x)
            tma_load_2d(sv + x * (kVBytes / NS), &map_kv, vcol + 64 * x, beg + j * BN, b_v_full + 8 * st);
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ score issuer: S_j = Q K_j^T
    if (lane == 0) {
      constexpr uint32_t kIdescS = idesc_bf16(BM, BN, 0);
      bool ok = mbar_wait(b_q, 0, err, abort_flag);
      for (int j = 0; j < n_blocks && ok; ++j) {
        const int st = j % NK, b = j & 1, u = j >> 1;
        if (!mbar_wait(b_k_full + 8 * st, (j / NK) & 1, err, abort_flag)) break;
        // buffer b held S_{j-2} and then P_{j-2}; it is free once P_{j-2} V_{j-2} has completed
        if (!mbar_wait(b_s_empty + 8 * b, (u & 1) ^ 1, err, abort_flag)) break;
        const uint32_t sk = s_k + st * kKBytes;
        tc_fence_after();
#pragma unroll
        for (int kk = 0; kk < DH / 16; ++kk) {  // 16 head-dim elements per step; sub-tile switches at kk = 4
          const uint64_t da = smem_desc(s_q + (kk >> 2) * (kQBytes / NS) + (kk & 3) * 32, 16, 1024);
          const uint64_t db = smem_desc(sk + (kk >> 2) * (kKBytes / NS) + (kk & 3) * 32, 16, 1024);
          umma_bf16(t_s + b * BN, da, db, kIdescS, kk != 0);
        }
        umma_commit(b_s_full + 8 * b);
        umma_commit(b_k_empty + 8 * st);  // the K tile is free as soon as these MMAs have read it
      }
    }
  } else if (warp == 10) {
    // ------------------------------------------------------------------ output issuer: O += P_j V_j
    if (lane == 0) {
      constexpr uint32_t kIdescO = idesc_bf16(BM, DH, 1);
      for (int j = 0; j < n_blocks; ++j) {
        if (!mbar_wait(b_p_full, j & 1, err, abort_flag)) break;
        if (!mbar_wait(b_v_full + 8 * (j & 1), (j >> 1) & 1, err, abort_flag)) break;
        tc_fence_after();
        const uint32_t sv = s_v + (j & 1) * kVBytes;
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) {  // 16 keys per step: 8 packed columns of P, 16 rows of V
          const uint64_t db = smem_desc(sv + kk * 2048, kVBytes / NS, 1024);   // V: MN-major, DH/64 atoms of 64 dh
          umma_bf16_ts(t_o, t_s + (j & 1) * BN + kk * 8, db, kIdescO, (j | kk) != 0);
        }
        umma_commit(b_o_full);
        umma_commit(b_v_empty + 8 * (j & 1));
        umma_commit(b_s_empty + 8 * (j & 1));  // S/P buffer j&1 may be overwritten by Q K_{j+2}^T
      }
    }
  } else {
    // ------------------------------------------------------------------ softmax + output (128 rows x 2 column halves)
    const int quarter = warp & 3;
    const int colhalf = (warp - 2) >> 2;           // which 32 of a block's 64 keys / which half of the DH output columns
    const int r = quarter * 32 + lane;             // row inside the tile = TMEM lane
    const int qrow = qb * BM + r;                  // row inside the sequence
    const uint32_t lane_base = (uint32_t)(quarter * 32) << 16;
    const int pair_bar = 1 + quarter;              // named barrier of the two warps that share these rows
    float m_ref = 0.f, l = 0.f;                    // reference maximum (raw score units), this thread's partial sum
    bool ok = true;
    for (int j = 0; j < n_blocks; ++j) {
      const int b = j & 1, u = j >> 1;
      if (!mbar_wait(b_s_full + 8 * b, u & 1, err, abort_flag)) { ok = false; break; }
      tc_fence_after();
      uint32_t sr[32];
      tmem_ld32(t_s + lane_base + b * BN + colhalf * 32, sr);
      tmem_ld_wait();
      const int key0 = j * BN + colhalf * 32;
      if ((causal && j * BN + BN - 1 > qb * BM) || j * BN + BN > len) {
#pragma unroll
        for (int c = 0; c < 32; ++c) {
          const int key = key0 + c;
          if (key >= len || (causal && key > qrow)) sr[c] = 0xff800000u;  // -inf
        }
      }
      float bm = -INFINITY;
#pragma unroll
      for (int c = 0; c < 32; ++c) bm = fmaxf(bm, __uint_as_float(sr[c]));
      // Row maximum over both halves.  The value only serves as a reference for the exponentials, so it
      // is exchanged rounded up to bf16; both threads of a row use the same two rounded numbers.
      const __nv_bfloat16 bmr = __float2bfloat16_ru(bm);
      xch[colhalf * 128 + r] = bmr;
      asm volatile("bar.sync %0, 64;" ::"r"(pair_bar) : "memory");
      bm = fmaxf(__bfloat162float(bmr), __bfloat162float(xch[(colhalf ^ 1) * 128 + r]));
      asm volatile("bar.sync %0, 64;" ::"r"(pair_bar) : "memory");  // both have read before the next block writes
      bool saw_pv = false;  // has this thread already observed the completion of P_{j-1} V_{j-1}?
      if (j == 0) {
        m_ref = (bm == -INFINITY) ? 0.f : bm;
      } else {
        // Rescale O only when this row's maximum outgrew the reference by more than 2^8 (rare).  Both
        // threads of a row see the same bm and m_ref, so both warps of the pair take the same branch.
        const bool need = (bm - m_ref) * scale_log2 > 8.f;
        if (__any_sync(0xffffffffu, need)) {
          if (!mbar_wait(b_o_full, (j - 1) & 1, err, abort_flag)) { ok = false; break; }
          saw_pv = true;
          tc_fence_after();
          const float m_new = need ? bm : m_ref;
          const float f = exp2f((m_ref - m_new) * scale_log2);
#pragma unroll 1
          for (int c = 0; c < NS; ++c) {
            uint32_t o[32];
            tmem_ld32(t_o + lane_base + colhalf * (DH / 2) + c * 32, o);
            tmem_ld_wait();
#pragma unroll
            for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * f);
            tmem_st32(t_o + lane_base + colhalf * (DH / 2) + c * 32, o);
          }
          tmem_st_wait();
          l *= f;
          m_ref = m_new;
        }
      }
      const float ms = m_ref * scale_log2;
      uint32_t pk[16];
      const uint64_t sc2 = f2_pack(scale_log2, scale_log2), nm2 = f2_pack(-ms, -ms);
      uint64_t rs2 = f2_pack(0.f, 0.f);
#pragma unroll
      for (int c = 0; c < 16; ++c) {
        float x0, x1;
        f2_unpack(f2_fma(f2_pack(__uint_as_float(sr[2 * c]), __uint_as_float(sr[2 * c + 1])), sc2, nm2), x0, x1);
        const float p0 = ex2(x0), p1 = ex2(x1);
        rs2 = f2_add(rs2, f2_pack(p0, p1));
        pk[c] = pack_bf16(p0, p1);  // key 2c in the low half, key 2c+1 in the high half
      }
      float rs, rs_hi;
      f2_unpack(rs2, rs, rs_hi);
      rs += rs_hi;
      l += rs;
      // P_j (packed bf16) goes over the first 32 columns of the S_j buffer: both threads of the row have
      // loaded their S values (they met at the pair barrier above), and Q K_{j+2}^T is only issued once
      // P_j V_j has completed (s_empty), so nothing else touches these columns meanwhile.
      tmem_st16(t_s + lane_base + b * BN + colhalf * 16, pk);
      tmem_st_wait();
      tc_fence_before();
      // mbarrier parity only tells the current phase from the previous one, so every thread observes
      // every phase, in order, while the next one cannot complete yet: P_j V_j needs this thread's
      // arrival below, hence the o_full barrier is at phase j-1 or j here and the wait is unambiguous
      // (P_{j-1} V_{j-1} was issued a whole block ago, so it has normally finished).  Likewise p_full:
      // a warp that runs ahead must not have its arrival for block j counted in block j-1's phase.
      if (j > 0 && !saw_pv && !mbar_wait(b_o_full, (j - 1) & 1, err, abort_flag)) { ok = false; break; }
      if (j > 0 && !mbar_wait(b_p_full, (j - 1) & 1, err, abort_flag)) { ok = false; break; }
      __syncwarp();
      if (lane == 0) mbar_arrive(b_p_full);  // one arrival per warp
    }
    if (ok && mbar_wait(b_o_full, (n_blocks - 1) & 1, err, abort_flag)) {
      tc_fence_after();
      xch_l[colhalf * 128 + r] = l;  // the row's sum is the sum of the two partial sums
      asm volatile("bar.sync %0, 64;" ::"r"(pair_bar) : "memory");
      const float inv = 1.f / (l + xch_l[(colhalf ^ 1) * 128 + r]);
      __nv_bfloat16* orow = out + (size_t)(beg + qrow) * ((size_t)hq * DH) + (size_t)h * DH + colhalf * (DH / 2);
#pragma unroll 1
      for (int c = 0; c < NS; ++c) {
        uint32_t o[32];
        tmem_ld32(t_o + lane_base + colhalf * (DH / 2) + c * 32, o);
        tmem_ld_wait();
        if (qrow < len) {
#pragma unroll
          for (int v = 0; v < 4; ++v) {
            uint4 pk;
            pk.x = pack_bf16(__uint_as_float(o[v * 8 + 0]) * inv, __uint_as_float(o[v * 8 + 1]) * inv);
            pk.y = pack_bf16(__uint_as_float(o[v * 8 + 2]) * inv, __uint_as_float(o[v * 8 + 3]) * inv);
            pk.z = pack_bf16(__uint_as_float(o[v * 8 + 4]) * inv, __uint_as_float(o[v * 8 + 5]) * inv);
            pk.w = pack_bf16(__uint_as_float(o[v * 8 + 6]) * inv, __uint_as_float(o[v * 8 + 7]) * inv);
            *reinterpret_cast<uint4*>(orow + c * 32 + v * 8) = pk;
          }
        }
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols));
  }
}

}  // namespace

cudaError_t launch_attention_tc(const void* qkv, void* out, const int* cu, int seq0, int nseq, int row0, int rows,
                                int max_len, int n_q_heads, int n_kv_heads, int causal, int* err, cudaStream_t st,
                                int head_dim) {
  if (nseq <= 0 || max_len <= 0 || rows <= 0) return cudaSuccess;
  if (head_dim != 128 && head_dim != 64) return cudaErrorInvalidValue;
  const int DH = head_dim;
  static std::atomic<unsigned long long> smem_set[2];
  if (cudaError_t e = DH == 128 ? ensure_dynamic_smem(k_attention_tc<128>, smem_bytes_of(128), smem_set[0])
                                : ensure_dynamic_smem(k_attention_tc<64>, smem_bytes_of(64), smem_set[1]))
    return e;
  // Exactly `rows` rows are described, so tiles that run past the batch read zeros, never stale memory.
  const uint64_t ld = (uint64_t)(n_q_heads + 2 * n_kv_heads) * DH;
  TmaDesc mq, mkv;
  cudaError_t e = make_tma_2d_bf16(&mq, qkv, (uint64_t)rows, ld, BM, 64);
  if (e == cudaSuccess) e = make_tma_2d_bf16(&mkv, qkv, (uint64_t)rows, ld, BN, 64);
  if (e != cudaSuccess) return e;
  dim3 grid((max_len + BM - 1) / BM, n_q_heads, nseq);
  const float scale_log2 = 1.4426950408889634f / sqrtf((float)DH);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = smem_bytes_of(DH);
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl_for(rows) ? 1 : 0;
  const CUtensorMap& m0 = reinterpret_cast<const CUtensorMap&>(mq);
  const CUtensorMap& m1 = reinterpret_cast<const CUtensorMap&>(mkv);
  cudaError_t le = DH == 128 ? cudaLaunchKernelEx(&cfg, k_attention_tc<128>, m0, m1, (__nv_bfloat16*)out, cu, seq0, row0, n_q_heads,
                                                  n_kv_heads, causal, scale_log2, err)
                             : cudaLaunchKernelEx(&cfg, k_attention_tc<64>, m0, m1, (__nv_bfloat16*)out, cu, seq0, row0, n_q_heads,
                                                  n_kv_heads, causal, scale_log2, err);
  if (le != cudaSuccess) return le;
  return cudaGetLastError();
}

}  // namespace prism
