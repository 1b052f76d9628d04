// The single-CTA version of the projection GEMMs (PRISM_IMPL_SOLO; the default is the CTA-pair kernel of
// gemm_tc2.cu, which this file also serves with the tensor-map builders).
// Projection GEMMs of the decoder block on the 5th-generation tensor cores (sm_100a):
//   C[M,N] = A[M,K] * B[N,K]^T, bf16 operands (both K-major), fp32 accumulation in tensor memory.
//
// One persistent CTA per SM, warp-specialised:
//   warp 0      TMA producer: 128x64 A tile + 256x64 B tile per stage, 128-byte swizzle, 4 stages
//   warp 1      MMA issuer: one elected lane issues tcgen05.mma (M=128, N=256, K=16) into one of two
//               256-column TMEM accumulators, commits stage-release and accumulator-ready barriers
//   warps 2..9  epilogue: two warps per 32-row TMEM lane quarter, each taking one half of the tile's
//               columns; tcgen05.ld the accumulator (one row per thread), apply the fused epilogue
//               while the MMA warp fills the other buffer:
//                 store     bf16 store
//                 residual  x += acc through shared memory and a TMA reduce-add (asynchronous, no read of
//                           x by the SM, one add per element so the result is deterministic)
//                 SwiGLU    silu(gate) * up
//                 QKV       per-head RMSNorm (QK-norm) and rotary embedding on the q and k heads before
//                           the bf16 store (a 256-column tile is exactly two heads of 128)
// Every tile uses the same shape and the same K order whatever M is, so a row's result does not
// depend on where it sits in the batch (duplicated candidates give bit-identical scores).
//
// Every mbarrier wait is bounded: on expiry the kernel records kErrTimeout and all roles drain to
// the common exit, which frees the tensor memory.  Every TMA load is a plain per-CTA load.
#include "tc_common.cuh"

namespace prism {

namespace {

using namespace tc;

constexpr int BM = 128, BN = 256, BK = 64, UMMA_K = 16;
constexpr int kStages = 4;
constexpr int kABytes = BM * BK * 2;           // 16 KB
constexpr int kBBytes = BN * BK * 2;           // 32 KB
constexpr int kStageBytes = kABytes + kBBytes; // 48 KB
constexpr int kEpiBufBytes = 32 * 32 * 4;      // one 32x32 fp32 sub-tile staged for a TMA reduce-add
constexpr int kEpiStageBytes = 4 * 2 * kEpiBufBytes;  // 4 epilogue warps x 2 buffers
constexpr int kSmemBytes = kStages * kStageBytes + kEpiStageBytes + 1024 /*alignment slack*/ + 256 /*barriers*/;
constexpr int kThreads = 320;  // TMA warp, MMA warp, 8 epilogue warps


// kind::f16 instruction descriptor: D fp32, A/B bf16, both K-major, M=128, N=256.
constexpr uint32_t kIdesc = idesc_bf16(BM, BN, 0);

template <int kEpi>
__global__ void __launch_bounds__(kThreads, 1)
k_gemm_tc(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b0,
          const __grid_constant__ CUtensorMap map_b1, const __grid_constant__ CUtensorMap map_r,
          __nv_bfloat16* __restrict__ out, int m, int n, int k, const QkvRopeArgs qa, int* __restrict__ err) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t tiles = (raw + 1023u) & ~1023u;  // swizzled tiles need 1024-byte alignment
  unsigned char* gen_tiles = smem_raw + (tiles - raw);
  const uint32_t epi_stage = tiles + kStages * kStageBytes;  // 1024-byte aligned
  uint64_t* bars = reinterpret_cast<uint64_t*>(gen_tiles + kStages * kStageBytes + kEpiStageBytes);
  // bars: full[kStages], empty[kStages], acc_full[2], acc_empty[2]; then tmem base and abort flag
  const uint32_t bar_full = smem_u32(bars), bar_empty = smem_u32(bars + kStages);
  const uint32_t bar_acc_full = smem_u32(bars + 2 * kStages), bar_acc_empty = smem_u32(bars + 2 * kStages + 2);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * kStages + 4);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // Output tile width: SwiGLU tiles hold 128 gate + 128 up columns and produce 128 outputs.
  constexpr int kOutCols = (kEpi == kEpiSwiGLU) ? 128 : 256;
  (void)epi_stage;
  const int m_tiles = (m + BM - 1) / BM, n_tiles = (n + kOutCols - 1) / kOutCols;
  const int num_tiles = m_tiles * n_tiles, num_kb = (k + BK - 1) / BK;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(bar_full + 8 * s, 1);
      mbar_init(bar_empty + 8 * s, 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(bar_acc_full + 8 * a, 1);
      mbar_init(bar_acc_empty + 8 * a, 8);
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {  // allocate all 512 tensor-memory columns (two 256-column accumulators)
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(512));
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::);
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      uint32_t stage = 0, phase = 0, armed = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
        const int mt = tile / n_tiles, nt = tile % n_tiles;
        const int row_a = mt * BM;
        const int row_b0 = (kEpi == kEpiSwiGLU) ? nt * 128 : nt * BN;
        const int row_b1 = (kEpi == kEpiSwiGLU) ? nt * 128 : nt * BN + 128;
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!mbar_wait(bar_empty + 8 * stage, phase ^ 1, err, abort_flag)) { ok = false; break; }
          const uint32_t sa = tiles + stage * kStageBytes, sb = sa + kABytes;
          mbar_expect_tx(bar_full + 8 * stage, kStageBytes);
          tma_load_2d(sa, &map_a, kb * BK, row_a, bar_full + 8 * stage);
          tma_load_2d(sb, &map_b0, kb * BK, row_b0, bar_full + 8 * stage);
          tma_load_2d(sb + kBBytes / 2, &map_b1, kb * BK, row_b1, bar_full + 8 * stage);
          armed |= 1u << stage;
          if (++stage == kStages) { stage = 0; phase ^= 1; }
        }
      }
      if (!ok) {
        // Let copies already in flight land before shared memory is released (bounded).
        for (int s = 0; s < kStages; ++s) {
          if (!(armed & (1u << s))) continue;
          const uint32_t par = (s < (int)stage) ? phase : (phase ^ 1);
          const unsigned long long t0 = clock64();
          while (!mbar_try(bar_full + 8 * s, par) && clock64() - t0 < kWaitCycles / 8) {}
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      uint32_t stage = 0, phase = 0;
      bool ok = true;
      int it = 0;
      for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++it) {
        const uint32_t acc = it & 1, acc_phase = (it >> 1) & 1;
        if (!mbar_wait(bar_acc_empty + 8 * acc, acc_phase ^ 1, err, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + acc * BN;
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!mbar_wait(bar_full + 8 * stage, phase, err, abort_flag)) { ok = false; break; }
          tc_fence_after();
          const uint32_t sa = tiles + stage * kStageBytes, sb = sa + kABytes;
          const uint64_t da = smem_desc(sa, 16, 1024), db = smem_desc(sb, 16, 1024);
#pragma unroll
          for (int kk = 0; kk < BK / UMMA_K; ++kk) {
            // advancing K by 16 bf16 = 32 bytes inside the swizzle atom: +2 in 16-byte units
            umma_bf16(d_tmem, da + 2 * kk, db + 2 * kk, kIdesc, (kb | kk) != 0);
          }
          umma_commit(bar_empty + 8 * stage);  // stage is free once these MMAs have read it
          if (++stage == kStages) { stage = 0; phase ^= 1; }
        }
        if (ok) umma_commit(bar_acc_full + 8 * acc);  // accumulator complete
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (8 warps, 128 rows x 2 column halves)
    const int quarter = warp & 3;        // TMEM lane quarter this warp may read
    const int colhalf = (warp - 2) >> 2;  // 0: first half of the tile's columns, 1: second half
    bool ok = true;
    int it = 0;
    // QKV epilogue: the row's position and the first half of its rotary table rows do not depend on the
    // accumulator, so they are requested before the wait for it (their L2 latency hides behind the MMAs).
    [[maybe_unused]] int rope_pos = 0;
    [[maybe_unused]] float4 tv[8];
    [[maybe_unused]] auto rope_row_pos = [&](int t) {
      const int rw = (t / n_tiles) * BM + quarter * 32 + lane;
      return qa.pos[rw < m ? rw : 0];
    };
    [[maybe_unused]] auto rope_fetch = [&](int half) {
#pragma unroll
      for (int i8 = 0; i8 < 8; ++i8) {
        const int rr = (colhalf * 8 + i8) * 2 + (lane >> 4);  // this warp fetches 16 of the quarter's 32 rows
        const int p = __shfl_sync(0xffffffffu, rope_pos, rr);
        tv[i8] = __ldg(reinterpret_cast<const float4*>(qa.tab + (size_t)p * 128 + half * 64) + (lane & 15));
      }
    };
    if constexpr (kEpi == kEpiQkvRope) {
      if ((int)blockIdx.x < num_tiles) rope_pos = rope_row_pos(blockIdx.x);
    }
    for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++it) {
      const uint32_t acc = it & 1, acc_phase = (it >> 1) & 1;
      const int mt = tile / n_tiles, nt = tile % n_tiles;
      [[maybe_unused]] int rope_pos_next = 0;
      if constexpr (kEpi == kEpiQkvRope) {
        if (nt * 2 < qa.hq + qa.hkv) rope_fetch(0);
        if (tile + (int)gridDim.x < num_tiles) rope_pos_next = rope_row_pos(tile + gridDim.x);
      }
      if (!mbar_wait(bar_acc_full + 8 * acc, acc_phase, err, abort_flag)) { ok = false; break; }
      tc_fence_after();
      const int row = mt * BM + quarter * 32 + lane;
      const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + acc * BN;
      const int col0 = nt * kOutCols;
      if constexpr (kEpi == kEpiSwiGLU) {
#pragma unroll 1
        for (int cc = 0; cc < 2; ++cc) {
          const int c = colhalf * 2 + cc;  // 32 of the tile's 128 outputs: gate columns c*32.., up columns 128 + c*32..
          uint32_t g[32], u[32];
          tmem_ld32(taddr + c * 32, g);
          tmem_ld32(taddr + 128 + c * 32, u);
          tmem_ld_wait();
          if (row < m) {
            __nv_bfloat16* o = out + (size_t)row * n + col0 + c * 32;
#pragma unroll
            for (int v = 0; v < 4; ++v) {
              if (col0 + c * 32 + v * 8 < n) {
                uint32_t pk[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                  const float g0 = __uint_as_float(g[v * 8 + 2 * e]), g1 = __uint_as_float(g[v * 8 + 2 * e + 1]);
                  const float u0 = __uint_as_float(u[v * 8 + 2 * e]), u1 = __uint_as_float(u[v * 8 + 2 * e + 1]);
                  pk[e] = pack_bf16(__fdividef(g0, 1.f + __expf(-g0)) * u0, __fdividef(g1, 1.f + __expf(-g1)) * u1);
                }
                *reinterpret_cast<uint4*>(o + v * 8) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
              }
            }
          }
        }
      } else if constexpr (kEpi == kEpiResidual) {
        // 32x32 fp32 sub-tiles go through this warp's staging buffer (128-byte swizzle) into a TMA reduce-add.
        const uint32_t buf = epi_stage + (uint32_t)(warp - 2) * kEpiBufBytes;
#pragma unroll 1
        for (int cc = 0; cc < 4; ++cc) {
          const int c = colhalf * 4 + cc;
          // sub-tiles outside the matrix are skipped (warp-uniform)
          if (col0 + c * 32 >= n || mt * BM + quarter * 32 >= m) break;
          uint32_t r[32];
          tmem_ld32(taddr + c * 32, r);
          if (lane == 0) bulk_wait_read<0>();  // the previous reduce has finished reading the buffer
          __syncwarp();
          tmem_ld_wait();
#pragma unroll
          for (int v = 0; v < 8; ++v) {
            const uint32_t dst = buf + lane * 128 + ((v ^ (lane & 7)) << 4);
            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(r[4 * v]), "r"(r[4 * v + 1]),
                         "r"(r[4 * v + 2]), "r"(r[4 * v + 3]) : "memory");
          }
          fence_async_smem();
          __syncwarp();
          if (lane == 0) {
            tma_reduce_add_2d(&map_r, buf, col0 + c * 32, mt * BM + quarter * 32);
            bulk_commit();
          }
        }
      } else if constexpr (kEpi == kEpiQkvRope) {
        // A 256-column tile is two heads; this warp owns head `colhalf` of the tile.  q and k heads:
        // optional RMSNorm over the head, then the rotation of pairs (i, i+64); v heads are stored as
        // they are.  The rotary table rows of the quarter's 32 rows are fetched coalesced (256 bytes per
        // row and half) into a staging buffer shared by the two warps of the quarter, 16-byte chunks
        // XOR-swizzled by row so that every thread reads its own row without bank conflicts.
        const uint32_t stage = epi_stage + (uint32_t)quarter * 2 * kEpiBufBytes;  // 8 KB = 32 rows x 256 B
        const int pair_bar = 1 + quarter;                                         // named barrier of the two warps
        const int head = nt * 2 + colhalf;
        const bool live = head * 128 < n;
        const bool rot = live && head < qa.hq + qa.hkv;
        const bool any_rot = nt * 2 < qa.hq + qa.hkv;  // same for both warps of the pair
        const uint32_t th = taddr + colhalf * 128;
        auto stage_table = [&]() {
#pragma unroll
          for (int i8 = 0; i8 < 8; ++i8) {
            const int rr = (colhalf * 8 + i8) * 2 + (lane >> 4), ch = lane & 15;
            const uint32_t dst = stage + rr * 256 + ((ch ^ (rr & 7)) << 4);
            asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "f"(tv[i8].x), "f"(tv[i8].y), "f"(tv[i8].z),
                         "f"(tv[i8].w) : "memory");
          }
        };
        float rnh = 1.f;
        if (rot && qa.qk_norm) {
          float ss = 0.f;
#pragma unroll 1
          for (int c = 0; c < 4; ++c) {
            uint32_t r[32];
            tmem_ld32(th + c * 32, r);
            tmem_ld_wait();
#pragma unroll
            for (int e = 0; e < 32; ++e) ss = fmaf(__uint_as_float(r[e]), __uint_as_float(r[e]), ss);
          }
          rnh = 1.0f / sqrtf(ss * (1.f / 128.f) + qa.eps);
        }
        __nv_bfloat16* o = out + (size_t)row * n + (size_t)head * 128;
        const __nv_bfloat16* gain = head < qa.hq ? qa.g_q : qa.g_k;
#pragma unroll 1
        for (int half = 0; half < 2; ++half) {
          if (any_rot) {
            // both warps are done reading the previous half before it is overwritten
            asm volatile("bar.sync %0, 64;" ::"r"(pair_bar) : "memory");
            stage_table();
            asm volatile("bar.sync %0, 64;" ::"r"(pair_bar) : "memory");
            if (half == 0) rope_fetch(1);
          }
          if (!live) continue;
          uint32_t a[32], b[32];
          tmem_ld32(th + half * 32, a);
          tmem_ld32(th + 64 + half * 32, b);
          tmem_ld_wait();
          if (!rot) {  // v head: plain store of the two 32-column pieces
            if (row < m) {
#pragma unroll
              for (int v = 0; v < 4; ++v) {
                uint4 pa, pb;
                pa.x = pack_bf16(__uint_as_float(a[v * 8 + 0]), __uint_as_float(a[v * 8 + 1]));
                pa.y = pack_bf16(__uint_as_float(a[v * 8 + 2]), __uint_as_float(a[v * 8 + 3]));
                pa.z = pack_bf16(__uint_as_float(a[v * 8 + 4]), __uint_as_float(a[v * 8 + 5]));
                pa.w = pack_bf16(__uint_as_float(a[v * 8 + 6]), __uint_as_float(a[v * 8 + 7]));
                pb.x = pack_bf16(__uint_as_float(b[v * 8 + 0]), __uint_as_float(b[v * 8 + 1]));
                pb.y = pack_bf16(__uint_as_float(b[v * 8 + 2]), __uint_as_float(b[v * 8 + 3]));
                pb.z = pack_bf16(__uint_as_float(b[v * 8 + 4]), __uint_as_float(b[v * 8 + 5]));
                pb.w = pack_bf16(__uint_as_float(b[v * 8 + 6]), __uint_as_float(b[v * 8 + 7]));
                *reinterpret_cast<uint4*>(o + half * 32 + v * 8) = pa;
                *reinterpret_cast<uint4*>(o + 64 + half * 32 + v * 8) = pb;
              }
            }
            continue;
          }
#pragma unroll
          for (int v = 0; v < 4; ++v) {
            float x0[8], x1[8], cs[8], sn[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) {
              x0[e] = __uint_as_float(a[v * 8 + e]);
              x1[e] = __uint_as_float(b[v * 8 + e]);
            }
            if (qa.qk_norm) {
              const uint4 g0 = __ldg(reinterpret_cast<const uint4*>(gain + half * 32 + v * 8));
              const uint4 g1 = __ldg(reinterpret_cast<const uint4*>(gain + 64 + half * 32 + v * 8));
              const __nv_bfloat16* p0 = reinterpret_cast<const __nv_bfloat16*>(&g0);
              const __nv_bfloat16* p1 = reinterpret_cast<const __nv_bfloat16*>(&g1);
#pragma unroll
              for (int e = 0; e < 8; ++e) {
                x0[e] = x0[e] * rnh * __bfloat162float(p0[e]);
                x1[e] = x1[e] * rnh * __bfloat162float(p1[e]);
              }
            }
            // staged row: chunks 0..7 = cos(32*half + 0..31), chunks 8..15 = sin
#pragma unroll
            for (int q4 = 0; q4 < 2; ++q4) {
              const int cc = v * 2 + q4;
              const uint32_t ca = stage + lane * 256 + ((cc ^ (lane & 7)) << 4);
              const uint32_t sa = stage + lane * 256 + (((cc + 8) ^ (lane & 7)) << 4);
              asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];"
                           : "=f"(cs[q4 * 4]), "=f"(cs[q4 * 4 + 1]), "=f"(cs[q4 * 4 + 2]), "=f"(cs[q4 * 4 + 3]) : "r"(ca));
              asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];"
                           : "=f"(sn[q4 * 4]), "=f"(sn[q4 * 4 + 1]), "=f"(sn[q4 * 4 + 2]), "=f"(sn[q4 * 4 + 3]) : "r"(sa));
            }
            uint32_t lo[4], hi[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const float y0 = x0[2 * e] * cs[2 * e] - x1[2 * e] * sn[2 * e];
              const float y1 = x0[2 * e + 1] * cs[2 * e + 1] - x1[2 * e + 1] * sn[2 * e + 1];
              const float z0 = x1[2 * e] * cs[2 * e] + x0[2 * e] * sn[2 * e];
              const float z1 = x1[2 * e + 1] * cs[2 * e + 1] + x0[2 * e + 1] * sn[2 * e + 1];
              lo[e] = pack_bf16(y0, y1);
              hi[e] = pack_bf16(z0, z1);
            }
            if (row < m) {
              *reinterpret_cast<uint4*>(o + half * 32 + v * 8) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
              *reinterpret_cast<uint4*>(o + 64 + half * 32 + v * 8) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
            }
          }
        }
      } else {
#pragma unroll 1
        for (int cc = 0; cc < 4; ++cc) {
          const int c = colhalf * 4 + cc;
          uint32_t r[32];
          tmem_ld32(taddr + c * 32, r);
          tmem_ld_wait();
          if (row < m) {
            __nv_bfloat16* o = out + (size_t)row * n + col0 + c * 32;
#pragma unroll
            for (int v = 0; v < 4; ++v) {
              if (col0 + c * 32 + v * 8 < n) {
                uint4 pk;
                pk.x = pack_bf16(__uint_as_float(r[v * 8 + 0]), __uint_as_float(r[v * 8 + 1]));
                pk.y = pack_bf16(__uint_as_float(r[v * 8 + 2]), __uint_as_float(r[v * 8 + 3]));
                pk.z = pack_bf16(__uint_as_float(r[v * 8 + 4]), __uint_as_float(r[v * 8 + 5]));
                pk.w = pack_bf16(__uint_as_float(r[v * 8 + 6]), __uint_as_float(r[v * 8 + 7]));
                *reinterpret_cast<uint4*>(o + v * 8) = pk;
              }
            }
          }
        }
      }
      if constexpr (kEpi == kEpiQkvRope) rope_pos = rope_pos_next;
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_acc_empty + 8 * acc);
    }
    if constexpr (kEpi == kEpiResidual) {
      if (lane == 0) bulk_wait<0>();  // all reduce-adds of this warp have completed
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512));
  }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// A tensor map is a pure function of (kind, base, rows, cols, box); the layer loop asks for the same few maps
// again and again (the handle's buffers are fixed and the row count changes only at a compaction), so each host
// thread keeps the most recent ones.  Direct-mapped, 64 entries; a miss encodes and replaces.
struct MapKey {
  int kind;
  const void* base;
  uint64_t rows, cols;
  uint32_t box_rows, box_cols;
  bool operator==(const MapKey& o) const {
    return kind == o.kind && base == o.base && rows == o.rows && cols == o.cols && box_rows == o.box_rows &&
           box_cols == o.box_cols;
  }
};
struct MapSlot {
  MapKey key;
  TmaDesc desc;
  bool valid;
};
constexpr int kMapSlots = 64;

template <typename Encode>
cudaError_t cached_map(TmaDesc* out, const MapKey& key, Encode encode) {
  thread_local MapSlot slots[kMapSlots] = {};
  uint64_t h = reinterpret_cast<uintptr_t>(key.base) * 0x9E3779B97F4A7C15ull;
  h ^= (key.rows + 0x632BE59BD9B4E019ull) * 0xC2B2AE3D27D4EB4Full;
  h ^= (key.cols * 31 + key.box_rows * 7 + key.box_cols + (uint64_t)key.kind * 1315423911ull) * 0x165667B19E3779F9ull;
  MapSlot& s = slots[(h >> 40) % kMapSlots];
  if (s.valid && s.key == key) {
    *out = s.desc;
    return cudaSuccess;
  }
  const cudaError_t e = encode(out);
  if (e == cudaSuccess) {
    s.key = key;
    s.desc = *out;
    s.valid = true;
  }
  return e;
}

}  // namespace

static_assert(sizeof(CUtensorMap) == sizeof(TmaDesc), "TmaDesc must mirror CUtensorMap");

cudaError_t make_tma_2d_bf16(TmaDesc* out, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows,
                             uint32_t box_cols) {
  EncodeTiledFn enc = get_encode();
  if (!enc) return cudaErrorNotSupported;
  if ((reinterpret_cast<uintptr_t>(base) & 15) || (cols * 2) % 16 || box_cols * 2 != 128 || box_rows > 256)
    return cudaErrorInvalidValue;
  return cached_map(out, MapKey{0, base, rows, cols, box_rows, box_cols}, [&](TmaDesc* d) {
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {cols * 2};
    cuuint32_t box[2] = {box_cols, box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = enc(reinterpret_cast<CUtensorMap*>(d), CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base),
                     dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                     CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
  });
}

int gemm_tc_sm_count() {
  static std::atomic<int> cached{0};  // every GPU of a node is the same part
  int sms = cached.load(std::memory_order_relaxed);
  if (!sms) {
    int dev = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (sms <= 0) sms = 148;
    cached.store(sms, std::memory_order_relaxed);
  }
  return sms;
}

cudaError_t make_tma_2d_f32_box32(TmaDesc* out, const void* base, uint64_t rows, uint64_t cols) {
  EncodeTiledFn enc = get_encode();
  if (!enc) return cudaErrorNotSupported;
  if ((reinterpret_cast<uintptr_t>(base) & 15) || (cols * 4) % 16) return cudaErrorInvalidValue;
  return cached_map(out, MapKey{1, base, rows, cols, 32, 32}, [&](TmaDesc* d) {
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {cols * 4};
    cuuint32_t box[2] = {32, 32};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = enc(reinterpret_cast<CUtensorMap*>(d), CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<void*>(base),
                     dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                     CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
  });
}

cudaError_t make_tma_2d_bf16_box32_sw64(TmaDesc* out, const void* base, uint64_t rows, uint64_t cols) {
  EncodeTiledFn enc = get_encode();
  if (!enc) return cudaErrorNotSupported;
  if ((reinterpret_cast<uintptr_t>(base) & 15) || (cols * 2) % 16) return cudaErrorInvalidValue;
  return cached_map(out, MapKey{2, base, rows, cols, 32, 32}, [&](TmaDesc* d) {
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {cols * 2};
    cuuint32_t box[2] = {32, 32};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = enc(reinterpret_cast<CUtensorMap*>(d), CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base),
                     dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_64B,
                     CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
  });
}

cudaError_t launch_gemm_tc(const TmaDesc& a, const TmaDesc& b0, const TmaDesc& b1, void* out, float* resid, int m,
                           int n, int k, int epilogue, const QkvRopeArgs* qa, int* err, cudaStream_t st) {
  if (m <= 0 || n <= 0) return cudaSuccess;
  if (k <= 0 || (k % 8) || (n % 8)) return cudaErrorInvalidValue;
  static std::atomic<unsigned long long> smem_set[4];
  {
    cudaError_t e = cudaErrorInvalidValue;
    if (epilogue == kEpiStore) e = ensure_dynamic_smem(k_gemm_tc<kEpiStore>, kSmemBytes, smem_set[0]);
    else if (epilogue == kEpiResidual) e = ensure_dynamic_smem(k_gemm_tc<kEpiResidual>, kSmemBytes, smem_set[1]);
    else if (epilogue == kEpiSwiGLU) e = ensure_dynamic_smem(k_gemm_tc<kEpiSwiGLU>, kSmemBytes, smem_set[2]);
    else if (epilogue == kEpiQkvRope) e = ensure_dynamic_smem(k_gemm_tc<kEpiQkvRope>, kSmemBytes, smem_set[3]);
    if (e != cudaSuccess) return e;
  }
  const int out_cols = epilogue == kEpiSwiGLU ? 128 : 256;
  const long long tiles = (long long)((m + BM - 1) / BM) * ((n + out_cols - 1) / out_cols);
  const int sms = gemm_tc_sm_count();
  const int grid = (int)(tiles < sms ? tiles : sms);
  const CUtensorMap& ma = reinterpret_cast<const CUtensorMap&>(a);
  const CUtensorMap& mb0 = reinterpret_cast<const CUtensorMap&>(b0);
  const CUtensorMap& mb1 = reinterpret_cast<const CUtensorMap&>(b1);
  TmaDesc rdesc = a;  // placeholder for the epilogues that do not use it
  QkvRopeArgs q{};
  if (epilogue == kEpiResidual) {
    // the residual rows of this launch, exactly m of them, so that the TMA unit clips the ragged last tile
    cudaError_t e = make_tma_2d_f32_box32(&rdesc, resid, (uint64_t)m, (uint64_t)n);
    if (e != cudaSuccess) return e;
  }
  if (epilogue == kEpiQkvRope) {
    if (!qa || n % 128) return cudaErrorInvalidValue;
    q = *qa;
  }
  const CUtensorMap& mr = reinterpret_cast<const CUtensorMap&>(rdesc);
  __nv_bfloat16* o = (__nv_bfloat16*)out;
  if (epilogue == kEpiStore)
    k_gemm_tc<kEpiStore><<<grid, kThreads, kSmemBytes, st>>>(ma, mb0, mb1, mr, o, m, n, k, q, err);
  else if (epilogue == kEpiResidual)
    k_gemm_tc<kEpiResidual><<<grid, kThreads, kSmemBytes, st>>>(ma, mb0, mb1, mr, o, m, n, k, q, err);
  else if (epilogue == kEpiSwiGLU)
    k_gemm_tc<kEpiSwiGLU><<<grid, kThreads, kSmemBytes, st>>>(ma, mb0, mb1, mr, o, m, n, k, q, err);
  else if (epilogue == kEpiQkvRope)
    k_gemm_tc<kEpiQkvRope><<<grid, kThreads, kSmemBytes, st>>>(ma, mb0, mb1, mr, o, m, n, k, q, err);
  else
    return cudaErrorInvalidValue;
  return cudaGetLastError();
}

}  // namespace prism
