// The projection GEMMs of gemm_tc.cu on CTA PAIRS (tcgen05 cta_group::2): a cluster of two CTAs computes a
// 256x256 tile; each CTA loads its own 128 rows of A and ONE HALF (128 rows) of the B tile, the leader's
// elected thread issues M256 N256 K16 MMAs that read both CTAs' shared memory, and each CTA's tensor
// memory receives its own 128 accumulator rows.  Per SM this halves the B operand traffic through shared
// memory, which is the co-limit of the single-CTA kernel.
//
// Epilogues (8 warps per CTA, one accumulator row per thread) compute what gemm_tc.cu's do, but every result
// leaves through a swizzled shared-memory staging buffer and a TMA operation whose tensor map has exactly M
// rows (the ragged last tile is clipped by the TMA unit):
//   store     bf16, 32-row x 128-byte boxes, two buffers per warp
//   residual  x += acc as a TMA reduce-add (no read of x by the SM, one add per element: deterministic)
//   SwiGLU    rank 0 of the pair loads the tile's gate rows, rank 1 the up rows, so each CTA's accumulator
//             holds gate and up of its rows side by side; silu(gate) * up, one 64-column box per warp and tile
//   QKV       per-head RMSNorm (QK-norm) and rotary embedding on the q and k heads (a 256-column tile is two
//             heads of 128); rotary-table rows staged per 32-row quarter; 32x32 boxes with the 64-byte swizzle
// Every tile has the same shape and K order whatever M is, and the row tiles can be walked in either
// direction, so a row's result does not depend on where it sits in the batch or on the direction.
//
// Protocol: full[s] lives in the leader and counts the bytes of BOTH CTAs' TMA loads; empty[s] and
// acc_full[a] exist in both CTAs and are signalled by commits that arrive in both CTAs; acc_empty[a] lives in the leader
// and is arrived on by the epilogue warps of both CTAs.  Every TMA load is a plain per-CTA load.  Every wait is bounded.
#include "tc_common.cuh"

namespace prism {

namespace {

using namespace tc;

constexpr int BM = 128, BN = 256, BK = 64, UMMA_K = 16;
constexpr int kABytes = BM * BK * 2;           // 16 KB
constexpr int kBBytes = (BN / 2) * BK * 2;     // 16 KB: this CTA's half of the B tile
constexpr int kStageBytes = kABytes + kBBytes; // 32 KB
constexpr int kEpiBufBytes = 32 * 32 * 4;      // one 32-row, 128-byte-wide sub-tile staged for a TMA store or reduce-add
// Operand ring and epilogue staging share 224 KB: the residual and SwiGLU epilogues stage one 4 KB sub-tile per
// warp and keep six operand stages; the plain store stages 8 KB per warp (two buffers), the QKV epilogue 32 KB
// of rotary-table rows and 4 KB of output per warp, and these keep five.
__host__ __device__ constexpr int stages_of(int epi) {
  return (epi == kEpiResidual || epi == kEpiResidualBias || epi == kEpiSwiGLU) ? 6 : 5;
}
__host__ __device__ constexpr int epi_stage_bytes_of(int epi) { return (7 - stages_of(epi)) * kStageBytes; }
constexpr int kSmemBytes = 7 * kStageBytes + 1024 /*alignment slack*/ + 256 /*barriers*/;
constexpr int kThreads = 320;  // TMA warp, MMA warp, 8 epilogue warps


__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// Address of the same shared-memory offset in CTA `rank` of the cluster.
__device__ __forceinline__ uint32_t map_to_cta(uint32_t addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void cluster_sync() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// TMA tile load of the pair form: data lands in this CTA, the byte count is reported to `bar`, which may
// be a barrier of the other CTA of the pair (a shared::cluster address).
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(bar)
      : "memory");
}
__device__ __forceinline__ void umma_bf16_pair(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc,
                                               uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate)
      : "memory");
}
// Arrives on the barrier at this offset in BOTH CTAs once all MMAs issued so far have completed.
__device__ __forceinline__ void umma_commit_pair(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(bar), "h"((uint16_t)3) : "memory");
}

// gelu(x) = x Phi(x) without a branch: Phi from the rational-times-Gaussian form of erfc (Abramowitz & Stegun
// 7.1.26, absolute error below 5e-7, far under the bf16 rounding of the result): one reciprocal, one exp2 and a
// handful of FMAs per element, so that the epilogue keeps up with the MMAs.  Two values at once, the polynomial and
// the products in packed fp32 arithmetic (half the FMA issue slots); the factor 0.5 of the tail is folded into the
// coefficients.
__device__ __forceinline__ void gelu_fast2(float x0, float x1, float& y0, float& y1) {
  const float c = 0.70710678118654752f;
  const uint64_t z = f2_pack(fabsf(x0) * c, fabsf(x1) * c);
  float d0, d1, t0, t1;
  f2_unpack(f2_fma(f2_pack(0.3275911f, 0.3275911f), z, f2_pack(1.f, 1.f)), d0, d1);
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(t0) : "f"(d0));
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(t1) : "f"(d1));
  const uint64_t t = f2_pack(t0, t1);
  uint64_t p = f2_fma(f2_pack(0.5f * 1.061405429f, 0.5f * 1.061405429f), t, f2_pack(0.5f * -1.453152027f, 0.5f * -1.453152027f));
  p = f2_fma(p, t, f2_pack(0.5f * 1.421413741f, 0.5f * 1.421413741f));
  p = f2_fma(p, t, f2_pack(0.5f * -0.284496736f, 0.5f * -0.284496736f));
  p = f2_fma(p, t, f2_pack(0.5f * 0.254829592f, 0.5f * 0.254829592f));
  float a0, a1, e0, e1;
  f2_unpack(f2_mul(f2_mul(z, z), f2_pack(-1.4426950408889634f, -1.4426950408889634f)), a0, a1);
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e0) : "f"(a0));
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e1) : "f"(a1));
  float q0, q1;  // x * Phi(-|x|)
  f2_unpack(f2_mul(f2_mul(f2_mul(p, t), f2_pack(e0, e1)), f2_pack(x0, x1)), q0, q1);
  y0 = x0 >= 0.f ? x0 - q0 : q0;
  y1 = x1 >= 0.f ? x1 - q1 : q1;
}

// kind::f16 instruction descriptor: D fp32, A/B bf16, both K-major, M=128, N=256.
constexpr uint32_t kIdesc = idesc_bf16(2 * BM, BN, 0);  // the pair's instruction: M = 256

template <int kEpi>
__global__ void __launch_bounds__(kThreads, 1)
k_gemm_tc2(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b0,
          const __grid_constant__ CUtensorMap map_b1, const __grid_constant__ CUtensorMap map_r,
          __nv_bfloat16* __restrict__ out, int m, int n, int k, const QkvRopeArgs qa, int reverse,
          int* __restrict__ err, const float* __restrict__ bias) {
  // the bias variants share the staging and the TMA path of the plain store and of the residual reduce-add
  constexpr bool kHasBias = kEpi == kEpiStoreBias || kEpi == kEpiGeluBias || kEpi == kEpiResidualBias;
  constexpr bool kIsResidual = kEpi == kEpiResidual || kEpi == kEpiResidualBias;
  constexpr int kStages = stages_of(kEpi), kEpiStageBytes = epi_stage_bytes_of(kEpi);
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
  // A pair works on 256 rows: its tile index t names rows [256*(t / n_tiles), +256), of which this CTA owns
  // the half selected by its rank in the cluster.
  const uint32_t rank = cluster_ctarank();
  const bool leader = rank == 0;
  const int pair_id = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
  const int m_tiles2 = (m + 2 * BM - 1) / (2 * BM), n_tiles = (n + kOutCols - 1) / kOutCols;
  const int num_tiles = m_tiles2 * n_tiles, num_kb = (k + BK - 1) / BK;
  // reverse: the row tiles are taken from the end of the matrix backwards (launch_gemm_tc2 says why)
  auto my_m_tile = [&](int t) {  // in units of 128 rows
    const int mrow2 = t / n_tiles;
    return (reverse ? m_tiles2 - 1 - mrow2 : mrow2) * 2 + (int)rank;
  };

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(bar_full + 8 * s, 1);
      mbar_init(bar_empty + 8 * s, 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(bar_acc_full + 8 * a, 1);
      mbar_init(bar_acc_empty + 8 * a, 16);  // 8 epilogue warps of each CTA of the pair (used in the leader)
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  cluster_sync();  // both CTAs' barriers exist before anything can signal them
  if (warp == 1) {  // both CTAs of the pair allocate all 512 tensor-memory columns (two 256-column accumulators)
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(512));
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::);
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  pdl_sync();  // set-up done: the kernel before this one has to be complete from here on
  const uint32_t tmem_base = *tmem_slot;
  const uint32_t leader_full = map_to_cta(bar_full, 0);            // full[] of the leader, as seen from this CTA
  const uint32_t leader_acc_empty = map_to_cta(bar_acc_empty, 0);  // acc_empty[] of the leader

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer (one per CTA)
    if (lane == 0) {
      uint32_t stage = 0, phase = 0;
      bool ok = true;
      for (int tile = pair_id; tile < num_tiles && ok; tile += n_pairs) {
        const int mt = my_m_tile(tile), nt = tile % n_tiles;
        const int row_a = mt * BM;
        // this CTA's half of the B tile: rows [128*rank, +128) of the 256-row tile, or for SwiGLU the gate
        // rows (rank 0) / the up rows (rank 1) of the tile's 128 outputs
        const CUtensorMap* map_b = (kEpi == kEpiSwiGLU && rank == 1) ? &map_b1 : &map_b0;
        const int row_b = (kEpi == kEpiSwiGLU) ? nt * 128 : nt * BN + (int)rank * 128;
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!mbar_wait(bar_empty + 8 * stage, phase ^ 1, err, abort_flag)) { ok = false; break; }
          const uint32_t sa = tiles + stage * kStageBytes, sb = sa + kABytes;
          // the leader's barrier collects the bytes of both CTAs
          if (leader) mbar_expect_tx(bar_full + 8 * stage, 2 * kStageBytes);
          tma_load_2d_pair(sa, &map_a, kb * BK, row_a, leader_full + 8 * stage);
          tma_load_2d_pair(sb, map_b, kb * BK, row_b, leader_full + 8 * stage);
          if (++stage == kStages) { stage = 0; phase ^= 1; }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer (leader CTA only)
    if (lane == 0 && leader) {
      uint32_t stage = 0, phase = 0;
      bool ok = true;
      int it = 0;
      for (int tile = pair_id; tile < num_tiles && ok; tile += n_pairs, ++it) {
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
            umma_bf16_pair(d_tmem, da + 2 * kk, db + 2 * kk, kIdesc, (kb | kk) != 0);
          }
          umma_commit_pair(bar_empty + 8 * stage);  // the stage is free in both CTAs once these MMAs have read it
          if (++stage == kStages) { stage = 0; phase ^= 1; }
        }
        if (ok) umma_commit_pair(bar_acc_full + 8 * acc);  // both CTAs' halves of the accumulator are complete
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (8 warps, 128 rows x 2 column halves)
    const int quarter = warp & 3;        // TMEM lane quarter this warp may read
    const int colhalf = (warp - 2) >> 2;  // 0: first half of the tile's columns, 1: second half
    bool ok = true;
    int it = 0;
    [[maybe_unused]] uint32_t n_stores = 0;  // TMA stores issued by this warp (selects its staging buffer)
    // QKV epilogue: the row's position and the first half of its rotary table rows do not depend on the
    // accumulator, so they are requested before the wait for it (their L2 latency hides behind the MMAs).
    [[maybe_unused]] int rope_pos = 0;
    [[maybe_unused]] float4 tv[8];
    [[maybe_unused]] auto rope_row_pos = [&](int t) {
      const int rw = my_m_tile(t) * BM + quarter * 32 + lane;
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
      if (pair_id < num_tiles) rope_pos = rope_row_pos(pair_id);
    }
    for (int tile = pair_id; tile < num_tiles && ok; tile += n_pairs, ++it) {
      const uint32_t acc = it & 1, acc_phase = (it >> 1) & 1;
      const int mt = my_m_tile(tile), nt = tile % n_tiles;
      [[maybe_unused]] int rope_pos_next = 0;
      if constexpr (kEpi == kEpiQkvRope) {
        if (nt * 2 < qa.hq + qa.hkv) rope_fetch(0);
        if (tile + n_pairs < num_tiles) rope_pos_next = rope_row_pos(tile + n_pairs);
      }
      if (!mbar_wait(bar_acc_full + 8 * acc, acc_phase, err, abort_flag)) { ok = false; break; }
      tc_fence_after();
      [[maybe_unused]] const int row = mt * BM + quarter * 32 + lane;
      const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + acc * BN;
      const int col0 = nt * kOutCols;
      if constexpr (kEpi == kEpiSwiGLU) {
        // This warp's 32 rows x 64 outputs (columns colhalf*64.. of the tile's 128) are staged as bf16 in its
        // buffer (128-byte rows, 128-byte swizzle) and leave as one TMA store per tile.
        if (col0 + colhalf * 64 < n && mt * BM + quarter * 32 < m) {
          const uint32_t buf = epi_stage + (uint32_t)(warp - 2) * kEpiBufBytes;
          if (lane == 0) bulk_wait_read<0>();  // the previous tile's store has read the buffer
          __syncwarp();
#pragma unroll 1
          for (int cc = 0; cc < 2; ++cc) {
            const int c = colhalf * 2 + cc;  // 32 of the tile's 128 outputs: gate columns c*32.., up columns 128 + c*32..
            uint32_t g[32], u[32];
            tmem_ld32(taddr + c * 32, g);
            tmem_ld32(taddr + 128 + c * 32, u);
            tmem_ld_wait();
#pragma unroll
            for (int v = 0; v < 4; ++v) {
              uint32_t pk[4];
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                const float g0 = __uint_as_float(g[v * 8 + 2 * e]), g1 = __uint_as_float(g[v * 8 + 2 * e + 1]);
                const float u0 = __uint_as_float(u[v * 8 + 2 * e]), u1 = __uint_as_float(u[v * 8 + 2 * e + 1]);
                pk[e] = pack_bf16(__fdividef(g0, 1.f + __expf(-g0)) * u0, __fdividef(g1, 1.f + __expf(-g1)) * u1);
              }
              const uint32_t dst = buf + lane * 128 + (((cc * 4 + v) ^ (lane & 7)) << 4);
              asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(pk[0]), "r"(pk[1]), "r"(pk[2]), "r"(pk[3])
                           : "memory");
            }
          }
          fence_async_smem();
          __syncwarp();
          if (lane == 0) {
            tma_store_2d(&map_r, buf, col0 + colhalf * 64, mt * BM + quarter * 32);
            bulk_commit();
          }
        }
      } else if constexpr (kIsResidual) {
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
          if constexpr (kHasBias) {  // the same 32 bias values for every row: warp-uniform loads
#pragma unroll
            for (int v = 0; v < 8; ++v) {
              const int cb = col0 + c * 32 + v * 4;
              if (cb < n) {
                const float4 bv = __ldg(reinterpret_cast<const float4*>(bias + cb));
                r[4 * v] = __float_as_uint(__uint_as_float(r[4 * v]) + bv.x);
                r[4 * v + 1] = __float_as_uint(__uint_as_float(r[4 * v + 1]) + bv.y);
                r[4 * v + 2] = __float_as_uint(__uint_as_float(r[4 * v + 2]) + bv.z);
                r[4 * v + 3] = __float_as_uint(__uint_as_float(r[4 * v + 3]) + bv.w);
              }
            }
          }
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
        const uint32_t out_stage = epi_stage + 8 * kEpiBufBytes + (uint32_t)(warp - 2) * kEpiBufBytes;  // 2 boxes of 2 KB
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
          if (!live || mt * BM + quarter * 32 >= m) continue;  // warp-uniform
          uint32_t a[32], b[32];
          tmem_ld32(th + half * 32, a);
          tmem_ld32(th + 64 + half * 32, b);
          if (lane == 0) bulk_wait_read<0>();  // the previous half's stores have read the two output boxes
          __syncwarp();
          tmem_ld_wait();
          // output columns [32*half, +32) and [64 + 32*half, +32) of the head: two 32-row x 64-byte boxes
          // (64-byte swizzle), each leaving as one TMA store
          const uint32_t box_lo = out_stage + lane * 64, box_hi = box_lo + 2048;
          const uint32_t sw = (uint32_t)(lane >> 1) & 3u;
          if (!rot) {  // v head: stored as it is
#pragma unroll
            for (int v = 0; v < 4; ++v) {
              asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(box_lo + ((v ^ sw) << 4)),
                           "r"(pack_bf16(__uint_as_float(a[v * 8 + 0]), __uint_as_float(a[v * 8 + 1]))),
                           "r"(pack_bf16(__uint_as_float(a[v * 8 + 2]), __uint_as_float(a[v * 8 + 3]))),
                           "r"(pack_bf16(__uint_as_float(a[v * 8 + 4]), __uint_as_float(a[v * 8 + 5]))),
                           "r"(pack_bf16(__uint_as_float(a[v * 8 + 6]), __uint_as_float(a[v * 8 + 7])))
                           : "memory");
              asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(box_hi + ((v ^ sw) << 4)),
                           "r"(pack_bf16(__uint_as_float(b[v * 8 + 0]), __uint_as_float(b[v * 8 + 1]))),
                           "r"(pack_bf16(__uint_as_float(b[v * 8 + 2]), __uint_as_float(b[v * 8 + 3]))),
                           "r"(pack_bf16(__uint_as_float(b[v * 8 + 4]), __uint_as_float(b[v * 8 + 5]))),
                           "r"(pack_bf16(__uint_as_float(b[v * 8 + 6]), __uint_as_float(b[v * 8 + 7])))
                           : "memory");
            }
          } else {
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
            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(box_lo + ((v ^ sw) << 4)), "r"(lo[0]), "r"(lo[1]),
                         "r"(lo[2]), "r"(lo[3]) : "memory");
            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(box_hi + ((v ^ sw) << 4)), "r"(hi[0]), "r"(hi[1]),
                         "r"(hi[2]), "r"(hi[3]) : "memory");
          }
          }
          fence_async_smem();
          __syncwarp();
          if (lane == 0) {
            tma_store_2d(&map_r, out_stage, head * 128 + half * 32, mt * BM + quarter * 32);
            tma_store_2d(&map_r, out_stage + 2048, head * 128 + 64 + half * 32, mt * BM + quarter * 32);
            bulk_commit();
          }
        }
      } else {
        // 32 rows x 64 columns at a time: bf16 into one of the warp's two staging buffers (128-byte rows,
        // 128-byte swizzle), then one TMA store, which clips the ragged edges of the matrix.
#pragma unroll 1
        for (int cc = 0; cc < 2; ++cc) {
          const int c = colhalf * 2 + cc;  // 64-column piece of the tile
          if (col0 + c * 64 >= n || mt * BM + quarter * 32 >= m) break;  // warp-uniform; later pieces are outside too
          uint32_t r[64];
          tmem_ld32(taddr + c * 64, r);
          tmem_ld32(taddr + c * 64 + 32, r + 32);
          const uint32_t buf = epi_stage + (uint32_t)(warp - 2) * 2 * kEpiBufBytes + (n_stores & 1) * kEpiBufBytes;
          if (lane == 0) bulk_wait_read<1>();  // the store that last used this buffer has read it
          __syncwarp();
          tmem_ld_wait();
          if constexpr (kHasBias) {
#pragma unroll
            for (int v = 0; v < 16; ++v) {
              const int cb = col0 + c * 64 + v * 4;
              float4 bv = make_float4(0.f, 0.f, 0.f, 0.f);
              if (cb < n) bv = __ldg(reinterpret_cast<const float4*>(bias + cb));  // warp-uniform address
              float y[4] = {__uint_as_float(r[4 * v]) + bv.x, __uint_as_float(r[4 * v + 1]) + bv.y,
                            __uint_as_float(r[4 * v + 2]) + bv.z, __uint_as_float(r[4 * v + 3]) + bv.w};
              if constexpr (kEpi == kEpiGeluBias) {
                gelu_fast2(y[0], y[1], y[0], y[1]);
                gelu_fast2(y[2], y[3], y[2], y[3]);
              }
#pragma unroll
              for (int e = 0; e < 4; ++e) r[4 * v + e] = __float_as_uint(y[e]);
            }
          }
#pragma unroll
          for (int v = 0; v < 8; ++v) {
            const uint32_t dst = buf + lane * 128 + ((v ^ (lane & 7)) << 4);
            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst),
                         "r"(pack_bf16(__uint_as_float(r[v * 8 + 0]), __uint_as_float(r[v * 8 + 1]))),
                         "r"(pack_bf16(__uint_as_float(r[v * 8 + 2]), __uint_as_float(r[v * 8 + 3]))),
                         "r"(pack_bf16(__uint_as_float(r[v * 8 + 4]), __uint_as_float(r[v * 8 + 5]))),
                         "r"(pack_bf16(__uint_as_float(r[v * 8 + 6]), __uint_as_float(r[v * 8 + 7])))
                         : "memory");
          }
          fence_async_smem();
          __syncwarp();
          if (lane == 0) {
            tma_store_2d(&map_r, buf, col0 + c * 64, mt * BM + quarter * 32);
            bulk_commit();
          }
          ++n_stores;
        }
      }
      if constexpr (kEpi == kEpiQkvRope) rope_pos = rope_pos_next;
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(leader_acc_empty + 8 * acc);  // the leader's MMA thread waits for both CTAs
    }
    if (lane == 0) bulk_wait<0>();  // all TMA stores / reduce-adds of this warp have completed
  }

  tc_fence_before();
  __syncthreads();
  cluster_sync();  // neither CTA frees its shared or tensor memory while the other may still use or signal it
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512));
  }
}

}  // namespace

// reverse: see launch_rmsnorm; the result is the same bit for bit in either direction (every tile has the same
// shape and K order, and each output element is written or reduced into exactly once).
cudaError_t launch_gemm_tc2(const TmaDesc& a, const TmaDesc& b0, const TmaDesc& b1, void* out, float* resid, int m,
                           int n, int k, int epilogue, const QkvRopeArgs* qa, int* err, cudaStream_t st, bool reverse,
                           const float* bias) {
  if (m <= 0 || n <= 0) return cudaSuccess;
  if (k <= 0 || (k % 8) || (n % 8)) return cudaErrorInvalidValue;
  static std::atomic<unsigned long long> smem_set[7];
  const bool has_bias = epilogue == kEpiStoreBias || epilogue == kEpiGeluBias || epilogue == kEpiResidualBias;
  if (has_bias && (!bias || (reinterpret_cast<uintptr_t>(bias) & 15))) return cudaErrorInvalidValue;
  {
    cudaError_t e = cudaErrorInvalidValue;
    if (epilogue == kEpiStore) e = ensure_dynamic_smem(k_gemm_tc2<kEpiStore>, kSmemBytes, smem_set[0]);
    else if (epilogue == kEpiResidual) e = ensure_dynamic_smem(k_gemm_tc2<kEpiResidual>, kSmemBytes, smem_set[1]);
    else if (epilogue == kEpiSwiGLU) e = ensure_dynamic_smem(k_gemm_tc2<kEpiSwiGLU>, kSmemBytes, smem_set[2]);
    else if (epilogue == kEpiQkvRope) e = ensure_dynamic_smem(k_gemm_tc2<kEpiQkvRope>, kSmemBytes, smem_set[3]);
    else if (epilogue == kEpiStoreBias) e = ensure_dynamic_smem(k_gemm_tc2<kEpiStoreBias>, kSmemBytes, smem_set[4]);
    else if (epilogue == kEpiGeluBias) e = ensure_dynamic_smem(k_gemm_tc2<kEpiGeluBias>, kSmemBytes, smem_set[5]);
    else if (epilogue == kEpiResidualBias) e = ensure_dynamic_smem(k_gemm_tc2<kEpiResidualBias>, kSmemBytes, smem_set[6]);
    if (e != cudaSuccess) return e;
  }
  const int out_cols = epilogue == kEpiSwiGLU ? 128 : 256;
  const long long tiles = (long long)((m + 2 * BM - 1) / (2 * BM)) * ((n + out_cols - 1) / out_cols);
  const int pairs = gemm_tc_sm_count() / 2;
  const int grid = 2 * (int)(tiles < pairs ? tiles : pairs);
  const CUtensorMap& ma = reinterpret_cast<const CUtensorMap&>(a);
  const CUtensorMap& mb0 = reinterpret_cast<const CUtensorMap&>(b0);
  const CUtensorMap& mb1 = reinterpret_cast<const CUtensorMap&>(b1);
  TmaDesc rdesc = a;  // the output (or residual) rows of this launch, exactly m of them: the TMA unit clips the ragged last tile
  QkvRopeArgs q{};
  if (epilogue == kEpiResidual || epilogue == kEpiResidualBias) {
    // the residual rows of this launch, exactly m of them, so that the TMA unit clips the ragged last tile
    cudaError_t e = make_tma_2d_f32_box32(&rdesc, resid, (uint64_t)m, (uint64_t)n);
    if (e != cudaSuccess) return e;
  }
  if (epilogue == kEpiQkvRope) {
    if (!qa || n % 128) return cudaErrorInvalidValue;
    q = *qa;
    cudaError_t e = make_tma_2d_bf16_box32_sw64(&rdesc, out, (uint64_t)m, (uint64_t)n);
    if (e != cudaSuccess) return e;
  }
  if (epilogue == kEpiStore || epilogue == kEpiSwiGLU || epilogue == kEpiStoreBias || epilogue == kEpiGeluBias) {
    cudaError_t e = make_tma_2d_bf16(&rdesc, out, (uint64_t)m, (uint64_t)n, 32, 64);
    if (e != cudaSuccess) return e;
  }
  const CUtensorMap& mr = reinterpret_cast<const CUtensorMap&>(rdesc);
  __nv_bfloat16* o = (__nv_bfloat16*)out;
  // clusters of two CTAs along x
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = kSmemBytes;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl_for(m) ? 2 : 1;
  cudaError_t le;
  if (epilogue == kEpiStore)
    le = cudaLaunchKernelEx(&cfg, k_gemm_tc2<kEpiStore>, ma, mb0, mb1, mr, o, m, n, k, q, reverse ? 1 : 0, err, bias);
  else if (epilogue == kEpiResidual)
    le = cudaLaunchKernelEx(&cfg, k_gemm_tc2<kEpiResidual>, ma, mb0, mb1, mr, o, m, n, k, q, reverse ? 1 : 0, err, bias);
  else if (epilogue == kEpiSwiGLU)
    le = cudaLaunchKernelEx(&cfg, k_gemm_tc2<kEpiSwiGLU>, ma, mb0, mb1, mr, o, m, n, k, q, reverse ? 1 : 0, err, bias);
  else if (epilogue == kEpiQkvRope)
    le = cudaLaunchKernelEx(&cfg, k_gemm_tc2<kEpiQkvRope>, ma, mb0, mb1, mr, o, m, n, k, q, reverse ? 1 : 0, err, bias);
  else if (epilogue == kEpiStoreBias)
    le = cudaLaunchKernelEx(&cfg, k_gemm_tc2<kEpiStoreBias>, ma, mb0, mb1, mr, o, m, n, k, q, reverse ? 1 : 0, err, bias);
  else if (epilogue == kEpiGeluBias)
    le = cudaLaunchKernelEx(&cfg, k_gemm_tc2<kEpiGeluBias>, ma, mb0, mb1, mr, o, m, n, k, q, reverse ? 1 : 0, err, bias);
  else if (epilogue == kEpiResidualBias)
    le = cudaLaunchKernelEx(&cfg, k_gemm_tc2<kEpiResidualBias>, ma, mb0, mb1, mr, o, m, n, k, q, reverse ? 1 : 0, err, bias);
  else
    return cudaErrorInvalidValue;
  if (le != cudaSuccess) return le;
  return cudaGetLastError();
}

}  // namespace prism
