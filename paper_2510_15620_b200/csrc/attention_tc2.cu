// S5 on the 5th-generation tensor cores, two query heads per CTA: varlen flash attention over packed
// sequences, bf16, causal or bidirectional; head_dim 128 for grouped-query models with an even group size, head_dim 64
// for even group sizes and for one key/value head per query head (the encoder stack).
//
// A work item is (sequence, PAIR of query heads, 128-query-row block).  With an even group size the pair shares a
// key/value head: the two heads' Q tiles ("A" and "B") use the same K_j / V_j tiles (128 keys each), which are
// fetched once.  With one key/value head per query head (head_dim 64 only) a ring stage holds both heads' tiles.
// One persistent CTA per SM walks the items, heaviest query blocks first; nothing but the item's end
// separates consecutive items, so the loads and the first scores of the next item run under the tail of
// the current one.  Warp-specialised, 576 threads:
//   warp 0      TMA producer: Q_A, K_0, Q_B, then K_t and V_{t-1} alternately (K ring 2, V ring 2)
//   warp 1      the only MMA issuer: S_x = Q_x K_j^T (SS form, M128 N128 K16 x 8) and O_x += P_x V_j (TS form: P
//               is read from TENSOR MEMORY, V is an MN-major shared-memory operand), in the order
//               PV_A(g) S_A(g+1) PV_B(g) S_B(g+1): while one head's softmax runs, the other head's MMAs do
//   warps 2..9  softmax of head A, warps 10..17 softmax of head B: two threads per query row (TMEM lane), each
//               taking two of a block's four 32-key chunks: exponentials against a per-row reference that
//               is the row's score on key 0 (no row maximum on the common path; the two threads of a row
//               exchange one vote per block), P as packed bf16 back over the first 64 columns of S_x; O_x
//               stays in tensor memory and is rescaled (read-modify-write, by an exact power of two) only
//               when a row sum threatens fp32 range; at the item's end the same threads normalise O_x
//               and store it through swizzled staging rows in 64-byte pieces.
// Tensor memory: S_A, S_B, O_A, O_B, 128 columns each.  S_x(g+1) overwrites the columns P_x(g) occupies;
// it is issued after PV_x(g) by the same thread with the same instruction shape, and such MMAs execute
// in issue order.  Every mbarrier wait is bounded; on expiry the kernel records kErrTimeout, all roles
// drain to the common exit and the tensor memory is freed.  Every TMA load is a plain per-CTA load.
#include "tc_common.cuh"

namespace prism {

namespace {

using namespace tc;

constexpr int BM = 128, BN = 128;
constexpr int NK = 2, NV = 2;
constexpr int kStageBytes = 32 * 64;  // per softmax warp: 32 rows x 32 bf16 of output on their way to global memory
// One [128 x DH] tile (Q, K and V tiles alike): DH / 64 swizzled [128 x 64] sub-tiles, 32 KB at head_dim 128.
__host__ __device__ constexpr int tile_bytes(int dh) { return 128 * dh * 2; }
// kShare: the two query heads of an item read the same K / V head (a grouped-query pair), so a ring stage holds one
// tile; otherwise (one K / V head per query head) it holds the two heads' tiles side by side.
__host__ __device__ constexpr int smem_bytes(int dh, bool share) {
  return (2 + (NK + NV) * (share ? 1 : 2)) * tile_bytes(dh) + 16 * kStageBytes + 1024 /*alignment slack*/ + 512 /*barriers, flags*/;
}
static_assert(smem_bytes(128, true) <= 232448 && smem_bytes(64, false) <= 232448, "exceeds the shared memory one CTA may have");
constexpr float kBigSum = 1.2089258e24f;  // 2^80: row sums of one block beyond this move the reference
constexpr int kThreads = 576;  // TMA warp, MMA warp, 2 x 8 softmax warps
constexpr int kTmemCols = 512;

__device__ __forceinline__ float ex2(float x) {  // 2^x on the special-function unit; -inf -> 0
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// 2^x for a pair of exponents.  All softmax warps of the SM share its special-function unit, so kEmulated of
// every 8 pairs can take the FMA pipe instead: x = n + f with n = round(x) (the 1.5 * 2^23 trick leaves n in the low
// bits of t), 2^f by a cubic whose relative error (7.5e-5) is far below bf16 rounding, and n is added to the exponent
// field.  x is clamped to [-125, 126]: masked scores (-inf) come out as 2^-125 instead of 0 (every row sum is at least
// 1), and exponents beyond fp32 range still produce a sum that the range check catches.
// Measured in one call on the three benchmark shape sets: 0 of 8 -> 371 / 650 / 844 TFLOP/s, 1 -> 372 / 649 / 842,
// 2 -> 371 / 641 / 834, 3 -> 362 / 625 / 815: the special-function pipe is about 20 % busy, so taking work off it
// buys nothing and the extra instructions cost a little.  All exponentials therefore go to ex2.approx.
constexpr int kEmulated = 0;
__device__ __forceinline__ void exp2_pair(uint64_t xv, bool emulate, float& p0, float& p1) {
  float x0, x1;
  f2_unpack(xv, x0, x1);
  if (!emulate) {
    p0 = ex2(x0);
    p1 = ex2(x1);
    return;
  }
  const float kMagic = 12582912.f;
  const uint64_t xc = f2_pack(fminf(fmaxf(x0, -125.f), 126.f), fminf(fmaxf(x1, -125.f), 126.f));
  const uint64_t t = f2_add(xc, f2_pack(kMagic, kMagic));
  const uint64_t nf = f2_add(t, f2_pack(-kMagic, -kMagic));
  const uint64_t fr = f2_fma(nf, f2_pack(-1.f, -1.f), xc);
  uint64_t p = f2_fma(f2_pack(0.055171408f, 0.055171408f), fr, f2_pack(0.24261075f, 0.24261075f));
  p = f2_fma(p, fr, f2_pack(0.69326097f, 0.69326097f));
  p = f2_fma(p, fr, f2_pack(0.99992812f, 0.99992812f));
  float q0, q1, t0, t1;
  f2_unpack(p, q0, q1);
  f2_unpack(t, t0, t1);
  p0 = __uint_as_float(__float_as_uint(q0) + (__float_as_uint(t0) << 23));
  p1 = __uint_as_float(__float_as_uint(q1) + (__float_as_uint(t1) << 23));
}

__device__ __forceinline__ void tmem_ld1(uint32_t taddr, uint32_t& v) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x1.b32 {%0}, [%1];" : "=r"(v) : "r"(taddr));
}
// Work distribution.  Sequences are taken in groups of `gsz` (as many as keep their q/k/v rows well inside L2);
// candidate index i names (group, query block, sequence of the group, head pair) with the query block
// descending inside a group: a sequence's K and V rows are fetched from DRAM once and found in L2 by its
// other query blocks and head pairs, and the last items of the launch are the light ones.
// Candidates whose block lies beyond the sequence's end are skipped.  CTAs draw candidates from a device-wide
// counter (the items differ in cost by the number of key blocks, and a fixed assignment leaves a quarter of
// the SMs idle at the end).  The producer thread draws, and publishes each item through a small ring in
// shared memory to the other roles, which read the ring in order.
struct ItemRec {
  int qb, pair, beg, len, n_blocks;  // n_blocks == 0: no more items
  int first;                         // the launch's first sequence (it stores the rows of a shared prefix)
};
constexpr int NI = 4;  // ring depth

struct ItemReader {
  volatile ItemRec* ring;
  uint32_t b_full, b_empty, n;
  int qb, pair, beg, len, n_blocks, first;  // the current item
  __device__ __forceinline__ void init(ItemRec* ring_, uint32_t b_full_, uint32_t b_empty_) {
    ring = ring_, b_full = b_full_, b_empty = b_empty_, n = 0;
    n_blocks = 0;
  }
  // Moves to the next item; false at the end of the work or when the wait gave up.
  __device__ __forceinline__ bool next(int* err, volatile int* abort_flag) {
    const uint32_t slot = n % NI;
    if (!mbar_wait(b_full + 8 * slot, (n / NI) & 1, err, abort_flag)) return false;
    qb = ring[slot].qb, pair = ring[slot].pair, beg = ring[slot].beg, len = ring[slot].len;
    n_blocks = ring[slot].n_blocks;
    first = ring[slot].first;
    return n_blocks > 0;
  }
  // The caller (one thread per arriving party) is done with the current item's record.
  __device__ __forceinline__ void release() { mbar_arrive(b_empty + 8 * (n % NI)); }
  __device__ __forceinline__ void advance() { ++n; }
};

template <int DH, bool kShare>
__global__ void __launch_bounds__(kThreads, 1)
k_attention_tc2(const __grid_constant__ CUtensorMap map_qkv, const __grid_constant__ CUtensorMap map_pre,
                const __grid_constant__ CUtensorMap map_rest, __nv_bfloat16* __restrict__ out,
                const int* __restrict__ cu, int seq0, int nseq, int row0, int nqb, int gsz, int hq, int hkv,
                int causal, int reverse, int prefix, int write_prefix, float scale_log2, int* __restrict__ sched,
                int* __restrict__ err) {
  extern __shared__ unsigned char smem_raw[];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  unsigned char* gen = smem_raw + (base - raw);
  constexpr int kTile = tile_bytes(DH), kSub = DH / 64;   // bytes per tile, [128 x 64] sub-tiles per tile
  constexpr int kStage = (kShare ? 1 : 2) * kTile;         // one K (or V) ring stage
  const uint32_t s_q = base, s_k = base + 2 * kTile, s_v = s_k + NK * kStage, s_o = s_v + NV * kStage;
  uint64_t* bars = reinterpret_cast<uint64_t*>(gen + 2 * kTile + (NK + NV) * kStage + 16 * kStageBytes);
  // q_full[2], q_empty[2], k_full[2], k_empty[2], v_full[2], v_empty[2], s_full[2], p_full[2], o_full[2]
  const uint32_t b_q_full = smem_u32(bars), b_q_empty = smem_u32(bars + 2);
  const uint32_t b_k_full = smem_u32(bars + 4), b_k_empty = smem_u32(bars + 6);
  const uint32_t b_v_full = smem_u32(bars + 8), b_v_empty = smem_u32(bars + 10);
  const uint32_t b_s_full = smem_u32(bars + 12), b_p_full = smem_u32(bars + 14), b_o_full = smem_u32(bars + 16);
  // pair[8]: one barrier per (head, lane quarter), arrived on by the two softmax warps that share those rows;
  // votes[8][3]: what they vote on, three slots in rotation
  const uint32_t b_pair = smem_u32(bars + 18);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 26);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  uint32_t* votes = tmem_slot + 2;
  // item_full[NI] (the producer), item_empty[NI] (the MMA thread and the 16 softmax warps), the ring itself
  const uint32_t b_item_full = smem_u32(votes + 24), b_item_empty = b_item_full + 8 * NI;
  ItemRec* ring = reinterpret_cast<ItemRec*>(votes + 24 + 4 * NI);
  static_assert(26 * 8 + 8 + 24 * 4 + 2 * NI * 8 + NI * sizeof(ItemRec) <= 512, "barrier area too small");

  if (threadIdx.x == 0) {
    for (int i = 0; i < 14; ++i) mbar_init(b_q_full + 8 * i, 1);  // everything up to s_full: one arrival
    for (int i = 0; i < 2; ++i) {
      mbar_init(b_p_full + 8 * i, 8);  // the eight warps of a head's softmax group
      mbar_init(b_o_full + 8 * i, 1);
    }
    for (int i = 0; i < 8; ++i) mbar_init(b_pair + 8 * i, 2);
    for (int i = 0; i < 24; ++i) votes[i] = 0;
    for (int i = 0; i < NI; ++i) {
      mbar_init(b_item_full + 8 * i, 1);
      mbar_init(b_item_empty + 8 * i, 17);
    }
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
  pdl_sync();  // set-up done: the kernel before this one (it may still own the work counters) has to be complete
  const uint32_t tmem = *tmem_slot;
  const int group = hq / hkv, npairs = hq / 2;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      ItemRec it;
      const int per_qb = gsz * npairs, per_group = nqb * per_qb;
      const int total = ((nseq + gsz - 1) / gsz) * per_group;
      uint32_t kc = 0, vc = 0, ic = 0;  // K tiles, V tiles, items issued so far
      bool ok = true;
      while (ok) {
        // draw candidates until one is a real item
        it.n_blocks = 0;
        for (int i = atomicAdd(sched, 1); i < total; i = atomicAdd(sched, 1)) {
          const int n_groups = (nseq + gsz - 1) / gsz, grp = reverse ? n_groups - 1 - i / per_group : i / per_group;
          const int in_group = i % per_group, rem = in_group % per_qb, sl = grp * gsz + rem / npairs;
          if (sl >= nseq) continue;
          const int s = seq0 + sl;
          it.qb = nqb - 1 - in_group / per_qb;
          it.pair = rem % npairs;
          // Shared query prefix: rows 0 .. prefix-1 of the batch belong to every sequence, cu[s] is the first row
          // of the sequence's own part.  Row v of the sequence is batch row v (v < prefix) or beg + v - prefix.
          const int b = __ldg(cu + s);
          const int own = __ldg(cu + s + 1) - b;
          it.len = prefix + own;
          if (it.qb * BM >= it.len) continue;
          // a sequence without rows of its own (an empty document, or another rank's candidate) needs no item:
          // the prefix rows it would compute are the ones the launch's first sequence writes
          if (prefix > 0 && own == 0 && !(write_prefix && sl == 0)) continue;
          it.beg = b - row0;
          it.first = write_prefix && sl == 0;
          const int kv_end = causal ? min(it.len, (it.qb + 1) * BM) : it.len;
          it.n_blocks = (kv_end + BN - 1) / BN;
          break;
        }
        // publish it (or the end marker) once every reader has left the slot's previous record
        const uint32_t slot = ic % NI;
        if (!mbar_wait(b_item_empty + 8 * slot, ((ic / NI) & 1) ^ 1, err, abort_flag)) break;
        ring[slot] = it;
        mbar_arrive(b_item_full + 8 * slot);
        if (it.n_blocks == 0) break;
        const int h0 = it.pair * 2;
        // 128 rows of the sequence starting at row 128 * blk, columns col .. col + 127, as two 64-column
        // sub-tiles.  The block that holds a shared prefix is put together from two row ranges (prefix rows, then
        // the sequence's own first 128 - prefix rows; prefix is a multiple of 8, so the second part starts on a
        // swizzle-atom boundary); the boxes add up to a full tile, so the byte count is the same.
        auto load_tile = [&](uint32_t dst, int col, int blk, uint32_t bar) {
          if (prefix > 0 && blk == 0) {
#pragma unroll
            for (int sb = 0; sb < kSub; ++sb) {
              tma_load_2d(dst + sb * (128 * 128), &map_pre, col + 64 * sb, 0, bar);
              tma_load_2d(dst + sb * (128 * 128) + prefix * 128, &map_rest, col + 64 * sb, it.beg, bar);
            }
          } else {
            const int row = it.beg + blk * 128 - prefix;
#pragma unroll
            for (int sb = 0; sb < kSub; ++sb) tma_load_2d(dst + sb * (128 * 128), &map_qkv, col + 64 * sb, row, bar);
          }
        };
        auto load_q = [&](int x) {
          if (!mbar_wait(b_q_empty + 8 * x, (ic & 1) ^ 1, err, abort_flag)) return false;
          mbar_expect_tx(b_q_full + 8 * x, kTile);
          load_tile(s_q + x * kTile, (h0 + x) * DH, it.qb, b_q_full + 8 * x);
          return true;
        };
        // K (first = hq) or V (first = hq + hkv) of key block t into the next stage of its ring: one tile for a pair that
        // shares its K / V head, else one tile per head, under one barrier
        auto load_kv = [&](int first, int t, uint32_t ring, uint32_t b_full, uint32_t b_empty, uint32_t& cnt, int depth) {
          const uint32_t st = cnt % depth, u = cnt / depth;
          if (!mbar_wait(b_empty + 8 * st, (u & 1) ^ 1, err, abort_flag)) return false;
          mbar_expect_tx(b_full + 8 * st, kStage);
          load_tile(ring + st * kStage, (first + h0 / group) * DH, t, b_full + 8 * st);
          if (!kShare) load_tile(ring + st * kStage + kTile, (first + (h0 + 1) / group) * DH, t, b_full + 8 * st);
          ++cnt;
          return true;
        };
        const int kcol = hq, vcol = hq + hkv;
        ok = load_q(0) && load_kv(kcol, 0, s_k, b_k_full, b_k_empty, kc, NK) && load_q(1);
        for (int t = 1; ok && t <= it.n_blocks; ++t) {
          if (t < it.n_blocks) ok = load_kv(kcol, t, s_k, b_k_full, b_k_empty, kc, NK);
          if (ok) ok = load_kv(vcol, t - 1, s_v, b_v_full, b_v_empty, vc, NV);
        }
        ++ic;
      }
      // The CTA that checks out last rearms the counter for the next launch that is given it.
      __threadfence();
      if (atomicAdd(sched + 1, 1) == (int)gridDim.x - 1) {
        atomicExch(sched, 0);
        atomicExch(sched + 1, 0);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t kIdescS = idesc_bf16(BM, BN, 0), kIdescO = idesc_bf16(BM, DH, 1);
      constexpr int kDepthSteps = DH / 16;  // MMA steps over head_dim for the scores
      ItemReader its, itp;  // the block whose scores are issued next; the block whose P V is issued next
      its.init(ring, b_item_full, b_item_empty);
      itp.init(ring, b_item_full, b_item_empty);
      bool s_has = its.next(err, abort_flag), p_has = itp.next(err, abort_flag);
      int sj = 0, pj = 0;                // block index inside its / itp
      uint32_t sic = 0;                  // items started on the score side
      uint32_t kc = 0, vc = 0, pc = 0;   // K tiles consumed, V tiles consumed, blocks whose P V has been issued
      bool ok = true;
      // S_x of block (its, sj).  x = 1 also releases the K tile and moves the score cursor on.
      auto issue_s = [&](int x) {
        const uint32_t st = kc % NK;
        if (sj == 0 && !mbar_wait(b_q_full + 8 * x, sic & 1, err, abort_flag)) return false;
        if (x == 0 && !mbar_wait(b_k_full + 8 * st, (kc / NK) & 1, err, abort_flag)) return false;
        tc_fence_after();
        const uint32_t sq = s_q + x * kTile, sk = s_k + st * kStage + (kShare ? 0 : x * kTile);
#pragma unroll
        for (int kk = 0; kk < kDepthSteps; ++kk) {  // 16 head-dim elements per step; the sub-tile switches at kk = 4
          const uint64_t da = smem_desc(sq + (kk >> 2) * (128 * 128) + (kk & 3) * 32, 16, 1024);
          const uint64_t db = smem_desc(sk + (kk >> 2) * (128 * 128) + (kk & 3) * 32, 16, 1024);
          umma_bf16(tmem + x * BN, da, db, kIdescS, kk != 0);
        }
        umma_commit(b_s_full + 8 * x);
        if (sj == its.n_blocks - 1) umma_commit(b_q_empty + 8 * x);  // the item's last use of Q_x
        if (x == 1) {
          umma_commit(b_k_empty + 8 * st);
          ++kc;
          if (++sj == its.n_blocks) {
            sj = 0;
            ++sic;
            its.advance();
            s_has = its.next(err, abort_flag);
          }
        }
        return true;
      };
      auto issue_pv = [&](int x) {
        const uint32_t st = vc % NV;
        if (!mbar_wait(b_p_full + 8 * x, pc & 1, err, abort_flag)) return false;
        if (x == 0 && !mbar_wait(b_v_full + 8 * st, (vc / NV) & 1, err, abort_flag)) return false;
        tc_fence_after();
        const uint32_t sv = s_v + st * kStage + (kShare ? 0 : x * kTile);
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) {  // 16 keys per step: 8 packed columns of P, 16 rows of V
          const uint64_t db = smem_desc(sv + kk * 2048, 128 * 128, 1024);  // V: MN-major, DH / 64 dh atoms of 64
          umma_bf16_ts(tmem + 2 * BN + x * DH, tmem + x * BN + kk * 8, db, kIdescO, (pj | kk) != 0);
        }
        umma_commit(b_o_full + 8 * x);
        if (x == 1) umma_commit(b_v_empty + 8 * st);
        return true;
      };
      if (s_has) ok = issue_s(0) && issue_s(1);
      while (ok && p_has) {
        ok = issue_pv(0);
        if (ok && s_has) ok = issue_s(0);
        if (ok) ok = issue_pv(1);
        if (ok && s_has) ok = issue_s(1);
        ++vc;
        ++pc;
        if (++pj == itp.n_blocks) {
          pj = 0;
          itp.release();  // the score cursor is past this item too
          itp.advance();
          p_has = itp.next(err, abort_flag);
        }
      }
    }
  } else {
    // ------------------------------------------------------------------ softmax + output, two threads per query row
    const int x = (warp - 2) >> 3;        // head A or B of the pair
    const int hf = ((warp - 2) >> 2) & 1; // which chunks of a block / which 64 output columns this thread takes
    const int quarter = warp & 3;         // the TMEM lane quarter this warp may access
    const int r = quarter * 32 + lane;    // row inside the tile = TMEM lane
    const uint32_t lane_base = (uint32_t)(quarter * 32) << 16;
    const uint32_t t_s = tmem + lane_base + x * BN, t_o = tmem + lane_base + 2 * BN + x * DH + hf * (DH / 2);
    const uint32_t bar_s = b_s_full + 8 * x, bar_p = b_p_full + 8 * x, bar_o = b_o_full + 8 * x;
    // Meeting point of the two warps that share these 32 rows: an mbarrier with two arrivals (bounded wait, like
    // every other wait here) that also carries a vote.  Slot (u + 1) % 3 is cleared before the arrival at
    // meeting u: both warps read it after meeting u - 2 and before arriving at u - 1, and nobody writes it
    // before passing u.  Returns -1 if the wait gave up, else whether any of the 64 threads voted yes.
    const uint32_t pair_mb = b_pair + 8 * (x * 4 + quarter);
    volatile uint32_t* my_votes = votes + 3 * (x * 4 + quarter);
    uint32_t meet = 0;
    auto pair_meet = [&](bool flag) -> int {
      __syncwarp();  // the other lanes' shared-memory writes precede lane 0's arrival
      const bool any = __any_sync(0xffffffffu, flag);
      if (lane == 0) {
        if (hf == 0) my_votes[(meet + 1) % 3] = 0;
        if (any) my_votes[meet % 3] = 1;
        mbar_arrive(pair_mb);
      }
      if (!mbar_wait(pair_mb, meet & 1, err, abort_flag)) return -1;
      const int v = (int)my_votes[meet % 3];
      ++meet;
      return v;
    };
    const uint32_t stg = s_o + (uint32_t)(warp - 2) * kStageBytes;          // this warp's staging rows
    const uint32_t stg_other = s_o + (uint32_t)((warp - 2) ^ 4) * kStageBytes;  // the partner warp's
    const int c0 = hf, c1 = hf + 2;       // this thread's two 32-key chunks of every block
    ItemReader it;
    it.init(ring, b_item_full, b_item_empty);
    uint32_t gc = 0;  // blocks of this head handled so far (phase counter of s_full / p_full / o_full)
    bool ok = true;
    while (ok && it.next(err, abort_flag)) {
      const int qrow = it.qb * BM + r;
      // p = 2^(s * scale_log2 - ms).  The reference ms is NOT the running maximum: it starts as the row's score
      // against key 0 of the sequence (visible to every row, so the row sum is at least 1) and moves, by a
      // whole number of powers of two, only when a row sum leaves the range fp32 holds comfortably.  bf16
      // probabilities and fp32 sums keep their relative precision at any magnitude, so the common path needs
      // no row maximum and the two threads of a row exchange nothing but one vote per block.
      float ms = 0.f, l = 0.f;  // l: this thread's part of the row sum
      for (int j = 0; j < it.n_blocks; ++j, ++gc) {
        if (!mbar_wait(bar_s, gc & 1, err, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const bool diag = causal && j == it.qb;         // BN == BM: only the diagonal block is cut by causality
        const bool tail = j * BN + BN > it.len;         // keys beyond the sequence's end
        uint32_t sa[32], pk[32];
        tmem_ld32(t_s + c0 * 32, sa);
        if (j == 0) {
          uint32_t s00;
          tmem_ld1(t_s, s00);
          tmem_ld_wait();
          ms = __uint_as_float(s00) * scale_log2;
        } else {
          tmem_ld_wait();
        }
        const uint64_t sc2 = f2_pack(scale_log2, scale_log2);
        uint64_t rs2;
        // exponentials of one 32-key chunk into 16 packed bf16 pairs (key 2c in the low half) and the row sum
        auto chunk = [&](int ch, uint32_t* cur, uint32_t* out16) {
          if ((diag && ch > quarter) || j * BN + ch * 32 >= it.len) {  // beyond every row of this warp, or beyond the end
#pragma unroll
            for (int c = 0; c < 16; ++c) out16[c] = 0u;
            return;
          }
          if ((diag && ch == quarter) || tail) {
#pragma unroll
            for (int c = 0; c < 32; ++c) {
              const int key = j * BN + ch * 32 + c;
              if (key >= it.len || (causal && key > qrow)) cur[c] = 0xff800000u;  // -inf
            }
          }
          const uint64_t nm2 = f2_pack(-ms, -ms);
#pragma unroll
          for (int c = 0; c < 16; ++c) {
            float p0, p1;
            exp2_pair(f2_fma(f2_pack(__uint_as_float(cur[2 * c]), __uint_as_float(cur[2 * c + 1])), sc2, nm2),
                      (c & 7) < kEmulated, p0, p1);
            rs2 = f2_add(rs2, f2_pack(p0, p1));
            out16[c] = pack_bf16(p0, p1);
          }
        };
        rs2 = f2_pack(0.f, 0.f);
        chunk(c0, sa, pk);
        tmem_ld32(t_s + c1 * 32, sa);
        tmem_ld_wait();
        chunk(c1, sa, pk + 16);
        float rlo, rhi;
        f2_unpack(rs2, rlo, rhi);
        float rs = rlo + rhi;
        // One barrier of the row's two warps per block.  It carries the vote "some row sum is out of range", and
        // it orders the P stores below after BOTH threads' score loads: P chunks overwrite score columns of the
        // other thread's chunks.
        const int vote = pair_meet(!(rs <= kBigSum));
        if (vote < 0) { ok = false; break; }
        if (vote) {
          // Rare: rows whose largest exponent is beyond 2^64 move their reference up by d = ceil(that exponent)
          // powers of two; what was accumulated under the old reference is scaled by 2^-d (exact).  Nothing of
          // this block has been stored yet, so the scores are still in tensor memory.
          float xmax = -INFINITY;
#pragma unroll 1
          for (int w = 0; w < 2; ++w) {
            const int ch = w ? c1 : c0;
            tmem_ld32(t_s + ch * 32, sa);
            tmem_ld_wait();
#pragma unroll
            for (int c = 0; c < 32; ++c) {
              const int key = j * BN + ch * 32 + c;
              if (!(key >= it.len || (causal && key > qrow)))
                xmax = fmaxf(xmax, fmaf(__uint_as_float(sa[c]), scale_log2, -ms));
            }
          }
          asm volatile("st.shared.f32 [%0], %1;" ::"r"(stg + lane * 4), "f"(xmax) : "memory");
          if (pair_meet(false) < 0) { ok = false; break; }
          float xo;
          asm volatile("ld.shared.f32 %0, [%1];" : "=f"(xo) : "r"(stg_other + lane * 4) : "memory");
          xmax = fmaxf(xmax, xo);
          const float d = xmax > 64.f ? ceilf(xmax) : 0.f;
          const float f = exp2f(-d);
          if (j > 0) {
            if (!mbar_wait(bar_o, (gc - 1) & 1, err, abort_flag)) { ok = false; break; }  // complete already
            tc_fence_after();
#pragma unroll 1
            for (int c = 0; c < DH / 64; ++c) {  // this thread's DH / 2 columns of O
              uint32_t o[32];
              tmem_ld32(t_o + c * 32, o);
              tmem_ld_wait();
#pragma unroll
              for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * f);
              tmem_st32(t_o + c * 32, o);
            }
          }
          l *= f;
          ms += d;
          rs2 = f2_pack(0.f, 0.f);
          tmem_ld32(t_s + c0 * 32, sa);
          tmem_ld_wait();
          chunk(c0, sa, pk);
          tmem_ld32(t_s + c1 * 32, sa);
          tmem_ld_wait();
          chunk(c1, sa, pk + 16);
          f2_unpack(rs2, rlo, rhi);
          rs = rlo + rhi;
          // the partner, too, has re-read its scores (and this thread's xmax slot) before P overwrites them
          if (pair_meet(false) < 0) { ok = false; break; }
        }
        l += rs;
        tmem_st16(t_s + c0 * 16, pk);
        tmem_st16(t_s + c1 * 16, pk + 16);
        tmem_st_wait();
        tc_fence_before();
        // No wait is needed to keep the barrier phases apart.  The scores of block gc were issued after the
        // wait for p_full(gc - 1), so that phase is over before any warp gets here; and s_full(gc), which this
        // thread has observed, completes only after every earlier MMA of this head, so o_full stands at phase
        // gc - 1 exactly until this thread's arrival below lets P V(gc) be issued.
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_p);  // one arrival per warp
      }
      if (!ok) break;
      if (!mbar_wait(bar_o, (gc - 1) & 1, err, abort_flag)) { ok = false; break; }
      tc_fence_after();
      // the row sum is the sum of the two threads' parts
      asm volatile("st.shared.f32 [%0], %1;" ::"r"(stg + lane * 4), "f"(l) : "memory");
      if (pair_meet(false) < 0) { ok = false; break; }
      float lo;
      asm volatile("ld.shared.f32 %0, [%1];" : "=f"(lo) : "r"(stg_other + lane * 4) : "memory");
      if (pair_meet(false) < 0) { ok = false; break; }  // read before either warp stages output there
      const float inv = 1.f / (l + lo);
      // This thread's 64 columns of O_x / l as bf16, 32 columns at a time through the warp's staging rows
      // (64 bytes each, 16-byte chunks XOR-swizzled), so that global stores are 64 contiguous bytes per row.
      const int row_w = it.qb * BM + quarter * 32;  // first row of this warp inside the sequence
      __nv_bfloat16* ocol = out + (size_t)(it.pair * 2 + x) * DH + hf * (DH / 2);
#pragma unroll 1
      for (int part = 0; part < DH / 64; ++part) {
        uint32_t o[32];
        tmem_ld32(t_o + part * 32, o);
        tmem_ld_wait();
#pragma unroll
        for (int v = 0; v < 4; ++v) {
          const uint32_t dst = stg + lane * 64 + ((v ^ ((lane >> 1) & 3)) << 4);
          asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst),
                       "r"(pack_bf16(__uint_as_float(o[v * 8 + 0]) * inv, __uint_as_float(o[v * 8 + 1]) * inv)),
                       "r"(pack_bf16(__uint_as_float(o[v * 8 + 2]) * inv, __uint_as_float(o[v * 8 + 3]) * inv)),
                       "r"(pack_bf16(__uint_as_float(o[v * 8 + 4]) * inv, __uint_as_float(o[v * 8 + 5]) * inv)),
                       "r"(pack_bf16(__uint_as_float(o[v * 8 + 6]) * inv, __uint_as_float(o[v * 8 + 7]) * inv))
                       : "memory");
        }
        __syncwarp();
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int rr = i * 8 + (lane >> 2), chn = lane & 3;
          uint4 val;
          asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];"
                       : "=r"(val.x), "=r"(val.y), "=r"(val.z), "=r"(val.w)
                       : "r"(stg + rr * 64 + ((chn ^ ((rr >> 1) & 3)) << 4)));
          // row v of the sequence: its own row beg + v - prefix, or row v of the shared prefix, which only the
          // launch's first sequence writes (every sequence computes the same values for it)
          const int v = row_w + rr;
          if (v < it.len && (v >= prefix || it.first)) {
            const size_t prow = v < prefix ? (size_t)v : (size_t)(it.beg + v - prefix);
            *reinterpret_cast<uint4*>(ocol + prow * ((size_t)hq * DH) + part * 32 + chn * 8) = val;
          }
        }
        __syncwarp();
      }
      // The next item's first P V (which overwrites O_x) is issued only after this thread's arrival for that
      // block, which follows these loads in program order.
      tc_fence_before();
      __syncwarp();
      if (lane == 0) it.release();
      it.advance();
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

namespace {
// Work counters {next candidate, CTAs checked out}, one pair per launch in flight; a launch takes the next
// pair in rotation and leaves it zeroed.  Zero-initialised at module load.
constexpr int kTickets = 1024;
__device__ int g_sched[kTickets][2];
}  // namespace

cudaError_t launch_attention_tc2(const void* qkv, void* out, const int* cu, int seq0, int nseq, int row0, int rows,
                                 int max_len, int n_q_heads, int n_kv_heads, int causal, int* err, cudaStream_t st,
                                 bool reverse, int prefix, const void* qkv_prefix, bool write_prefix, int head_dim) {
  if (nseq <= 0 || max_len <= 0 || rows <= 0) return cudaSuccess;
  if (n_kv_heads < 1 || n_q_heads % n_kv_heads || (n_q_heads & 1)) return cudaErrorInvalidValue;
  // Pairs of query heads: with an even group size both heads of a pair read one K / V head (tiles shared); with one
  // K / V head per query head (head_dim 64 only: two tiles per stage fit) each head of the pair reads its own.
  const int group = n_q_heads / n_kv_heads;
  const bool share = (group & 1) == 0;
  if (!share && group != 1) return cudaErrorInvalidValue;
  if (!(head_dim == 128 && share) && head_dim != 64) return cudaErrorInvalidValue;
  const int DH = head_dim;
  const int kSmemBytes = smem_bytes(DH, share);
  static std::atomic<unsigned long long> smem_set[3];
  {
    cudaError_t e = DH == 128 ? ensure_dynamic_smem(k_attention_tc2<128, true>, kSmemBytes, smem_set[0])
                    : share   ? ensure_dynamic_smem(k_attention_tc2<64, true>, kSmemBytes, smem_set[1])
                              : ensure_dynamic_smem(k_attention_tc2<64, false>, kSmemBytes, smem_set[2]);
    if (e != cudaSuccess) return e;
  }
  // Exactly `rows` rows are described, so tiles that run past the batch read zeros, never stale memory.
  const uint64_t ld = (uint64_t)(n_q_heads + 2 * n_kv_heads) * DH;
  TmaDesc mq, mpre, mrest;
  cudaError_t e = make_tma_2d_bf16(&mq, qkv, (uint64_t)rows, ld, 128, 64);
  if (e != cudaSuccess) return e;
  mpre = mq;
  mrest = mq;
  if (prefix) {
    // shared query prefix: max_len counts prefix + own rows; the first block of every tile is two boxes
    // qkv_prefix: the q/k/v rows of the prefix (row 0 of that buffer is prefix row 0); null: they are the first rows
    // of qkv.  write_prefix: this launch's first sequence stores the prefix rows of the output (rows 0.. of out).
    if (prefix < 8 || prefix > 120 || (prefix & 7) || !causal) return cudaErrorInvalidValue;
    if (!qkv_prefix && row0 != 0) return cudaErrorInvalidValue;
    e = qkv_prefix ? make_tma_2d_bf16(&mpre, qkv_prefix, (uint64_t)prefix, ld, (uint32_t)prefix, 64)
                   : make_tma_2d_bf16(&mpre, qkv, (uint64_t)rows, ld, (uint32_t)prefix, 64);
    if (e == cudaSuccess) e = make_tma_2d_bf16(&mrest, qkv, (uint64_t)rows, ld, (uint32_t)(128 - prefix), 64);
    if (e != cudaSuccess) return e;
  }
  const int nqb = (max_len + BM - 1) / BM;
  // sequences per scheduling group: their q/k/v rows (at most max_len each) stay within 48 MB
  const long long seq_bytes = (long long)nqb * BM * (long long)ld * 2;
  int gsz = (int)((48ll << 20) / seq_bytes);
  gsz = gsz < 1 ? 1 : (gsz > nseq ? nseq : gsz);
  const long long total = (long long)((nseq + gsz - 1) / gsz) * gsz * nqb * (n_q_heads / 2);
  if (total > 0x7fffffffLL) return cudaErrorInvalidValue;
  const int sms = gemm_tc_sm_count();
  const int grid = (int)(total < sms ? total : sms);
  static std::atomic<unsigned> ticket{0};
  static std::atomic<int*> sched_base[64];  // per device
  int dev = 0;
  if (cudaError_t e2 = cudaGetDevice(&dev)) return e2;
  if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  int* sb = sched_base[dev].load(std::memory_order_acquire);
  if (!sb) {
    void* p = nullptr;
    if (cudaError_t e2 = cudaGetSymbolAddress(&p, g_sched)) return e2;
    sb = static_cast<int*>(p);
    sched_base[dev].store(sb, std::memory_order_release);
  }
  int* sched = sb + 2 * (ticket.fetch_add(1, std::memory_order_relaxed) % kTickets);
  const float scale_log2 = 1.4426950408889634f / sqrtf((float)DH);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = kSmemBytes;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl_for(rows) ? 1 : 0;
  const CUtensorMap& m0 = reinterpret_cast<const CUtensorMap&>(mq);
  const CUtensorMap& m1 = reinterpret_cast<const CUtensorMap&>(mpre);
  const CUtensorMap& m2 = reinterpret_cast<const CUtensorMap&>(mrest);
#define PRISM_ATTN2(D, S)                                                                                             \
  cudaLaunchKernelEx(&cfg, k_attention_tc2<D, S>, m0, m1, m2, (__nv_bfloat16*)out, cu, seq0, nseq, row0, nqb, gsz,    \
                     n_q_heads, n_kv_heads, causal, reverse ? 1 : 0, prefix, write_prefix ? 1 : 0, scale_log2, sched, err)
  const cudaError_t le = DH == 128 ? PRISM_ATTN2(128, true) : share ? PRISM_ATTN2(64, true) : PRISM_ATTN2(64, false);
#undef PRISM_ATTN2
  if (le != cudaSuccess) return le;
  return cudaGetLastError();
}

}  // namespace prism
