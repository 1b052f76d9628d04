// S11/S13: rank, dispersion (CV), optimal 1-D clustering, three-way routing, survivor offsets and
// the final top-K, for one scored layer.  One thread block decides; n <= 4096 candidates.  From 512 candidates on
// the block is the first of a cluster of eight whose other blocks only help with the quadratic part, the rows of
// the clustering's cost table (one warp per row, rows dealt round-robin over all warps of the cluster).
//
// The decision arithmetic is fp64 on fp32 scores in a fixed left-to-right order with explicitly
// rounded operations (no FMA contraction), so that the integer outcome (cuts, survivor set, new
// offsets, top-K order) is a pure function of the scores.
#include "../../include/prism_ops.h"
#include "common.cuh"

namespace prism {

namespace {

constexpr int kThreads = 1024;

struct Shared {
  float score[kMaxCandidates];
  int id[kMaxCandidates];
  int rank[kMaxCandidates];
  float by_rank[kMaxCandidates];  // the scores in rank order (read by the sequential fp64 sums)
  int warp_a[32], warp_b[32];
  int carry_a, carry_b;
  int lo_keep, hi_keep;  // ranks [lo_keep, hi_keep) survive
  int n_cuts;
  int cuts[kMaxClusters];
  int k_eff;
  int do_cluster;
  int n_owned;      // active candidates this rank runs (candidate-sharded runs with a shared prefix)
  int n_owned_new;  // the same among the survivors
};

// Inclusive warp scan.
__device__ __forceinline__ int warp_scan(int v, int lane) {
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    int u = __shfl_up_sync(0xffffffffu, v, o);
    if (lane >= o) v += u;
  }
  return v;
}

__device__ __forceinline__ double dsub(double a, double b) { return __dsub_rn(a, b); }
__device__ __forceinline__ double dadd(double a, double b) { return __dadd_rn(a, b); }
__device__ __forceinline__ double dmul(double a, double b) { return __dmul_rn(a, b); }
__device__ __forceinline__ double ddiv(double a, double b) { return __ddiv_rn(a, b); }

// Sum of squared deviations of ranks [i, j) from their mean, from centred prefix sums.
__device__ __forceinline__ double group_cost(const double* p1, const double* p2, int i, int j) {
  const double s1 = dsub(p1[j], p1[i]);
  const double s2 = dsub(p2[j], p2[i]);
  return dsub(s2, ddiv(dmul(s1, s1), (double)(j - i)));
}

__device__ __forceinline__ uint32_t cluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}

// Row c of the cost table: D[c][j] = min over i of D[c-1][i] + cost(i, j), the smallest such i in arg.  One warp per
// j; the lanes stride over i and keep their first strict minimum, the warp takes the smallest (cost, i) pair, which
// is the i a left-to-right scan with `<` would keep.
__device__ __forceinline__ void dp_row(int c, int n, const double* __restrict__ p1, const double* __restrict__ p2,
                                       const int* __restrict__ valid, const double* __restrict__ dprev,
                                       double* __restrict__ dcur, int* __restrict__ arg_row, int warp_id, int n_warps,
                                       int lane) {
  const double inf = __longlong_as_double(0x7ff0000000000000LL);
  for (int j = warp_id; j <= n; j += n_warps) {
    double best = inf;
    int bi = 0;
    if (j >= c && valid[j]) {
      for (int i = c - 1 + lane; i < j; i += 32) {
        const double dp = dprev[i];
        if (dp == inf) continue;
        const double tot = dadd(dp, group_cost(p1, p2, i, j));
        if (tot < best) { best = tot; bi = i; }
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        const double ob = __shfl_xor_sync(0xffffffffu, best, o);
        const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
        if (ob < best || (ob == best && ob != inf && oi < bi)) { best = ob; bi = oi; }
      }
      if (best == inf) bi = 0;
    }
    if (lane == 0) {
      dcur[j] = best;
      arg_row[j] = bi;
    }
  }
}

__global__ void __launch_bounds__(kThreads) k_route(const float* __restrict__ scores, const int* __restrict__ cu_old,
                                                    const int* __restrict__ seq2orig_old, int n, RouteParams p,
                                                    int* __restrict__ cu_new, int* __restrict__ seq2orig_new,
                                                    int* __restrict__ old_of_new, RouteState* __restrict__ state,
                                                    int* __restrict__ res_idx, float* __restrict__ res_score,
                                                    ProbeRecordDev* __restrict__ rec, float* __restrict__ trace_scores,
                                                    int* __restrict__ trace_ids, unsigned char* __restrict__ scratch,
                                                    int n_cta) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  Shared& sh = *reinterpret_cast<Shared*>(smem_raw);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int crank = n_cta > 1 ? (int)cluster_rank() : 0;
  const int n_warps = n_cta * (kThreads / 32), warp_id = warp * n_cta + crank;  // rows dealt round-robin over the cluster
  const int np1 = n + 1;
  double* p1 = reinterpret_cast<double*>(scratch);
  double* p2 = p1 + np1;
  double* dbuf0 = p2 + np1;
  double* dbuf1 = dbuf0 + np1;
  int* arg = reinterpret_cast<int*>(dbuf1 + np1);  // [kMaxClusters][np1]
  int* valid = arg + (size_t)kMaxClusters * np1;   // [np1]
  int* sorted = valid + np1;                       // [np1] batch position of each rank
  volatile int* flags = sorted + np1;              // [2] in the scratch's tail: cluster? and with how many groups

  int* rank_g = arg + (size_t)(kMaxClusters - 1) * np1;  // the table's last row is never a cost-table row (c - 2 <= 6)

  // Every block of the cluster holds the scores and ids; the deciding block also records them for the trace.
  for (int i = tid; i < n; i += kThreads) {
    const float raw = scores[i];
    sh.score[i] = (raw != raw) ? -INFINITY : raw;  // a NaN score ranks last instead of breaking the order
    sh.id[i] = seq2orig_old[i];
  }
  __syncthreads();
  // ---- rank by (score descending, original index ascending); with a cluster, candidate i is ranked by block i mod 8
  for (int i = tid * n_cta + crank; i < n; i += kThreads * n_cta) {
    const float si = sh.score[i];
    const int ii = sh.id[i];
    int r = 0;
    for (int j = 0; j < n; ++j) {
      const float sj = sh.score[j];
      r += (sj > si) || (sj == si && sh.id[j] < ii);
    }
    if (n_cta > 1) rank_g[i] = r; else sh.rank[i] = r;
    sorted[r] = i;
  }
  if (n_cta > 1) {
    __syncthreads();
    cluster_sync_all();  // all ranks are written
  }

  if (crank != 0) {
    // Helper block: wait for the deciding block's verdict, then compute its share of every row of the cost table.
    cluster_sync_all();
    if (flags[0]) {
      const int k = flags[1];
      double* dprev = dbuf0;
      double* dcur = dbuf1;
      for (int c = 2; c <= k; ++c) {
        dp_row(c, n, p1, p2, valid, dprev, dcur, arg + (size_t)(c - 2) * np1, warp_id, n_warps, lane);
        cluster_sync_all();
        double* t = dprev; dprev = dcur; dcur = t;
      }
    }
    return;
  }
  bool verdict_out = false;  // has this block published flags and met the helpers?

  const int k_rem = state->k_rem;
  const int n_result = state->n_result;
  if (tid == 0) sh.n_owned = 0;
  __syncthreads();
  for (int i = tid; i < n; i += kThreads) {
    if (trace_scores) trace_scores[i] = scores[i];
    if (trace_ids) trace_ids[i] = seq2orig_old[i];
    if (n_cta > 1) sh.rank[i] = rank_g[i];
    if (p.prefix && p.owned && p.owned[sh.id[i]]) atomicAdd(&sh.n_owned, 1);
  }
  if (tid == 0) {
    sh.lo_keep = 0;
    sh.hi_keep = n;
    sh.n_cuts = 0;
    sh.do_cluster = 0;
    sh.k_eff = 1;
  }
  __syncthreads();

  for (int r = tid; r < n; r += kThreads) sh.by_rank[r] = sh.score[sorted[r]];
  __syncthreads();
  // with a shared query prefix the batch holds the prefix rows once: report query + document per sequence this
  // rank runs (all of them, unless the candidates are sharded over ranks)
  const int tokens_before = p.prefix ? (cu_old[n] - p.prefix) + (p.owned ? sh.n_owned : n) * p.prefix : cu_old[n];

  int fired = 0, n_selected = 0, n_dropped = 0, n_deferred = n, append_lo = 0, append_hi = 0;
  int k_after = k_rem, done = 0;
  double cv = 0.0;

  const bool take_all = (n <= k_rem);
  if (p.is_final || take_all) {
    // Last layer, or nothing left to decide: the best k_rem (all, if fewer) leave in rank order.
    const int cnt = n < k_rem ? n : k_rem;
    append_lo = 0;
    append_hi = cnt;
    k_after = k_rem - cnt;
    done = 1;
    if (tid == 0) { sh.lo_keep = 0; sh.hi_keep = 0; }
  } else if (p.mode == 1) {  // FIXED_KEEP
    if (p.keep_count < n) {
      fired = 1;
      n_dropped = n - p.keep_count;
      n_deferred = p.keep_count;
      if (tid == 0) { sh.lo_keep = 0; sh.hi_keep = p.keep_count; }
    }
  } else if (p.mode == 2) {  // CLUSTER
    // Sequential fp64 prefix sums over the ranked scores (thread 0): mean, then centred sums.
    if (tid == 0) {
      double acc = 0.0;
      for (int r = 0; r < n; ++r) {
        const double s = (double)sh.by_rank[r];
        acc = (r == 0) ? s : dadd(acc, s);
      }
      const double mu = ddiv(acc, (double)n);
      double a1 = 0.0, a2 = 0.0;
      p1[0] = 0.0;
      p2[0] = 0.0;
      int distinct = 1;
      valid[0] = 0;
      for (int r = 0; r < n; ++r) {
        const float sr = sh.by_rank[r];
        const double z = dsub((double)sr, mu);
        const double zz = dmul(z, z);
        a1 = (r == 0) ? z : dadd(a1, z);
        a2 = (r == 0) ? zz : dadd(a2, zz);
        p1[r + 1] = a1;
        p2[r + 1] = a2;
        if (r > 0) {
          const int v = sh.by_rank[r - 1] != sr;
          valid[r] = v;
          distinct += v;
        }
      }
      valid[n] = 1;
      const double denom = (double)(n - p.ddof);
      double c = 0.0;
      if (denom > 0.0) {
        const double sigma = __dsqrt_rn(ddiv(a2, denom));
        if (sigma == 0.0) c = 0.0;
        else if (mu == 0.0) c = __longlong_as_double(0x7ff0000000000000LL);
        else c = ddiv(sigma, fabs(mu));
      }
      sh.k_eff = distinct < p.n_clusters ? distinct : p.n_clusters;
      sh.do_cluster = (c > p.cv_threshold) && (sh.k_eff > 1);
      // stash cv where every thread can read it
      dbuf1[0] = c;
    }
    __syncthreads();
    cv = dbuf1[0];
    __syncthreads();
    if (sh.do_cluster) {
      const int k = sh.k_eff;
      const double inf = __longlong_as_double(0x7ff0000000000000LL);
      // D[1][j]
      for (int j = tid; j <= n; j += kThreads)
        dbuf0[j] = (j >= 1 && valid[j]) ? group_cost(p1, p2, 0, j) : inf;
      if (tid == 0) {
        flags[0] = 1;
        flags[1] = k;
      }
      __syncthreads();
      if (n_cta > 1) cluster_sync_all();  // the helpers see the prefix sums, the first row and the verdict
      verdict_out = true;
      double* dprev = dbuf0;
      double* dcur = dbuf1;
      for (int c = 2; c <= k; ++c) {
        dp_row(c, n, p1, p2, valid, dprev, dcur, arg + (size_t)(c - 2) * np1, warp_id, n_warps, lane);
        __syncthreads();
        if (n_cta > 1) cluster_sync_all();  // every block's rows are written before the next row reads them
        double* t = dprev; dprev = dcur; dcur = t;
      }
      if (tid == 0) {
        int j = n;
        for (int c = k; c >= 2; --c) {
          j = arg[(size_t)(c - 2) * np1 + j];
          sh.cuts[c - 2] = j;
        }
        sh.n_cuts = k - 1;
        // boundary group: bounds[g] < k_rem <= bounds[g+1]
        int lo = 0, hi = n;
        for (int g = 0; g < k; ++g) {
          const int b0 = g == 0 ? 0 : sh.cuts[g - 1];
          const int b1 = g == k - 1 ? n : sh.cuts[g];
          if (b0 < k_rem && k_rem <= b1) { lo = b0; hi = b1; break; }
        }
        sh.lo_keep = p.select_winners ? lo : 0;
        sh.hi_keep = hi;
        sh.carry_a = lo;  // group start, reused below
      }
      __syncthreads();
      fired = 1;
      const int lo = sh.carry_a, hi = sh.hi_keep;
      n_dropped = n - hi;
      if (p.select_winners) {
        n_selected = lo;
        n_deferred = hi - lo;
        append_lo = 0;
        append_hi = lo;  // selected leave now, in rank order
        k_after = k_rem - lo;
      } else {
        n_deferred = hi;
      }
    }
  }
  __syncthreads();
  if (n_cta > 1 && !verdict_out) {  // nothing to cluster: release the helpers
    if (tid == 0) flags[0] = 0;
    __syncthreads();
    cluster_sync_all();
  }

  // ranks [lo_keep, hi_keep) survive; clamped so that no argument can make the survivor count negative
  const int lo_keep = min(max(sh.lo_keep, 0), n), hi_keep = min(max(sh.hi_keep, lo_keep), n);
  int n_new = hi_keep - lo_keep;
  // Terminal condition: the survivors exactly fill the open slots.
  const bool terminal = !done && (n_new == k_after);
  if (terminal) done = 1;

  // ---- append leavers (rank order) ----------------------------------------------------------
  for (int r = append_lo + tid; r < append_hi; r += kThreads) {
    const int pos = sorted[r];
    res_idx[n_result + (r - append_lo)] = sh.id[pos];
    res_score[n_result + (r - append_lo)] = sh.score[pos];
  }
  int n_res_after = n_result + (append_hi - append_lo);
  if (terminal) {
    for (int r = lo_keep + tid; r < hi_keep; r += kThreads) {
      const int pos = sorted[r];
      res_idx[n_res_after + (r - lo_keep)] = sh.id[pos];
      res_score[n_res_after + (r - lo_keep)] = sh.score[pos];
    }
    n_res_after += n_new;
    k_after = 0;
  }

  // ---- survivor offsets: stable compaction in batch order ---------------------------------
  int total_new = 0;
  if (!done) {
    if (tid == 0) { sh.carry_a = 0; sh.carry_b = p.prefix; sh.n_owned_new = 0; }  // the prefix rows stay in front
    __syncthreads();
    for (int base = 0; base < n; base += kThreads) {
      const int i = base + tid;
      int keep = 0, len = 0;
      if (i < n) {
        const int r = sh.rank[i];
        keep = (r >= lo_keep && r < hi_keep);
        len = keep ? (cu_old[i + 1] - cu_old[i]) : 0;
      }
      int a = warp_scan(keep, lane), b = warp_scan(len, lane);
      if (lane == 31) { sh.warp_a[warp] = a; sh.warp_b[warp] = b; }
      __syncthreads();
      if (warp == 0) {
        int ta = warp_scan(sh.warp_a[lane], lane), tb = warp_scan(sh.warp_b[lane], lane);
        sh.warp_a[lane] = ta;
        sh.warp_b[lane] = tb;
      }
      __syncthreads();
      const int ea = sh.carry_a + (warp ? sh.warp_a[warp - 1] : 0) + a - keep;
      const int eb = sh.carry_b + (warp ? sh.warp_b[warp - 1] : 0) + b - len;
      if (keep) {
        cu_new[ea] = eb;
        seq2orig_new[ea] = sh.id[i];
        old_of_new[ea] = i;
        if (p.owned && p.owned[sh.id[i]]) atomicAdd(&sh.n_owned_new, 1);
      }
      __syncthreads();
      if (tid == kThreads - 1) { sh.carry_a += sh.warp_a[31]; sh.carry_b += sh.warp_b[31]; }
      __syncthreads();
    }
    total_new = sh.carry_b;
    if (tid == 0) cu_new[n_new] = total_new;
  } else {
    n_new = 0;
    if (tid == 0) cu_new[0] = 0;
  }

  if (tid == 0) {
    state->n_active = n_new;
    state->n_tokens = total_new;
    state->k_rem = k_after;
    state->n_result = n_res_after;
    state->done = done;
    state->pad0 = (!done && p.owned) ? sh.n_owned_new : n_new;  // survivors this rank runs
    if (rec) {
      rec->layer = p.layer;
      rec->n_active_before = n;
      rec->fired = fired;
      rec->n_selected = n_selected;
      rec->n_dropped = n_dropped;
      rec->n_deferred = n_deferred;
      rec->k_rem_after = k_after;
      rec->n_cuts = sh.n_cuts;
      for (int c = 0; c < kMaxClusters; ++c) rec->cuts[c] = c < sh.n_cuts ? sh.cuts[c] : 0;
      rec->tokens_before = tokens_before;
      rec->cv = cv;
    }
  }
}

}  // namespace

cudaError_t launch_route(const float* scores, const int* cu_old, const int* seq2orig_old, int n,
                         const RouteParams& p, int* cu_new, int* seq2orig_new, int* old_of_new,
                         RouteState* state, int* res_idx, float* res_score, ProbeRecordDev* rec,
                         float* trace_scores, int* trace_ids, void* scratch, cudaStream_t st) {
  static std::atomic<unsigned long long> smem_set{0};
  if (cudaError_t e = ensure_dynamic_smem(k_route, (int)sizeof(Shared), smem_set)) return e;
  if (n < 0 || n > kMaxCandidates) return cudaErrorInvalidValue;
  // the quadratic part (n^2 / 2 group costs per cost-table row, an fp64 division each) is shared by a cluster of
  // eight blocks once it dominates
  const int n_cta = (n >= 512 && p.mode == 2 && !p.is_final) ? 8 : 1;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(n_cta);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = sizeof(Shared);
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = n_cta;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  unsigned char* scr = (unsigned char*)scratch;
  cudaError_t e = cudaLaunchKernelEx(&cfg, k_route, scores, cu_old, seq2orig_old, n, p, cu_new, seq2orig_new, old_of_new, state,
                                     res_idx, res_score, rec, trace_scores, trace_ids, scr, n_cta);
  return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace prism

// ------------------------------------------------------------------------------------------------
// prism_op_route_static: the pruning decision for callers that cannot allocate device memory.
//
// The scratch the kernel needs (prefix sums, the two cost rows and the argmin table of the
// clustering) lives in a fixed array inside the library image instead of a cudaMalloc'd buffer.
// Every GPU that loads the library holds these bytes until the process exits.
namespace {

constexpr int kStaticRouteMaxN = PRISM_ROUTE_STATIC_MAX_CANDIDATES;
constexpr size_t kStaticRouteBytes = (prism::route_scratch_bytes(kStaticRouteMaxN) + 255) / 256 * 256;

static __device__ __align__(256) unsigned char g_route_static_scratch[kStaticRouteBytes];

constexpr int kMaxDevices = 64;
std::atomic<void*> g_route_static_ptr[kMaxDevices] = {};  // device address of the array, per device, filled on first use

}  // namespace

extern "C" int prism_op_route_static(const float* scores, const int32_t* cu_old, const int32_t* seq2orig_old,
                                     int32_t n, int32_t mode, int32_t keep_count, double cv_threshold,
                                     int32_t n_clusters, int32_t std_ddof, int32_t select_winners, int32_t is_final,
                                     int32_t layer, int32_t* cu_new, int32_t* seq2orig_new, int32_t* old_of_new,
                                     int32_t* state, int32_t* res_idx, float* res_score, prism_probe_record* rec,
                                     void* stream) {
  using namespace prism;
  if (!scores || !cu_old || !seq2orig_old || !cu_new || !seq2orig_new || !old_of_new || !state || !res_idx || !res_score)
    return PRISM_ERR_INVALID_ARG;
  if (!route_args_ok(n, mode, keep_count, n_clusters, std_ddof, kMaxCandidates)) return PRISM_ERR_INVALID_ARG;
  if (n > kStaticRouteMaxN) return PRISM_ERR_SHAPE_LIMIT;  // the built-in scratch is sized for this many candidates
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return PRISM_ERR_CUDA;
  void* scratch = g_route_static_ptr[dev].load(std::memory_order_acquire);
  if (!scratch) {
    // In host code the array's name is only a handle; the kernel needs the address it has on THIS device.
    // Two host threads may both get here: they look up, and store, the same address.
    if (cudaGetSymbolAddress(&scratch, g_route_static_scratch) != cudaSuccess || !scratch) return PRISM_ERR_CUDA;
    g_route_static_ptr[dev].store(scratch, std::memory_order_release);
  }
  RouteParams prm{};
  prm.mode = mode;
  prm.keep_count = keep_count;
  prm.cv_threshold = cv_threshold;
  prm.n_clusters = n_clusters;
  prm.ddof = std_ddof;
  prm.select_winners = select_winners;
  prm.is_final = is_final;
  prm.layer = layer;
  cudaError_t e = launch_route(scores, cu_old, seq2orig_old, n, prm, cu_new, seq2orig_new, old_of_new,
                               reinterpret_cast<RouteState*>(state), res_idx, res_score,
                               reinterpret_cast<ProbeRecordDev*>(rec), nullptr, nullptr, scratch,
                               reinterpret_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? PRISM_OK : PRISM_ERR_CUDA;
}
