/*
 * prism.h -- C ABI of the PRISM hot path on one NVIDIA B200 (sm_100a).
 *
 * The library computes semantic top-K selection the way the paper's "monolithic forwarding"
 * does (Sec. 3.3): all N query||candidate sequences of one request advance through the layers
 * of a decoder cross-encoder reranker together, as ONE padding-free packed batch.  After the
 * designated layers a relevance score is probed per candidate with the model's own classifier
 * (Sec. 3.1, 4.1); the dispersion CV = |std/mean| of the scores decides whether clustering runs;
 * clusters above the one holding the K-th ranked candidate are *selected*, clusters below it are
 * *dropped*, the boundary cluster is *deferred* and is the only part that keeps computing
 * (Sec. 4.1, Fig. 4); the survivors are stream-compacted before the next layer; the forward
 * stops when #deferred equals the remaining top-K slots (Sec. 4.1, 4.5).  Chunked execution
 * (Sec. 4.3) and overlapped layer streaming (Sec. 4.2) are options of the handle.
 *
 * Conventions
 *   - plain C, no exceptions, nothing printed; every call returns a prism_status (0 = OK).
 *   - "device pointer" = CUDA global memory of the current device; "host pointer" = CPU memory.
 *   - matrices are row-major [out_features, in_features] (both GEMM operands are K-major).
 *   - element type of every weight tensor is cfg.dtype (PRISM_FP32: float, PRISM_BF16: bfloat16).
 *   - a handle serves one request at a time (not re-entrant); different handles are independent.
 *   - the library never takes ownership of caller memory and never frees it.
 */
#ifndef PRISM_H_
#define PRISM_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define PRISM_API __attribute__((visibility("default")))
#else
#define PRISM_API
#endif

#define PRISM_MAX_CLUSTERS 8      /* upper bound for prism_prune_schedule.n_clusters          */
#define PRISM_MAX_CANDIDATES 4096 /* upper bound for prism_model_cfg.max_candidates           */
#define PRISM_MAX_LAYERS 128

typedef enum {
  PRISM_OK = 0,
  PRISM_ERR_INVALID_ARG = -1, /* null pointer, negative size, K < 1, malformed schedule/config          */
  PRISM_ERR_SHAPE_LIMIT = -2, /* N, a sequence length or the token total exceeds the handle's maxima    */
  PRISM_ERR_BAD_INPUT = -3,   /* token id outside [0, vocab) or non-monotone offsets (found on device)  */
  PRISM_ERR_BUDGET = -4,      /* activation budget cannot hold the hidden states plus one sequence      */
  PRISM_ERR_CUDA = -5,        /* a CUDA call failed; text via prism_last_error                          */
  PRISM_ERR_TIMEOUT = -6,     /* a bounded device-side wait expired (kernel returned, context usable)   */
  PRISM_ERR_NOMEM = -7,       /* device or host allocation failed                                       */
  PRISM_ERR_UNSUPPORTED = -8  /* shape not supported by the kernels (e.g. head_dim, alignment)          */
} prism_status;

enum { PRISM_FP32 = 0, PRISM_BF16 = 1 };
enum { PRISM_WEIGHTS_DEVICE = 0, PRISM_WEIGHTS_HOST_STREAMED = 1 };
enum { PRISM_PRUNE_NONE = 0, PRISM_PRUNE_FIXED_KEEP = 1, PRISM_PRUNE_CLUSTER = 2 };
/* Implementation selectors (validation): AUTO picks the tcgen05 tensor-core kernels in bf16 mode (the GEMM on
 * CTA pairs: cta_group::2, one 256x256 tile per two-CTA cluster), SIMT the CUDA-core kernels, MMA (attention
 * only) the warp-level mma.sync flash-attention kernel, SOLO (GEMM only) the single-CTA tcgen05 kernel with
 * 128x256 tiles. */
enum { PRISM_IMPL_AUTO = 0, PRISM_IMPL_SIMT = 1, PRISM_IMPL_MMA = 2, PRISM_IMPL_SOLO = 3 };

/* weight_format of prism_model_cfg.  PLAIN: matrices in the element type of cfg.dtype.  W4: the quantised arm of
 * the paper's evaluation (Sec. 6.1: the method composed with 4-bit weight-only quantisation, 16-bit activations).
 * The five matrices of every layer (w_qkv, w_o, w_gate, w_up, w_down; for the encoder stack w_qkv, w_o, w_ffn1, w_ffn2)
 * are packed blobs; for an [N, K] matrix and
 * group size G = quant_group, every section starting on a 16-byte boundary:
 *     codes   N*K/2 bytes, row-major; byte (n, k/2) holds code(n,k) in its low nibble for even k, high nibble for odd k
 *     scales  N*K/G bf16, row-major [N, K/G]
 *     zeros   N*K/G bytes (0..15), row-major
 *     value(n,k) = bf16( float(scale[n,k/G]) * (code(n,k) - zero[n,k/G]) )
 * Before a layer runs, its matrices are rebuilt as bf16 into one layer-sized device scratch and the usual GEMMs read
 * that; with PRISM_WEIGHTS_HOST_STREAMED the PACKED layer crosses the host link (a quarter of the bytes).  Results
 * equal those of a PLAIN handle given the dequantised matrices, bit for bit.  Norm gains, embedding and score head
 * stay plain. */
enum { PRISM_WFMT_PLAIN = 0, PRISM_WFMT_W4 = 1 };

/* arch of prism_model_cfg.  DECODER: the pre-norm blocks described at prism_model_cfg, created by prism_create.
 * ENCODER: the encoder-only reranker the paper evaluates next to them (BGE-M3's, an XLM-RoBERTa stack; Sec. 6.1,
 * Table 1), created by prism_create_encoder: token + learned position + token-type embedding, LayerNorm, then
 * post-norm blocks x = LN1(x + O(attention(QKV x))), x = LN2(x + W2 gelu(W1 x + b1) + b2) with a bias on every
 * linear map and the exact GELU x Phi(x); the classifier reads the FIRST token. */
enum { PRISM_ARCH_DECODER = 0, PRISM_ARCH_ENCODER = 1 };

/* shared_prefix of prism_model_cfg */
enum { PRISM_PREFIX_AUTO = 0, PRISM_PREFIX_OFF = 1 };

typedef struct prism_handle prism_handle;

/* Model description: a pre-norm decoder block stack (RMSNorm -> GQA attention with optional
 * per-head QK-norm and rotary embedding -> residual -> RMSNorm -> SwiGLU -> residual), the
 * architecture of the rerankers the paper evaluates (Sec. 6.1, Table 1). */
typedef struct {
  int32_t n_layers;   /* 1..PRISM_MAX_LAYERS */
  int32_t hidden;     /* D <= 8192; multiple of 8 in bf16 mode, of 4 in fp32 mode */
  int32_t n_q_heads;  /* Hq, multiple of n_kv_heads */
  int32_t n_kv_heads; /* Hkv */
  int32_t head_dim;   /* dh: 128 for the tensor-core attention kernels (bf16, attention_impl AUTO or MMA);
                         even and <= 256 for the CUDA-core path (fp32 mode, or attention_impl SIMT) */
  int32_t ffn;        /* F; multiple of 128 for the tensor-core GEMM (bf16, gemm_impl AUTO), of 8 otherwise in bf16 */
  int32_t vocab;
  float rope_theta;
  float rms_eps;
  int32_t causal;  /* 1 = decoder (causal) attention, 0 = bidirectional */
  int32_t qk_norm; /* 1 = RMSNorm over head_dim on q and k before the rotary embedding */
  int32_t dtype;   /* PRISM_FP32 or PRISM_BF16: weights, activations and GEMM inputs; the residual
                      stream, accumulators, norms, softmax and scores are always fp32 */
  int32_t max_seq_len;      /* max query_len + doc length of one sequence */
  int32_t max_candidates;   /* max N (<= PRISM_MAX_CANDIDATES) */
  int32_t max_total_tokens; /* max sum over candidates of (query_len + doc length) */
  int64_t activation_budget_bytes; /* 0 = unlimited.  Otherwise chunked execution (Sec. 4.3): the
                      hidden states of all sequences plus the intermediates of ONE chunk stay
                      within this many bytes; chunks are cut on sequence boundaries */
  int32_t weight_residency; /* PRISM_WEIGHTS_DEVICE, or PRISM_WEIGHTS_HOST_STREAMED: layer tensors
                      are pinned host memory, two device slots, layer l+1 is copied on a side
                      stream while layer l computes (overlapped layer streaming, Sec. 4.2) */
  int32_t gemm_impl;      /* PRISM_IMPL_* */
  int32_t attention_impl; /* PRISM_IMPL_* */
  int32_t embed_cache_rows; /* 0: `embed` is a device table.  > 0: embedding table caching (Sec. 4.4): `embed` is
                      the complete table in PINNED HOST memory and the device holds this many of its rows,
                      replaced least-recently-used first.  Every request first collects its distinct tokens
                      (one device-to-host copy of the token ids) and brings the missing rows into the cache
                      before the layers start.  A request with more distinct tokens than rows fails with
                      PRISM_ERR_SHAPE_LIMIT.  The paper sizes the cache at 10 % of the vocabulary. */
  int32_t hidden_offload;   /* 1: dynamic offloading of the hidden states (Sec. 4.3): the hidden states of all
                      sequences live in pinned host memory (allocated by the library) and at most three chunks
                      are on the device at a time: the one being computed, the one being written back and the
                      one being fetched.  Needs activation_budget_bytes > 0, which then has to hold three
                      chunks of hidden states plus one chunk's intermediates.  Embedding, probe and compaction
                      work on the host copy directly.  0: hidden states stay on the device. */
  int32_t shared_prefix;    /* PRISM_PREFIX_AUTO (0): under causal attention the query's rows do not depend on the
                      document behind them, so the batch stores and computes them ONCE, in front of all documents,
                      and every sequence attends to those rows followed by its own (Sec. 3.1's batch, minus the
                      N - 1 repeated copies of the query).  Scores, selections and traces are bit-identical to the
                      batch with one query copy per sequence; tokens_per_layer and tokens_before keep counting
                      query_len + document length per sequence.  Taken when: causal, bf16 tensor-core path with an
                      even Hq / Hkv, 8 <= query_len <= 120 and query_len a multiple of 8, N >= 2
                      (under chunked execution and hidden_offload the first chunk of a layer carries the query
                      rows; with prism_select_sharded every rank holds them).  Otherwise, or with
                      PRISM_PREFIX_OFF (1), every sequence carries its own copy of the query. */
  int32_t arch;             /* PRISM_ARCH_*.  For PRISM_ARCH_ENCODER: rms_eps is the LayerNorm epsilon; rope_theta and
                      qk_norm are ignored (qk_norm must be 0); causal is normally 0; head_dim is 64 or 128 on the
                      tensor-core path; ffn a multiple of 8; gemm_impl AUTO or SIMT, attention_impl AUTO, SOLO or SIMT.
                      With PRISM_WEIGHTS_HOST_STREAMED the four matrices of a block are streamed; its vectors are
                      read once at creation. */
  int32_t max_positions;    /* encoder: rows of the learned position table; max_seq_len + pos_offset <= max_positions */
  int32_t pos_offset;       /* encoder: token p of a sequence reads position row p + pos_offset (2 for XLM-RoBERTa) */
  int32_t weight_format;    /* PRISM_WFMT_*; W4 needs dtype PRISM_BF16 */
  int32_t quant_group;      /* W4: input channels per scale / zero point: 32, 64 or 128, dividing hidden, ffn and
                               n_q_heads * head_dim */
} prism_model_cfg;

typedef struct {
  const void* g_attn; /* [D] */
  const void* w_qkv;  /* [(Hq+2Hkv)*dh, D]: all q heads, then k heads, then v heads */
  const void* g_q;    /* [dh], used when qk_norm */
  const void* g_k;    /* [dh], used when qk_norm */
  const void* w_o;    /* [D, Hq*dh] */
  const void* g_ffn;  /* [D] */
  const void* w_gate; /* [F, D] */
  const void* w_up;   /* [F, D] */
  const void* w_down; /* [D, F] */
} prism_layer_weights;

/* Pointers only.  embed/g_final/score_head are device pointers.  The layer tensors are device
 * pointers (PRISM_WEIGHTS_DEVICE) or pinned host pointers (PRISM_WEIGHTS_HOST_STREAMED); each
 * must be 16-byte aligned.  The caller keeps all of them alive and unchanged until
 * prism_destroy.  `layers` itself is a host array of n_layers structs, read during
 * prism_create only. */
typedef struct {
  const void* embed;      /* [vocab, D] */
  const void* g_final;    /* [D] final RMSNorm gain */
  const void* score_head; /* [2, D]: row 0 = "yes" logit row, row 1 = "no"; score = yes - no */
  const prism_layer_weights* layers;
} prism_weights;

/* Weights of one encoder block.  Matrices have the element type of cfg.dtype and are device pointers, 16-byte
 * aligned (pinned host pointers with PRISM_WEIGHTS_HOST_STREAMED); the vectors (biases, LayerNorm gain and shift)
 * have the same element type, may live in device or pinned host memory, and are widened to fp32 device copies
 * inside prism_create_encoder. */
typedef struct {
  const void* w_qkv;  /* [(Hq+2Hkv)*dh, D]: all q heads, then k heads, then v heads */
  const void* b_qkv;  /* [(Hq+2Hkv)*dh] */
  const void* w_o;    /* [D, Hq*dh] */
  const void* b_o;    /* [D] */
  const void* ln1_g;  /* [D] LayerNorm after the attention residual */
  const void* ln1_b;  /* [D] */
  const void* w_ffn1; /* [F, D] */
  const void* b_ffn1; /* [F] */
  const void* w_ffn2; /* [D, F] */
  const void* b_ffn2; /* [D] */
  const void* ln2_g;  /* [D] LayerNorm after the FFN residual */
  const void* ln2_b;  /* [D] */
} prism_encoder_layer_weights;

typedef struct {
  const void* embed;        /* [vocab, D] */
  const void* pos_embed;    /* [max_positions, D] */
  const void* type_embed;   /* [D]: the token-type-0 row */
  const void* emb_ln_g;     /* [D] LayerNorm of the embedding sum */
  const void* emb_ln_b;     /* [D] */
  const void* head_dense_w; /* [D, D] classifier: dense + tanh ... */
  const void* head_dense_b; /* [D] */
  const void* head_out_w;   /* [D] ... then one logit, which is the score */
  const void* head_out_b;   /* [1] */
  const prism_encoder_layer_weights* layers; /* host array of n_layers structs, read during creation only */
} prism_encoder_weights;

/* When and how to prune (Sec. 4.1).  probe_layers[j] counts completed layers (1-based),
 * strictly increasing, each < n_layers; the last layer is always scored and never prunes.
 *   NONE        no probes; the result is the exact top-K by final score.
 *   FIXED_KEEP  at probe j keep the keep_counts[j] best (each >= K).
 *   CLUSTER     if CV > cv_threshold: split the ranked scores into n_clusters contiguous groups of
 *               minimum within-group variance, route selected / deferred / dropped around the
 *               group that holds rank K_rem.  select_winners = 0 is the drop-only variant (Sec. 7):
 *               contenders above the boundary keep computing, so every returned score is a
 *               final-layer score. */
typedef struct {
  int32_t mode;
  int32_t n_probes;
  const int32_t* probe_layers; /* host */
  const int32_t* keep_counts;  /* host, FIXED_KEEP only */
  double cv_threshold;
  int32_t n_clusters;     /* 2..PRISM_MAX_CLUSTERS (0 = default 3) */
  int32_t std_ddof;       /* 0 population std (default), 1 sample std */
  int32_t select_winners; /* 1 three-way routing, 0 drop-only */
} prism_prune_schedule;

typedef struct {
  int32_t layer;           /* completed layers when the scores were probed */
  int32_t n_active_before; /* candidates scored */
  int32_t fired;           /* 1 if candidates were removed at this probe */
  int32_t n_selected, n_dropped, n_deferred;
  int32_t k_rem_after; /* top-K slots still open after the probe */
  int32_t n_cuts;
  int32_t cuts[PRISM_MAX_CLUSTERS]; /* cluster boundaries in rank space */
  int32_t tokens_before;            /* live tokens entering the probe */
  double cv;
} prism_probe_record;

/* Optional per-request record, all host memory owned by the caller.  Scored layers are written in
 * order: every probe layer reached, then the final layer if it was reached (fired = 0 there). */
typedef struct {
  int32_t capacity;            /* in: records available in `records` (and rows in scores/ids) */
  int32_t n_records;           /* out */
  prism_probe_record* records; /* out [capacity] */
  float* scores;               /* out, nullable: [capacity, N] probe scores, batch order */
  int32_t* ids;                /* out, nullable: [capacity, N] original candidate index per score */
  int32_t layers_run;          /* out: layers executed before the forward stopped */
  int32_t* tokens_per_layer;   /* out, nullable: [n_layers] live tokens forwarded through each layer */
  int32_t n_chunks_max;        /* out: largest number of chunks used for one layer */
  int64_t workspace_bytes;     /* out: device bytes held by the handle */
  int32_t shared_prefix_rows;  /* out: query rows stored once for all sequences (0: one copy per sequence) */
  int32_t reserved;
} prism_trace;

/* Validate cfg, take the weight pointers, allocate every workspace the handle will ever need
 * (no allocation happens later), build TMA descriptors and the rotary table.
 * Errors: INVALID_ARG, UNSUPPORTED, BUDGET (budget below hidden states + one max_seq_len sequence),
 * NOMEM, CUDA.  On error *out = NULL. */
PRISM_API int prism_create(const prism_model_cfg* cfg, const prism_weights* w, prism_handle** out);

/* The same for the encoder stack (cfg->arch must be PRISM_ARCH_ENCODER).  The handle serves prism_select,
 * prism_select_host, prism_select_calibrated and prism_select_sharded exactly like a decoder handle: packing,
 * chunked execution, probe schedule, routing, compaction and the final top-K are shared; the probe after block l
 * applies the classifier to the first token of block l's output.  Errors as prism_create. */
PRISM_API int prism_create_encoder(const prism_model_cfg* cfg, const prism_encoder_weights* w, prism_handle** out);

/* Top-K selection for one request (problem statement Sec. 2.1; method Sec. 3.3-4.3).
 *   query_tokens  device int32[query_len]
 *   cand_tokens   device int32[cand_offsets[N]]   document token ids, concatenated
 *   cand_offsets  device int32[N+1], cand_offsets[0] = 0, non-decreasing
 *   topk_idx      device int32[K]   original candidate indices
 *   topk_scores   device float[K]   score each had when it left the computation
 *   n_out         host   int32      min(K, N) on success, 0 on error
 *   trace         host, nullable
 *   cuda_stream   a cudaStream_t (NULL = default stream); work is enqueued there and the call
 *                 returns after the stream has drained.
 * Sequence i is query_tokens followed by document i, positions restart at 0.  Output order:
 * candidates selected at earlier probes first (within a probe: score descending, index
 * ascending), then the final fill in the same order.  K > N is not an error.
 * Errors: INVALID_ARG, SHAPE_LIMIT, BAD_INPUT, BUDGET, CUDA, TIMEOUT; outputs are then unspecified. */
PRISM_API int prism_select(prism_handle* h, const int32_t* query_tokens, int32_t query_len,
                 const int32_t* cand_tokens, const int32_t* cand_offsets, int32_t N, int32_t K,
                 const prism_prune_schedule* sched, int32_t* topk_idx, float* topk_scores,
                 int32_t* n_out, prism_trace* trace, void* cuda_stream);

/* One request over several GPUs, one process (rank) per GPU: the candidates are partitioned over the ranks (the
 * sequences never attend to each other, so a candidate's hidden states and scores do not depend on which rank
 * runs it), every rank runs the layers on its own candidates only, and the one global step of the method, the
 * prune decision after a probe (Sec. 4.1), is taken by every rank on the same complete score vector.
 *   owned      host uint8[N]: 1 for the candidates this rank runs.  Every candidate must be owned by exactly
 *              one rank; the library cannot check that.
 *   exchange   device float[N], caller-owned.  Before every prune decision the library writes the scores of
 *              the n still-active candidates to exchange[0..n) on cuda_stream (0 for candidates of other
 *              ranks) and calls reduce.
 *   reduce     must replace exchange[0..n) by its element-wise sum over all ranks, ordered after the work
 *              already enqueued on cuda_stream and before work enqueued there later (an all-reduce on that
 *              stream, or a stream synchronisation around a host-side reduction); returns 0 on success.  n is
 *              the same on every rank.  The sum is exact (one non-zero term per element), so all ranks
 *              decide on bit-identical numbers and stay in step without any other communication.
 * All other arguments, the outputs (identical on every rank) and the errors are those of prism_select; every
 * rank passes the complete cand_tokens / cand_offsets.  max_total_tokens bounds the rank's own tokens.
 * The paper runs on one device and has no counterpart of this entry point. */
typedef int (*prism_exchange_fn)(void* ctx, int32_t n, void* cuda_stream);
PRISM_API int prism_select_sharded(prism_handle* h, const int32_t* query_tokens, int32_t query_len,
                 const int32_t* cand_tokens, const int32_t* cand_offsets, int32_t N, int32_t K,
                 const prism_prune_schedule* sched, const uint8_t* owned, float* exchange,
                 prism_exchange_fn reduce, void* ctx, int32_t* topk_idx, float* topk_scores,
                 int32_t* n_out, prism_trace* trace, void* cuda_stream);

/* Counters of the embedding-row cache since prism_create: rows found in the cache, rows fetched from the host
 * table, and fetched rows that replaced another token's row.  All zero when embed_cache_rows == 0. */
PRISM_API int prism_embed_cache_stats(const prism_handle* h, int64_t* hits, int64_t* misses, int64_t* evictions);

/* Same request with HOST buffers: copies the three inputs to the device, runs prism_select's path
 * and copies topk_idx / topk_scores back (all on cuda_stream, inside the call).  Pinned buffers
 * make the copies asynchronous; pageable ones work too. */
PRISM_API int prism_select_host(prism_handle* h, const int32_t* query_tokens, int32_t query_len,
                      const int32_t* cand_tokens, const int32_t* cand_offsets, int32_t N, int32_t K,
                      const prism_prune_schedule* sched, int32_t* topk_idx, float* topk_scores,
                      int32_t* n_out, prism_trace* trace, void* cuda_stream);

/* Automatic calibration of the dispersion threshold (Sec. 4.1, last paragraph): the user states a
 * minimum precision; requests are sampled at a fixed frequency, the sampled ones are re-run without
 * pruning to obtain the ground-truth top-K, and after every `window` samples the mean
 * precision = |top-K with pruning  intersect  top-K without| / min(K, N) is compared with the target:
 * below it the threshold is raised (more conservative), otherwise lowered (more pruning).
 * The paper does not say by how much; here the threshold is multiplied by raise_factor (> 1) or
 * lower_factor (< 1) and clamped to [min_threshold, max_threshold].  The re-run happens inside the
 * call (the paper defers it to idle time); the caller owns the struct and may persist it. */
typedef struct {
  double threshold;         /* in/out: dispersion threshold used for the next request */
  double target_precision;  /* in: e.g. 0.99 */
  double raise_factor;      /* in: > 1 */
  double lower_factor;      /* in: in (0, 1) */
  double min_threshold;     /* in */
  double max_threshold;     /* in */
  int32_t sample_every;     /* in: every sample_every-th request is also run unpruned (>= 1) */
  int32_t window;           /* in: samples per adjustment (>= 1) */
  int32_t n_in_window;      /* state: samples collected since the last adjustment */
  int32_t n_adjustments;    /* out: adjustments made so far */
  int64_t n_requests;       /* out: requests served */
  int64_t n_sampled;        /* out: requests re-run unpruned */
  double precision_sum;     /* state: sum of the window's precisions */
  double last_precision;    /* out: precision of the last sampled request */
  double last_window_precision; /* out: mean precision of the last completed window */
} prism_calibrator;

/* prism_select with the threshold taken from (and maintained in) `cal`.  sched must be a
 * PRISM_PRUNE_CLUSTER schedule; its cv_threshold field is ignored.  Outputs are those of the pruned
 * run.  Errors: those of prism_select, plus INVALID_ARG for a malformed calibrator. */
PRISM_API int prism_select_calibrated(prism_handle* h, const int32_t* query_tokens, int32_t query_len,
                                      const int32_t* cand_tokens, const int32_t* cand_offsets, int32_t N, int32_t K,
                                      const prism_prune_schedule* sched, prism_calibrator* cal, int32_t* topk_idx,
                                      float* topk_scores, int32_t* n_out, prism_trace* trace, void* cuda_stream);

/* Free the handle and its workspaces (NULL is allowed).  Caller memory is untouched. */
PRISM_API void prism_destroy(prism_handle* h);

/* Text of the last error on this handle ("" if none); valid until the next call on the handle. */
PRISM_API const char* prism_last_error(const prism_handle* h);

/* Static name of a status code. */
PRISM_API const char* prism_status_str(int status);

/* Number of kernels this library launched since the handle was created (for launch accounting). */
PRISM_API int64_t prism_launch_count(const prism_handle* h);

/* Per-kernel timing of the steps prism_select chains.  While enabled, every kernel launch of a request
 * is bracketed by CUDA events on the request's stream (this adds a few microseconds per launch, so
 * latency figures are taken with profiling off).  `work` accumulates the ALGORITHMIC work the driver
 * asked of the class: flops for the GEMM and attention classes (2*M*N*K; causal attention
 * 2*L^2*Hq*dh per sequence), bytes that must move for all others. */
enum {
  PRISM_K_PACK = 0, PRISM_K_EMBED, PRISM_K_RMSNORM, PRISM_K_GEMM_QKV, PRISM_K_ROPE, PRISM_K_ATTENTION,
  PRISM_K_GEMM_O, PRISM_K_GEMM_GATEUP, PRISM_K_GEMM_DOWN, PRISM_K_PROBE, PRISM_K_ROUTE, PRISM_K_COMPACT,
  PRISM_K_DEQUANT, /* W4 -> bf16 of a layer's matrices (weight_format PRISM_WFMT_W4) */
  PRISM_N_KERNEL_CLASSES
};
typedef struct {
  double ms;        /* summed device time between the bracketing events */
  double work;      /* flops or bytes, see above */
  int64_t launches;
} prism_kernel_stat;
PRISM_API int prism_profile(prism_handle* h, int enable);
/* Copy the accumulated statistics to out[PRISM_N_KERNEL_CLASSES] (host); reset != 0 clears them. */
PRISM_API int prism_profile_read(prism_handle* h, prism_kernel_stat* out, int reset);

#ifdef __cplusplus
}
#endif
#endif /* PRISM_H_ */
