/*
 * maaso.h — C ABI of the placement-scoring library.
 *
 * The library scores many candidate placements of heterogeneous model instances against
 * one request trace, the inner loop of a simulator-guided placer (paper: Alg. 1 evaluates
 * Phi(I', R_x) once per tentative instance list; the simulator is described in Sec. V-A
 * "Simulator Implementation", the distributor in Sec. IV-F, the profiler model in
 * Sec. IV-B Eq. 1).  Everything runs in CUDA kernels on one GPU; there is no CPU fallback.
 *
 * Conventions
 *   - All times are int64 microseconds.  All results are integers; the same inputs give
 *     byte-identical outputs whatever the launch shape, stream or mapping.
 *   - "host" / "device" below says where a pointer must live.  The caller owns every
 *     buffer it passes; the library copies what it keeps (profile, trace) and never frees
 *     or retains caller memory beyond the stream work of the call.
 *   - Every function returns 0 on success or a negative MAASO_E* code; maaso_strerror()
 *     gives a text.  Nothing throws, aborts or traps.  A bad *candidate* never fails a
 *     call: its record carries a non-zero `status` (MAASO_CAND_*) and zeroed statistics.
 *   - Calls on one context are not thread-safe.  maaso_eval_placements / maaso_topk only
 *     enqueue work on the given stream; outputs are valid once that stream is synchronised.
 *     Successive calls on one context share its scratch memory, so their device work must
 *     not overlap: use one stream, or synchronise between calls on different streams.
 */
#ifndef MAASO_H
#define MAASO_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define MAASO_API __attribute__((visibility("default")))
#else
#define MAASO_API
#endif

#define MAASO_WMAX 64           /* largest batch cap; latency tables have this many columns */
#define MAASO_MAX_INSTANCES 128 /* most instances in one candidate */
#define MAASO_MAX_MODELS 16
#define MAASO_MAX_STRATEGIES 256
#define MAASO_MAX_ROWS 256      /* n_models * n_strategies */
#define MAASO_MAX_CLASSES 256
#define MAASO_MAX_STEP_US (1 << 30)
#define MAASO_MAX_TOPK 1024
#define MAASO_TTFT_BINS 64     /* bins of the optional time-to-first-token histogram */

/* return codes */
#define MAASO_OK 0
#define MAASO_EINVAL (-1) /* null pointer, size or range violation, unsorted trace, unknown model/class */
#define MAASO_ESTATE (-2) /* profile not loaded, trace belongs to another context, ... */
#define MAASO_ENOMEM (-3)
#define MAASO_ECUDA (-4)  /* a CUDA runtime call failed; text via maaso_last_error() */
#define MAASO_ETOOBIG (-5) /* size beyond the fixed capacity of an entry point that cannot allocate */

/* per-candidate status bits (maaso_result.status) */
#define MAASO_CAND_EBUDGET 1u   /* devices used exceed the budget: constraint (c), Sec. IV-C */
#define MAASO_CAND_EMEMFIT 2u   /* an instance has fewer devices than its model needs: constraint (d) */
#define MAASO_CAND_ETOOMANY 4u  /* more than MAASO_MAX_INSTANCES instances */
#define MAASO_CAND_EBADINST 8u  /* unknown model/strategy, batch cap outside 1..64, reserved bits set */
#define MAASO_CAND_ETIMEOUT 16u /* a bounded device-side wait ran out; the candidate was not scored */
#define MAASO_CAND_ELOOP 32u    /* more than 2 + 128*64 distributor attempts for one request */

/* maaso_eval_opts.flags */
#define MAASO_FLAG_PRED_OPTIMISTIC 1u /* distributor predicts with the step time right after admission
                                         instead of the worst case F(M,P,B_I) of Sec. IV-F step 3 */

#define MAASO_FLAG_ENGINE_FROZEN 2u /* replay with the engine that fixes a request's decode speed at its
                                      admission (Sec. IV-C read literally: the concurrency W_i "when
                                      request r arrives"; virtual slots of Sec. V-A): a slot is busy from
                                      admission to the request's finish time, first token = admission +
                                      prefill, one token every step[running + 1] afterwards; later
                                      admissions slow nobody down and prefills stall nobody.  Same
                                      distributor.  Lane-group code only: MAASO_MAP_BLOCK and
                                      MAASO_MAP_THREAD are refused; a placement with more than 32 instances
                                      (up to MAASO_MAX_INSTANCES) is replayed by one warp, four instances
                                      per lane; finish times must stay below 2^57 us (else
                                      MAASO_CAND_ELOOP). */

#define MAASO_FLAG_TBT_MAXGAP 4u /* the TBT term of the hit test (Phi_S indicator) looks at the largest gap
                                    between two consecutive tokens of a request, prefill stalls included,
                                    instead of the mean gap; a request of one token has no gap.  The
                                    distributor's prediction is unchanged.  Same limits as
                                    MAASO_FLAG_ENGINE_FROZEN (lane-group code; one warp per placement
                                    beyond 32 instances). */

#define MAASO_FLAG_INSTANCE_QUEUES 8u /* a request whose chosen instance is full queues THERE (Sec. II-A: requests
                                        beyond the batch cap wait in the instance's queue) instead of at the
                                        dispatcher: it takes the slot that frees first (lowest slot among equal
                                        finish times), starts at that time with the speed of the level then
                                        (1 + the other slots still busy), and the dispatcher goes on to the
                                        next request at once: one distributor round per request.  Implies the
                                        engine of MAASO_FLAG_ENGINE_FROZEN (a queued request's times must be
                                        known when it is handed over) and has its limits. */

#define MAASO_FLAG_TEST_STALL 0x80000000u /* test hook for the bounded device-side waits: the trace copies
                                             are never issued and every wait is limited to about 0.1 s, so
                                             each valid candidate must come back with MAASO_CAND_ETIMEOUT
                                             and the call must return normally */

/* maaso_eval_opts.mapping */
#define MAASO_MAP_AUTO 0u   /* the library routes the batch: threads for large batches of placements the trace
                               overloads (default engine), else lane groups; see maaso_eval_placements */
#define MAASO_MAP_BLOCK 1u  /* one thread block per candidate, one warp per instance, lanes = slots */
#define MAASO_MAP_GROUP 2u  /* one lane per instance, groups of lanes per candidate (<= 32 instances; beyond
                               that one warp per candidate with four instances per lane) */
#define MAASO_MAP_THREAD 3u /* one thread per candidate, looping over the instances of the request's model;
                               default engine only (flags 0 or MAASO_FLAG_PRED_OPTIMISTIC), any instance count */

typedef struct maaso_ctx maaso_ctx;
typedef struct maaso_trace maaso_trace;

/* One request of the trace (16 bytes).  Requests are sorted by arrival; equal arrivals
 * are served in index order.  out_tokens >= 1 (S_r, the decode length of Sec. IV-C). */
typedef struct {
    int64_t arrival_us;
    uint32_t in_tokens;
    uint16_t out_tokens;
    uint8_t cls;   /* index into the SLO class table */
    uint8_t model; /* which model the request is for */
} maaso_request;

/* One SLO class; a negative limit means "no limit".  The deadline tau_r = d_r*theta_r*theta
 * of Sec. III-C is the tbt term: finish - first_token <= (S-1) * tbt_us. */
typedef struct {
    int64_t ttft_us; /* first token - arrival */
    int64_t tbt_us;  /* mean time between tokens */
    int64_t e2e_us;  /* finish - arrival */
} maaso_slo_class;

/* Latency tables, all host pointers, int32, copied by maaso_load_profile.
 * Row (m, s) = model m under parallelism strategy s. */
typedef struct {
    uint32_t n_models;     /* 1..MAASO_MAX_MODELS */
    uint32_t n_strategies; /* 1..MAASO_MAX_STRATEGIES, n_models*n_strategies <= MAASO_MAX_ROWS */
    uint32_t wmax;         /* must be MAASO_WMAX */
    const int32_t *devices;         /* [S]  N(P): devices one instance occupies, >= 1 */
    const int32_t *min_devices;     /* [M]  fewest devices a model fits in */
    const int32_t *prefill_base_us; /* [M][S] >= 0 */
    const int32_t *prefill_q16;     /* [M][S] >= 0, microseconds per input token in Q16 */
    const int32_t *step_us;         /* [M][S][wmax]: one decode step with w running requests is
                                       entry w-1, 1..MAASO_MAX_STEP_US (Eq. 1 as a table:
                                       step = 1 / F(M,P,B,W) at W = w <= B) */
} maaso_profile_desc;

/* A batch of candidates in CSR form; device pointers (host pointers for the *_host call).
 * inst word: bits 0-3 model, 4-11 strategy, 12-19 batch cap B, 20-31 zero.
 * class_mask (may be NULL): bit k set = requests of class k belong to the request subset
 * this placement is scored on (sub-cluster mapping, Sec. IV-F step 1); ignored when the
 * trace has more than 32 classes. */
typedef struct {
    const uint32_t *offsets;    /* [n_cand + 1], offsets[0] = 0, non-decreasing */
    const uint32_t *inst;       /* [n_inst] */
    const uint32_t *class_mask; /* [n_cand] or NULL */
    uint64_t n_cand;
    uint64_t n_inst;            /* = offsets[n_cand] */
    uint32_t budget;            /* modeled devices available, N(G) */
    uint32_t reserved;
} maaso_cand_batch;

/* Options; NULL means all zero.  The dump buffers (device, each [dump_n][n_requests], any
 * may be NULL) receive per-request times for the candidates listed in dump_cand_idx
 * (device, [dump_n], distinct): finish time, first-token time, serving instance;
 * -1 = rejected, -2 = not counted (masked out, or the candidate is invalid). */
typedef struct {
    uint32_t flags;
    uint32_t mapping;
    uint32_t dump_n;
    uint32_t reserved;
    const uint32_t *dump_cand_idx;
    int64_t *dump_finish_us;
    int64_t *dump_first_us;
    int32_t *dump_inst;
    uint32_t *rejected_by_model; /* device, [n_cand][MAASO_MAX_MODELS] or NULL: requests of each model
                                    the placement left unserved (R_res of Alg. 1); zero for invalid ones */
    uint32_t *ttft_hist;         /* device, [n_cand][MAASO_TTFT_BINS] or NULL: histogram of the time to
                                    first token of the served requests (the "response latency" of
                                    Sec. V-A), overwritten by the call.  Bin 0 holds t < 1024 us; for
                                    t >= 1024 with e = floor(log2 t) and h = the bit below the leading
                                    one, bin = min(63, 1 + 2 (e - 10) + h): two bins per octave.
                                    All zero for an invalid candidate. */
} maaso_eval_opts;

/* Per-candidate result (128 bytes).  Statistics are over served requests unless noted. */
typedef struct {
    uint32_t status;      /* 0 = scored */
    uint32_t n_counted;   /* requests of the subset (after class_mask) */
    uint32_t n_served;
    uint32_t n_hit;       /* Phi_S: served within every limit of their class */
    uint32_t n_rejected;  /* blocked by overflow protection; count as SLO misses */
    uint32_t n_cascade;   /* admitted as feasible but finished late (cascaded timeout, Sec. III-B) */
    uint32_t hit_by_class[8]; /* classes >= 7 share the last bin */
    int64_t sum_ttft_us, max_ttft_us; /* response latency = time to first token (Sec. V-A) */
    int64_t sum_e2e_us, max_e2e_us;
    int64_t makespan_us;  /* last completion time */
    uint64_t tokens_out;  /* decode throughput = tokens_out / makespan */
    uint64_t checksum;    /* order-independent hash of (request, instance, first token, finish) */
    uint64_t attempts;    /* distributor attempts over all counted requests */
    uint64_t reserved;
} maaso_result;

/* Create / destroy a context bound to one CUDA device.  maaso_destroy frees the profile,
 * every trace loaded through the context and its scratch memory. */
MAASO_API int maaso_create(maaso_ctx **out, int cuda_device);
MAASO_API void maaso_destroy(maaso_ctx *ctx);

/* Copy and validate the latency tables (profiler output, Sec. IV-B).  Replaces any earlier
 * profile; traces loaded before stay valid only if n_models did not shrink below their
 * largest model index (checked at eval).  Synchronous. */
MAASO_API int maaso_load_profile(maaso_ctx *ctx, const maaso_profile_desc *desc);

/* Copy and validate a trace (R_x of Alg. 1) with its SLO class table.  `reqs` may be a host
 * or a device pointer, `classes` is a host pointer.  Checks: n >= 0, n < 2^32, arrivals
 * non-negative and non-decreasing, out_tokens >= 1, cls < n_classes, model < n_models of
 * the loaded profile (MAASO_ESTATE if none).  Synchronous.  *out must be released with
 * maaso_free_trace (or by maaso_destroy). */
MAASO_API int maaso_load_trace(maaso_ctx *ctx, const maaso_request *reqs, uint64_t n,
                     const maaso_slo_class *classes, uint32_t n_classes, maaso_trace **out);
MAASO_API void maaso_free_trace(maaso_ctx *ctx, maaso_trace *trace);

/* Score every candidate of `cands` (device pointers) against `trace`: replay the trace
 * through the distributor (Sec. IV-F) and per-instance continuous batching with virtual
 * slots (Sec. V-A), and write one record per candidate to out_results (device,
 * [n_cand]).  Work is enqueued on `cuda_stream` (a cudaStream_t, NULL = default stream).
 * opts->mapping chooses the kernel: MAASO_MAP_AUTO (default) lets the library route the batch (large
 * batches of placements that the trace overloads go to the thread kernel, the rest to the lane groups,
 * where a placement of more than 32 instances gets a warp of its own); the records do not depend on it.
 * The context's scratch memory grows on demand (this may allocate and synchronise on the
 * first call or when a batch is larger than any before). */
MAASO_API int maaso_eval_placements(maaso_ctx *ctx, const maaso_trace *trace, const maaso_cand_batch *cands,
                          const maaso_eval_opts *opts, maaso_result *out_results, void *cuda_stream);

/* The same batch of candidates scored against several traces in ONE pass (the load sweep of a
 * placement study: the same candidate space under different arrival rates or burstiness).  traces:
 * host array of n_traces <= 16 handles of this context, all loaded with the same SLO class table;
 * out_results (device): n_traces blocks of n_cand records, record c of trace t at
 * out_results[t * n_cand + c]; opts->rejected_by_model and opts->ttft_hist, if given, are laid out
 * the same way ([n_traces * n_cand][...]).  Each record equals what maaso_eval_placements returns
 * for that trace alone; scoring them together lets small candidate sets fill the GPU.  Lane-group
 * and thread mappings only: dump buffers and MAASO_MAP_BLOCK are refused.  A placement of more than 32
 * instances is scored by the thread kernel where the batch goes there, else one warp replays it with the
 * lane-group code (four instances per lane).  No engine and no mapping refuses a placement of
 * MAASO_MAX_INSTANCES instances or fewer.  Enqueued on cuda_stream. */
MAASO_API int maaso_eval_placements_multi(maaso_ctx *ctx, const maaso_trace *const *traces, uint32_t n_traces,
                                          const maaso_cand_batch *cands, const maaso_eval_opts *opts,
                                          maaso_result *out_results, void *cuda_stream);

/* Same scoring with HOST buffers: copies the candidate batch to the device, scores it,
 * copies the records back into out_results (host, [n_cand]) and synchronises.  Dump
 * buffers, per-model counts and histograms are not supported here (opts->dump_n must be 0,
 * opts->rejected_by_model and opts->ttft_hist NULL). */
MAASO_API int maaso_eval_placements_host(maaso_ctx *ctx, const maaso_trace *trace, const maaso_cand_batch *cands,
                               const maaso_eval_opts *opts, maaso_result *out_results);

/* Select the k best records (the "keep the best solution per GPU count" step of Alg. 1,
 * and the argmax of a sweep).  order 0: scored candidates before invalid ones; more n_hit first; then lower
 * mean time to first token, sum_ttft_us / n_served compared exactly by 128-bit
 * cross-multiplication (a candidate that served nothing ranks after one that served
 * something); then lower index.  out_idx (device, [k]) gets candidate indices, best
 * first, padded with 0xFFFFFFFF when k > n_cand; out_res (device, [k], may be NULL) the
 * matching records (zeroed padding).  k <= MAASO_MAX_TOPK.  Enqueued on cuda_stream. */
MAASO_API int maaso_topk(maaso_ctx *ctx, const maaso_result *results, uint64_t n_cand, uint32_t k,
               uint32_t order, uint32_t *out_idx, maaso_result *out_res, void *cuda_stream);

/* Composite serving score of Sec. IV-D, one double per record (device, [n_cand]):
 *   Phi = alpha * PhiS_n + beta * PhiT_n + (1 - beta) * PhiL_n
 *   PhiS_n = n_hit / n_counted (SLO satisfaction ratio),
 *   PhiT_n = min(tokens_out / makespan [tokens/s], gamma_t) / gamma_t,
 *   PhiL_n = max(gamma_l - mean time to first token [s], 0) / gamma_l.
 * A record that counted nothing has PhiS_n = 0, one that served nothing has PhiT_n = PhiL_n = 0,
 * an invalid candidate scores -1.  Computed in IEEE double without fused operations.
 * gamma_t, gamma_l must be positive and finite.  (The paper uses alpha = 4, beta = 0.3, and
 * alpha = 10 for its MaaSO* variant, Sec. V-A.)  Enqueued on cuda_stream. */
typedef struct {
    double alpha, beta, gamma_t, gamma_l;
} maaso_score_params;

/* Latency percentiles from the histograms maaso_eval_placements filled (opts.ttft_hist): for
 * every candidate c and every requested rank permille[j] (1..1000, host array, n_p <= 16),
 * out[c * n_p + j] (device, int64) = the upper edge in microseconds of the first bin at which the
 * cumulative count reaches ceil(permille[j] * served / 1000), i.e. an upper bound of that
 * percentile that is tight to a factor 1.5; INT64_MAX if it falls in the open last bin, -1 if
 * the candidate served nothing.  The paper reports the mean response latency only (Sec. V-A);
 * tail percentiles are an addition for comparing placements.  Enqueued on cuda_stream. */
MAASO_API int maaso_ttft_percentiles(maaso_ctx *ctx, const uint32_t *ttft_hist, uint64_t n_cand,
                                     const uint32_t *permille, uint32_t n_p, int64_t *out, void *cuda_stream);
MAASO_API int maaso_score(maaso_ctx *ctx, const maaso_result *results, uint64_t n_cand,
                          const maaso_score_params *params, double *out_scores, void *cuda_stream);

/* Top-k by score (the "if phi > Phi*[k]" selection of Alg. 1 over a batch): higher score first,
 * then lower index; NaN scores rank last.  Outputs as maaso_topk. */
MAASO_API int maaso_topk_scores(maaso_ctx *ctx, const maaso_result *results, const double *scores,
                                uint64_t n_cand, uint32_t k, uint32_t *out_idx, maaso_result *out_res,
                                void *cuda_stream);

/* Alg. 1, "Simulator-Based Instance Configuration": greedy instance deployment for one
 * sub-cluster of `gpus` devices, scored on the requests of `trace` whose class bit is set in
 * class_mask (all requests if use_mask == 0).  For every configuration (strategy, batch cap) of the
 * caller's (already pruned) list, starting from the empty placement: while devices remain and a
 * model is not saturated, add an instance of the non-saturated model with the most unserved
 * requests (ties: lowest index), evaluate the tentative placement (maaso_eval_placements +
 * maaso_score), accept it if the score improved, else mark the model saturated; the best score
 * and placement per device count are kept.  All configurations advance together, so each greedy
 * step is ONE batch of tentative placements on the GPU.  The device count k that indexes the outputs
 * is that of the placement stored there (Sec. IV-E: "solutions for all possible GPU allocations k"),
 * so istar_inst[k] occupies exactly k devices; the listing's k, taken before the tentative instance
 * is added, would file an accepted placement under fewer devices than it needs.
 * A tentative placement that violates a constraint scores -1 and is never accepted.
 * Host pointers: configs[n_configs]; outputs phi_star[gpus+1], istar_len[gpus+1],
 * istar_inst[(gpus+1) * MAASO_MAX_INSTANCES] (packed instance words).  Synchronous; uses the
 * context's own stream and scratch memory.  gpus <= 4096. */
typedef struct {
    uint32_t strategy;
    uint32_t batch;
} maaso_config;
MAASO_API int maaso_ins_deploy(maaso_ctx *ctx, const maaso_trace *trace, uint32_t gpus,
                               const maaso_config *configs, uint32_t n_configs, int use_mask,
                               uint32_t class_mask, const maaso_score_params *score, uint32_t flags,
                               double *phi_star, uint32_t *istar_len, uint32_t *istar_inst);

/* getPrunedConfigs of Alg. 1: the configuration tree (Sec. III-C) after the two pruning rules of
 * Sec. IV-D.  (1) On the tables: a strategy is dropped if another one needs no more devices, hosts
 * every model it hosts and is at least as fast for those models at every decode level and in
 * prefill (identical rows keep the lower index), or if no model fits on it.  (2) By simulation on the trace (class_mask as in
 * maaso_ins_deploy): for each remaining strategy and each batch cap of `batches`, a probe placement
 * with one instance of every model that fits is scored (all probes in one batch); a cap is kept
 * iff no other cap of the strategy has >= SLO hits and <= mean time to first token with one of
 * them strictly better (exact comparison; equal outcomes keep the smaller cap).
 * Result in tree order (strategies by increasing level-1 decode step of model 0, caps ascending):
 * out_configs (host, capacity n_strategies * n_batches), *out_n.  Synchronous. */
MAASO_API int maaso_prune_configs(maaso_ctx *ctx, const maaso_trace *trace, int use_mask, uint32_t class_mask,
                                  const uint32_t *batches, uint32_t n_batches, uint32_t flags,
                                  maaso_config *out_configs, uint32_t *out_n);

/* Alg. 2, "Dynamic Resource Partition", for two sub-clusters: R_t / R_l are the requests whose
 * class bit is set in mask_t / mask_l.  G'_l = floor(|R_l| * gpus / (|R_t| + |R_l|));
 * maaso_ins_deploy on (R_l, G'_l) and on (R_t, gpus); Phi_opt starts at the best score of
 * maaso_ins_deploy on (R_t + R_l, gpus) if `baseline` is non-zero (homogeneous fallback), else
 * at 0; then g_l = 1..G'_l, g_t = gpus - g_l, keeping the pair with the largest
 * Phi_t*[g_t] + Phi_l*[g_l] if it is strictly better.  Host outputs: out_g[2] = (g_t, g_l), both 0
 * when no partition beat Phi_opt; *out_phi; the two placements (packed words, up to
 * MAASO_MAX_INSTANCES each) with their lengths.  Synchronous. */
MAASO_API int maaso_partition(maaso_ctx *ctx, const maaso_trace *trace, uint32_t mask_t, uint32_t mask_l,
                              uint32_t gpus, const maaso_config *configs, uint32_t n_configs,
                              const maaso_score_params *score, uint32_t flags, int baseline, uint32_t *out_g,
                              double *out_phi, uint32_t *len_t, uint32_t *inst_t, uint32_t *len_l,
                              uint32_t *inst_l);

/* Top-k without any allocation.  (The paper has no counterpart; this is a deployment
 * variant of maaso_topk.)  It is meant for callers that must not allocate device memory
 * while they run: code inside a memory-pool or arena framework that owns all device memory,
 * a latency-critical serving loop where an allocation would synchronise the device, or a
 * process that is already close to its memory limit.  Same inputs, outputs and ordering
 * as maaso_topk, no context needed; the partial lists of the selection passes live in a
 * fixed array of about 0.8 MB inside the library image (every GPU that loads the library
 * holds it until the process exits) instead of context scratch memory.
 * Limits: n_cand <= MAASO_NOALLOC_MAX_CAND and k <= MAASO_NOALLOC_MAX_K; anything larger
 * returns MAASO_ETOOBIG and does nothing.  The call uses the current CUDA device and calls
 * no cudaMalloc / cudaFree or other allocating routine.  Every call looks up the array's address
 * on the current device (nothing is cached, so a re-created context or several host threads are
 * fine); the first call on a device may make the runtime load the library's device code, so make
 * that first call before starting any stream capture.
 * All calls on a device share the one array: two calls whose kernels may overlap on the
 * GPU (different streams, no ordering between them) race on it, so order them.  Nothing
 * in the array needs clearing between calls: each pass overwrites what the next one reads. */
#define MAASO_NOALLOC_MAX_CAND (1u << 20)
#define MAASO_NOALLOC_MAX_K 64
MAASO_API int maaso_topk_noalloc(const maaso_result *results, uint64_t n_cand, uint32_t k, uint32_t order,
                                 uint32_t *out_idx, maaso_result *out_res, void *cuda_stream);

/* Optional device timing.  While enabled, maaso_eval_placements and maaso_topk record CUDA
 * events on the caller's stream around each kernel family; maaso_get_timing waits for the
 * events of the most recent calls and reports milliseconds (0 for a family that did not
 * run).  Off by default; costs a few event records per call when on. */
typedef struct {
    float prep_ms;  /* validation, routing + bucket sort (+ dump buffer fill) */
    float group_ms; /* lane-group scoring kernel */
    float block_ms; /* block-layout scoring kernels and the one-warp-per-placement kernel for more than 32 instances */
    float topk_ms;  /* all passes of the last maaso_topk */
    float thread_ms; /* thread-mapping scoring kernel */
} maaso_timing;
MAASO_API int maaso_set_timing(maaso_ctx *ctx, int enabled);
MAASO_API int maaso_get_timing(maaso_ctx *ctx, maaso_timing *out);

/* Number of kernels this context has launched so far (for accounting in benchmarks). */
MAASO_API uint64_t maaso_launch_count(const maaso_ctx *ctx);

/* Test hook for the out-of-memory paths (no counterpart in the paper): the next `count` times the
 * context would grow one of its scratch buffers, the growth is refused as if the device had no
 * memory left.  The call that needed it returns MAASO_ENOMEM and enqueues nothing; the context
 * keeps the buffers it had, stays usable, and the next call allocates normally.  count = 0
 * switches the hook off. */
MAASO_API int maaso_test_fail_allocs(maaso_ctx *ctx, int count);

/* Text for a return code; for MAASO_ECUDA the context keeps the CUDA error string. */
MAASO_API const char *maaso_strerror(int code);
MAASO_API const char *maaso_last_error(const maaso_ctx *ctx);

#ifdef __cplusplus
}
#endif
#endif /* MAASO_H */
