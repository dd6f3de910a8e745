// C ABI of the placement-scoring library: handles, validation, host<->device copies and
// kernel launches.  Semantics of every entry point are documented in include/maaso.h.
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <string>
#include <vector>

#include "common.cuh"

namespace maaso {
cudaError_t launch_prep(const EvalParams& P, const uint32_t* dump_idx, cudaStream_t stream, int* launches);
cudaError_t launch_rej_hash(uint64_t* out, uint32_t n);
cudaError_t launch_cook_trace(const uint4* reqs, const int64_t* classes, uint4* out, uint32_t n);
cudaError_t launch_scan_trace(const uint4* reqs, const int64_t* classes, uint4* scan, uint32_t n);
size_t scan_trace_units(uint32_t n);
cudaError_t launch_eval_group(const EvalParams& P, int grid, int tile_recs, int blocks_per_sm, int smem_per_sm,
                              cudaStream_t stream);
int occupancy_eval_group(const EvalParams& P, int tile_recs, int blocks_per_sm, int smem_per_sm);
size_t group_scratch_per_lane();
cudaError_t launch_eval_thread(const EvalParams& P, int grid, uint32_t pool_bytes, uint32_t hot_bytes, uint32_t theta,
                               void* arena, cudaStream_t stream);
int occupancy_eval_thread(const EvalParams& P, uint32_t pool_bytes, uint32_t hot_bytes, bool in_smem);
size_t thread_scratch_per_warp(uint32_t pool_bytes);
uint32_t thread_fixed_smem(uint32_t n_models, uint32_t n_rows);
cudaError_t launch_eval_wide(const EvalParams& P, int grid, cudaStream_t stream);
int occupancy_eval_wide(const EvalParams& P);
size_t wide_scratch_per_warp();
cudaError_t launch_eval_block(const EvalParams& P, int bucket, int grid, int tile_recs, cudaStream_t stream);
cudaError_t launch_eval_block_reg(const EvalParams& P, int bucket, int grid, int tile_recs, cudaStream_t stream);
int occupancy_eval_block_reg(const EvalParams& P, int bucket, int tile_recs);
int occupancy_eval_block(const EvalParams& P, int bucket, int tile_recs);
size_t block_payload_per_cta(int bucket);
size_t topk_scratch_bytes(uint64_t n_cand, uint32_t k);
cudaError_t launch_topk(const maaso_result* results, uint64_t n_cand, uint32_t k, void* scratch,
                        uint32_t* out_idx, maaso_result* out_res, cudaStream_t stream, int* launches,
                        const double* scores);
cudaError_t launch_score(const maaso_result* res, uint64_t n, const maaso_score_params& p, double* out,
                         cudaStream_t stream);
cudaError_t launch_ttft_percentiles(const uint32_t* hist, uint64_t n, const uint32_t* permille, uint32_t n_p,
                                    int64_t* out, cudaStream_t stream);
}  // namespace maaso

using namespace maaso;

struct maaso_trace {
    maaso_ctx* owner;
    uint4* d_reqs;
    int64_t* d_classes;
    uint64_t* d_rej_hash;
    uint4* d_cooked;  // prepared records for the lane-group kernel
    uint4* d_scan;    // scan records for the thread mapping
    uint64_t* d_class_tot;  // per class: number of requests, sum of their "rejected" checksum terms
    std::vector<int64_t> h_classes;  // host copy of the class table (several traces in one call must agree on it)
    uint64_t n;
    uint32_t n_classes;
    uint32_t max_model;
    double tok_rate;  // output tokens per second the trace asks for (routing hint of MAASO_MAP_AUTO)
};

struct maaso_ctx {
    int device;
    int sm_count;
    bool has_profile;
    uint32_t n_models, n_strategies, n_rows;
    int32_t* d_rows;
    int32_t* d_devices;
    int32_t* d_min_devices;
    std::vector<int32_t> h_devices;  // host copies for the Alg. 1 driver and the pruning rules
    std::vector<int32_t> h_min_devices;
    std::vector<int32_t> h_rows;
    std::vector<maaso_trace*> traces;
    void* scratch;
    size_t scratch_bytes;
    void* topk_scratch;
    size_t topk_scratch_bytes;
    // staging for the host-buffer entry point
    void* stage;
    size_t stage_bytes;
    void* deploy;
    size_t deploy_bytes;
    cudaStream_t own_stream;
    uint64_t launches;
    int tile_recs;
    int group_blocks;  // blocks of the lane-group kernel per SM its key pool is sized for; 0 = by batch size
    int smem_per_sm;
    int promote_pct;  // share of the spare resident warps the planner may use for promotions
    int thread_arena_kb;  // thread mapping: KB of global memory per warp for the cold part of the placements' state, 0 = shared memory
    int thread_hot_kb;    // with an arena: KB of shared memory per warp for the hot part
    bool thread_blocks_set;  // MAASO_THREAD_BLOCKS was given: also caps the resident warps per SM in arena mode
    int thread_blocks;   // one-warp blocks of the thread-mapping kernel per SM its pool is sized for
    uint32_t thread_theta;     // waiting lanes of a warp that trigger a distributor round in the thread mapping
    uint32_t thread_min_cand;  // MAASO_MAP_AUTO takes the thread mapping from this many candidates on
    uint32_t last_mapping;     // mapping the most recent scoring call resolved to
    int fail_allocs;           // test hook: this many of the next scratch allocations are refused
    bool timing;
    cudaEvent_t ev[7];   // eval: start, after prep, after group, after block; topk: start, end; eval: after thread
    bool ev_eval, ev_topk;
    std::string last_error;
};

namespace {

struct DeviceGuard {
    int prev;
    bool ok;
    explicit DeviceGuard(int dev) : prev(-1), ok(true) {
        if (cudaGetDevice(&prev) != cudaSuccess) prev = -1;
        if (prev != dev) ok = cudaSetDevice(dev) == cudaSuccess;
    }
    ~DeviceGuard() {
        if (prev >= 0) cudaSetDevice(prev);
    }
};

int cuda_fail(maaso_ctx* ctx, cudaError_t e, const char* what) {
    if (ctx) ctx->last_error = std::string(what) + ": " + cudaGetErrorString(e);
    cudaGetLastError();  // clear the sticky-free error state
    return e == cudaErrorMemoryAllocation ? MAASO_ENOMEM : MAASO_ECUDA;
}

int fail(maaso_ctx* ctx, int code, const char* what) {
    if (ctx) ctx->last_error = what;
    return code;
}

int grow(maaso_ctx* ctx, void** buf, size_t* have, size_t need) {
    if (need <= *have) return MAASO_OK;
    if (ctx && ctx->fail_allocs > 0) {  // test hook: behave as if the allocation had been refused
        ctx->fail_allocs--;
        return fail(ctx, MAASO_ENOMEM, "scratch allocation refused (test hook)");
    }
    cudaError_t e = cudaDeviceSynchronize();
    if (e != cudaSuccess) return cuda_fail(ctx, e, "synchronize before growing scratch");
    if (*buf) cudaFree(*buf);
    *buf = nullptr;
    *have = 0;
    need = (need + (size_t)(1 << 20) - 1) & ~((size_t)(1 << 20) - 1);
    e = cudaMalloc(buf, need);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "scratch allocation");
    *have = need;
    return MAASO_OK;
}

size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// Checksum term of "request r was rejected": the SplitMix64 output mixer (public domain) of
// r * 0x9E3779B97F4A7C15 ^ all-ones, as the kernels compute it.
uint64_t host_rejected_hash(uint32_t r) {
    uint64_t z = (uint64_t)r * 0x9E3779B97F4A7C15ull ^ ~0ull;
    z ^= z >> 30; z *= 0xBF58476D1CE4E5B9ull;
    z ^= z >> 27; z *= 0x94D049BB133111EBull;
    z ^= z >> 31;
    return z;
}

}  // namespace

extern "C" {

MAASO_API int maaso_create(maaso_ctx** out, int cuda_device) {
    if (!out) return MAASO_EINVAL;
    *out = nullptr;
    int count = 0;
    cudaError_t e = cudaGetDeviceCount(&count);
    if (e != cudaSuccess) return cuda_fail(nullptr, e, "cudaGetDeviceCount");
    if (cuda_device < 0 || cuda_device >= count) return MAASO_EINVAL;
    maaso_ctx* ctx = new (std::nothrow) maaso_ctx();
    if (!ctx) return MAASO_ENOMEM;
    ctx->device = cuda_device;
    ctx->has_profile = false;
    ctx->d_rows = ctx->d_devices = ctx->d_min_devices = nullptr;
    ctx->scratch = ctx->topk_scratch = ctx->stage = ctx->deploy = nullptr;
    ctx->scratch_bytes = ctx->topk_scratch_bytes = ctx->stage_bytes = ctx->deploy_bytes = 0;
    ctx->launches = 0;
    ctx->tile_recs = 64;
    ctx->group_blocks = 0;
    ctx->own_stream = nullptr;
    ctx->timing = false;
    ctx->ev_eval = ctx->ev_topk = false;
    for (int i = 0; i < 7; i++) ctx->ev[i] = nullptr;
    DeviceGuard g(cuda_device);
    cudaDeviceProp prop;
    e = cudaGetDeviceProperties(&prop, cuda_device);
    if (e != cudaSuccess || !g.ok) {
        delete ctx;
        return cuda_fail(nullptr, e, "cudaGetDeviceProperties");
    }
    if (prop.major < 10) {  // the kernels are built for sm_100a only
        delete ctx;
        return MAASO_ESTATE;
    }
    ctx->sm_count = prop.multiProcessorCount;
    ctx->smem_per_sm = (int)prop.sharedMemPerMultiprocessor;
    e = cudaStreamCreateWithFlags(&ctx->own_stream, cudaStreamNonBlocking);
    if (e != cudaSuccess) {
        delete ctx;
        return cuda_fail(nullptr, e, "cudaStreamCreate");
    }
    ctx->promote_pct = 100;
    const char* pp = getenv("MAASO_PROMOTE_PCT");
    if (pp) {
        int v = atoi(pp);
        if (v >= 0 && v <= 100) ctx->promote_pct = v;
    }
    const char* env = getenv("MAASO_TILE_RECS");
    if (env) {
        int v = atoi(env);
        if (v >= 16 && v <= 2048) ctx->tile_recs = v & ~1;  // even: tiles of 8-byte terms stay 16-byte aligned
    }

    ctx->thread_arena_kb = 128;
    const char* ta = getenv("MAASO_THREAD_ARENA_KB");
    if (ta) {
        int v = atoi(ta);
        if (v >= 0 && v <= 1023) ctx->thread_arena_kb = v;
    }
    ctx->thread_hot_kb = 10;
    const char* thk = getenv("MAASO_THREAD_HOT_KB");
    if (thk) {
        int v = atoi(thk);
        if (v >= 2 && v <= 128) ctx->thread_hot_kb = v;
    }
    ctx->thread_blocks = 6;
    ctx->thread_blocks_set = false;
    const char* tb = getenv("MAASO_THREAD_BLOCKS");
    if (tb) {
        int v = atoi(tb);
        if (v >= 1 && v <= 16) { ctx->thread_blocks = v; ctx->thread_blocks_set = true; }
    }
    ctx->thread_theta = 8;
    const char* tt = getenv("MAASO_THREAD_THETA");
    if (tt) {
        int v = atoi(tt);
        if (v >= 1 && v <= 32) ctx->thread_theta = (uint32_t)v;
    }
    ctx->thread_min_cand = 16384;  // fewer loaded placements than this do not fill the GPU one per lane
    const char* tm = getenv("MAASO_THREAD_MIN_CAND");
    if (tm) {
        long v = atol(tm);
        if (v >= 0) ctx->thread_min_cand = (uint32_t)v;
    }
    ctx->last_mapping = MAASO_MAP_GROUP;
    ctx->fail_allocs = 0;
    const char* gb = getenv("MAASO_GROUP_BLOCKS");
    if (gb) {
        int v = atoi(gb);
        if (v >= 0 && v <= 8) ctx->group_blocks = v;
    }
    *out = ctx;
    return MAASO_OK;
}

MAASO_API void maaso_free_trace(maaso_ctx* ctx, maaso_trace* trace) {
    if (!ctx || !trace || trace->owner != ctx) return;
    DeviceGuard g(ctx->device);
    cudaDeviceSynchronize();
    for (size_t i = 0; i < ctx->traces.size(); i++)
        if (ctx->traces[i] == trace) {
            ctx->traces.erase(ctx->traces.begin() + i);
            break;
        }
    if (trace->d_reqs) cudaFree(trace->d_reqs);
    if (trace->d_classes) cudaFree(trace->d_classes);
    if (trace->d_rej_hash) cudaFree(trace->d_rej_hash);
    if (trace->d_cooked) cudaFree(trace->d_cooked);
    if (trace->d_scan) cudaFree(trace->d_scan);
    if (trace->d_class_tot) cudaFree(trace->d_class_tot);
    delete trace;
}

MAASO_API void maaso_destroy(maaso_ctx* ctx) {
    if (!ctx) return;
    DeviceGuard g(ctx->device);
    cudaDeviceSynchronize();
    while (!ctx->traces.empty()) maaso_free_trace(ctx, ctx->traces.back());
    if (ctx->d_rows) cudaFree(ctx->d_rows);
    if (ctx->d_devices) cudaFree(ctx->d_devices);
    if (ctx->d_min_devices) cudaFree(ctx->d_min_devices);
    if (ctx->scratch) cudaFree(ctx->scratch);
    if (ctx->topk_scratch) cudaFree(ctx->topk_scratch);
    if (ctx->stage) cudaFree(ctx->stage);
    if (ctx->deploy) cudaFree(ctx->deploy);
    if (ctx->own_stream) cudaStreamDestroy(ctx->own_stream);
    for (int i = 0; i < 7; i++)
        if (ctx->ev[i]) cudaEventDestroy(ctx->ev[i]);
    delete ctx;
}

MAASO_API int maaso_load_profile(maaso_ctx* ctx, const maaso_profile_desc* d) {
    if (!ctx || !d) return MAASO_EINVAL;
    if (!d->devices || !d->min_devices || !d->prefill_base_us || !d->prefill_q16 || !d->step_us)
        return fail(ctx, MAASO_EINVAL, "profile: null table");
    if (d->n_models < 1 || d->n_models > MAASO_MAX_MODELS || d->n_strategies < 1 ||
        d->n_strategies > MAASO_MAX_STRATEGIES || d->n_models * d->n_strategies > MAASO_MAX_ROWS ||
        d->wmax != MAASO_WMAX)
        return fail(ctx, MAASO_EINVAL, "profile: table shape out of range");
    const uint32_t M = d->n_models, S = d->n_strategies, R = M * S;
    for (uint32_t s = 0; s < S; s++)
        if (d->devices[s] < 1) return fail(ctx, MAASO_EINVAL, "profile: devices[s] < 1");
    for (uint32_t m = 0; m < M; m++)
        if (d->min_devices[m] < 0) return fail(ctx, MAASO_EINVAL, "profile: min_devices[m] < 0");
    std::vector<int32_t> rows((size_t)R * kRowStride);
    for (uint32_t r = 0; r < R; r++) {
        if (d->prefill_base_us[r] < 0 || d->prefill_q16[r] < 0)
            return fail(ctx, MAASO_EINVAL, "profile: negative prefill cost");
        rows[(size_t)r * kRowStride + 0] = d->prefill_base_us[r];
        rows[(size_t)r * kRowStride + 1] = d->prefill_q16[r];
        for (uint32_t w = 0; w < MAASO_WMAX; w++) {
            const int32_t v = d->step_us[(size_t)r * MAASO_WMAX + w];
            if (v < 1 || v > MAASO_MAX_STEP_US) return fail(ctx, MAASO_EINVAL, "profile: step_us out of range");
            rows[(size_t)r * kRowStride + 2 + w] = v;
        }
    }
    DeviceGuard g(ctx->device);
    cudaError_t e = cudaDeviceSynchronize();
    if (e != cudaSuccess) return cuda_fail(ctx, e, "synchronize");
    if (ctx->d_rows) cudaFree(ctx->d_rows);
    if (ctx->d_devices) cudaFree(ctx->d_devices);
    if (ctx->d_min_devices) cudaFree(ctx->d_min_devices);
    ctx->d_rows = ctx->d_devices = ctx->d_min_devices = nullptr;
    ctx->has_profile = false;
    if ((e = cudaMalloc(&ctx->d_rows, rows.size() * 4)) != cudaSuccess) return cuda_fail(ctx, e, "profile alloc");
    if ((e = cudaMalloc(&ctx->d_devices, S * 4)) != cudaSuccess) return cuda_fail(ctx, e, "profile alloc");
    if ((e = cudaMalloc(&ctx->d_min_devices, M * 4)) != cudaSuccess) return cuda_fail(ctx, e, "profile alloc");
    if ((e = cudaMemcpy(ctx->d_rows, rows.data(), rows.size() * 4, cudaMemcpyHostToDevice)) != cudaSuccess ||
        (e = cudaMemcpy(ctx->d_devices, d->devices, S * 4, cudaMemcpyHostToDevice)) != cudaSuccess ||
        (e = cudaMemcpy(ctx->d_min_devices, d->min_devices, M * 4, cudaMemcpyHostToDevice)) != cudaSuccess)
        return cuda_fail(ctx, e, "profile copy");
    ctx->h_devices.assign(d->devices, d->devices + S);
    ctx->h_min_devices.assign(d->min_devices, d->min_devices + M);
    ctx->h_rows = rows;
    ctx->n_models = M;
    ctx->n_strategies = S;
    ctx->n_rows = R;
    ctx->has_profile = true;
    return MAASO_OK;
}

MAASO_API int maaso_load_trace(maaso_ctx* ctx, const maaso_request* reqs, uint64_t n, const maaso_slo_class* classes,
                     uint32_t n_classes, maaso_trace** out) {
    if (!ctx || !out) return MAASO_EINVAL;
    *out = nullptr;
    if (!ctx->has_profile) return fail(ctx, MAASO_ESTATE, "trace: load a profile first");
    if ((!reqs && n) || !classes || n_classes < 1 || n_classes > MAASO_MAX_CLASSES || n >= 0xFFFFFFFFull)
        return fail(ctx, MAASO_EINVAL, "trace: null pointer or size out of range");
    const int64_t kLimMax = (int64_t)1 << 40;
    std::vector<int64_t> cls((size_t)n_classes * 3);
    for (uint32_t k = 0; k < n_classes; k++) {
        const int64_t v[3] = {classes[k].ttft_us, classes[k].tbt_us, classes[k].e2e_us};
        for (int j = 0; j < 3; j++) {
            if (v[j] > kLimMax) return fail(ctx, MAASO_EINVAL, "trace: SLO limit above 2^40 us");
            cls[(size_t)k * 3 + j] = v[j] < 0 ? -1 : v[j];
        }
    }
    DeviceGuard g(ctx->device);
    // the requests may live on the host or on the device; validate on a host copy
    const maaso_request* host = reqs;
    std::vector<maaso_request> tmp;
    bool on_device = false;
    if (n) {
        cudaPointerAttributes attr;
        cudaError_t pe = cudaPointerGetAttributes(&attr, reqs);
        if (pe != cudaSuccess) cudaGetLastError();
        on_device = pe == cudaSuccess && (attr.type == cudaMemoryTypeDevice || attr.type == cudaMemoryTypeManaged);
        if (on_device) {
            tmp.resize(n);
            cudaError_t e = cudaMemcpy(tmp.data(), reqs, n * sizeof(maaso_request), cudaMemcpyDeviceToHost);
            if (e != cudaSuccess) return cuda_fail(ctx, e, "trace copy to host");
            host = tmp.data();
        }
    }
    int64_t prev = 0;
    uint32_t max_model = 0;
    const int64_t kArrMax = (int64_t)1 << 50;
    // per class: how many requests, and the sum of their checksum terms as rejected requests (the thread
    // mapping starts from "everything counted was rejected" and takes the served ones out)
    std::vector<uint64_t> class_tot((size_t)n_classes * 2, 0);
    uint64_t tok_sum = 0;
    for (uint64_t r = 0; r < n; r++) {
        const maaso_request& q = host[r];
        if (q.arrival_us < prev || q.arrival_us > kArrMax)
            return fail(ctx, MAASO_EINVAL, "trace: arrivals must be non-negative, non-decreasing, below 2^50");
        prev = q.arrival_us;
        if (q.out_tokens < 1) return fail(ctx, MAASO_EINVAL, "trace: out_tokens must be >= 1");
        if (q.cls >= n_classes) return fail(ctx, MAASO_EINVAL, "trace: unknown SLO class");
        if (q.model >= ctx->n_models) return fail(ctx, MAASO_EINVAL, "trace: unknown model");
        if (q.model > max_model) max_model = q.model;
        tok_sum += q.out_tokens;
        class_tot[(size_t)q.cls * 2] += 1;
        class_tot[(size_t)q.cls * 2 + 1] += host_rejected_hash((uint32_t)r);
    }
    maaso_trace* t = new (std::nothrow) maaso_trace();
    if (!t) return MAASO_ENOMEM;
    t->owner = ctx;
    t->d_reqs = nullptr;
    t->d_classes = nullptr;
    t->d_rej_hash = nullptr;
    t->d_cooked = nullptr;
    t->d_scan = nullptr;
    t->d_class_tot = nullptr;
    t->n = n;
    t->n_classes = n_classes;
    t->max_model = max_model;
    {
        const double span_s = n > 1 ? (double)(host[n - 1].arrival_us - host[0].arrival_us) * 1e-6 : 0.0;
        t->tok_rate = span_s > 0.0 ? (double)tok_sum / span_s : 0.0;
    }
    t->h_classes = cls;
    cudaError_t e = cudaMalloc(&t->d_reqs, (n ? n : 1) * sizeof(maaso_request));
    if (e == cudaSuccess) e = cudaMalloc(&t->d_classes, cls.size() * 8);
    if (e == cudaSuccess) e = cudaMalloc(&t->d_rej_hash, (n ? n : 1) * 8);
    if (e == cudaSuccess) e = cudaMalloc(&t->d_cooked, (n ? n : 1) * 16 * kCookedWords);
    if (e == cudaSuccess) e = cudaMalloc(&t->d_scan, scan_trace_units((uint32_t)n) * 16);
    if (e == cudaSuccess) e = cudaMalloc(&t->d_class_tot, (size_t)n_classes * 16);
    if (e == cudaSuccess) e = cudaMemcpy(t->d_class_tot, class_tot.data(), (size_t)n_classes * 16, cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = launch_rej_hash(t->d_rej_hash, (uint32_t)n);
    if (e == cudaSuccess) e = cudaDeviceSynchronize();
    if (e == cudaSuccess && n)
        e = cudaMemcpy(t->d_reqs, reqs, n * sizeof(maaso_request),
                       on_device ? cudaMemcpyDeviceToDevice : cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaMemcpy(t->d_classes, cls.data(), cls.size() * 8, cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = launch_cook_trace(t->d_reqs, t->d_classes, t->d_cooked, (uint32_t)n);
    if (e == cudaSuccess) e = launch_scan_trace(t->d_reqs, t->d_classes, t->d_scan, (uint32_t)n);
    if (e == cudaSuccess) e = cudaDeviceSynchronize();
    if (e != cudaSuccess) {
        if (t->d_cooked) cudaFree(t->d_cooked);
        if (t->d_scan) cudaFree(t->d_scan);
        if (t->d_class_tot) cudaFree(t->d_class_tot);
        if (t->d_reqs) cudaFree(t->d_reqs);
        if (t->d_classes) cudaFree(t->d_classes);
        if (t->d_rej_hash) cudaFree(t->d_rej_hash);
        delete t;
        return cuda_fail(ctx, e, "trace upload");
    }
    ctx->traces.push_back(t);
    *out = t;
    return MAASO_OK;
}

// Scoring of one candidate batch against n_traces traces (1 = the plain call).
static int eval_impl(maaso_ctx* ctx, const maaso_trace* const* traces, uint32_t n_traces,
                     const maaso_cand_batch* cands, const maaso_eval_opts* opts, maaso_result* out_results,
                     void* cuda_stream) {
    if (!ctx || !traces || !cands || n_traces < 1 || n_traces > (uint32_t)kMaxTraces) return MAASO_EINVAL;
    if (!ctx->has_profile) return fail(ctx, MAASO_ESTATE, "eval: no profile loaded");
    const maaso_trace* trace = traces[0];
    uint64_t n_max = 0;
    for (uint32_t t = 0; t < n_traces; t++) {
        const maaso_trace* x = traces[t];
        if (!x) return MAASO_EINVAL;
        if (x->owner != ctx) return fail(ctx, MAASO_ESTATE, "eval: trace belongs to another context");
        if (x->n && x->max_model >= ctx->n_models)
            return fail(ctx, MAASO_ESTATE, "eval: trace refers to a model the current profile lacks");
        if (x->h_classes != trace->h_classes)
            return fail(ctx, MAASO_EINVAL, "eval: traces scored in one call must have the same SLO classes");
        if (x->n > n_max) n_max = x->n;
    }
    if (cands->n_cand == 0) return MAASO_OK;
    if ((uint64_t)cands->n_cand * n_traces >= 0xFFFFFFFFull)
        return fail(ctx, MAASO_EINVAL, "eval: candidates x traces out of range");
    if (!cands->offsets || !out_results || (cands->n_inst && !cands->inst) || cands->n_cand >= 0xFFFFFFFFull ||
        cands->n_inst >= 0xFFFFFFFFull)
        return fail(ctx, MAASO_EINVAL, "eval: null pointer or size out of range");
    maaso_eval_opts o;
    memset(&o, 0, sizeof(o));
    if (opts) o = *opts;
    if (o.mapping > MAASO_MAP_THREAD) return fail(ctx, MAASO_EINVAL, "eval: unknown mapping");
    if (o.dump_n && !o.dump_cand_idx) return fail(ctx, MAASO_EINVAL, "eval: dump_n without dump_cand_idx");
    if (n_traces > 1 && (o.dump_n || o.mapping == MAASO_MAP_BLOCK))
        return fail(ctx, MAASO_EINVAL, "eval: several traces in one call allow no dump buffers and no block mapping");
    if (o.flags & ~(MAASO_FLAG_PRED_OPTIMISTIC | MAASO_FLAG_ENGINE_FROZEN | MAASO_FLAG_TBT_MAXGAP | MAASO_FLAG_INSTANCE_QUEUES |
                    MAASO_FLAG_TEST_STALL))
        return fail(ctx, MAASO_EINVAL, "eval: unknown flag");
    if ((o.flags & (MAASO_FLAG_ENGINE_FROZEN | MAASO_FLAG_TBT_MAXGAP | MAASO_FLAG_INSTANCE_QUEUES)) &&
        o.mapping == MAASO_MAP_BLOCK)
        return fail(ctx, MAASO_EINVAL,
                    "eval: the fixed-speed engine, per-instance queues and the largest-gap test have no block mapping");
    const bool variant = (o.flags & (MAASO_FLAG_ENGINE_FROZEN | MAASO_FLAG_TBT_MAXGAP | MAASO_FLAG_INSTANCE_QUEUES)) != 0;
    if (variant && o.mapping == MAASO_MAP_THREAD)
        return fail(ctx, MAASO_EINVAL,
                    "eval: the fixed-speed engine, per-instance queues and the largest-gap test have no thread mapping");
    // MAASO_MAP_AUTO: the other engines exist in the lane-group kernel only; for the default engine both the
    // lane-group and the thread kernel are launched and the validation kernels route the batch
    if (o.mapping == MAASO_MAP_AUTO && variant) o.mapping = MAASO_MAP_GROUP;
    ctx->last_mapping = o.mapping;

    DeviceGuard g(ctx->device);
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    const uint32_t C = (uint32_t)cands->n_cand;
    const int tile = ctx->tile_recs;

    EvalParams P;
    memset(&P, 0, sizeof(P));
    P.reqs = trace->d_reqs;
    P.n_req = (uint32_t)trace->n;
    P.n_classes = trace->n_classes;
    P.classes = trace->d_classes;
    P.rej_hash = trace->d_rej_hash;
    P.cooked = trace->d_cooked;
    P.n_traces = n_traces;
    for (uint32_t t = 0; t < n_traces; t++) {
        P.trace_cooked[t] = traces[t]->d_cooked;
        P.trace_scan[t] = traces[t]->d_scan;
        P.trace_class_tot[t] = traces[t]->d_class_tot;
        P.trace_n[t] = (uint32_t)traces[t]->n;
    }
    P.rows = ctx->d_rows;
    P.devices = ctx->d_devices;
    P.min_devices = ctx->d_min_devices;
    P.n_rows = ctx->n_rows;
    P.n_models = ctx->n_models;
    P.n_strategies = ctx->n_strategies;
    P.budget = cands->budget;
    P.offsets = cands->offsets;
    P.inst = cands->inst;
    P.class_mask = cands->class_mask;
    P.n_cand = C;
    P.n_inst = (uint32_t)cands->n_inst;
    P.flags = o.flags & ~MAASO_FLAG_TEST_STALL;
    P.stall_test = (o.flags & MAASO_FLAG_TEST_STALL) ? 1u : 0u;
    P.wait_cycles = P.stall_test ? 200000000ll : kWaitCycles;
    P.mapping = o.mapping;
    P.out = out_results;
    P.dump_n = o.dump_n;
    P.dump_finish = o.dump_finish_us;
    P.dump_first = o.dump_first_us;
    P.dump_inst = o.dump_inst;
    P.rej_by_model = o.rejected_by_model;
    P.ttft_hist = o.ttft_hist;

    // launch shapes: persistent grids bounded by what the batch can use
    // Blocks per SM of the lane-group kernel.  A batch that three blocks per SM can hold in one
    // wave is bound by its longest dependent chains, which run faster with fewer warps sharing a
    // scheduler; a larger batch is bound by instruction issue and wants all four.  Lanes needed
    // ~ instances x 1.3 (group widths are powers of two).
    const bool threads = o.mapping == MAASO_MAP_THREAD || o.mapping == MAASO_MAP_AUTO;
    const bool groups = o.mapping == MAASO_MAP_GROUP || o.mapping == MAASO_MAP_AUTO;
    int group_blocks = ctx->group_blocks;
    if (group_blocks == 0) {
        const uint64_t est_warps = ((cands->n_inst * 13 / 10 + 31) / 32 + 6) * n_traces;
        group_blocks = est_warps <= (uint64_t)ctx->sm_count * 3 * (kGroupThreads / 32) ? 3 : 4;
    }
    int grid_g = 0, grid_t = 0;
    uint32_t thread_pool = 0, thread_hot = 0;
    size_t pay_entries = 0, pay_thread = 0;  // scratch entries of the lane-group / block kernels, of the thread kernel
    static_assert(sizeof(Payload) == 32, "scratch is counted in 32-byte entries");
    if (threads) {
        // thread mapping: one-warp blocks; the pool is what is left of an SM's shared memory when
        // `thread_blocks` of them share it (1 KB per block is reserved by the system)
        // The hot part of the instances (what a prediction reads: 3 units each) is always in shared memory;
        // the cold part (slot masks and keys) is in shared memory too, or in a per-warp arena in global memory,
        // which leaves room for more resident warps.
        size_t pool, hot;
        if (ctx->thread_arena_kb > 0) {
            pool = (size_t)ctx->thread_arena_kb * 1024;
            hot = (size_t)ctx->thread_hot_kb * 1024;
        } else {
            size_t per_block = (size_t)ctx->smem_per_sm / (size_t)ctx->thread_blocks;
            per_block = per_block > 1024 ? per_block - 1024 : 0;
            if (per_block > 227u * 1024u) per_block = 227u * 1024u;
            const size_t fixed = thread_fixed_smem(ctx->n_models, ctx->n_rows);
            const size_t both = per_block > fixed ? per_block - fixed : 0;
            hot = both / 5;  // an instance has 2 hot units and about 9 cold ones
            hot -= hot % 512;
            pool = both - hot;
            pool -= pool % 512;
        }
        if (pool > 65535u * 16u) pool = 65535u * 16u - (65535u * 16u) % 512;  // unit offsets are 16-bit
        if (pool < 4096 || hot < 1536) return fail(ctx, MAASO_ESTATE, "eval: no shared memory for the thread mapping");
        thread_pool = (uint32_t)pool;
        thread_hot = (uint32_t)hot;
        P.thread_pool_units = thread_pool / 16u;
        P.thread_hot_units = thread_hot / 16u;
        int occ_t = occupancy_eval_thread(P, thread_pool, thread_hot, ctx->thread_arena_kb == 0);
        if (ctx->thread_arena_kb > 0 && ctx->thread_blocks_set && occ_t > ctx->thread_blocks) occ_t = ctx->thread_blocks;
        grid_t = ctx->sm_count * occ_t;
        const uint64_t max_items_t = ((uint64_t)C + 9) * n_traces;
        if ((uint64_t)grid_t > max_items_t) grid_t = (int)max_items_t;
        pay_thread = ((size_t)grid_t * (thread_scratch_per_warp(thread_pool) + (ctx->thread_arena_kb > 0 ? thread_pool : 0)) +
                      sizeof(Payload) - 1) / sizeof(Payload);
    }
    if (groups) {
        const int occ_g = occupancy_eval_group(P, tile, group_blocks, ctx->smem_per_sm);
        grid_g = ctx->sm_count * occ_g;
        // at most one work item per 4 candidates + bucket tails, once per trace
        const uint64_t max_items_g = ((uint64_t)C / 4 + 6) * n_traces;
        if ((uint64_t)grid_g > max_items_g) grid_g = (int)max_items_g;
        pay_entries = (size_t)grid_g * kGroupThreads * (group_scratch_per_lane() / sizeof(Payload));
    }
    int grid_b[4];
    for (int b = 6; b <= kGenericBlockBucket; b++) {
        // the block kernels run only when the block mapping is asked for
        grid_b[b - 6] = 0;
        if (!(n_traces == 1 && o.mapping == MAASO_MAP_BLOCK)) continue;
        // placements with at most 8 instances: one warp per instance with register-resident state
        int gb = ctx->sm_count * (b < kGenericBlockBucket ? occupancy_eval_block_reg(P, b, tile)
                                                        : occupancy_eval_block(P, b, tile));
        if ((uint64_t)gb > C) gb = (int)C;
        grid_b[b - 6] = gb;
        const size_t need = b < kGenericBlockBucket ? 0 : (size_t)gb * block_payload_per_cta(b);
        if (need > pay_entries) pay_entries = need;
    }

    // placements of more than 32 instances outside the thread kernel (the other engines; the default engine
    // unless the batch goes to the threads; whatever the thread kernel's pools cannot hold): one warp per
    // placement with the lane-group code
    int grid_w = 0;
    if (o.mapping != MAASO_MAP_BLOCK && cands->n_inst > 32) {
        // As many warps per SM as the registers allow (8) where the batch is made of large placements (more
        // than 16 instances per placement on average): the kernel waits on dependent chains, and four more
        // warps per SM are worth a third of its time.  Elsewhere 4 per SM, which needs no more scratch than
        // the lane-group kernel has anyway (a warp's scratch is a lane-group block's, 1 MB).
        int occ_w = occupancy_eval_wide(P);
        const int occ_cap = cands->n_inst > 16ull * C ? 8 : 4;
        if (occ_w > occ_cap) occ_w = occ_cap;
        grid_w = ctx->sm_count * occ_w;
        // a placement that needs this kernel has more than 32 instances (or, thread mapping forced, more state
        // than a warp's pools): the batch cannot hold more of them than instances / 33
        uint64_t max_items_w = (o.mapping == MAASO_MAP_THREAD ? (uint64_t)C : cands->n_inst / 33u) * n_traces;
        if (max_items_w < 1) max_items_w = 1;
        if ((uint64_t)grid_w > max_items_w) grid_w = (int)max_items_w;
        const size_t need = ((size_t)grid_w * wide_scratch_per_warp() + sizeof(Payload) - 1) / sizeof(Payload);
        if (need > pay_entries) pay_entries = need;
    }

    // scratch layout: counters | bucket lists | dump rows | payload
    size_t off = 0;
    const size_t off_counters = off; off = align_up(off + kCounterWords * 4, 256);
    const size_t off_code = off;     off = align_up(off + (size_t)C * 4, 256);
    const size_t off_code2 = off;    off = align_up(off + (size_t)C * 4, 256);
    const size_t off_lists = off;    off = align_up(off + (size_t)kNumBuckets * C * 4, 256);
    const size_t off_dump = off;     off = align_up(off + (o.dump_n ? (size_t)C * 4 : 0), 256);
    const size_t off_pay = off;      off = align_up(off + pay_entries * sizeof(Payload), 256);
    const size_t off_pay_t = off;    off = align_up(off + pay_thread * sizeof(Payload), 256);
    int rc = grow(ctx, &ctx->scratch, &ctx->scratch_bytes, off);
    if (rc != MAASO_OK) return rc;
    unsigned char* sb = static_cast<unsigned char*>(ctx->scratch);
    P.bucket_count = reinterpret_cast<uint32_t*>(sb + off_counters);
    P.work_ctr = P.bucket_count + 32;
    P.hist = P.bucket_count + 64;
    P.sm_ctr = P.hist + kHistRows * kCostBins;
    P.n_sm = (uint32_t)(ctx->sm_count < 1024 ? ctx->sm_count : 1024);
    P.code = reinterpret_cast<uint32_t*>(sb + off_code);
    P.code2 = reinterpret_cast<uint32_t*>(sb + off_code2);
    P.bucket_list = reinterpret_cast<uint32_t*>(sb + off_lists);
    P.dump_row = o.dump_n ? reinterpret_cast<int32_t*>(sb + off_dump) : nullptr;
    P.payload = reinterpret_cast<Payload*>(sb + off_pay);

    static_assert(64 + kHistRows * kCostBins + 1024 <= kCounterWords, "counter region");
    P.group_warps = (uint32_t)grid_g * (kGroupThreads / 32);
    P.mapping = o.mapping;  // block, lane groups, threads, or auto (routed by the validation kernels)
    P.thread_min_cand = ctx->thread_min_cand;
    {   // output tokens per second the trace(s) ask for (mean over the traces of the call)
        double d = 0.0;
        for (uint32_t t = 0; t < n_traces; t++) d += traces[t]->tok_rate;
        d /= n_traces;
        P.demand_tok_s = d >= 4.0e9 ? 4000000000u : (uint32_t)d;
    }
    P.promote_pct = (uint32_t)ctx->promote_pct;
    cudaError_t e = cudaMemsetAsync(sb + off_counters, 0, kCounterWords * 4, stream);
    if (e == cudaSuccess && o.ttft_hist)
        e = cudaMemsetAsync(o.ttft_hist, 0, (size_t)C * n_traces * MAASO_TTFT_BINS * 4, stream);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "memset");
    int launches = 0;
    if (ctx->timing) cudaEventRecord(ctx->ev[0], stream);
    e = launch_prep(P, o.dump_cand_idx, stream, &launches);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "prep launch");
    if (ctx->timing) cudaEventRecord(ctx->ev[1], stream);
    if (groups) {
        e = launch_eval_group(P, grid_g, tile, group_blocks, ctx->smem_per_sm, stream);
        launches++;
        if (e != cudaSuccess) return cuda_fail(ctx, e, "group kernel launch");
    }
    if (ctx->timing) cudaEventRecord(ctx->ev[2], stream);
    if (threads) {
        // the thread kernel has scratch of its own; its arena (if any) follows the entries of the running requests
        EvalParams PT = P;
        PT.payload = reinterpret_cast<Payload*>(sb + off_pay_t);
        void* arena = ctx->thread_arena_kb > 0
                          ? static_cast<void*>(sb + off_pay_t + (size_t)grid_t * thread_scratch_per_warp(thread_pool))
                          : nullptr;
        e = launch_eval_thread(PT, grid_t, thread_pool, thread_hot, ctx->thread_theta, arena, stream);
        launches++;
        if (e != cudaSuccess) return cuda_fail(ctx, e, "thread kernel launch");
    }
    if (ctx->timing) cudaEventRecord(ctx->ev[6], stream);
    if (grid_w > 0) {
        e = launch_eval_wide(P, grid_w, stream);
        launches++;
        if (e != cudaSuccess) return cuda_fail(ctx, e, "wide kernel launch");
    }
    for (int b = 6; b <= kGenericBlockBucket; b++) {
        if (grid_b[b - 6] == 0) continue;
        e = b < kGenericBlockBucket ? launch_eval_block_reg(P, b, grid_b[b - 6], tile, stream)
                  : launch_eval_block(P, b, grid_b[b - 6], tile, stream);
        launches++;
        if (e != cudaSuccess) return cuda_fail(ctx, e, "block kernel launch");
    }
    if (ctx->timing) {
        cudaEventRecord(ctx->ev[3], stream);
        ctx->ev_eval = true;
    }
    ctx->launches += (uint64_t)launches;
    return MAASO_OK;
}

MAASO_API int maaso_eval_placements(maaso_ctx* ctx, const maaso_trace* trace, const maaso_cand_batch* cands,
                                    const maaso_eval_opts* opts, maaso_result* out_results, void* cuda_stream) {
    if (!trace) return MAASO_EINVAL;
    return eval_impl(ctx, &trace, 1, cands, opts, out_results, cuda_stream);
}

MAASO_API int maaso_eval_placements_multi(maaso_ctx* ctx, const maaso_trace* const* traces, uint32_t n_traces,
                                          const maaso_cand_batch* cands, const maaso_eval_opts* opts,
                                          maaso_result* out_results, void* cuda_stream) {
    return eval_impl(ctx, traces, n_traces, cands, opts, out_results, cuda_stream);
}

MAASO_API int maaso_eval_placements_host(maaso_ctx* ctx, const maaso_trace* trace, const maaso_cand_batch* cands,
                               const maaso_eval_opts* opts, maaso_result* out_results) {
    if (!ctx || !trace || !cands) return MAASO_EINVAL;
    if (opts && (opts->dump_n || opts->rejected_by_model || opts->ttft_hist))
        return fail(ctx, MAASO_EINVAL, "eval_host: dump buffers, per-model counts and histograms are not supported");
    if (cands->n_cand == 0) return MAASO_OK;
    if (!cands->offsets || !out_results || (cands->n_inst && !cands->inst) || cands->n_cand >= 0xFFFFFFFFull ||
        cands->n_inst >= 0xFFFFFFFFull)
        return fail(ctx, MAASO_EINVAL, "eval_host: null pointer or size out of range");
    DeviceGuard g(ctx->device);
    const size_t C = cands->n_cand, NI = cands->n_inst;
    size_t off = 0;
    const size_t o_off = off; off = align_up(off + (C + 1) * 4, 256);
    const size_t o_inst = off; off = align_up(off + (NI ? NI : 1) * 4, 256);
    const size_t o_mask = off; off = align_up(off + C * 4, 256);
    const size_t o_res = off;  off = align_up(off + C * sizeof(maaso_result), 256);
    int rc = grow(ctx, &ctx->stage, &ctx->stage_bytes, off);
    if (rc != MAASO_OK) return rc;
    unsigned char* sb = static_cast<unsigned char*>(ctx->stage);
    cudaStream_t st = ctx->own_stream;
    cudaError_t e = cudaMemcpyAsync(sb + o_off, cands->offsets, (C + 1) * 4, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess && NI) e = cudaMemcpyAsync(sb + o_inst, cands->inst, NI * 4, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess && cands->class_mask)
        e = cudaMemcpyAsync(sb + o_mask, cands->class_mask, C * 4, cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "eval_host: upload");
    maaso_cand_batch dev = *cands;
    dev.offsets = reinterpret_cast<const uint32_t*>(sb + o_off);
    dev.inst = reinterpret_cast<const uint32_t*>(sb + o_inst);
    dev.class_mask = cands->class_mask ? reinterpret_cast<const uint32_t*>(sb + o_mask) : nullptr;
    rc = maaso_eval_placements(ctx, trace, &dev, opts, reinterpret_cast<maaso_result*>(sb + o_res), st);
    if (rc != MAASO_OK) return rc;
    e = cudaMemcpyAsync(out_results, sb + o_res, C * sizeof(maaso_result), cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "eval_host: download");
    return MAASO_OK;
}

MAASO_API int maaso_topk(maaso_ctx* ctx, const maaso_result* results, uint64_t n_cand, uint32_t k, uint32_t order,
               uint32_t* out_idx, maaso_result* out_res, void* cuda_stream) {
    if (!ctx) return MAASO_EINVAL;
    if (k == 0) return MAASO_OK;
    if (!out_idx || (!results && n_cand) || k > MAASO_MAX_TOPK || order != 0 || n_cand >= 0xFFFFFFFFull)
        return fail(ctx, MAASO_EINVAL, "topk: null pointer, k or order out of range");
    DeviceGuard g(ctx->device);
    int rc = grow(ctx, &ctx->topk_scratch, &ctx->topk_scratch_bytes, topk_scratch_bytes(n_cand, k));
    if (rc != MAASO_OK) return rc;
    int launches = 0;
    if (ctx->timing) cudaEventRecord(ctx->ev[4], (cudaStream_t)cuda_stream);
    cudaError_t e = launch_topk(results, n_cand, k, ctx->topk_scratch, out_idx, out_res,
                                (cudaStream_t)cuda_stream, &launches, nullptr);
    if (ctx->timing) {
        cudaEventRecord(ctx->ev[5], (cudaStream_t)cuda_stream);
        ctx->ev_topk = true;
    }
    ctx->launches += (uint64_t)launches;
    if (e != cudaSuccess) return cuda_fail(ctx, e, "topk launch");
    return MAASO_OK;
}

MAASO_API int maaso_score(maaso_ctx* ctx, const maaso_result* results, uint64_t n_cand,
                          const maaso_score_params* params, double* out_scores, void* cuda_stream) {
    if (!ctx || !params) return MAASO_EINVAL;
    if (n_cand == 0) return MAASO_OK;
    if (!results || !out_scores || !(params->gamma_t > 0.0) || !(params->gamma_l > 0.0) ||
        params->gamma_t > 1e300 || params->gamma_l > 1e300)
        return fail(ctx, MAASO_EINVAL, "score: null pointer or non-positive threshold");
    DeviceGuard g(ctx->device);
    cudaError_t e = launch_score(results, n_cand, *params, out_scores, (cudaStream_t)cuda_stream);
    ctx->launches++;
    if (e != cudaSuccess) return cuda_fail(ctx, e, "score launch");
    return MAASO_OK;
}

MAASO_API int maaso_ttft_percentiles(maaso_ctx* ctx, const uint32_t* ttft_hist, uint64_t n_cand,
                                     const uint32_t* permille, uint32_t n_p, int64_t* out, void* cuda_stream) {
    if (!ctx) return MAASO_EINVAL;
    if (n_cand == 0 || n_p == 0) return MAASO_OK;
    if (!ttft_hist || !permille || !out || n_p > 16) return fail(ctx, MAASO_EINVAL, "percentiles: null pointer or more than 16 ranks");
    for (uint32_t j = 0; j < n_p; j++)
        if (permille[j] < 1 || permille[j] > 1000) return fail(ctx, MAASO_EINVAL, "percentiles: rank outside 1..1000");
    DeviceGuard g(ctx->device);
    cudaError_t e = launch_ttft_percentiles(ttft_hist, n_cand, permille, n_p, out, (cudaStream_t)cuda_stream);
    ctx->launches++;
    if (e != cudaSuccess) return cuda_fail(ctx, e, "percentile launch");
    return MAASO_OK;
}

MAASO_API int maaso_topk_scores(maaso_ctx* ctx, const maaso_result* results, const double* scores,
                                uint64_t n_cand, uint32_t k, uint32_t* out_idx, maaso_result* out_res,
                                void* cuda_stream) {
    if (!ctx) return MAASO_EINVAL;
    if (k == 0) return MAASO_OK;
    if (!out_idx || ((!results || !scores) && n_cand) || k > MAASO_MAX_TOPK || n_cand >= 0xFFFFFFFFull)
        return fail(ctx, MAASO_EINVAL, "topk_scores: null pointer or k out of range");
    DeviceGuard g(ctx->device);
    int rc = grow(ctx, &ctx->topk_scratch, &ctx->topk_scratch_bytes, topk_scratch_bytes(n_cand, k));
    if (rc != MAASO_OK) return rc;
    int launches = 0;
    cudaError_t e = launch_topk(results, n_cand, k, ctx->topk_scratch, out_idx, out_res,
                                (cudaStream_t)cuda_stream, &launches, scores);
    ctx->launches += (uint64_t)launches;
    if (e != cudaSuccess) return cuda_fail(ctx, e, "topk_scores launch");
    return MAASO_OK;
}

// Alg. 1 as a host driver: every configuration runs its own greedy chain; the tentative
// placements of all chains in one greedy step are one candidate batch on the GPU.
// Alg. 1 for several independent problems at once (each with its own request subset and device
// count): every greedy chain of every problem proposes its next tentative placement, and all of
// them are scored in ONE batch, so a greedy step costs one trace replay however many problems
// run side by side.  Problem p writes phi_star[p][0..gpus[p]], istar_len[p][..], istar_inst[p][..].
struct DeployProblem {
    uint32_t gpus;
    int use_mask;
    uint32_t class_mask;
    double* phi_star;
    uint32_t* istar_len;
    uint32_t* istar_inst;
};

static int ins_deploy_multi(maaso_ctx* ctx, const maaso_trace* trace, const DeployProblem* prob, uint32_t n_prob,
                            const maaso_config* configs, uint32_t n_configs, const maaso_score_params* score,
                            uint32_t flags) {
    if (!ctx->has_profile) return fail(ctx, MAASO_ESTATE, "ins_deploy: no profile loaded");
    for (uint32_t c = 0; c < n_configs; c++)
        if (configs[c].strategy >= ctx->n_strategies || configs[c].batch < 1 || configs[c].batch > MAASO_WMAX)
            return fail(ctx, MAASO_EINVAL, "ins_deploy: configuration out of range");
    uint32_t max_gpus = 0;
    bool any_mask = false;
    for (uint32_t p = 0; p < n_prob; p++) {
        for (uint32_t k = 0; k <= prob[p].gpus; k++) { prob[p].phi_star[k] = 0.0; prob[p].istar_len[k] = 0; }
        if (prob[p].gpus > max_gpus) max_gpus = prob[p].gpus;
        any_mask = any_mask || prob[p].use_mask;
    }
    if (n_configs == 0 || n_prob == 0) return MAASO_OK;
    DeviceGuard g(ctx->device);

    // device staging: offsets | inst | mask | results | scores | rejected-by-model
    const size_t C = (size_t)n_configs * n_prob;
    const size_t cap_spec = 1u << 16;  // speculative follow-ups only while the batch stays this small
    const size_t per_chain = C * (2 + (size_t)ctx->n_models) <= cap_spec ? 2 + (size_t)ctx->n_models : 1;
    const size_t cap_cand = C * per_chain > n_prob ? C * per_chain : n_prob;
    const size_t cap_inst = cap_cand * (MAASO_MAX_INSTANCES + 2);
    size_t off = 0;
    const size_t o_off = off;  off = align_up(off + (cap_cand + 1) * 4, 256);
    const size_t o_inst = off; off = align_up(off + cap_inst * 4, 256);
    const size_t o_mask = off; off = align_up(off + cap_cand * 4, 256);
    const size_t o_res = off;  off = align_up(off + cap_cand * sizeof(maaso_result), 256);
    const size_t o_sc = off;   off = align_up(off + cap_cand * 8, 256);
    const size_t o_rbm = off;  off = align_up(off + cap_cand * MAASO_MAX_MODELS * 4, 256);
    int rc = grow(ctx, &ctx->deploy, &ctx->deploy_bytes, off);
    if (rc != MAASO_OK) return rc;
    unsigned char* sb = static_cast<unsigned char*>(ctx->deploy);
    cudaStream_t st = ctx->own_stream;

    std::vector<uint32_t> h_off(cap_cand + 1), h_inst, h_mask(cap_cand), h_rbm(cap_cand * MAASO_MAX_MODELS);
    std::vector<double> h_sc(cap_cand);
    auto run_batch = [&](uint32_t n_cand) -> int {
        cudaError_t e = cudaMemcpyAsync(sb + o_off, h_off.data(), (n_cand + 1) * 4, cudaMemcpyHostToDevice, st);
        if (e == cudaSuccess && !h_inst.empty())
            e = cudaMemcpyAsync(sb + o_inst, h_inst.data(), h_inst.size() * 4, cudaMemcpyHostToDevice, st);
        if (e == cudaSuccess && any_mask)
            e = cudaMemcpyAsync(sb + o_mask, h_mask.data(), n_cand * 4, cudaMemcpyHostToDevice, st);
        if (e != cudaSuccess) return cuda_fail(ctx, e, "ins_deploy: upload");
        maaso_cand_batch b;
        memset(&b, 0, sizeof(b));
        b.offsets = reinterpret_cast<const uint32_t*>(sb + o_off);
        b.inst = reinterpret_cast<const uint32_t*>(sb + o_inst);
        b.class_mask = any_mask ? reinterpret_cast<const uint32_t*>(sb + o_mask) : nullptr;
        b.n_cand = n_cand;
        b.n_inst = h_inst.size();
        b.budget = max_gpus;  // each chain's own device count is enforced below, on the host
        maaso_eval_opts o;
        memset(&o, 0, sizeof(o));
        o.flags = flags;
        o.rejected_by_model = reinterpret_cast<uint32_t*>(sb + o_rbm);
        int r = maaso_eval_placements(ctx, trace, &b, &o, reinterpret_cast<maaso_result*>(sb + o_res), st);
        if (r != MAASO_OK) return r;
        r = maaso_score(ctx, reinterpret_cast<const maaso_result*>(sb + o_res), n_cand, score,
                        reinterpret_cast<double*>(sb + o_sc), st);
        if (r != MAASO_OK) return r;
        e = cudaMemcpyAsync(h_sc.data(), sb + o_sc, n_cand * 8, cudaMemcpyDeviceToHost, st);
        if (e == cudaSuccess)
            e = cudaMemcpyAsync(h_rbm.data(), sb + o_rbm, (size_t)n_cand * MAASO_MAX_MODELS * 4,
                                cudaMemcpyDeviceToHost, st);
        if (e == cudaSuccess) e = cudaStreamSynchronize(st);
        if (e != cudaSuccess) return cuda_fail(ctx, e, "ins_deploy: download");
        return MAASO_OK;
    };
    // a problem without a mask counts every class (masks are ignored anyway beyond 32 classes)
    auto mask_of = [&](uint32_t p) { return prob[p].use_mask ? prob[p].class_mask : 0xFFFFFFFFu; };

    // R_res = R_x before anything is deployed: the empty placement rejects every request of R_x
    for (uint32_t p = 0; p <= n_prob; p++) h_off[p] = 0;
    for (uint32_t p = 0; p < n_prob; p++) h_mask[p] = mask_of(p);
    h_inst.clear();
    rc = run_batch(n_prob);
    if (rc != MAASO_OK) return rc;

    struct Step {
        uint32_t k;    // device count of the placement the step leaves (the one stored under Phi*[k], I*[k])
        uint32_t len;  // instances of the accepted placement after the step
        double phi;    // its score after the step
    };
    struct Chain {
        std::vector<uint32_t> inst;  // accepted placement I (instances are only ever appended)
        std::vector<Step> steps;
        bool sat[MAASO_MAX_MODELS];
        uint32_t unserved[MAASO_MAX_MODELS];
        double phi;
        uint32_t dev;
        uint32_t gpus;  // device count of the chain's problem
        uint32_t mask;
        int tentative;  // model of the tentative instance, -1 = chain finished
    };
    std::vector<Chain> chains(C);  // chain p * n_configs + c
    for (uint32_t p = 0; p < n_prob; p++)
        for (uint32_t c = 0; c < n_configs; c++) {
            Chain& ch = chains[(size_t)p * n_configs + c];
            memset(ch.sat, 0, sizeof(ch.sat));
            memcpy(ch.unserved, h_rbm.data() + (size_t)p * MAASO_MAX_MODELS, sizeof(ch.unserved));
            ch.phi = 0.0;
            ch.dev = (uint32_t)ctx->h_devices[configs[c].strategy];
            ch.gpus = prob[p].gpus;
            ch.mask = mask_of(p);
            ch.tentative = 0;
        }
    // Two greedy steps per batch.  Besides its tentative placement A = I + m' every chain also
    // proposes what its NEXT step would score, for both outcomes of this one: if A is rejected the
    // next tentative model is already known (m' becomes saturated, nothing else changes): B; if A is
    // accepted the unserved counts change, so the next model is not known: I + m' + m for every model
    // m still open.  After the batch the first step is taken with A's result and the second with the
    // speculative result that matches the actual state.  The batches are a few times larger, the
    // number of trace replays halves; the steps taken are those of the sequential algorithm.
    const uint32_t n_models = ctx->n_models;
    const bool speculate = C * (2 + (size_t)n_models) <= cap_spec;
    auto next_model = [&](const Chain& ch, const bool* sat, size_t len) -> int {
        int mp = -1;  // model with the most unserved requests among the non-saturated ones
        if ((uint64_t)len * ch.dev < ch.gpus && len <= MAASO_MAX_INSTANCES)
            for (uint32_t m = 0; m < n_models; m++)
                if (!sat[m] && (mp < 0 || ch.unserved[m] > ch.unserved[mp])) mp = (int)m;
        return mp;
    };
    uint32_t n_batch = 0;
    std::vector<char> batch_over;  // the placement needs more devices than its problem has
    auto propose = [&](const Chain& ch, const maaso_config& cf, int m1, int m2) -> int {
        // candidate I + m1 (+ m2); returns its index in the batch
        h_off[n_batch] = (uint32_t)h_inst.size();
        h_mask[n_batch] = ch.mask;
        h_inst.insert(h_inst.end(), ch.inst.begin(), ch.inst.end());
        const uint32_t w = ((cf.strategy & 0xFFu) << 4) | ((cf.batch & 0xFFu) << 12);
        h_inst.push_back(((uint32_t)m1 & 0xFu) | w);
        if (m2 >= 0) h_inst.push_back(((uint32_t)m2 & 0xFu) | w);
        batch_over.push_back(((uint64_t)ch.inst.size() + (m2 >= 0 ? 2 : 1)) * ch.dev > ch.gpus ? 1 : 0);
        return (int)n_batch++;
    };
    auto take_step = [&](Chain& ch, int model, uint32_t word, int j) {
        Step sp;
        // a placement beyond the problem's own device count is invalid (score -1), as it would be
        // if the problem were scored alone with its device count as the budget
        const double sc = batch_over[j] ? -1.0 : h_sc[j];
        bool accepted = false;
        if (sc > ch.phi) {  // accept the new instance
            ch.phi = sc;
            ch.inst.push_back(word);
            memcpy(ch.unserved, h_rbm.data() + (size_t)j * MAASO_MAX_MODELS, sizeof(ch.unserved));
            accepted = true;
        } else {
            ch.sat[model] = true;  // stop deploying this model
        }
        sp.len = (uint32_t)ch.inst.size();
        sp.k = sp.len * ch.dev;  // "all possible GPU allocations k" (Sec. IV-E): the devices the stored placement occupies
        sp.phi = ch.phi;
        ch.steps.push_back(sp);
        return accepted;
    };
    struct Plan {
        uint32_t chain;
        int m1, a;           // tentative model, batch index of A
        int mb, b;           // model and batch index of the "A rejected" follow-up (-1: none)
        int c[MAASO_MAX_MODELS];  // batch index of the "A accepted, then model m" follow-up (-1: none)
    };
    std::vector<Plan> plans;
    for (;;) {
        // every unfinished chain proposes its next tentative placement I' = I + (m', P, B)
        plans.clear();
        batch_over.clear();
        h_inst.clear();
        n_batch = 0;
        for (size_t x = 0; x < C; x++) {
            Chain& ch = chains[x];
            const maaso_config& cf = configs[x % n_configs];
            if (ch.tentative < 0) continue;
            const int mp = next_model(ch, ch.sat, ch.inst.size());
            ch.tentative = mp;
            if (mp < 0) continue;
            Plan pl;
            pl.chain = (uint32_t)x;
            pl.m1 = mp;
            pl.a = propose(ch, cf, mp, -1);
            pl.mb = -1;
            pl.b = -1;
            for (uint32_t m = 0; m < MAASO_MAX_MODELS; m++) pl.c[m] = -1;
            if (speculate) {
                bool sat2[MAASO_MAX_MODELS];
                memcpy(sat2, ch.sat, sizeof(sat2));
                sat2[mp] = true;
                pl.mb = next_model(ch, sat2, ch.inst.size());
                if (pl.mb >= 0) pl.b = propose(ch, cf, pl.mb, -1);
                const size_t len2 = ch.inst.size() + 1;
                if ((uint64_t)len2 * ch.dev < ch.gpus && len2 <= MAASO_MAX_INSTANCES)
                    for (uint32_t m = 0; m < n_models; m++)
                        if (!ch.sat[m]) pl.c[m] = propose(ch, cf, mp, (int)m);
            }
            plans.push_back(pl);
        }
        if (plans.empty()) break;
        h_off[n_batch] = (uint32_t)h_inst.size();
        rc = run_batch(n_batch);
        if (rc != MAASO_OK) return rc;
        for (const Plan& pl : plans) {
            Chain& ch = chains[pl.chain];
            const maaso_config& cf = configs[pl.chain % n_configs];
            const uint32_t w = ((cf.strategy & 0xFFu) << 4) | ((cf.batch & 0xFFu) << 12);
            const bool accepted = take_step(ch, pl.m1, ((uint32_t)pl.m1 & 0xFu) | w, pl.a);
            if (!speculate) continue;
            const int m2 = next_model(ch, ch.sat, ch.inst.size());  // from the state the first step left
            if (m2 < 0) continue;  // the chain ends; the next round marks it finished
            const int j = accepted ? pl.c[m2] : (m2 == pl.mb ? pl.b : -1);
            if (j >= 0) take_step(ch, m2, ((uint32_t)m2 & 0xFu) | w, j);
        }
    }
    // Phi*[k] / I*[k]: replay the steps configuration by configuration, as the sequential algorithm
    // would have met them ("first strictly better wins")
    for (uint32_t p = 0; p < n_prob; p++)
        for (uint32_t c = 0; c < n_configs; c++) {
            const Chain& ch = chains[(size_t)p * n_configs + c];
            for (const Step& sp : ch.steps)
                if (sp.k <= prob[p].gpus && sp.phi > prob[p].phi_star[sp.k]) {
                    prob[p].phi_star[sp.k] = sp.phi;
                    prob[p].istar_len[sp.k] = sp.len;
                    for (uint32_t i = 0; i < sp.len && i < MAASO_MAX_INSTANCES; i++)
                        prob[p].istar_inst[(size_t)sp.k * MAASO_MAX_INSTANCES + i] = ch.inst[i];
                }
        }
    return MAASO_OK;
}

MAASO_API int maaso_ins_deploy(maaso_ctx* ctx, const maaso_trace* trace, uint32_t gpus,
                               const maaso_config* configs, uint32_t n_configs, int use_mask,
                               uint32_t class_mask, const maaso_score_params* score, uint32_t flags,
                               double* phi_star, uint32_t* istar_len, uint32_t* istar_inst) {
    if (!ctx || !trace || !score || !phi_star || !istar_len || !istar_inst || (n_configs && !configs) ||
        gpus > 4096 || n_configs > (1u << 20))
        return MAASO_EINVAL;
    const DeployProblem one{gpus, use_mask, class_mask, phi_star, istar_len, istar_inst};
    return ins_deploy_multi(ctx, trace, &one, 1, configs, n_configs, score, flags);
}

// getPrunedConfigs: strategy dominance on the host copy of the tables, batch-cap Pareto front from
// one batch of probe placements.
MAASO_API int maaso_prune_configs(maaso_ctx* ctx, const maaso_trace* trace, int use_mask, uint32_t class_mask,
                                  const uint32_t* batches, uint32_t n_batches, uint32_t flags,
                                  maaso_config* out_configs, uint32_t* out_n) {
    if (!ctx || !trace || !out_configs || !out_n || (n_batches && !batches) || n_batches > MAASO_WMAX)
        return MAASO_EINVAL;
    *out_n = 0;
    if (!ctx->has_profile) return fail(ctx, MAASO_ESTATE, "prune: no profile loaded");
    for (uint32_t b = 0; b < n_batches; b++)
        if (batches[b] < 1 || batches[b] > MAASO_WMAX) return fail(ctx, MAASO_EINVAL, "prune: batch cap out of range");
    const uint32_t S = ctx->n_strategies, M = ctx->n_models;
    const int32_t* rows = ctx->h_rows.data();
    auto faster_or_equal = [&](uint32_t q, uint32_t s, bool& strict) {
        for (uint32_t m = 0; m < M; m++) {
            if (ctx->h_devices[s] < ctx->h_min_devices[m]) continue;    // s cannot host this model anyway
            if (ctx->h_devices[q] < ctx->h_min_devices[m]) return false;  // q cannot replace s for it
            const int32_t* rq = rows + (size_t)(m * S + q) * kRowStride;
            const int32_t* rs = rows + (size_t)(m * S + s) * kRowStride;
            if (rq[0] > rs[0] || (uint32_t)rq[1] > (uint32_t)rs[1]) return false;
            if (rq[0] < rs[0] || (uint32_t)rq[1] < (uint32_t)rs[1]) strict = true;
            for (int w = 0; w < MAASO_WMAX; w++) {
                if (rq[2 + w] > rs[2 + w]) return false;
                if (rq[2 + w] < rs[2 + w]) strict = true;
            }
        }
        return true;
    };
    std::vector<uint32_t> order;
    for (uint32_t s = 0; s < S; s++) {
        bool keep = false;
        for (uint32_t m = 0; m < M; m++) keep = keep || ctx->h_devices[s] >= ctx->h_min_devices[m];
        for (uint32_t q = 0; q < S && keep; q++) {
            if (q == s || ctx->h_devices[q] > ctx->h_devices[s]) continue;
            bool strict = false;
            if (!faster_or_equal(q, s, strict)) continue;
            if (strict || ctx->h_devices[q] < ctx->h_devices[s] || q < s) keep = false;
        }
        if (keep) order.push_back(s);
    }
    for (size_t i = 1; i < order.size(); i++)  // tree order: increasing level-1 step of model 0
        for (size_t j = i; j > 0; j--) {
            const uint32_t a = order[j - 1], b = order[j];
            const int32_t sa = rows[(size_t)a * kRowStride + 2], sb = rows[(size_t)b * kRowStride + 2];
            if (sa > sb || (sa == sb && a > b)) { order[j - 1] = b; order[j] = a; } else break;
        }
    if (order.empty() || n_batches == 0) return MAASO_OK;

    // one batch of probe placements: (strategy, cap) -> one instance of every model that fits
    const size_t C = order.size() * n_batches;
    std::vector<uint32_t> h_off(C + 1), h_inst, h_mask(C, class_mask);
    for (size_t i = 0; i < order.size(); i++)
        for (uint32_t b = 0; b < n_batches; b++) {
            h_off[i * n_batches + b] = (uint32_t)h_inst.size();
            for (uint32_t m = 0; m < M; m++)
                if (ctx->h_devices[order[i]] >= ctx->h_min_devices[m])
                    h_inst.push_back((m & 0xFu) | ((order[i] & 0xFFu) << 4) | ((batches[b] & 0xFFu) << 12));
        }
    h_off[C] = (uint32_t)h_inst.size();
    DeviceGuard g(ctx->device);
    size_t off = 0;
    const size_t o_off = off;  off = align_up(off + (C + 1) * 4, 256);
    const size_t o_inst = off; off = align_up(off + h_inst.size() * 4 + 4, 256);
    const size_t o_mask = off; off = align_up(off + C * 4, 256);
    const size_t o_res = off;  off = align_up(off + C * sizeof(maaso_result), 256);
    int rc = grow(ctx, &ctx->deploy, &ctx->deploy_bytes, off);
    if (rc != MAASO_OK) return rc;
    unsigned char* sb = static_cast<unsigned char*>(ctx->deploy);
    cudaStream_t st = ctx->own_stream;
    cudaError_t e = cudaMemcpyAsync(sb + o_off, h_off.data(), (C + 1) * 4, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(sb + o_inst, h_inst.data(), h_inst.size() * 4, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess && use_mask) e = cudaMemcpyAsync(sb + o_mask, h_mask.data(), C * 4, cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "prune: upload");
    maaso_cand_batch bt;
    memset(&bt, 0, sizeof(bt));
    bt.offsets = reinterpret_cast<const uint32_t*>(sb + o_off);
    bt.inst = reinterpret_cast<const uint32_t*>(sb + o_inst);
    bt.class_mask = use_mask ? reinterpret_cast<const uint32_t*>(sb + o_mask) : nullptr;
    bt.n_cand = C;
    bt.n_inst = h_inst.size();
    bt.budget = 0xFFFFFFFFu;  // a probe, not a deployment
    maaso_eval_opts o;
    memset(&o, 0, sizeof(o));
    o.flags = flags;
    rc = maaso_eval_placements(ctx, trace, &bt, &o, reinterpret_cast<maaso_result*>(sb + o_res), st);
    if (rc != MAASO_OK) return rc;
    std::vector<maaso_result> res(C);
    e = cudaMemcpyAsync(res.data(), sb + o_res, C * sizeof(maaso_result), cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "prune: download");
    for (size_t i = 0; i < order.size(); i++) {
        const maaso_result* r = res.data() + i * n_batches;
        for (uint32_t b = 0; b < n_batches; b++) {
            bool dominated = r[b].status != 0;
            for (uint32_t c = 0; c < n_batches && !dominated; c++) {
                if (c == b || r[c].status != 0) continue;
                bool lat_le, lat_lt;  // mean time to first token of c vs b; nothing served = infinite
                if (r[c].n_served == 0) { lat_le = r[b].n_served == 0; lat_lt = false; }
                else if (r[b].n_served == 0) { lat_le = true; lat_lt = true; }
                else {
                    const unsigned __int128 l = (unsigned __int128)(uint64_t)r[c].sum_ttft_us * r[b].n_served;
                    const unsigned __int128 rr = (unsigned __int128)(uint64_t)r[b].sum_ttft_us * r[c].n_served;
                    lat_le = l <= rr; lat_lt = l < rr;
                }
                const bool hit_ge = r[c].n_hit >= r[b].n_hit, hit_gt = r[c].n_hit > r[b].n_hit;
                if (hit_ge && lat_le && (hit_gt || lat_lt)) dominated = true;
                else if (hit_ge && lat_le && batches[c] < batches[b]) dominated = true;  // equal outcome
            }
            if (!dominated) {
                out_configs[*out_n].strategy = order[i];
                out_configs[*out_n].batch = batches[b];
                (*out_n)++;
            }
        }
    }
    return MAASO_OK;
}

// Alg. 2 for two sub-clusters on top of maaso_ins_deploy.
MAASO_API int maaso_partition(maaso_ctx* ctx, const maaso_trace* trace, uint32_t mask_t, uint32_t mask_l,
                              uint32_t gpus, const maaso_config* configs, uint32_t n_configs,
                              const maaso_score_params* score, uint32_t flags, int baseline, uint32_t* out_g,
                              double* out_phi, uint32_t* len_t, uint32_t* inst_t, uint32_t* len_l,
                              uint32_t* inst_l) {
    if (!ctx || !trace || !out_g || !out_phi || !len_t || !inst_t || !len_l || !inst_l || gpus > 4096)
        return MAASO_EINVAL;
    if (trace->owner != ctx) return fail(ctx, MAASO_ESTATE, "partition: trace belongs to another context");
    // |R_t|, |R_l|: what the empty placement counts under each mask
    DeviceGuard g(ctx->device);
    int rc = grow(ctx, &ctx->deploy, &ctx->deploy_bytes, 4096);
    if (rc != MAASO_OK) return rc;
    unsigned char* sb = static_cast<unsigned char*>(ctx->deploy);
    const uint32_t h_off[3] = {0, 0, 0}, h_mask[2] = {mask_t, mask_l};
    maaso_result h_res[2];
    cudaStream_t st = ctx->own_stream;
    cudaError_t e = cudaMemcpyAsync(sb, h_off, sizeof(h_off), cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(sb + 256, h_mask, sizeof(h_mask), cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "partition: upload");
    maaso_cand_batch b;
    memset(&b, 0, sizeof(b));
    b.offsets = reinterpret_cast<const uint32_t*>(sb);
    b.inst = reinterpret_cast<const uint32_t*>(sb + 512);
    b.class_mask = reinterpret_cast<const uint32_t*>(sb + 256);
    b.n_cand = 2;
    b.budget = gpus;
    rc = maaso_eval_placements(ctx, trace, &b, nullptr, reinterpret_cast<maaso_result*>(sb + 1024), st);
    if (rc != MAASO_OK) return rc;
    e = cudaMemcpyAsync(h_res, sb + 1024, sizeof(h_res), cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "partition: download");
    const uint64_t n_t = h_res[0].n_counted, n_l = h_res[1].n_counted;
    const uint32_t gl_max = (n_t + n_l) ? (uint32_t)((n_l * (uint64_t)gpus) / (n_t + n_l)) : 0;

    const size_t cells = (size_t)gpus + 1;
    std::vector<double> phi_t(cells), phi_l(cells), phi_h(cells);
    std::vector<uint32_t> ln_t(cells), ln_l(cells), ln_h(cells);
    std::vector<uint32_t> in_t(cells * MAASO_MAX_INSTANCES), in_l(cells * MAASO_MAX_INSTANCES),
        in_h(cells * MAASO_MAX_INSTANCES);
    // the loose, the tight and (if asked) the homogeneous problem are independent: their greedy
    // chains advance side by side, one batch per step for all of them
    if (!score || (n_configs && !configs) || n_configs > (1u << 20)) return MAASO_EINVAL;
    DeployProblem probs[3] = {
        {gl_max, 1, mask_l, phi_l.data(), ln_l.data(), in_l.data()},
        {gpus, 1, mask_t, phi_t.data(), ln_t.data(), in_t.data()},
        {gpus, 1, mask_t | mask_l, phi_h.data(), ln_h.data(), in_h.data()},
    };
    rc = ins_deploy_multi(ctx, trace, probs, baseline ? 3u : 2u, configs, n_configs, score, flags);
    double phi_opt = 0.0;
    if (rc == MAASO_OK && baseline)  // homogeneous deployment as the fallback
        for (uint32_t k = 0; k <= gpus; k++)
            if (phi_h[k] > phi_opt) phi_opt = phi_h[k];
    if (rc != MAASO_OK) return rc;
    out_g[0] = out_g[1] = 0;
    *len_t = *len_l = 0;
    for (uint32_t gl = 1; gl <= gl_max; gl++) {
        const uint32_t gt = gpus - gl;
        if (phi_t[gt] + phi_l[gl] > phi_opt) {
            phi_opt = phi_t[gt] + phi_l[gl];
            out_g[0] = gt;
            out_g[1] = gl;
            *len_t = ln_t[gt];
            *len_l = ln_l[gl];
            memcpy(inst_t, in_t.data() + (size_t)gt * MAASO_MAX_INSTANCES, ln_t[gt] * 4);
            memcpy(inst_l, in_l.data() + (size_t)gl * MAASO_MAX_INSTANCES, ln_l[gl] * 4);
        }
    }
    *out_phi = phi_opt;
    return MAASO_OK;
}

MAASO_API int maaso_set_timing(maaso_ctx* ctx, int enabled) {
    if (!ctx) return MAASO_EINVAL;
    DeviceGuard g(ctx->device);
    if (enabled)
        for (int i = 0; i < 7; i++)
            if (!ctx->ev[i]) {
                cudaError_t e = cudaEventCreate(&ctx->ev[i]);
                if (e != cudaSuccess) return cuda_fail(ctx, e, "cudaEventCreate");
            }
    ctx->timing = enabled != 0;
    ctx->ev_eval = ctx->ev_topk = false;
    return MAASO_OK;
}

MAASO_API int maaso_get_timing(maaso_ctx* ctx, maaso_timing* out) {
    if (!ctx || !out) return MAASO_EINVAL;
    memset(out, 0, sizeof(*out));
    if (!ctx->timing) return fail(ctx, MAASO_ESTATE, "timing is not enabled");
    DeviceGuard g(ctx->device);
    cudaError_t e = cudaSuccess;
    if (ctx->ev_eval) {
        e = cudaEventSynchronize(ctx->ev[3]);
        if (e == cudaSuccess) e = cudaEventElapsedTime(&out->prep_ms, ctx->ev[0], ctx->ev[1]);
        if (e == cudaSuccess) e = cudaEventElapsedTime(&out->group_ms, ctx->ev[1], ctx->ev[2]);
        if (e == cudaSuccess) e = cudaEventElapsedTime(&out->thread_ms, ctx->ev[2], ctx->ev[6]);
        if (e == cudaSuccess) e = cudaEventElapsedTime(&out->block_ms, ctx->ev[6], ctx->ev[3]);
    }
    if (e == cudaSuccess && ctx->ev_topk) {
        e = cudaEventSynchronize(ctx->ev[5]);
        if (e == cudaSuccess) e = cudaEventElapsedTime(&out->topk_ms, ctx->ev[4], ctx->ev[5]);
    }
    if (e != cudaSuccess) return cuda_fail(ctx, e, "timing events");
    return MAASO_OK;
}

MAASO_API uint64_t maaso_launch_count(const maaso_ctx* ctx) { return ctx ? ctx->launches : 0; }

MAASO_API int maaso_test_fail_allocs(maaso_ctx* ctx, int count) {
    if (!ctx || count < 0) return MAASO_EINVAL;
    ctx->fail_allocs = count;
    return MAASO_OK;
}

MAASO_API const char* maaso_strerror(int code) {
    switch (code) {
        case MAASO_OK: return "ok";
        case MAASO_EINVAL: return "invalid argument";
        case MAASO_ESTATE: return "wrong state (no profile, foreign trace, unsupported device)";
        case MAASO_ENOMEM: return "out of memory";
        case MAASO_ECUDA: return "CUDA runtime error";
        case MAASO_ETOOBIG: return "size beyond the fixed capacity of this entry point";
        default: return "unknown error";
    }
}

MAASO_API const char* maaso_last_error(const maaso_ctx* ctx) { return ctx ? ctx->last_error.c_str() : ""; }

}  // extern "C"
