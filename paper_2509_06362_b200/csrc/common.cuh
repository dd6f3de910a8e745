// Device-side building blocks shared by the scoring kernels: request decode, slot payload,
// per-lane statistics, completion accounting, mbarrier / bulk-copy wrappers.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>
#include "../../include/maaso.h"

namespace maaso {

constexpr uint32_t kAttemptCap = 2u + MAASO_MAX_INSTANCES * MAASO_WMAX;
constexpr int kRowStride = 66;  // int32 per profile row: prefill base, prefill q16, 64 steps
constexpr uint64_t kKeyInf = ~0ull;
constexpr long long kWaitCycles = 4000000000ll;  // bound on any device-side wait (~2 s)

// Buckets the validation kernel sorts candidates into.
// 0..5: lane groups of 1,2,4,8,16,32 lanes (one lane per instance)
// 6..8: block layout with 2, 4, 8 warps, one warp per instance, state in registers
// 9:    block layout with 16 warps striding over up to 128 instances, state in shared memory
// 10..18: thread mapping, by how many lanes of a warp work at a time (32, 24, 16, 12, 8, 6, 4, 2, 1:
//        the larger the placements, the fewer fit the warp's pools)
constexpr int kNumBuckets = 20;
constexpr int kGenericBlockBucket = 9;
constexpr int kThreadBucket0 = 10;  // buckets 10..18: the thread mapping, by lanes per warp
constexpr int kThreadBuckets = 9;
constexpr int kWideBucket = 19;     // 33..128 instances under the engines of the lane-group code: one warp per placement
constexpr int kCostBins = 256;   // bin 0 = most expensive (largest total batch cap)
constexpr int kCounterWords = 17408;  // counters | work counters | histograms + cursors, cleared per call
// histogram sets (rows of kCostBins words in EvalParams::hist): candidates that can only go to a lane-group
// or block bucket, only to a thread bucket, or either way (counted once per side); then the write cursors
constexpr int kHistOnlyG = 0, kHistBothG = 10, kHistOnlyT = 20, kHistBothT = 29, kHistWide = 38, kHistBothW = 39, kHistCursor = 40;
constexpr int kHistRows = kHistCursor + kNumBuckets;
// counters beside the bucket counts (EvalParams::bucket_count[0..31])
constexpr int kCtrBoth = 24, kCtrLoaded = 25, kCtrCut = 26, kCtrUseThreads = 27;
constexpr int kGroupThreads = 128;
constexpr int kScanTile = 256;       // requests per scan tile of the thread mapping
constexpr int kScanHdrUnits = 40;    // 16-byte units of a scan tile's header (see scan_trace_kernel)
constexpr int kScanHdrBase = 4;      // unit of the tile's base arrival time
constexpr int kScanHdrClassBits = 5; // first unit of the 8 per-class bitmaps (2 units = 256 bits each)
constexpr int kScanHdrModelBits = 21; // first unit of the 8 per-model bitmaps
constexpr int kMaxTraces = 16;  // traces one call of the lane-group kernel can replay side by side

struct Request {
    int64_t arrival;
    uint32_t in_tokens;
    uint32_t S;
    uint32_t cls;
    uint32_t model;
};

__device__ __forceinline__ Request decode_request(uint4 v) {
    Request q;
    q.arrival = (int64_t)(((uint64_t)v.y << 32) | v.x);
    q.in_tokens = v.z;
    q.S = v.w & 0xFFFFu;
    q.cls = (v.w >> 16) & 0xFFu;
    q.model = v.w >> 24;
    return q;
}

// A trace record prepared once per trace for the lane-group kernel (48 bytes, three 16-byte
// words): everything about a request that does not depend on the candidate.
//   word 0: arrival time, latest first-token time (arrival + TTFT limit, INT64_MAX if none)
//   word 1: latest finish time (arrival + end-to-end limit, INT64_MAX if none), input tokens,
//           TBT limit clamped to 32 bits (0xFFFFFFFF = none; step times are below 2^31)
//   word 2: checksum term of "this request was rejected", S - 1 | cls << 16 | model << 24, 0
constexpr int kCookedWords = 3;

// What a running request must remember until it completes (32 bytes, two 16-byte words).
struct Payload {
    int64_t first_tok;
    int64_t arrival;
    uint32_t req;
    uint32_t s_cls;  // S | cls << 16
    uint64_t pad;
};
static_assert(sizeof(Payload) == 32, "payload is two 16-byte words");

__device__ __forceinline__ void store_payload(Payload* p, int64_t first_tok, int64_t arrival,
                                              uint32_t req, uint32_t S, uint32_t cls) {
    uint4 a, b;
    a.x = (uint32_t)first_tok; a.y = (uint32_t)((uint64_t)first_tok >> 32);
    a.z = (uint32_t)arrival;   a.w = (uint32_t)((uint64_t)arrival >> 32);
    b.x = req; b.y = S | (cls << 16); b.z = 0; b.w = 0;
    reinterpret_cast<uint4*>(p)[0] = a;
    reinterpret_cast<uint4*>(p)[1] = b;
}

struct Stats {
    uint32_t served, hit;
    int64_t sum_ttft, max_ttft, sum_e2e, max_e2e, makespan;
    uint64_t tokens, checksum;
    __device__ __forceinline__ void clear() {
        served = hit = 0;
        sum_ttft = max_ttft = sum_e2e = max_e2e = makespan = 0;
        tokens = checksum = 0;
    }
};

// SplitMix64 output mixer (public domain)
__device__ __forceinline__ uint64_t mix64(uint64_t z) {
    z ^= z >> 30; z *= 0xBF58476D1CE4E5B9ull;
    z ^= z >> 27; z *= 0x94D049BB133111EBull;
    z ^= z >> 31;
    return z;
}
__device__ __forceinline__ uint64_t served_hash(uint32_t req, int64_t t_fin, int64_t first_tok,
                                                uint32_t inst) {
    uint64_t f = (uint64_t)first_tok;
    return mix64((uint64_t)req * 0x9E3779B97F4A7C15ull ^ (uint64_t)t_fin ^ ((f << 32) | (f >> 32)) ^
                 ((uint64_t)inst << 56));
}
__device__ __forceinline__ uint64_t rejected_hash(uint32_t req) {
    return mix64((uint64_t)req * 0x9E3779B97F4A7C15ull ^ ~0ull);
}

// Where per-request times of a dumped candidate go (all null / row < 0 when not dumped).
struct Dump {
    int64_t* finish;
    int64_t* first;
    int32_t* inst;
    uint32_t* hist;  // this candidate's time-to-first-token histogram, or null
};

// Histogram bin of a time to first token: bin 0 below 1024 us, then two bins per octave.
__device__ __forceinline__ uint32_t ttft_bin(int64_t t) {
    if (t < 1024) return 0;
    const int e = 63 - __clzll(t);
    const uint32_t b = 1u + 2u * (uint32_t)(e - 10) + (uint32_t)((t >> (e - 1)) & 1);
    return b > (uint32_t)(MAASO_TTFT_BINS - 1) ? (uint32_t)(MAASO_TTFT_BINS - 1) : b;
}

// A request leaves the system served at t_fin (Phi_S indicator and the latency / throughput sums).
// `classes` holds (ttft, tbt, e2e) per class, negative = no limit.  Returns whether it was a hit.
// max_gap: largest gap between two consecutive tokens of the request if the TBT term is to be
// checked on it (MAASO_FLAG_TBT_MAXGAP), negative for the mean-gap form.
__device__ __forceinline__ bool account_completion(Stats& st, const int64_t* classes, uint32_t inst,
                                                   uint32_t req, int64_t arrival, int64_t first_tok,
                                                   int64_t t_fin, uint32_t S, uint32_t cls,
                                                   const Dump& dump, int64_t max_gap) {
    const int64_t lim_ttft = classes[cls * 3 + 0];
    const int64_t lim_tbt = classes[cls * 3 + 1];
    const int64_t lim_e2e = classes[cls * 3 + 2];
    const int64_t ttft = first_tok - arrival, e2e = t_fin - arrival, span = t_fin - first_tok;
    // TBT term: the mean gap between tokens, or (max_gap >= 0) the largest single gap
    const bool tbt_ok = lim_tbt < 0 || (max_gap >= 0 ? max_gap <= lim_tbt : span <= (int64_t)(S - 1) * lim_tbt);
    const bool hit = (lim_ttft < 0 || ttft <= lim_ttft) && tbt_ok && (lim_e2e < 0 || e2e <= lim_e2e);
    st.served++;
    st.hit += hit ? 1u : 0u;
    st.sum_ttft += ttft; st.max_ttft = max(st.max_ttft, ttft);
    st.sum_e2e += e2e;   st.max_e2e = max(st.max_e2e, e2e);
    st.makespan = max(st.makespan, t_fin);
    st.tokens += S;
    st.checksum += served_hash(req, t_fin, first_tok, inst);
    if (dump.finish) dump.finish[req] = t_fin;
    if (dump.first) dump.first[req] = first_tok;
    if (dump.inst) dump.inst[req] = (int32_t)inst;
    if (dump.hist) atomicAdd(dump.hist + ttft_bin(ttft), 1u);
    return hit;
}

// ceil(dt / s) for dt >= 1, s >= 1
__device__ __forceinline__ uint32_t ceil_div_steps(int64_t dt, uint32_t s) {
    if (((uint64_t)dt >> 32) == 0) return ((uint32_t)dt - 1u) / s + 1u;
    return (uint32_t)(((uint64_t)dt - 1ull) / s) + 1u;
}

// ceil(dt / s) when the quotient is known to be below 2^16 and rs = 1/s in float, exact to a
// few units in the last place: the float estimate is then within one of the true quotient
// and is fixed up exactly.
__device__ __forceinline__ uint32_t ceil_div_small(int64_t dt, uint32_t s, float rs) {
    if (((uint64_t)dt >> 32) != 0) return (uint32_t)(((uint64_t)dt - 1ull) / s) + 1u;
    uint32_t q = (uint32_t)(__uint2float_rz((uint32_t)dt) * rs);
    int64_t r = dt - (int64_t)q * (int64_t)s;
    if (r < 0) { q--; r += s; }
    else if (r >= (int64_t)s) { q++; r -= s; }
    return q + (r > 0 ? 1u : 0u);
}

__device__ __forceinline__ float rcp_approx(float x) {
    float r;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x));
    return r;
}

__device__ __forceinline__ int64_t prefill_us(uint32_t base, uint32_t q16, uint32_t in_tokens) {
    return (int64_t)base + (int64_t)(((uint64_t)q16 * in_tokens + 32768u) >> 16);
}

// ---- mbarrier + 1-D bulk copy (TMA) -----------------------------------------------------------
__device__ __forceinline__ uint32_t smem_addr(const void* p) {
    return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void fence_barrier_init() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void fence_proxy_async() {
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_addr(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait: false if the barrier did not complete within kWaitCycles.
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity, long long limit = kWaitCycles) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    while (!mbar_try_wait(bar, parity)) {
        if (clock64() - t0 > limit) return false;
    }
    return true;
}
// Plain bulk copy global -> this CTA's own shared memory (one destination CTA); 16-byte aligned, size % 16 == 0.
__device__ __forceinline__ void bulk_load(void* dst_smem, const void* src_gmem, uint32_t bytes,
                                          uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
            smem_addr(dst_smem)),
        "l"(src_gmem), "r"(bytes), "r"(smem_addr(bar))
        : "memory");
}

// Everything a scoring kernel needs, passed by value.
struct EvalParams {
    const uint4* reqs;
    uint32_t n_req;
    uint32_t n_classes;
    const int64_t* classes;  // [n_classes][3]
    const uint4* cooked;     // [n_req][kCookedWords] prepared records (lane-group kernel)
    // several traces in one launch (lane-group kernel only): trace t of n_traces > 1 has
    // trace_n[t] prepared records at trace_cooked[t]; record c of trace t goes to out[t * n_cand + c]
    // (and likewise for the per-model counts and the histograms).  n_traces = 1: cooked / n_req.
    uint32_t n_traces;
    const uint4* trace_cooked[kMaxTraces];
    // thread mapping: scan tiles (header + 16-byte records, see scan_trace_kernel) and per-class totals
    // {requests, sum of the checksum terms of "rejected"} of each trace (index 0 when there is only one)
    const uint4* trace_scan[kMaxTraces];
    const uint64_t* trace_class_tot[kMaxTraces];  // [n_classes][2]: count, checksum sum
    uint32_t trace_n[kMaxTraces];
    const uint64_t* rej_hash;  // [n_req] checksum term of "request r was rejected" (same for every candidate)
    const int32_t* rows;     // [n_rows][kRowStride]
    const int32_t* devices;
    const int32_t* min_devices;
    uint32_t n_rows, n_models, n_strategies;
    uint32_t budget;
    const uint32_t* offsets;
    const uint32_t* inst;
    const uint32_t* class_mask;  // null, or ignored when n_classes > 32
    uint32_t n_cand;
    uint32_t n_inst;
    uint32_t flags;
    uint32_t mapping;
    maaso_result* out;
    uint32_t* bucket_count;  // [32]: candidates per bucket after planning, and the kCtr* counters
    uint32_t* bucket_list;   // [kNumBuckets][n_cand], each bucket sorted by decreasing cost estimate
    uint32_t* work_ctr;      // [16]: next work item of the block kernels [1..4], of the thread buckets [5..13], of the wide kernel [14]
    uint32_t* hist;          // [kHistRows][kCostBins]: candidates per cost bin by set, then write cursors
    uint32_t* code;          // [n_cand] lane-group / block bucket << 8 | cost bin, 0xFFFFFFFF if none
    uint32_t* code2;         // [n_cand] thread bucket << 8 | cost bin, 0xFFFFFFFF if none
    uint32_t demand_tok_s;   // output tokens per second the trace(s) ask for
    uint32_t thread_min_cand; // MAASO_MAP_AUTO: fewest loaded candidates for which the thread mapping is chosen
    uint32_t group_warps;    // warps the lane-group grid keeps resident (capacity for promotions)
    uint32_t* sm_ctr;        // [n_sm] next work item of each SM's share (lane-group kernel)
    uint32_t n_sm;
    uint32_t promote_pct;
    uint32_t thread_pool_units;  // thread mapping: 16-byte units one warp has for the cold part of its placements' state
    uint32_t thread_hot_units;   // and for the hot part (3 units per instance, shared memory)
    long long wait_cycles;   // bound of every device-side wait
    uint32_t stall_test;     // test hook: never issue the trace copies
    int32_t* dump_row;       // [n_cand] or null
    uint32_t dump_n;
    int64_t* dump_finish;
    int64_t* dump_first;
    int32_t* dump_inst;
    Payload* payload;        // scratch for running requests
    uint32_t* rej_by_model;  // [n_cand][MAASO_MAX_MODELS] or null
    uint32_t* ttft_hist;     // [n_cand][MAASO_TTFT_BINS] or null (zeroed before the kernels run)
};

// The usual form: TBT term on the mean gap.
__device__ __forceinline__ bool account_completion(Stats& st, const int64_t* classes, uint32_t inst,
                                                   uint32_t req, int64_t arrival, int64_t first_tok,
                                                   int64_t t_fin, uint32_t S, uint32_t cls,
                                                   const Dump& dump) {
    return account_completion(st, classes, inst, req, arrival, first_tok, t_fin, S, cls, dump, (int64_t)-1);
}

// `cand`: index of the candidate's record in the output (trace index * n_cand + candidate index
// when several traces are replayed in one launch; dump rows exist for one trace only).
__device__ __forceinline__ Dump dump_for(const EvalParams& P, uint32_t cand) {
    Dump d{nullptr, nullptr, nullptr, nullptr};
    if (P.ttft_hist) d.hist = P.ttft_hist + (size_t)cand * MAASO_TTFT_BINS;
    if (P.n_traces > 1) return d;
    if (P.dump_row) {
        int32_t row = P.dump_row[cand];
        if (row >= 0) {
            size_t off = (size_t)row * P.n_req;
            if (P.dump_finish) d.finish = P.dump_finish + off;
            if (P.dump_first) d.first = P.dump_first + off;
            if (P.dump_inst) d.inst = P.dump_inst + off;
        }
    }
    return d;
}

__device__ __forceinline__ void write_result(maaso_result* out, uint32_t status, uint32_t n_counted,
                                             uint32_t n_rejected, uint64_t attempts, const Stats& st,
                                             const uint32_t* hit_by_class) {
    uint4* o = reinterpret_cast<uint4*>(out);
    if (status) {
        o[0] = make_uint4(status, 0, 0, 0);
        for (int i = 1; i < 8; i++) o[i] = make_uint4(0, 0, 0, 0);
        return;
    }
    auto lo = [](uint64_t v) { return (uint32_t)v; };
    auto hi = [](uint64_t v) { return (uint32_t)(v >> 32); };
    o[0] = make_uint4(0, n_counted, st.served, st.hit);
    o[1] = make_uint4(n_rejected, st.served - st.hit, hit_by_class[0], hit_by_class[1]);
    o[2] = make_uint4(hit_by_class[2], hit_by_class[3], hit_by_class[4], hit_by_class[5]);
    o[3] = make_uint4(hit_by_class[6], hit_by_class[7], lo(st.sum_ttft), hi(st.sum_ttft));
    o[4] = make_uint4(lo(st.max_ttft), hi(st.max_ttft), lo(st.sum_e2e), hi(st.sum_e2e));
    o[5] = make_uint4(lo(st.max_e2e), hi(st.max_e2e), lo(st.makespan), hi(st.makespan));
    o[6] = make_uint4(lo(st.tokens), hi(st.tokens), lo(st.checksum), hi(st.checksum));
    o[7] = make_uint4(lo(attempts), hi(attempts), 0, 0);
}

}  // namespace maaso
