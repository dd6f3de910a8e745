// Scoring kernel, lane-group mapping: a candidate with I <= 32 instances is replayed by a
// group of G = 2^ceil(log2 I) lanes of one warp, one lane per simulated instance.  All
// instance state lives in registers; slot keys and the data of running requests in a
// shared-memory pool; the distributor's argmin is a shuffle butterfly inside the group.
// The trace (and the per-request checksum term of a rejection) is staged once per thread
// block in shared-memory tiles by 1-D bulk copies (TMA) and shared by every candidate of
// the block.  No global memory access sits on the per-request path.
#include "lane_frozen.cuh"

namespace maaso {

constexpr int kStages = 3;
constexpr uint32_t kFullMask = 0xFFFFFFFFu;

__device__ __forceinline__ uint64_t shfl_xor_u64(uint64_t v, int off, uint32_t mask) {
    uint32_t lo = __shfl_xor_sync(mask, (uint32_t)v, off);
    uint32_t hi = __shfl_xor_sync(mask, (uint32_t)(v >> 32), off);
    return ((uint64_t)hi << 32) | lo;
}
__device__ __forceinline__ uint64_t shfl_u64(uint64_t v, int src, uint32_t mask) {
    uint32_t lo = __shfl_sync(mask, (uint32_t)v, src);
    uint32_t hi = __shfl_sync(mask, (uint32_t)(v >> 32), src);
    return ((uint64_t)hi << 32) | lo;
}

struct ArgMin {
    bool found;
    uint32_t tier;
    int winner;  // lane
};

// Distributor's choice inside a lane group: smallest (tier, predicted first token), lowest lane
// among equals.  Called by all 32 lanes.  The comparison runs on the 32-bit keys of lane_predict;
// only if the group's minimum is a clamped key (a first token 2^31 us or more ahead: rare) the
// group repeats the reduction on (tier, first token) in 64 bits, with its own lane mask.
// `own`: the warp holds a single candidate, so one full-warp reduction replaces the butterfly.
__device__ __forceinline__ ArgMin group_argmin(uint32_t k32, int64_t first, uint32_t gmask, uint32_t G, bool own) {
    ArgMin r;
    uint32_t best = k32;
    if (own) {
        best = __reduce_min_sync(kFullMask, k32);
    } else {
        for (uint32_t o = 1; o < G; o <<= 1) best = min(best, __shfl_xor_sync(kFullMask, best, (int)o));
    }
    bool eq = k32 == best;
    if ((best & 0x7FFFFFFFu) == kOffSat) {
        const uint64_t key = k32 == kKey32Inf ? kKeyInf : (((uint64_t)(k32 >> 31) << 63) | (uint64_t)first);
        uint64_t b64 = key;
        for (uint32_t o = 1; o < G; o <<= 1) b64 = min(b64, shfl_xor_u64(b64, (int)o, gmask));
        eq = key == b64;
    }
    __syncwarp();
    r.found = best != kKey32Inf;
    r.tier = best >> 31;
    const uint32_t votes = __ballot_sync(kFullMask, eq) & gmask;
    r.winner = r.found ? __ffs((int)votes) - 1 : (int)(threadIdx.x & 31u);
    return r;
}

// Per-request side outputs of a rejection (dump rows, per-model counts); rare.
__device__ __forceinline__ void reject_side(const EvalParams& P, uint32_t oc, uint32_t req, uint32_t model) {
    const Dump dump = dump_for(P, oc);
    if (P.rej_by_model) atomicAdd(&P.rej_by_model[(size_t)oc * MAASO_MAX_MODELS + model], 1u);
    if (dump.finish) dump.finish[req] = -1;
    if (dump.first) dump.first[req] = -1;
    if (dump.inst) dump.inst[req] = -1;
}

struct GroupSmem {
    uint4* tiles;        // [kStages][tile_recs][kCookedWords] prepared request records
    unsigned char* pool; // slot keys + block minima, carved per work item in 32-byte units
    uint4* qa;           // [kQueue][kGroupThreads] queued completions: first-token time, arrival time
    uint2* qb;           // [kQueue][kGroupThreads] request index, S | cls << 16
    int64_t* qf;         // [kQueue][kGroupThreads] finish time
    int64_t* qg;         // [kQueue][kGroupThreads] largest token gap (largest-gap mode)
    int64_t* classes;    // [n_classes][3], negative = no limit (completion accounting)
    uint64_t* full_bar;  // [kStages]
    int32_t* steps;      // [n_rows][64]
    uint32_t* empty_cnt; // [kStages]
    uint32_t* work;      // [2]
    uint32_t* wsum;      // [warps] pool units each warp asks for
};

__host__ __device__ inline size_t group_smem_static(uint32_t n_rows, uint32_t n_classes, int tile_recs, bool maxgap) {
    size_t b = (size_t)kStages * tile_recs * 16 * kCookedWords;
    b += (size_t)kQueue * kGroupThreads * (16 + 8 + 8 + (maxgap ? 8 : 0));
    b += (size_t)n_classes * 24;
    b += kStages * 8;
    b += (size_t)n_rows * 64 * 4;
    b += kStages * 4 + 8 + 16 + 32;
    return (b + 31) & ~(size_t)31;
}

__device__ __forceinline__ GroupSmem carve(unsigned char* base, uint32_t n_rows, uint32_t n_classes,
                                           int tile_recs, uint32_t pool_bytes, bool maxgap) {
    GroupSmem s;
    // every part that is read in 16-byte words first (all sizes are multiples of 16 bytes)
    s.pool = base;
    base += pool_bytes;
    s.tiles = reinterpret_cast<uint4*>(base);
    base += (size_t)kStages * tile_recs * 16 * kCookedWords;
    s.qa = reinterpret_cast<uint4*>(base);
    base += (size_t)kQueue * kGroupThreads * 16;
    s.qb = reinterpret_cast<uint2*>(base);
    base += (size_t)kQueue * kGroupThreads * 8;
    s.qf = reinterpret_cast<int64_t*>(base);
    base += (size_t)kQueue * kGroupThreads * 8;
    s.qg = reinterpret_cast<int64_t*>(base);
    if (maxgap) base += (size_t)kQueue * kGroupThreads * 8;
    s.classes = reinterpret_cast<int64_t*>(base);
    base += (size_t)n_classes * 24;
    s.full_bar = reinterpret_cast<uint64_t*>(base);
    base += kStages * 8;
    s.steps = reinterpret_cast<int32_t*>(base);
    base += (size_t)n_rows * 64 * 4;
    s.empty_cnt = reinterpret_cast<uint32_t*>(base);
    base += kStages * 4;
    s.work = reinterpret_cast<uint32_t*>(base);
    base += 8;
    s.wsum = reinterpret_cast<uint32_t*>(base);
    return s;
}

// One tile of prepared records (48 bytes each, so every copy is a multiple of 16 bytes and
// starts on a 16-byte boundary).
__device__ __forceinline__ void issue_tile(const GroupSmem& sm, const uint4* cooked, uint32_t n_req, uint32_t stage,
                                           uint32_t tile, int tile_recs) {
    const uint32_t recs = min((uint32_t)tile_recs, n_req - tile * tile_recs);
    const uint32_t bytes = recs * 16u * kCookedWords;
    mbar_expect_tx(&sm.full_bar[stage], bytes);
    bulk_load(sm.tiles + (size_t)stage * tile_recs * kCookedWords, cooked + (size_t)tile * tile_recs * kCookedWords,
              bytes, &sm.full_bar[stage]);
}

// Account the queued completions of the whole warp once some lane holds kFlushAt of them.
// The side-output pointers of the candidate (dump rows, histogram) are looked up here, when the
// queues are accounted, instead of being carried through the replay loop in registers.
// oc: index of the candidate's record in the output, or a negative value for a lane without one.
template <bool MAXGAP>
__device__ __forceinline__ void flush_now(uint32_t& qn, LaneStats& ls, const LaneEnv& env, const int64_t* classes,
                                          uint32_t sub, const EvalParams& P, int64_t oc) {
    Dump dump{nullptr, nullptr, nullptr, nullptr};
    if (oc >= 0) dump = dump_for(P, (uint32_t)oc);
    if (MAXGAP)
        flush_queue_maxgap(&ls, env.qf, env.qa, env.qb, env.ovf, qn, classes, sub, dump.finish, dump.first, dump.inst,
                           dump.hist);
    else
        flush_queue(&ls, env.qf, env.qa, env.qb, env.ovf, qn, classes, sub, dump.finish, dump.first, dump.inst,
                    dump.hist);
    qn = 0;
}
template <bool MAXGAP>
__device__ __forceinline__ void flush_if_due(uint32_t& qn, LaneStats& ls, const LaneEnv& env, const int64_t* classes,
                                             uint32_t sub, const EvalParams& P, int64_t oc) {
    if (__any_sync(kFullMask, qn >= (uint32_t)kFlushAt)) flush_now<MAXGAP>(qn, ls, env, classes, sub, P, oc);
}

// OPT: the distributor predicts with the step time right after admission (optimistic estimate).
// Inst: LaneInst (default engine: decode speed follows the running count), FrozenInst (speed
// fixed at admission) or QueueInst (FrozenInst with a queue in front of every instance).
// MAXGAP: the TBT term of the hit test looks at the largest token gap.  MINB: blocks per SM the
// register budget must allow: 4 for batches of many waves (127 registers), 3 for batches of one
// wave, which are bound by their longest dependent chains and run a little faster with fewer
// warps per scheduler and 144 registers.
template <bool OPT, class Inst, int MINB, bool MAXGAP>
__global__ void __launch_bounds__(kGroupThreads, MINB)
eval_group_kernel(const EvalParams P, const int tile_recs, const uint32_t pool_bytes) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    const GroupSmem sm = carve(smem_raw, P.n_rows, P.n_classes, tile_recs, pool_bytes, MAXGAP);
    const uint32_t tid = threadIdx.x, lane = tid & 31u, warp = tid >> 5;
    constexpr uint32_t kWarps = kGroupThreads / 32;
    // a wait is followed by a new choice, unless the engine and the estimate make that round redundant
    constexpr bool LOOP = OPT || Inst::kAlwaysLoop;

    // profile residency: decode-step tables and SLO classes into shared memory
    for (uint32_t i = tid; i < P.n_rows * 64u; i += kGroupThreads)
        sm.steps[i] = P.rows[(i >> 6) * kRowStride + 2 + (i & 63u)];
    for (uint32_t i = tid; i < P.n_classes * 3u; i += kGroupThreads) {
        sm.classes[i] = P.classes[i];
    }
    if (tid == 0) {
        for (int s = 0; s < kStages; s++) {
            mbar_init(&sm.full_bar[s], 1);
            sm.empty_cnt[s] = 0;
        }
        sm.work[1] = 0;  // set when a bounded wait ran out: the block stops taking work
        fence_barrier_init();
    }
    __syncthreads();

    unsigned char* const lane_scratch =
        reinterpret_cast<unsigned char*>(P.payload) + ((size_t)blockIdx.x * kGroupThreads + tid) * kLaneScratchBytes;
    LaneEnv env;
    env.qf = sm.qf + tid;
    env.qa = sm.qa + tid;
    env.qb = sm.qb + tid;
    env.pay_a = reinterpret_cast<uint4*>(lane_scratch + kLaneScratchA);
    env.pay_b = reinterpret_cast<uint2*>(lane_scratch + kLaneScratchB);
    env.ovf = lane_scratch + kLaneScratchOvf;
    env.qg = MAXGAP ? sm.qg + tid : nullptr;
    env.mg = nullptr;
    env.dl = nullptr;
    env.first = nullptr;
    env.stk = nullptr;
    const bool use_mask = P.class_mask != nullptr && P.n_classes <= 32;
    const uint32_t n_traces = P.n_traces > 1 ? P.n_traces : 1u;
    uint32_t tile_seq = 0;  // tiles consumed so far by this warp (same in every warp)

    // how many work items (4 warps each) every bucket contributes (largest groups first)
    uint32_t items[6];
    uint32_t total_items = 0;
    for (int b = 5; b >= 0; b--) {
        const uint32_t gpw = 32u >> b;                                 // groups per warp
        const uint32_t n_warps = (P.bucket_count[b] + gpw - 1) / gpw;
        items[b] = (n_warps + kWarps - 1) / kWarps;
        total_items += items[b];
    }
    // with several traces every work item exists once per trace: item index = item * n_traces + trace
    const uint32_t total_all = total_items * n_traces;

    for (;;) {
        __syncthreads();  // everyone is done with the previous batch (tiles, work slot)
        if (tid == 0) {
            // Work items are ordered from expensive to cheap.  SM s owns items s, s + n_sm, ...:
            // every SM gets the same share of each cost class however blocks were placed; a
            // block whose SM has run out takes from the other SMs' shares.
            uint32_t item = 0xFFFFFFFFu;
            if (!sm.work[1]) {
                uint32_t my_sm;
                asm volatile("mov.u32 %0, %%smid;" : "=r"(my_sm));
                for (uint32_t k = 0; k < P.n_sm && item == 0xFFFFFFFFu; k++) {
                    const uint32_t s = (my_sm + k) % P.n_sm;
                    if (*(volatile uint32_t*)&P.sm_ctr[s] * P.n_sm >= total_all) continue;  // exhausted
                    // snake order: odd rounds run backwards, so the SM that got the most expensive
                    // item of one round gets the cheapest of the next
                    const uint32_t j = atomicAdd(&P.sm_ctr[s], 1u);
                    const uint32_t it = j * P.n_sm + ((j & 1u) ? P.n_sm - 1u - s : s);
                    if (it < total_all) item = it;
                }
            }
            sm.work[0] = item;
        }
        __syncthreads();
        uint32_t wi = sm.work[0];
        if (wi >= total_all) break;
        const uint32_t tr = wi % n_traces;  // which trace this item replays
        wi /= n_traces;
        const uint4* const cooked = P.n_traces > 1 ? P.trace_cooked[tr] : P.cooked;
        const uint32_t n_req = P.n_traces > 1 ? P.trace_n[tr] : P.n_req;
        const uint32_t n_tiles = (n_req + tile_recs - 1) / tile_recs;
        const uint32_t out_base = tr * P.n_cand;  // this trace's block of records
        int b = 5;
        while (wi >= items[b]) { wi -= items[b]; b--; }
        const uint32_t G = 1u << b;
        const bool own = b == 5;  // the warp holds one candidate
        const uint32_t sub = tid & (G - 1u);
        // The bucket list is sorted by decreasing cost estimate.  Group slot j of warp x takes
        // position j * n_warps + x: every warp gets one candidate of each cost quantile, so the
        // expensive ones (whose events serialise inside a warp) are dealt one per warp, and the
        // most expensive warps start first.
        const uint32_t cnt = P.bucket_count[b];
        const uint32_t gpw = 32u >> b;
        const uint32_t n_warps = (cnt + gpw - 1) / gpw;
        const uint32_t warp_x = wi * kWarps + warp;
        const uint32_t pos = (lane >> b) * n_warps + warp_x;
        const bool valid = warp_x < n_warps && pos < cnt;
        const uint32_t cand = valid ? P.bucket_list[(size_t)b * P.n_cand + pos] : 0u;
        const uint32_t gmask = (G == 32u) ? kFullMask : (((1u << G) - 1u) << (lane & ~(G - 1u)));

        uint32_t n_i = 0, lo = 0;
        if (valid) { lo = P.offsets[cand]; n_i = P.offsets[cand + 1] - lo; }
        const bool has = valid && sub < n_i;
        Inst in;
        lane_reset(in, sm.steps);
        if (has) {
            const uint32_t word = P.inst[lo + sub];
            in.model = word & 0xFu;
            in.B = (word >> 12) & 0xFFu;
            const uint32_t row = in.model * P.n_strategies + ((word >> 4) & 0xFFu);
            in.step = sm.steps + row * 64u;
            in.stepB = (uint32_t)in.step[in.B - 1];
            in.pre_base = (uint32_t)P.rows[row * kRowStride + 0];
            in.pre_q16 = (uint32_t)P.rows[row * kRowStride + 1];
            in.mask = in.B >= 64u ? 0ull : (~0ull << in.B);
        }
        // key storage: every lane takes one 32-byte unit per block of 8 slots of its batch cap,
        // plus one for the block minima, from the thread block's pool, in thread order; lanes the
        // pool cannot hold use their global scratch instead
        {
            const uint32_t nblk = has ? (in.B + 7u) >> 3 : 0u;
            // largest-gap mode of the default engine: per slot two 8-byte words and one 4-byte word after the
            // minima (8 slots x words x 4 B = `words` units per block), then the lane's list of stretch gaps
            const uint32_t gap_units = (MAXGAP && Inst::kGapWords) ? nblk * Inst::kGapWords + Inst::kGapListUnits : 0u;
            const uint32_t units = has ? (nblk + 1u) * Inst::kKeyWords + gap_units : 0u;
            uint32_t incl = units;
            for (uint32_t o = 1; o < 32u; o <<= 1) {
                const uint32_t v = __shfl_up_sync(kFullMask, incl, o);
                if (lane >= o) incl += v;
            }
            if (lane == 31u) sm.wsum[warp] = incl;
            __syncthreads();
            uint32_t start = incl - units;
            for (uint32_t i = 0; i < warp; i++) start += sm.wsum[i];
            unsigned char* region = ((size_t)(start + units) * kKeyUnitBytes <= pool_bytes)
                                        ? sm.pool + (size_t)start * kKeyUnitBytes
                                        : lane_scratch + kLaneScratchKeys;
            env.keys_shared = region != lane_scratch + kLaneScratchKeys;
            env.keys = reinterpret_cast<uint32_t*>(region);
            env.bm_lo = reinterpret_cast<uint4*>(region + (size_t)nblk * kKeyUnitBytes * Inst::kKeyWords);
            env.bm_hi = env.bm_lo + 1;
            if (MAXGAP && Inst::kGapWords) {
                env.mg = reinterpret_cast<uint64_t*>(region + (size_t)(nblk + 1u) * kKeyUnitBytes * Inst::kKeyWords);
                env.dl = env.mg + 8u * nblk;
                env.first = reinterpret_cast<uint32_t*>(env.dl + 8u * nblk);
                env.stk = reinterpret_cast<uint4*>(env.first + 8u * nblk);
            }
            const uint4 e4 = make_uint4(kKeyEmpty, kKeyEmpty, kKeyEmpty, kKeyEmpty);
            for (uint32_t i = 0; i < 2u * units; i++) reinterpret_cast<uint4*>(region)[i] = e4;
        }
        const bool warp_has_work = __any_sync(kFullMask, valid);
        // models the group's placement has an instance of
        uint32_t gmodels = has ? (1u << in.model) : 0u;
        for (uint32_t o = 1; o < G; o <<= 1) gmodels |= __shfl_xor_sync(kFullMask, gmodels, (int)o);
        const uint32_t cmask = (valid && use_mask) ? P.class_mask[cand] : 0xFFFFFFFFu;
        // index of the candidate's record; the side outputs hang on it (dump rows, histogram)
        const int64_t oc = valid ? (int64_t)(out_base + cand) : -1;
        // per-request side outputs of a rejection (dump rows, per-model counts) are rare: one flag guards them
        bool side = P.rej_by_model != nullptr;
        if (valid && P.dump_row) side = side || P.dump_row[cand] >= 0;
        LaneStats ls;
        ls.st.clear();
        for (int i = 0; i < 8; i++) ls.hbc[i] = 0;
        ls.qg = env.qg;  // read by the largest-gap form of the flush only
        uint64_t rej_sum = 0;  // checksum terms of rejected requests
        int64_t now = 0;
        uint32_t n_counted = 0, n_rejected = 0, status = 0;
        uint64_t attempts = 0;   // distributor rounds beyond the first of each counted request

        // trace staging: first tiles of this batch
        if (tid == 0 && !P.stall_test) {
            for (uint32_t j = 0; j < (uint32_t)kStages && j < n_tiles; j++)
                issue_tile(sm, cooked, n_req, (tile_seq + j) % kStages, j, tile_recs);
        }

        for (uint32_t t = 0; t < n_tiles; t++) {
            const uint32_t s = tile_seq % kStages, parity = (tile_seq / kStages) & 1u;
            const bool arrived = mbar_wait_bounded(&sm.full_bar[s], parity, P.wait_cycles);
            if (!__all_sync(kFullMask, arrived)) {
                mbar_wait_bounded(&sm.full_bar[s], parity, P.wait_cycles);  // give copies in flight one more bounded chance
                // and the later tiles of this item that may have been issued already: no bulk copy
                // should land in this block's shared memory after the block has left
                if (!P.stall_test)
                    for (uint32_t x = 1; x < (uint32_t)kStages && t + x < n_tiles; x++) {
                        const uint32_t ts = tile_seq + x;
                        mbar_wait_bounded(&sm.full_bar[ts % kStages], (ts / kStages) & 1u, P.wait_cycles);
                    }
                status = MAASO_CAND_ETIMEOUT;
                sm.work[1] = 1;
                break;
            }
            const uint4* tile = sm.tiles + (size_t)s * tile_recs * kCookedWords;
            const uint32_t recs = min((uint32_t)tile_recs, n_req - t * tile_recs);
            // a warp without a candidate only keeps the tile pipeline going
            for (uint32_t ri = warp_has_work ? 0u : recs; ri < recs; ri++) {
                // statistics of completed requests: every fourth request, if some lane's queue is nearly full
                if ((ri & 3u) == 0u) flush_if_due<MAXGAP>(in.qn, ls, env, sm.classes, sub, P, oc);
                const uint4* rec = tile + (size_t)ri * kCookedWords;
                const uint4 r0 = rec[0], r1 = rec[1], r2 = rec[2];
                // All 32 lanes walk the trace together and every warp-level operation below uses
                // the full mask (segmented by the group width), so the groups of a warp share one
                // instruction stream; only events (retire, admit) diverge.
                const CookedReq q = decode_cooked(r0, r1, r2);
                const uint32_t req = t * tile_recs + ri;
                bool pending = valid && status == 0 && ((cmask >> (q.cls & 31u)) & 1u);
                if (pending) {
                    n_counted++;
                    now = max(now, q.arrival);  // pending time: the dispatcher never goes back
                    // The plain rejections need no look at any instance: the placement has no instance
                    // of the model, or the dispatcher's clock has already passed the request's
                    // first-token or end-to-end deadline (every predicted first token lies at or after
                    // `now`).  The instances are not advanced either: their clocks catch up lazily.
                    if (!((gmodels >> q.model) & 1u) || q.dl_ttft < now || q.dl_e2e < now) {
                        if (LOOP) attempts++;
                        n_rejected++;
                        if (sub == 0) {
                            rej_sum += q.rej;
                            if (side) reject_side(P, out_base + cand, req, q.model);
                        }
                        pending = false;
                    }
                }
                if (!__any_sync(kFullMask, pending)) continue;  // nothing for the distributor in this warp
                const int64_t pre = prefill_us(in.pre_base, in.pre_q16, q.in_tokens);
                const bool elig = has && in.model == q.model;
                uint32_t tries = 0;
                do {
                    uint32_t key = kKey32Inf;
                    int64_t t0 = 0, first = 0;
                    if (LOOP && pending) {
                        attempts++;
                        tries++;
                    }
                    if (pending && elig) {
                        lane_advance<MAXGAP>(in, now, false, env, status);
                        key = lane_predict(in, q, pre, now, OPT, t0, first);
                    }
                    const ArgMin am = group_argmin(key, first, gmask, G, own);
                    if (pending) {
                        if (!am.found) {
                            // overflow protection: nobody can meet the deadline -> rejected
                            n_rejected++;
                            if (sub == 0) {
                                rej_sum += q.rej;
                                if (side) reject_side(P, out_base + cand, req, q.model);
                            }
                            pending = false;
                        } else if (am.tier == 0) {
                            if ((int)lane == am.winner) lane_admit<MAXGAP>(in, q, req, pre, now, env, status);
                            pending = false;
                        } else if constexpr (Inst::kQueues) {
                            // every capable instance is full: the request queues at the chosen one
                            if ((int)lane == am.winner) lane_admit_queued<MAXGAP>(in, q, req, pre, env, status);
                            pending = false;
                        } else {
                            // every capable instance is full: wait until the chosen slot frees (the
                            // outcome is the same for all lanes of the group, so they are all here)
                            now = (int64_t)shfl_u64((uint64_t)t0, am.winner, gmask);
                            if (!LOOP) {
                                // With the worst-case estimate the next round cannot choose differently:
                                // at that time the winner has a free slot with the same predicted first
                                // token, and no other instance's prediction can have become earlier or
                                // feasible.  The second round is only counted; other clocks catch up lazily.
                                attempts++;  // the second round, counted only
                                if ((int)lane == am.winner) {
                                    lane_advance<MAXGAP>(in, now, false, env, status);
                                    lane_admit<MAXGAP>(in, q, req, pre, now, env, status);
                                }
                                pending = false;
                            } else if (tries >= kAttemptCap) {
                                status = MAASO_CAND_ELOOP;
                                pending = false;
                            }
                        }
                    }
                } while (LOOP && __any_sync(kFullMask, pending));
                // An admission can flag its candidate on the winner's lane alone (a time or a queue
                // beyond what the lane state can hold).  Every lane of the group must see the flag
                // before the next request, or `pending` would differ inside the group and a group
                // shuffle would name lanes that are not there.
                if (__any_sync(kFullMask, status != 0u))
                    for (uint32_t o = 1; o < G; o <<= 1) status |= __shfl_xor_sync(kFullMask, status, (int)o);
            }
            // release the stage; the warp that arrives last refills it
            __syncwarp();
            if (lane == 0) {
                __threadfence_block();
                const uint32_t old = atomicAdd(&sm.empty_cnt[s], 1u);
                if (old == kWarps - 1) {
                    sm.empty_cnt[s] = 0;
                    const uint32_t nt = t + kStages;
                    if (nt < n_tiles) {
                        fence_proxy_async();
                        issue_tile(sm, cooked, n_req, s, nt, tile_recs);
                    }
                }
            }
            tile_seq++;
        }

        // drain, account what is still queued, reduce over the group, write the record
        __syncwarp();
        flush_now<MAXGAP>(in.qn, ls, env, sm.classes, sub, P, oc);
        if (has && status == 0) lane_advance<MAXGAP>(in, 0, true, env, status);
        __syncwarp();
        flush_now<MAXGAP>(in.qn, ls, env, sm.classes, sub, P, oc);
        Stats st = ls.st;
        st.checksum += rej_sum;
        uint32_t h[8];
        for (int i = 0; i < 8; i++) h[i] = ls.hbc[i];
        for (uint32_t off = 1; off < G; off <<= 1) {
            for (int i = 0; i < 8; i++) h[i] += __shfl_xor_sync(kFullMask, h[i], (int)off);
            status |= __shfl_xor_sync(kFullMask, status, (int)off);
            st.served += __shfl_xor_sync(kFullMask, st.served, (int)off);
            st.hit += __shfl_xor_sync(kFullMask, st.hit, (int)off);
            st.sum_ttft += (int64_t)shfl_xor_u64((uint64_t)st.sum_ttft, (int)off, kFullMask);
            st.sum_e2e += (int64_t)shfl_xor_u64((uint64_t)st.sum_e2e, (int)off, kFullMask);
            st.tokens += shfl_xor_u64(st.tokens, (int)off, kFullMask);
            st.checksum += shfl_xor_u64(st.checksum, (int)off, kFullMask);
            st.max_ttft = max(st.max_ttft, (int64_t)shfl_xor_u64((uint64_t)st.max_ttft, (int)off, kFullMask));
            st.max_e2e = max(st.max_e2e, (int64_t)shfl_xor_u64((uint64_t)st.max_e2e, (int)off, kFullMask));
            st.makespan = max(st.makespan, (int64_t)shfl_xor_u64((uint64_t)st.makespan, (int)off, kFullMask));
        }
        __syncwarp();
        if (valid && sub == 0) {
            // worst-case mode: one round per counted request plus the counted second rounds
            write_result(P.out + out_base + cand, status, n_counted, n_rejected, LOOP ? attempts : attempts + n_counted, st, h);
        }
    }
}

using GroupKernel = void (*)(const EvalParams, const int, const uint32_t);
template <int MINB, bool MAXGAP>
static GroupKernel group_kernel_of(uint32_t flags) {
    const bool opt = (flags & MAASO_FLAG_PRED_OPTIMISTIC) != 0;
    if (flags & MAASO_FLAG_ENGINE_FROZEN)
        return opt ? eval_group_kernel<true, FrozenInst, MINB, MAXGAP> : eval_group_kernel<false, FrozenInst, MINB, MAXGAP>;
    return opt ? eval_group_kernel<true, LaneInst, MINB, MAXGAP> : eval_group_kernel<false, LaneInst, MINB, MAXGAP>;
}
template <bool MAXGAP>
static GroupKernel queue_kernel_of(uint32_t flags) {
    return (flags & MAASO_FLAG_PRED_OPTIMISTIC) ? eval_group_kernel<true, QueueInst, 4, MAXGAP>
                                                : eval_group_kernel<false, QueueInst, 4, MAXGAP>;
}
static GroupKernel group_kernel_for(uint32_t flags, int blocks_per_sm) {
    if (flags & MAASO_FLAG_INSTANCE_QUEUES)  // one register budget for this mode
        return (flags & MAASO_FLAG_TBT_MAXGAP) ? queue_kernel_of<true>(flags) : queue_kernel_of<false>(flags);
    if (flags & MAASO_FLAG_TBT_MAXGAP) return group_kernel_of<4, true>(flags);  // one register budget for this mode
    return blocks_per_sm >= 4 ? group_kernel_of<4, false>(flags) : group_kernel_of<3, false>(flags);
}

// Shared memory of one block: the fixed parts plus a key pool that fills what is left when
// `blocks_per_sm` blocks share an SM (1 KB per block is reserved by the system), at most what
// 128 lanes with 64 slots each can use.
static size_t group_smem_bytes(const EvalParams& P, int tile_recs, int blocks_per_sm, int smem_per_sm,
                               uint32_t* pool_bytes) {
    const size_t fixed = group_smem_static(P.n_rows, P.n_classes, tile_recs, (P.flags & MAASO_FLAG_TBT_MAXGAP) != 0);
    size_t budget = (size_t)smem_per_sm / (size_t)blocks_per_sm;
    budget = budget > 1024 ? budget - 1024 : 0;
    if (budget > 227u * 1024u) budget = 227u * 1024u;
    size_t pool = budget > fixed ? budget - fixed : 0;
    pool -= pool % 128;
    size_t lane_units = 9;  // 8 key blocks + the block minima
    if (P.flags & (MAASO_FLAG_ENGINE_FROZEN | MAASO_FLAG_INSTANCE_QUEUES)) lane_units = 18;
    else if (P.flags & MAASO_FLAG_TBT_MAXGAP) lane_units = 9 + 5 * 8 + 8;
    const size_t all = (size_t)kGroupThreads * lane_units * kKeyUnitBytes;
    if (pool > all) pool = all;
    *pool_bytes = (uint32_t)pool;
    return fixed + pool;
}

cudaError_t launch_eval_group(const EvalParams& P, int grid, int tile_recs, int blocks_per_sm, int smem_per_sm,
                              cudaStream_t stream) {
    uint32_t pool = 0;
    const size_t smem = group_smem_bytes(P, tile_recs, blocks_per_sm, smem_per_sm, &pool);
    auto kernel = group_kernel_for(P.flags, blocks_per_sm);
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    kernel<<<grid, kGroupThreads, smem, stream>>>(P, tile_recs, pool);
    return cudaGetLastError();
}

size_t group_scratch_per_lane() { return kLaneScratchBytes; }

int occupancy_eval_group(const EvalParams& P, int tile_recs, int blocks_per_sm, int smem_per_sm) {
    uint32_t pool = 0;
    const size_t smem = group_smem_bytes(P, tile_recs, blocks_per_sm, smem_per_sm, &pool);
    auto kernel = group_kernel_for(P.flags, blocks_per_sm);
    cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    int n = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, kernel, kGroupThreads, smem) != cudaSuccess) return 1;
    return n < 1 ? 1 : n;
}

}  // namespace maaso
