// Scoring kernel, lane-group mapping: a candidate with I <= 32 instances is replayed by a
// group of G = 2^ceil(log2 I) lanes of one warp, one lane per simulated instance.  All
// instance state lives in registers; slot keys in shared memory; the distributor's argmin
// is a shuffle butterfly inside the group.  The trace is staged once per thread block in
// shared-memory tiles by 1-D bulk copies (TMA) and shared by every candidate of the block.
#include "lane_sim.cuh"

namespace maaso {

constexpr int kStages = 3;

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
// among equals.  Called by all 32 lanes; every operation uses the full mask and stays inside
// the group because xor offsets are below G.  G may be smaller than the group when only its
// first G lanes hold instances: the other lanes then see "nothing found", which is harmless
// because only lanes with instances and the group's first lane act on the result.
__device__ __forceinline__ ArgMin group_argmin(uint64_t key, uint32_t gmask, uint32_t G) {
    ArgMin r;
    uint64_t best = key;
    for (uint32_t off = 1; off < G; off <<= 1) best = min(best, shfl_xor_u64(best, (int)off, 0xFFFFFFFFu));
    r.found = best != kKeyInf;
    r.tier = (uint32_t)(best >> 63);
    const uint32_t votes = __ballot_sync(0xFFFFFFFFu, key == best) & gmask;
    r.winner = r.found ? __ffs((int)votes) - 1 : (int)(threadIdx.x & 31u);
    return r;
}

struct GroupSmem {
    uint4* tiles;        // [kStages][tile_recs]
    int32_t* steps;      // [n_rows][64]
    int64_t* classes;    // [n_classes][3], negative = no limit (completion accounting)
    int64_t* plimits;    // [n_classes][3], INT64_MAX = no limit (distributor prediction)
    uint16_t* keys;      // [kGroupThreads][kKeyStride]
    uint32_t* hbc;       // [kGroupThreads][8]
    uint64_t* full_bar;  // [kStages]
    uint32_t* empty_cnt; // [kStages]
    uint32_t* work;      // [2]
};

__host__ __device__ inline size_t group_smem_bytes(uint32_t n_rows, uint32_t n_classes, int tile_recs) {
    size_t b = (size_t)kStages * tile_recs * 16;
    b += (size_t)n_rows * 64 * 4;
    b += (size_t)n_classes * 48;
    b += (size_t)kGroupThreads * kKeyStride * 2;
    b += (size_t)kGroupThreads * 8 * 4;
    b += kStages * 8 + kStages * 4 + 8 + 32;
    return (b + 15) & ~(size_t)15;
}

__device__ __forceinline__ GroupSmem carve(unsigned char* base, uint32_t n_rows, uint32_t n_classes,
                                           int tile_recs) {
    GroupSmem s;
    // 16-byte aligned parts first (tiles, slot keys are read as 16-byte words)
    s.tiles = reinterpret_cast<uint4*>(base);
    base += (size_t)kStages * tile_recs * 16;
    s.keys = reinterpret_cast<uint16_t*>(base);
    base += (size_t)kGroupThreads * kKeyStride * 2;
    s.hbc = reinterpret_cast<uint32_t*>(base);
    base += (size_t)kGroupThreads * 8 * 4;
    s.classes = reinterpret_cast<int64_t*>(base);
    base += (size_t)n_classes * 24;
    s.plimits = reinterpret_cast<int64_t*>(base);
    base += (size_t)n_classes * 24;
    s.full_bar = reinterpret_cast<uint64_t*>(base);
    base += kStages * 8;
    s.steps = reinterpret_cast<int32_t*>(base);
    base += (size_t)n_rows * 64 * 4;
    s.empty_cnt = reinterpret_cast<uint32_t*>(base);
    base += kStages * 4;
    s.work = reinterpret_cast<uint32_t*>(base);
    return s;
}

// OPT: the distributor predicts with the step time right after admission (optimistic estimate)
template <bool OPT>
__global__ void __launch_bounds__(kGroupThreads)
eval_group_kernel(const EvalParams P, const int tile_recs) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const GroupSmem sm = carve(smem_raw, P.n_rows, P.n_classes, tile_recs);
    const uint32_t tid = threadIdx.x, lane = tid & 31u;
    constexpr uint32_t kWarps = kGroupThreads / 32;

    // profile residency: decode-step tables and SLO classes into shared memory
    for (uint32_t i = tid; i < P.n_rows * 64u; i += kGroupThreads)
        sm.steps[i] = P.rows[(i >> 6) * kRowStride + 2 + (i & 63u)];
    for (uint32_t i = tid; i < P.n_classes * 3u; i += kGroupThreads) {
        const int64_t v = P.classes[i];
        sm.classes[i] = v;
        sm.plimits[i] = v < 0 ? INT64_MAX : v;
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

    LaneEnv env;
    env.keys = sm.keys + tid * kKeyStride;
    env.hbc = sm.hbc + tid * 8;
    env.pay = P.payload + ((size_t)blockIdx.x * kGroupThreads + tid) * MAASO_WMAX;
    env.classes = sm.classes;
    uint32_t* const hbc = env.hbc;
    const bool use_mask = P.class_mask != nullptr && P.n_classes <= 32;
    const uint32_t n_tiles = (P.n_req + tile_recs - 1) / tile_recs;
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
                    if (*(volatile uint32_t*)&P.sm_ctr[s] * P.n_sm >= total_items) continue;  // exhausted
                    // snake order: odd rounds run backwards, so the SM that got the most expensive
                    // item of one round gets the cheapest of the next
                    const uint32_t j = atomicAdd(&P.sm_ctr[s], 1u);
                    const uint32_t it = j * P.n_sm + ((j & 1u) ? P.n_sm - 1u - s : s);
                    if (it < total_items) item = it;
                }
            }
            sm.work[0] = item;
        }
        __syncthreads();
        uint32_t wi = sm.work[0];
        if (wi >= total_items) break;
        int b = 5;
        while (wi >= items[b]) { wi -= items[b]; b--; }
        const uint32_t G = 1u << b;
        const uint32_t sub = tid & (G - 1u);
        // The bucket list is sorted by decreasing cost estimate.  Group slot j of warp x takes
        // position j * n_warps + x: every warp gets one candidate of each cost quantile, so the
        // expensive ones (whose events serialise inside a warp) are dealt one per warp, and the
        // most expensive warps start first.
        const uint32_t cnt = P.bucket_count[b];
        const uint32_t gpw = 32u >> b;
        const uint32_t n_warps = (cnt + gpw - 1) / gpw;
        const uint32_t warp_x = wi * kWarps + (tid >> 5);
        const uint32_t pos = (lane >> b) * n_warps + warp_x;
        const bool valid = warp_x < n_warps && pos < cnt;
        const uint32_t cand = valid ? P.bucket_list[(size_t)b * P.n_cand + pos] : 0u;
        const uint32_t gmask = (G == 32u) ? 0xFFFFFFFFu : (((1u << G) - 1u) << (lane & ~(G - 1u)));

        uint32_t n_i = 0, lo = 0;
        if (valid) { lo = P.offsets[cand]; n_i = P.offsets[cand + 1] - lo; }
        const bool has = valid && sub < n_i;
        LaneInst in;
        in.T = 0; in.tc = 0; in.K = 0; in.w = 0; in.kmin = 0; in.sw = 1; in.rsw = 1.0f; in.bslots = 0; in.mask = 0;
        in.B = 1; in.model = 0xFFFFFFFFu; in.step = sm.steps; in.stepB = 1; in.pre_base = 0; in.pre_q16 = 0;
        if (has) {
            const uint32_t word = P.inst[lo + sub];
            in.model = word & 0xFu;
            in.B = (word >> 12) & 0xFFu;
            const uint32_t row = in.model * P.n_strategies + ((word >> 4) & 0xFFu);
            in.step = sm.steps + row * 64u;
            in.stepB = (uint32_t)in.step[in.B - 1];
            in.pre_base = (uint32_t)P.rows[row * kRowStride + 0];
            in.pre_q16 = (uint32_t)P.rows[row * kRowStride + 1];
        }
        // A warp that holds a single candidate (bucket 5, possibly promoted there with few
        // instances) only needs as many butterfly rounds as it has instances.
        const uint32_t n_i_warp = __shfl_sync(0xFFFFFFFFu, n_i, 0);
        const uint32_t Geff = b == 5 ? (n_i_warp <= 1 ? 1u : 1u << (32 - __clz((int)(n_i_warp - 1)))) : G;
        const uint32_t cmask = (valid && use_mask) ? P.class_mask[cand] : 0xFFFFFFFFu;
        Dump dump{nullptr, nullptr, nullptr};
        if (valid) dump = dump_for(P, cand);
        env.dump = dump;
        env.inst_idx = sub;
        Stats st; st.clear();
        for (int i = 0; i < 8; i++) hbc[i] = 0;
        int64_t now = 0;
        uint32_t n_counted = 0, n_rejected = 0, status = 0;
        uint64_t attempts = 0;

        // trace staging: first tiles of this batch
        if (tid == 0 && !P.stall_test) {
            for (uint32_t j = 0; j < (uint32_t)kStages && j < n_tiles; j++) {
                const uint32_t s = (tile_seq + j) % kStages;
                const uint32_t recs = min((uint32_t)tile_recs, P.n_req - j * tile_recs);
                mbar_expect_tx(&sm.full_bar[s], recs * 16u);
                bulk_load(sm.tiles + (size_t)s * tile_recs, P.reqs + (size_t)j * tile_recs, recs * 16u,
                          &sm.full_bar[s]);
            }
        }

        for (uint32_t t = 0; t < n_tiles; t++) {
            const uint32_t s = tile_seq % kStages, parity = (tile_seq / kStages) & 1u;
            const bool arrived = mbar_wait_bounded(&sm.full_bar[s], parity, P.wait_cycles);
            if (!__all_sync(0xFFFFFFFFu, arrived)) {
                mbar_wait_bounded(&sm.full_bar[s], parity, P.wait_cycles);  // give copies in flight one more bounded chance
                status = MAASO_CAND_ETIMEOUT;
                sm.work[1] = 1;
                break;
            }
            const uint4* tile = sm.tiles + (size_t)s * tile_recs;
            const uint32_t recs = min((uint32_t)tile_recs, P.n_req - t * tile_recs);
            uint4 raw_next = tile[0];
            for (uint32_t ri = 0; ri < recs; ri++) {
                const uint4 raw = raw_next;
                raw_next = tile[min(ri + 1, recs - 1)];  // read the next record ahead of its use
                // All 32 lanes walk the trace together and every warp-level operation below uses
                // the full mask (segmented by the group width), so the groups of a warp share one
                // instruction stream; only events (retire, admit) diverge.
                const Request q = decode_request(raw);
                const uint32_t req = t * tile_recs + ri;
                bool pending = valid && status == 0 && ((cmask >> (q.cls & 31u)) & 1u);
                if (pending) {
                    n_counted++;
                    now = max(now, q.arrival);  // pending time: the dispatcher never goes back
                }
                const int64_t pre = prefill_us(in.pre_base, in.pre_q16, q.in_tokens);
                const bool elig = has && in.model == q.model;
                const int64_t lim_ttft = sm.plimits[q.cls * 3 + 0];
                const int64_t lim_tbt = sm.plimits[q.cls * 3 + 1];
                const int64_t lim_e2e = sm.plimits[q.cls * 3 + 2];
                uint32_t tries = 0;
                do {
                    uint64_t key = kKeyInf;
                    int64_t t0 = 0;
                    if (pending) {
                        attempts++;
                        tries++;
                    }
                    if (pending && elig) {
                        lane_advance(in, now, false, env, st);
                        key = lane_predict(in, q, pre, lim_ttft, lim_tbt, lim_e2e, OPT, t0);
                    }
                    const ArgMin am = group_argmin(key, gmask, Geff);
                    const int64_t t0w = (int64_t)shfl_u64((uint64_t)t0, am.winner, 0xFFFFFFFFu);
                    if (pending) {
                        if (!am.found) {
                            // overflow protection: nobody can meet the deadline -> rejected
                            n_rejected++;
                            if (sub == 0) {
                                st.checksum += __ldg(P.rej_hash + req);
                                if (P.rej_by_model)
                                    atomicAdd(&P.rej_by_model[(size_t)cand * MAASO_MAX_MODELS + q.model], 1u);
                                if (dump.finish) dump.finish[req] = -1;
                                if (dump.first) dump.first[req] = -1;
                                if (dump.inst) dump.inst[req] = -1;
                            }
                            pending = false;
                        } else if (am.tier == 0) {
                            if ((int)lane == am.winner) lane_admit(in, q, req, pre, env, st);
                            pending = false;
                        } else {
                            // every capable instance is full: wait until the chosen slot frees
                            now = t0w;
                            if (!OPT) {
                                // With the worst-case estimate the next round cannot choose differently:
                                // at that time the winner has a free slot with the same predicted first
                                // token, and no other instance's prediction can have become earlier or
                                // feasible.  The second round is only counted; other clocks catch up lazily.
                                attempts++;
                                if ((int)lane == am.winner) {
                                    lane_advance(in, now, false, env, st);
                                    lane_admit(in, q, req, pre, env, st);
                                }
                                pending = false;
                            } else if (tries >= kAttemptCap) {
                                status = MAASO_CAND_ELOOP;
                                pending = false;
                            }
                        }
                    }
                } while (OPT && __any_sync(0xFFFFFFFFu, pending));
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
                        const uint32_t nrecs = min((uint32_t)tile_recs, P.n_req - nt * tile_recs);
                        fence_proxy_async();
                        mbar_expect_tx(&sm.full_bar[s], nrecs * 16u);
                        bulk_load(sm.tiles + (size_t)s * tile_recs, P.reqs + (size_t)nt * tile_recs,
                                  nrecs * 16u, &sm.full_bar[s]);
                    }
                }
            }
            tile_seq++;
        }

        // drain, reduce over the group, write the record
        if (has && status == 0) lane_advance(in, 0, true, env, st);
        __syncwarp();
        constexpr uint32_t kFull = 0xFFFFFFFFu;
        for (uint32_t off = 1; off < G; off <<= 1) {
            st.served += __shfl_xor_sync(kFull, st.served, (int)off);
            st.hit += __shfl_xor_sync(kFull, st.hit, (int)off);
            st.sum_ttft += (int64_t)shfl_xor_u64((uint64_t)st.sum_ttft, (int)off, kFull);
            st.sum_e2e += (int64_t)shfl_xor_u64((uint64_t)st.sum_e2e, (int)off, kFull);
            st.tokens += shfl_xor_u64(st.tokens, (int)off, kFull);
            st.checksum += shfl_xor_u64(st.checksum, (int)off, kFull);
            st.max_ttft = max(st.max_ttft, (int64_t)shfl_xor_u64((uint64_t)st.max_ttft, (int)off, kFull));
            st.max_e2e = max(st.max_e2e, (int64_t)shfl_xor_u64((uint64_t)st.max_e2e, (int)off, kFull));
            st.makespan = max(st.makespan, (int64_t)shfl_xor_u64((uint64_t)st.makespan, (int)off, kFull));
        }
        __syncwarp();
        if (valid && sub == 0) {
            uint32_t h[8];
            for (int i = 0; i < 8; i++) h[i] = 0;
            for (uint32_t g = 0; g < G; g++)
                for (int i = 0; i < 8; i++) h[i] += sm.hbc[(tid + g) * 8 + i];
            write_result(P.out + cand, status, n_counted, n_rejected, attempts, st, h);
        }
    }
}

cudaError_t launch_eval_group(const EvalParams& P, int grid, int tile_recs, cudaStream_t stream) {
    const size_t smem = group_smem_bytes(P.n_rows, P.n_classes, tile_recs);
    const bool opt = (P.flags & MAASO_FLAG_PRED_OPTIMISTIC) != 0;
    auto kernel = opt ? eval_group_kernel<true> : eval_group_kernel<false>;
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    kernel<<<grid, kGroupThreads, smem, stream>>>(P, tile_recs);
    return cudaGetLastError();
}

int occupancy_eval_group(const EvalParams& P, int tile_recs) {
    const size_t smem = group_smem_bytes(P.n_rows, P.n_classes, tile_recs);
    const bool opt = (P.flags & MAASO_FLAG_PRED_OPTIMISTIC) != 0;
    auto kernel = opt ? eval_group_kernel<true> : eval_group_kernel<false>;
    cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    int n = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, kernel, kGroupThreads, smem) != cudaSuccess) return 1;
    return n < 1 ? 1 : n;
}

}  // namespace maaso
