// Scoring kernel for placements of 33 to 128 instances under the engines that exist in the
// lane-group code only (the fixed-speed engine, per-instance queues, the largest-gap test; also the
// default engine when the lane-group mapping is forced with several traces in one pass): one warp
// replays one placement, lane l owns instances l, l + 32, l + 64, l + 96.  It reuses the
// per-instance code of the lane-group kernel (lane_sim.cuh, lane_frozen.cuh) unchanged: every
// (lane, stride) pair is a "virtual lane" with its own instance state, slot keys (in global
// scratch), scratch entries of running requests and completion-queue column.  The distributor's
// choice is a reduction over the four strides of each lane and then over the 32 lanes, on 64-bit
// keys (tier, predicted first token) with ties to the lowest instance index.
//
// This is the slow, plain member of the family: it reads the prepared trace records straight from
// global memory (one look-ahead record in registers) and keeps nothing but the queues and the
// tables in shared memory.  Placements of this size are rare in the sweeps; the default engine
// scores them in the thread kernel.
#include "lane_frozen.cuh"

namespace maaso {

constexpr int kWideStrides = MAASO_MAX_INSTANCES / 32;  // 4
constexpr uint32_t kFullMaskW = 0xFFFFFFFFu;
static_assert(kWideStrides * 32 == kGroupThreads, "a wide warp has as many virtual lanes as a lane-group block has threads");

struct WideSmem {
    uint4* qa;          // [kQueue][kGroupThreads] queued completions: first-token time, arrival time
    uint2* qb;          // [kQueue][kGroupThreads] request index, S | cls << 16
    int64_t* qf;        // [kQueue][kGroupThreads] finish time
    int64_t* qg;        // [kQueue][kGroupThreads] largest token gap (largest-gap mode)
    int64_t* classes;   // [n_classes][3]
    int32_t* steps;     // [n_rows][64]
};
__host__ __device__ inline size_t wide_smem_bytes(uint32_t n_rows, uint32_t n_classes, bool maxgap) {
    size_t b = (size_t)kQueue * kGroupThreads * (16 + 8 + 8 + (maxgap ? 8 : 0));
    b += (size_t)n_classes * 24;
    b += (size_t)n_rows * 64 * 4;
    return (b + 15) & ~(size_t)15;
}
__device__ __forceinline__ WideSmem wide_carve(unsigned char* base, uint32_t n_classes, bool maxgap) {
    WideSmem s;
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
    s.steps = reinterpret_cast<int32_t*>(base);
    return s;
}

__device__ __forceinline__ uint64_t wshfl_xor_u64(uint64_t v, int off) {
    const uint32_t lo = __shfl_xor_sync(kFullMaskW, (uint32_t)v, off);
    const uint32_t hi = __shfl_xor_sync(kFullMaskW, (uint32_t)(v >> 32), off);
    return ((uint64_t)hi << 32) | lo;
}
__device__ __forceinline__ uint64_t wshfl_u64(uint64_t v, int src) {
    const uint32_t lo = __shfl_sync(kFullMaskW, (uint32_t)v, src);
    const uint32_t hi = __shfl_sync(kFullMaskW, (uint32_t)(v >> 32), src);
    return ((uint64_t)hi << 32) | lo;
}

template <bool MAXGAP>
__device__ __forceinline__ void wide_flush(uint32_t& qn, LaneStats& ls, const LaneEnv& env, const int64_t* classes,
                                           uint32_t inst_idx, const EvalParams& P, uint32_t oc) {
    const Dump dump = dump_for(P, oc);
    if (MAXGAP) {
        ls.qg = env.qg;
        flush_queue_maxgap(&ls, env.qf, env.qa, env.qb, env.ovf, qn, classes, inst_idx, dump.finish, dump.first, dump.inst,
                           dump.hist);
    } else {
        flush_queue(&ls, env.qf, env.qa, env.qb, env.ovf, qn, classes, inst_idx, dump.finish, dump.first, dump.inst, dump.hist);
    }
    qn = 0;
}

template <bool OPT, class Inst, bool MAXGAP>
__global__ void __launch_bounds__(32) eval_wide_kernel(const __grid_constant__ EvalParams P) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    const WideSmem sm = wide_carve(smem_raw, P.n_classes, MAXGAP);
    const uint32_t lane = threadIdx.x;
    if (P.stall_test) return;  // test hook: nothing is scored, every valid candidate keeps its "not scored" mark
    for (uint32_t i = lane; i < P.n_rows * 64u; i += 32u) sm.steps[i] = P.rows[(i >> 6) * kRowStride + 2 + (i & 63u)];
    for (uint32_t i = lane; i < P.n_classes * 3u; i += 32u) sm.classes[i] = P.classes[i];
    __syncwarp();
    // a wait is followed by a new choice, unless the engine and the estimate make that round redundant
    constexpr bool LOOP = OPT || Inst::kAlwaysLoop;
    const bool use_mask = P.class_mask != nullptr && P.n_classes <= 32;
    const uint32_t n_traces = P.n_traces > 1 ? P.n_traces : 1u;
    const uint32_t cnt = P.bucket_count[kWideBucket];
    const uint64_t total = (uint64_t)cnt * n_traces;

    for (;;) {
        uint32_t wi = 0;
        if (lane == 0) wi = atomicAdd(&P.work_ctr[14], 1u);
        wi = __shfl_sync(kFullMaskW, wi, 0);
        if (wi >= total) break;
        const uint32_t tr = wi % n_traces;
        const uint32_t cand = P.bucket_list[(size_t)kWideBucket * P.n_cand + wi / n_traces];
        const uint4* const cooked = P.trace_cooked[tr];
        const uint32_t n_req = P.trace_n[tr];
        const uint32_t oc = tr * P.n_cand + cand;
        const uint32_t lo = P.offsets[cand], n_i = P.offsets[cand + 1] - lo;

        Inst ins[kWideStrides];
        LaneEnv envs[kWideStrides];
        bool has[kWideStrides];
        uint32_t gmodels = 0;
#pragma unroll
        for (int s = 0; s < kWideStrides; s++) {
            const uint32_t v = (uint32_t)s * 32u + lane;  // virtual lane = instance index
            Inst& in = ins[s];
            LaneEnv& env = envs[s];
            lane_reset(in, sm.steps);
            has[s] = v < n_i;
            unsigned char* const scratch =
                reinterpret_cast<unsigned char*>(P.payload) + ((size_t)blockIdx.x * kGroupThreads + v) * kLaneScratchBytes;
            env.qf = sm.qf + v;
            env.qa = sm.qa + v;
            env.qb = sm.qb + v;
            env.qg = MAXGAP ? sm.qg + v : nullptr;
            env.pay_a = reinterpret_cast<uint4*>(scratch + kLaneScratchA);
            env.pay_b = reinterpret_cast<uint2*>(scratch + kLaneScratchB);
            env.ovf = scratch + kLaneScratchOvf;
            env.mg = nullptr; env.dl = nullptr; env.first = nullptr; env.stk = nullptr;
            uint32_t nblk = 0;
            if (has[s]) {
                const uint32_t word = P.inst[lo + v];
                in.model = word & 0xFu;
                in.B = (word >> 12) & 0xFFu;
                const uint32_t row = in.model * P.n_strategies + ((word >> 4) & 0xFFu);
                in.step = sm.steps + row * 64u;
                in.stepB = (uint32_t)in.step[in.B - 1];
                in.pre_base = (uint32_t)P.rows[row * kRowStride + 0];
                in.pre_q16 = (uint32_t)P.rows[row * kRowStride + 1];
                in.mask = in.B >= 64u ? 0ull : (~0ull << in.B);
                nblk = (in.B + 7u) >> 3;
                gmodels |= 1u << in.model;
            }
            // slot keys, block minima and (largest-gap mode) gap data in the virtual lane's global scratch
            unsigned char* const region = scratch + kLaneScratchKeys;
            const uint32_t gap_units = (MAXGAP && Inst::kGapWords) ? nblk * Inst::kGapWords + Inst::kGapListUnits : 0u;
            const uint32_t units = has[s] ? (nblk + 1u) * Inst::kKeyWords + gap_units : 0u;
            env.keys_shared = false;
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
        for (uint32_t o = 1; o < 32u; o <<= 1) gmodels |= __shfl_xor_sync(kFullMaskW, gmodels, (int)o);
        const uint32_t cmask = use_mask ? P.class_mask[cand] : 0xFFFFFFFFu;
        bool side = P.rej_by_model != nullptr;
        if (P.dump_row) side = side || P.dump_row[cand] >= 0;
        LaneStats ls;
        ls.st.clear();
        for (int i = 0; i < 8; i++) ls.hbc[i] = 0;
        ls.qg = nullptr;
        uint64_t rej_sum = 0, attempts = 0;
        int64_t now = 0;
        uint32_t n_counted = 0, n_rejected = 0, status = 0;
        __syncwarp();

        uint4 r0 = make_uint4(0, 0, 0, 0), r1 = r0, r2 = r0;
        if (n_req) { r0 = __ldg(cooked); r1 = __ldg(cooked + 1); r2 = __ldg(cooked + 2); }
        for (uint32_t req = 0; req < n_req; req++) {
            const CookedReq q = decode_cooked(r0, r1, r2);
            if (req + 1 < n_req) {  // look-ahead: the next record is on its way while this one is handled
                const uint4* nx = cooked + (size_t)(req + 1) * kCookedWords;
                r0 = __ldg(nx); r1 = __ldg(nx + 1); r2 = __ldg(nx + 2);
            }
            // statistics of completed requests: every fourth request, if some queue is nearly full
            if ((req & 3u) == 0u) {
                bool due = false;
#pragma unroll
                for (int s = 0; s < kWideStrides; s++) due = due || ins[s].qn >= (uint32_t)kFlushAt;
                if (__any_sync(kFullMaskW, due)) {
#pragma unroll
                    for (int s = 0; s < kWideStrides; s++)
                        wide_flush<MAXGAP>(ins[s].qn, ls, envs[s], sm.classes, (uint32_t)s * 32u + lane, P, oc);
                }
            }
            bool pending = status == 0 && ((cmask >> (q.cls & 31u)) & 1u);
            if (!pending) continue;
            n_counted++;
            now = max(now, q.arrival);  // pending time: the dispatcher never goes back
            // the plain rejections: no instance of the model, or the clock has passed a deadline
            if (!((gmodels >> q.model) & 1u) || q.dl_ttft < now || q.dl_e2e < now) {
                if (LOOP) attempts++;
                n_rejected++;
                if (lane == 0) {
                    rej_sum += q.rej;
                    if (side) {
                        const Dump dump = dump_for(P, oc);
                        if (P.rej_by_model) atomicAdd(&P.rej_by_model[(size_t)oc * MAASO_MAX_MODELS + q.model], 1u);
                        if (dump.finish) dump.finish[req] = -1;
                        if (dump.first) dump.first[req] = -1;
                        if (dump.inst) dump.inst[req] = -1;
                    }
                }
                continue;
            }
            uint32_t tries = 0;
            do {
                if (LOOP) { attempts++; tries++; }
                // every virtual lane of the model: advance to `now`, predict; the lane keeps its best stride
                uint64_t key = kKeyInf;
                int64_t t0_best = 0;
                int s_best = 0;
#pragma unroll
                for (int s = 0; s < kWideStrides; s++) {
                    if (!(has[s] && ins[s].model == q.model)) continue;
                    const int64_t pre = prefill_us(ins[s].pre_base, ins[s].pre_q16, q.in_tokens);
                    int64_t t0 = 0, first = 0;
                    lane_advance<MAXGAP>(ins[s], now, false, envs[s], status);
                    const uint32_t k32 = lane_predict(ins[s], q, pre, now, OPT, t0, first);
                    if (k32 == kKey32Inf) continue;
                    const uint64_t k64 = ((uint64_t)(k32 >> 31) << 63) | (uint64_t)first;
                    if (k64 < key) { key = k64; t0_best = t0; s_best = s; }  // strict: the lower stride wins a tie
                }
                // over the lanes: smallest (tier, first token), then lowest instance index = lowest stride, lowest lane
                uint64_t best = key;
                for (int o = 1; o < 32; o <<= 1) best = min(best, wshfl_xor_u64(best, o));
                if (best == kKeyInf) {
                    // overflow protection: nobody can meet the deadline -> rejected
                    n_rejected++;
                    if (lane == 0) {
                        rej_sum += q.rej;
                        if (side) {
                            const Dump dump = dump_for(P, oc);
                            if (P.rej_by_model) atomicAdd(&P.rej_by_model[(size_t)oc * MAASO_MAX_MODELS + q.model], 1u);
                            if (dump.finish) dump.finish[req] = -1;
                            if (dump.first) dump.first[req] = -1;
                            if (dump.inst) dump.inst[req] = -1;
                        }
                    }
                    pending = false;
                } else {
                    uint32_t smin = key == best ? (uint32_t)s_best : 0xFFu;
                    for (int o = 1; o < 32; o <<= 1) smin = min(smin, __shfl_xor_sync(kFullMaskW, smin, o));
                    const uint32_t votes = __ballot_sync(kFullMaskW, key == best && (uint32_t)s_best == smin);
                    const int winner = __ffs((int)votes) - 1;
                    const bool mine = (int)lane == winner;
                    const uint32_t tier = (uint32_t)(best >> 63);
                    if (tier == 0) {
                        if (mine) {
#pragma unroll
                            for (int s = 0; s < kWideStrides; s++)
                                if (s == (int)smin)
                                    lane_admit<MAXGAP>(ins[s], q, req, prefill_us(ins[s].pre_base, ins[s].pre_q16, q.in_tokens), now,
                                                       envs[s], status);
                        }
                        pending = false;
                    } else if constexpr (Inst::kQueues) {
                        // every capable instance is full: the request queues at the chosen one
                        if (mine) {
#pragma unroll
                            for (int s = 0; s < kWideStrides; s++)
                                if (s == (int)smin)
                                    lane_admit_queued<MAXGAP>(ins[s], q, req, prefill_us(ins[s].pre_base, ins[s].pre_q16, q.in_tokens),
                                                              envs[s], status);
                        }
                        pending = false;
                    } else {
                        // every capable instance is full: wait until the chosen slot frees
                        now = (int64_t)wshfl_u64((uint64_t)t0_best, winner);
                        if (!LOOP) {
                            // under the worst-case estimate the round after the wait cannot choose differently
                            // (same argument as in the lane-group kernel): it is only counted
                            attempts++;
                            if (mine) {
#pragma unroll
                                for (int s = 0; s < kWideStrides; s++)
                                    if (s == (int)smin) {
                                        lane_advance<MAXGAP>(ins[s], now, false, envs[s], status);
                                        lane_admit<MAXGAP>(ins[s], q, req, prefill_us(ins[s].pre_base, ins[s].pre_q16, q.in_tokens),
                                                           now, envs[s], status);
                                    }
                            }
                            pending = false;
                        } else if (tries >= kAttemptCap) {
                            status = MAASO_CAND_ELOOP;
                            pending = false;
                        }
                    }
                }
                // a flag raised by one lane (a time beyond what the lane state can hold) ends the candidate for all
                if (__any_sync(kFullMaskW, status != 0u)) {
                    for (int o = 1; o < 32; o <<= 1) status |= __shfl_xor_sync(kFullMaskW, status, o);
                    pending = false;
                }
            } while (LOOP && pending);
        }

        // drain, account what is still queued, reduce over the warp, write the record
        __syncwarp();
#pragma unroll
        for (int s = 0; s < kWideStrides; s++) {
            wide_flush<MAXGAP>(ins[s].qn, ls, envs[s], sm.classes, (uint32_t)s * 32u + lane, P, oc);
            if (has[s] && status == 0) lane_advance<MAXGAP>(ins[s], 0, true, envs[s], status);
            wide_flush<MAXGAP>(ins[s].qn, ls, envs[s], sm.classes, (uint32_t)s * 32u + lane, P, oc);
        }
        Stats st = ls.st;
        uint32_t h[8];
        for (int i = 0; i < 8; i++) h[i] = ls.hbc[i];
        for (int off = 1; off < 32; off <<= 1) {
            for (int i = 0; i < 8; i++) h[i] += __shfl_xor_sync(kFullMaskW, h[i], off);
            status |= __shfl_xor_sync(kFullMaskW, status, off);
            st.served += __shfl_xor_sync(kFullMaskW, st.served, off);
            st.hit += __shfl_xor_sync(kFullMaskW, st.hit, off);
            st.sum_ttft += (int64_t)wshfl_xor_u64((uint64_t)st.sum_ttft, off);
            st.sum_e2e += (int64_t)wshfl_xor_u64((uint64_t)st.sum_e2e, off);
            st.tokens += wshfl_xor_u64(st.tokens, off);
            st.checksum += wshfl_xor_u64(st.checksum, off);
            st.max_ttft = max(st.max_ttft, (int64_t)wshfl_xor_u64((uint64_t)st.max_ttft, off));
            st.max_e2e = max(st.max_e2e, (int64_t)wshfl_xor_u64((uint64_t)st.max_e2e, off));
            st.makespan = max(st.makespan, (int64_t)wshfl_xor_u64((uint64_t)st.makespan, off));
        }
        if (lane == 0) {
            st.checksum += rej_sum;
            // worst-case mode: one round per counted request plus the counted second rounds
            write_result(P.out + oc, status, n_counted, n_rejected, LOOP ? attempts : attempts + n_counted, st, h);
        }
        __syncwarp();
    }
}

using WideKernel = void (*)(const EvalParams);
template <bool MAXGAP>
static WideKernel wide_kernel_of(uint32_t flags) {
    const bool opt = (flags & MAASO_FLAG_PRED_OPTIMISTIC) != 0;
    if (flags & MAASO_FLAG_INSTANCE_QUEUES)
        return opt ? eval_wide_kernel<true, QueueInst, MAXGAP> : eval_wide_kernel<false, QueueInst, MAXGAP>;
    if (flags & MAASO_FLAG_ENGINE_FROZEN)
        return opt ? eval_wide_kernel<true, FrozenInst, MAXGAP> : eval_wide_kernel<false, FrozenInst, MAXGAP>;
    return opt ? eval_wide_kernel<true, LaneInst, MAXGAP> : eval_wide_kernel<false, LaneInst, MAXGAP>;
}

cudaError_t launch_eval_wide(const EvalParams& P, int grid, cudaStream_t stream) {
    const bool maxgap = (P.flags & MAASO_FLAG_TBT_MAXGAP) != 0;
    auto kernel = maxgap ? wide_kernel_of<true>(P.flags) : wide_kernel_of<false>(P.flags);
    const size_t smem = wide_smem_bytes(P.n_rows, P.n_classes, maxgap);
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    kernel<<<grid, 32, smem, stream>>>(P);
    return cudaGetLastError();
}

int occupancy_eval_wide(const EvalParams& P) {
    const bool maxgap = (P.flags & MAASO_FLAG_TBT_MAXGAP) != 0;
    auto kernel = maxgap ? wide_kernel_of<true>(P.flags) : wide_kernel_of<false>(P.flags);
    const size_t smem = wide_smem_bytes(P.n_rows, P.n_classes, maxgap);
    cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    int n = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, kernel, 32, smem) != cudaSuccess) return 1;
    return n < 1 ? 1 : n;
}

// Global scratch one warp of the wide kernel needs: as much as a block of the lane-group kernel.
size_t wide_scratch_per_warp() { return (size_t)kGroupThreads * kLaneScratchBytes; }

}  // namespace maaso
