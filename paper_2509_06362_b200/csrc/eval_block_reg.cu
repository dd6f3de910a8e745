// Scoring kernel, block mapping for placements with at most W instances: one thread block per
// candidate, ONE WARP PER INSTANCE with the instance's state in that warp's registers (clock,
// step counter, level, cached next completion: warp-uniform) and its 64 virtual slots spread over
// the 32 lanes (two slot keys per lane, also in registers).  The next completion is one warp
// reduction, completions are accounted by the lanes that hold the finished slots, the
// distributor's keys meet in shared memory once per attempt (one block barrier, double-buffered)
// and every warp repeats the argmin.  Same lazy-clock and single-round rules as the lane-group
// kernel.  Placements with more instances than warps use the generic kernel in eval_block.cu.
#include "common.cuh"

namespace maaso {

constexpr int kRStages = 3;

__device__ __forceinline__ uint64_t rwarp_min_u64(uint64_t v) {
    const uint32_t hi = (uint32_t)(v >> 32);
    const uint32_t mh = __reduce_min_sync(0xFFFFFFFFu, hi);
    const uint32_t lo = hi == mh ? (uint32_t)v : 0xFFFFFFFFu;
    const uint32_t ml = __reduce_min_sync(0xFFFFFFFFu, lo);
    return ((uint64_t)mh << 32) | ml;
}
__device__ __forceinline__ uint64_t rwarp_sum_u64(uint64_t v) {
    for (int off = 16; off > 0; off >>= 1) {
        const uint32_t lo = __shfl_xor_sync(0xFFFFFFFFu, (uint32_t)v, off);
        const uint32_t hi = __shfl_xor_sync(0xFFFFFFFFu, (uint32_t)(v >> 32), off);
        v += ((uint64_t)hi << 32) | lo;
    }
    return v;
}
__device__ __forceinline__ int64_t rwarp_max_i64(int64_t v) {
    for (int off = 16; off > 0; off >>= 1) {
        const uint32_t lo = __shfl_xor_sync(0xFFFFFFFFu, (uint32_t)v, off);
        const uint32_t hi = __shfl_xor_sync(0xFFFFFFFFu, (uint32_t)((uint64_t)v >> 32), off);
        v = max(v, (int64_t)(((uint64_t)hi << 32) | lo));
    }
    return v;
}

template <int W>
__host__ __device__ inline size_t block_reg_smem_bytes(uint32_t n_rows, uint32_t n_classes, int tile_recs) {
    size_t b = (size_t)kRStages * tile_recs * 16;          // tiles
    b += (size_t)W * MAASO_WMAX * sizeof(Payload);         // payload of running requests
    b += (size_t)n_classes * 48;                           // class limits (accounting + prediction)
    b += kRStages * 8;                                     // full barriers
    b += (size_t)W * 32;                                   // distributor keys and start times, two buffers
    b += (size_t)W * 9 * 8;                                // per-warp reduction scratch
    b += (size_t)n_rows * 64 * 4;                          // decode-step tables
    b += kRStages * 4 + 8 * 4 + 16;                        // empty counters, hit-by-class, work slots
    return (b + 15) & ~(size_t)15;
}

// State of the warp's instance (identical in all 32 lanes) and the lane's two slot keys.
struct WarpInst {
    int64_t T, tc;
    uint64_t mask;
    uint32_t K, w, B, kfin, sw, stepB, pre_base, pre_q16, model;
    float rsw;
    const int32_t* step;
    uint32_t key0, key1;  // this lane's slots: lane and lane + 32
};

template <int W, bool OPT>
__global__ void __launch_bounds__(W * 32)
eval_block_reg_kernel(const EvalParams P, const int tile_recs, const int bucket) {
    constexpr int kThreads = W * 32;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    unsigned char* base = smem_raw;
    uint4* const tiles = reinterpret_cast<uint4*>(base);          base += (size_t)kRStages * tile_recs * 16;
    Payload* const spay = reinterpret_cast<Payload*>(base);       base += (size_t)W * MAASO_WMAX * sizeof(Payload);
    int64_t* const classes = reinterpret_cast<int64_t*>(base);    base += (size_t)P.n_classes * 24;
    int64_t* const plimits = reinterpret_cast<int64_t*>(base);    base += (size_t)P.n_classes * 24;
    uint64_t* const full_bar = reinterpret_cast<uint64_t*>(base); base += kRStages * 8;
    uint64_t* const dk = reinterpret_cast<uint64_t*>(base);       base += (size_t)W * 16;
    int64_t* const dt0 = reinterpret_cast<int64_t*>(base);        base += (size_t)W * 16;
    uint64_t* const red = reinterpret_cast<uint64_t*>(base);      base += (size_t)W * 9 * 8;
    int32_t* const steps = reinterpret_cast<int32_t*>(base);      base += (size_t)P.n_rows * 64 * 4;
    uint32_t* const empty_cnt = reinterpret_cast<uint32_t*>(base); base += kRStages * 4;
    uint32_t* const hbc = reinterpret_cast<uint32_t*>(base);      base += 8 * 4;
    uint32_t* const work = reinterpret_cast<uint32_t*>(base);

    const uint32_t tid = threadIdx.x, lane = tid & 31u, warp = tid >> 5;
    for (uint32_t i = tid; i < P.n_rows * 64u; i += kThreads) steps[i] = P.rows[(i >> 6) * kRowStride + 2 + (i & 63u)];
    for (uint32_t i = tid; i < P.n_classes * 3u; i += kThreads) {
        const int64_t v = P.classes[i];
        classes[i] = v;
        plimits[i] = v < 0 ? INT64_MAX : v;
    }
    if (tid == 0) {
        for (int s = 0; s < kRStages; s++) { mbar_init(&full_bar[s], 1); empty_cnt[s] = 0; }
        work[1] = 0;
        fence_barrier_init();
    }
    __syncthreads();

    Payload* const pay = spay + (size_t)warp * MAASO_WMAX;
    const bool use_mask = P.class_mask != nullptr && P.n_classes <= 32;
    const uint32_t n_tiles = (P.n_req + tile_recs - 1) / tile_recs;
    const uint32_t n_work = P.bucket_count[bucket];
    uint32_t tile_seq = 0;

    for (;;) {
        __syncthreads();
        if (tid == 0) work[0] = work[1] ? 0xFFFFFFFFu : atomicAdd(P.work_ctr + 1 + (bucket - 6), 1u);
        __syncthreads();
        const uint32_t wi = work[0];
        if (wi >= n_work) break;
        const uint32_t cand = P.bucket_list[(size_t)bucket * P.n_cand + wi];
        const uint32_t lo = P.offsets[cand];
        const uint32_t n_i = P.offsets[cand + 1] - lo;  // <= W
        const bool has = warp < n_i;
        WarpInst in;
        in.T = 0; in.tc = 0; in.mask = 0; in.K = 0; in.w = 0; in.B = 1; in.kfin = 0x10000u; in.sw = 1; in.rsw = 1.0f;
        in.stepB = 1; in.pre_base = 0; in.pre_q16 = 0; in.model = 0xFFFFFFFFu; in.step = steps; in.key0 = in.key1 = 0;
        if (has) {
            const uint32_t word = P.inst[lo + warp];
            in.model = word & 0xFu;
            in.B = (word >> 12) & 0xFFu;
            const uint32_t row = in.model * P.n_strategies + ((word >> 4) & 0xFFu);
            in.step = steps + row * 64u;
            in.stepB = (uint32_t)in.step[in.B - 1];
            in.pre_base = (uint32_t)P.rows[row * kRowStride + 0];
            in.pre_q16 = (uint32_t)P.rows[row * kRowStride + 1];
        }
        if (tid < 8) hbc[tid] = 0;
        const uint32_t cmask = use_mask ? P.class_mask[cand] : 0xFFFFFFFFu;
        const Dump dump = dump_for(P, cand);
        Stats st; st.clear();
        int64_t now = 0;
        uint32_t n_counted = 0, n_rejected = 0, status = 0, buf = 0;
        uint64_t attempts = 0, rej_sum = 0;
        if (tid == 0 && !P.stall_test) {
            for (uint32_t j = 0; j < (uint32_t)kRStages && j < n_tiles; j++) {
                const uint32_t s = (tile_seq + j) % kRStages;
                const uint32_t recs = min((uint32_t)tile_recs, P.n_req - j * tile_recs);
                mbar_expect_tx(&full_bar[s], recs * 16u);
                bulk_load(tiles + (size_t)s * tile_recs, P.reqs + (size_t)j * tile_recs, recs * 16u, &full_bar[s]);
            }
        }
        __syncthreads();

        // "reduce": run whole decode steps until the clock reaches t_now (drain: until empty); all 32
        // lanes take part, the state stays identical in all of them.
        auto advance = [&](int64_t t_now, bool drain) {
            while (in.w > 0 && (drain || in.T < t_now)) {
                if (!drain && t_now <= in.tc - (int64_t)in.sw) {
                    if (in.w < in.B) {  // a full instance keeps its clock until a slot frees
                        const uint32_t k = ceil_div_small(t_now - in.T, in.sw, in.rsw);
                        in.T += (int64_t)k * (int64_t)in.sw;
                        in.K += k;
                        in.kfin -= k;
                    }
                    break;
                }
                in.K += in.kfin;
                in.T = in.tc;
                const uint32_t K16 = in.K & 0xFFFFu;
                const bool have0 = (in.mask >> lane) & 1ull, have1 = (in.mask >> (lane + 32)) & 1ull;
                const uint32_t d0 = have0 ? ((in.key0 - K16) & 0xFFFFu) : 0x10000u;
                const uint32_t d1 = have1 ? ((in.key1 - K16) & 0xFFFFu) : 0x10000u;
                const bool done0 = d0 == 0, done1 = d1 == 0;
#pragma unroll 1
                for (int rep = 0; rep < 2; rep++) {
                    if (rep ? done1 : done0) {
                        const Payload* p = pay + lane + 32 * rep;
                        const uint4 a = reinterpret_cast<const uint4*>(p)[0];
                        const uint4 c = reinterpret_cast<const uint4*>(p)[1];
                        const int64_t first_tok = (int64_t)(((uint64_t)a.y << 32) | a.x);
                        const int64_t arrival = (int64_t)(((uint64_t)a.w << 32) | a.z);
                        const uint32_t cls = c.y >> 16;
                        if (account_completion(st, classes, warp, c.x, arrival, first_tok, in.T, c.y & 0xFFFFu, cls, dump))
                            atomicAdd(&hbc[cls < 7 ? cls : 7], 1u);
                    }
                }
                const uint32_t b0 = __ballot_sync(0xFFFFFFFFu, done0), b1 = __ballot_sync(0xFFFFFFFFu, done1);
                in.mask &= ~((uint64_t)b0 | ((uint64_t)b1 << 32));
                in.w -= __popc(b0) + __popc(b1);
                in.kfin = __reduce_min_sync(0xFFFFFFFFu, min(done0 ? 0x10000u : d0, done1 ? 0x10000u : d1));
                if (in.w > 0) {
                    in.sw = (uint32_t)in.step[in.w - 1];
                    in.rsw = __frcp_rn((float)in.sw);
                    in.tc = in.T + (int64_t)in.kfin * (int64_t)in.sw;
                }
            }
            if (!drain && in.w == 0 && in.T < t_now) in.T = t_now;
        };
        // "map": prefill at the boundary, then the request takes the lowest free slot
        auto admit = [&](const Request& q, uint32_t req, int64_t pre) {
            in.T += pre;
            if (q.S == 1) {
                in.tc += pre;
                if (lane == 0 && account_completion(st, classes, warp, req, q.arrival, in.T, in.T, 1, q.cls, dump))
                    atomicAdd(&hbc[q.cls < 7 ? q.cls : 7], 1u);
                return;
            }
            const int slot = __ffsll((long long)~in.mask) - 1;
            const uint32_t key = (in.K + q.S - 1) & 0xFFFFu;
            if ((int)lane == (slot & 31)) {
                if (slot < 32) in.key0 = key; else in.key1 = key;
                store_payload(pay + slot, in.T, q.arrival, req, q.S, q.cls);
            }
            const uint32_t dist = q.S - 1;
            if (in.w == 0 || dist < in.kfin) in.kfin = dist;
            in.mask |= 1ull << slot;
            in.w++;
            in.sw = (uint32_t)in.step[in.w - 1];
            in.rsw = __frcp_rn((float)in.sw);
            in.tc = in.T + (int64_t)in.kfin * (int64_t)in.sw;
            __syncwarp();
        };

        for (uint32_t t = 0; t < n_tiles; t++) {
            const uint32_t s = tile_seq % kRStages, parity = (tile_seq / kRStages) & 1u;
            const bool ok = mbar_wait_bounded(&full_bar[s], parity, P.wait_cycles);
            if (!__all_sync(0xFFFFFFFFu, ok)) {
                mbar_wait_bounded(&full_bar[s], parity, P.wait_cycles);
                status = MAASO_CAND_ETIMEOUT;
                work[1] = 1;  // the block stops taking work
            }
            if (__syncthreads_or(status != 0 && status != MAASO_CAND_ELOOP)) { status = MAASO_CAND_ETIMEOUT; break; }
            const uint4* tile = tiles + (size_t)s * tile_recs;
            const uint32_t recs = min((uint32_t)tile_recs, P.n_req - t * tile_recs);
            for (uint32_t ri = 0; ri < recs; ri++) {
                const Request q = decode_request(tile[ri]);
                const uint32_t req = t * tile_recs + ri;
                if (status != 0 || !((cmask >> (q.cls & 31u)) & 1u)) continue;  // uniform in the block
                n_counted++;
                now = max(now, q.arrival);
                const int64_t lim_ttft = plimits[q.cls * 3 + 0];
                const int64_t lim_tbt = plimits[q.cls * 3 + 1];
                const int64_t lim_e2e = plimits[q.cls * 3 + 2];
                const int64_t pre = prefill_us(in.pre_base, in.pre_q16, q.in_tokens);
                const bool elig = has && in.model == q.model;
                for (uint32_t tries = 1;; tries++) {
                    attempts++;
                    uint64_t key = kKeyInf;
                    int64_t t0 = 0;
                    if (elig) {
                        advance(now, false);
                        uint64_t tier;
                        int64_t sB = (int64_t)in.stepB;  // worst case F(M,P,B_I)
                        if (in.w < in.B) {
                            tier = 0; t0 = in.T;
                            if (OPT) sB = (int64_t)in.step[min(in.w + 1, in.B) - 1];
                        } else {
                            tier = 1; t0 = in.tc;
                        }
                        const int64_t first = t0 + pre;
                        const int64_t fin = first + (int64_t)(q.S - 1) * sB;
                        if (first - q.arrival <= lim_ttft && (q.S == 1 || sB <= lim_tbt) && fin - q.arrival <= lim_e2e)
                            key = (tier << 63) | (uint64_t)first;
                    }
                    if (lane == 0) { dk[buf * W + warp] = key; dt0[buf * W + warp] = t0; }
                    __syncthreads();
                    // every warp finds the winner itself: lowest instance among the smallest keys
                    const uint64_t mine = lane < (uint32_t)W ? dk[buf * W + lane] : kKeyInf;
                    const uint64_t best = rwarp_min_u64(mine);
                    if (best == kKeyInf) {  // overflow protection: nobody can meet the deadline
                        if (tid == 0) {
                            n_rejected++;
                            rej_sum += __ldg(P.rej_hash + req);
                            if (P.rej_by_model) atomicAdd(&P.rej_by_model[(size_t)cand * MAASO_MAX_MODELS + q.model], 1u);
                            if (dump.finish) dump.finish[req] = -1;
                            if (dump.first) dump.first[req] = -1;
                            if (dump.inst) dump.inst[req] = -1;
                        }
                        break;
                    }
                    const uint32_t win = __reduce_min_sync(0xFFFFFFFFu, mine == best ? lane : 0xFFFFFFFFu);
                    if ((best >> 63) == 0) {
                        if (warp == win) admit(q, req, pre);
                        break;
                    }
                    now = dt0[buf * W + win];  // every capable instance is full: wait for the winner's slot
                    if (!OPT) {
                        // under the worst-case estimate the next round cannot choose differently: it is
                        // only counted, the winner runs to that time and admits, other clocks catch up later
                        attempts++;
                        if (warp == win) { advance(now, false); admit(q, req, pre); }
                        break;
                    }
                    buf ^= 1u;  // the next attempt writes the other key buffer
                    if (tries >= kAttemptCap) { status = MAASO_CAND_ELOOP; break; }
                }
                buf ^= 1u;
            }
            __syncwarp();
            if (lane == 0) {
                __threadfence_block();
                const uint32_t old = atomicAdd(&empty_cnt[s], 1u);
                if (old == W - 1) {
                    empty_cnt[s] = 0;
                    const uint32_t nt = t + kRStages;
                    if (nt < n_tiles) {
                        const uint32_t nrecs = min((uint32_t)tile_recs, P.n_req - nt * tile_recs);
                        fence_proxy_async();
                        mbar_expect_tx(&full_bar[s], nrecs * 16u);
                        bulk_load(tiles + (size_t)s * tile_recs, P.reqs + (size_t)nt * tile_recs, nrecs * 16u, &full_bar[s]);
                    }
                }
            }
            tile_seq++;
        }

        if (status == 0 && has) advance(0, true);
        if (tid == 0) st.checksum += rej_sum;
        const uint64_t r_served = rwarp_sum_u64(st.served), r_hit = rwarp_sum_u64(st.hit);
        const uint64_t r_sttft = rwarp_sum_u64((uint64_t)st.sum_ttft), r_se2e = rwarp_sum_u64((uint64_t)st.sum_e2e);
        const uint64_t r_tok = rwarp_sum_u64(st.tokens), r_chk = rwarp_sum_u64(st.checksum);
        const int64_t r_mttft = rwarp_max_i64(st.max_ttft), r_me2e = rwarp_max_i64(st.max_e2e);
        const int64_t r_mk = rwarp_max_i64(st.makespan);
        if (lane == 0) {
            uint64_t* r = red + warp * 9;
            r[0] = r_served; r[1] = r_hit; r[2] = r_sttft; r[3] = r_se2e; r[4] = r_tok; r[5] = r_chk;
            r[6] = (uint64_t)r_mttft; r[7] = (uint64_t)r_me2e; r[8] = (uint64_t)r_mk;
        }
        __syncthreads();
        if (tid == 0) {
            Stats tot; tot.clear();
            for (int x = 0; x < W; x++) {
                const uint64_t* r = red + x * 9;
                tot.served += (uint32_t)r[0]; tot.hit += (uint32_t)r[1];
                tot.sum_ttft += (int64_t)r[2]; tot.sum_e2e += (int64_t)r[3];
                tot.tokens += r[4]; tot.checksum += r[5];
                tot.max_ttft = max(tot.max_ttft, (int64_t)r[6]);
                tot.max_e2e = max(tot.max_e2e, (int64_t)r[7]);
                tot.makespan = max(tot.makespan, (int64_t)r[8]);
            }
            uint32_t h[8];
            for (int x = 0; x < 8; x++) h[x] = hbc[x];
            write_result(P.out + cand, status, n_counted, n_rejected, attempts, tot, h);
        }
    }
}

template <int W>
static cudaError_t launch_reg(const EvalParams& P, int grid, int tile_recs, int bucket, cudaStream_t stream) {
    const size_t smem = block_reg_smem_bytes<W>(P.n_rows, P.n_classes, tile_recs);
    const bool opt = (P.flags & MAASO_FLAG_PRED_OPTIMISTIC) != 0;
    auto kernel = opt ? eval_block_reg_kernel<W, true> : eval_block_reg_kernel<W, false>;
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    kernel<<<grid, W * 32, smem, stream>>>(P, tile_recs, bucket);
    return cudaGetLastError();
}
template <int W>
static int occupancy_reg(const EvalParams& P, int tile_recs) {
    const size_t smem = block_reg_smem_bytes<W>(P.n_rows, P.n_classes, tile_recs);
    const bool opt = (P.flags & MAASO_FLAG_PRED_OPTIMISTIC) != 0;
    auto kernel = opt ? eval_block_reg_kernel<W, true> : eval_block_reg_kernel<W, false>;
    cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    int n = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, kernel, W * 32, smem) != cudaSuccess) return 1;
    return n < 1 ? 1 : n;
}

// bucket 6: <= 2 instances (2 warps), 7: <= 4 (4 warps), 8: <= 8 (8 warps)
cudaError_t launch_eval_block_reg(const EvalParams& P, int bucket, int grid, int tile_recs, cudaStream_t stream) {
    if (bucket == 6) return launch_reg<2>(P, grid, tile_recs, bucket, stream);
    if (bucket == 7) return launch_reg<4>(P, grid, tile_recs, bucket, stream);
    return launch_reg<8>(P, grid, tile_recs, bucket, stream);
}
int occupancy_eval_block_reg(const EvalParams& P, int bucket, int tile_recs) {
    if (bucket == 6) return occupancy_reg<2>(P, tile_recs);
    if (bucket == 7) return occupancy_reg<4>(P, tile_recs);
    return occupancy_reg<8>(P, tile_recs);
}

}  // namespace maaso
