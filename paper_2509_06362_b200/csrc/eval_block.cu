// Scoring kernel, block mapping: one thread block per candidate placement, one warp per
// simulated instance (warps stride over the instances when there are more instances than
// warps), the 32 lanes of a warp hold the instance's virtual slots (two per lane, B <= 64).
// Next-completion search and completion accounting are warp-parallel over the slots; the
// distributor's argmin goes through shared memory (keys of all instances) and a warp
// reduction that every warp repeats, so one block barrier per attempt is enough.
#include "common.cuh"

namespace maaso {

constexpr int kBStages = 3;

template <int W> struct BlockCfg {
    static constexpr int kMaxInst = (W == 2) ? 2 : (W == 8 ? 8 : MAASO_MAX_INSTANCES);
    static constexpr int kSmemPay = (W == 2) ? 2 : (W == 8 ? 8 : 32);  // instances with payload in smem
    static constexpr int kThreads = W * 32;
};

struct InstMeta {
    uint32_t model, B, stepB, pre_base, pre_q16, row;
};

template <int W>
__host__ __device__ inline size_t block_smem_bytes(uint32_t n_rows, uint32_t n_classes, int tile_recs) {
    using C = BlockCfg<W>;
    size_t b = (size_t)kBStages * tile_recs * 16;          // tiles
    b += (size_t)C::kSmemPay * MAASO_WMAX * sizeof(Payload); // payload
    b += (size_t)n_classes * 24;                           // classes
    b += kBStages * 8;                                     // full barriers
    b += (size_t)C::kMaxInst * (8 + 8 + 8 + 8 + 8 + 8);     // T, mask, dk[2], dt0[2]
    b += (size_t)W * 9 * 8;                                // per-warp reduction scratch
    b += (size_t)n_rows * 64 * 4;                          // steps
    b += (size_t)C::kMaxInst * (4 + 4 + sizeof(InstMeta)); // K, w, meta
    b += (size_t)C::kMaxInst * MAASO_WMAX * 2;             // keys
    b += kBStages * 4 + 8 * 4 + 16;                        // empty counters, hit_by_class, work
    return (b + 15) & ~(size_t)15;
}

__device__ __forceinline__ uint64_t warp_min_u64(uint64_t v) {
    const uint32_t hi = (uint32_t)(v >> 32);
    const uint32_t mh = __reduce_min_sync(0xFFFFFFFFu, hi);
    const uint32_t lo = hi == mh ? (uint32_t)v : 0xFFFFFFFFu;
    const uint32_t ml = __reduce_min_sync(0xFFFFFFFFu, lo);
    return ((uint64_t)mh << 32) | ml;
}
__device__ __forceinline__ uint64_t warp_sum_u64(uint64_t v) {
    for (int off = 16; off > 0; off >>= 1) {
        const uint32_t lo = __shfl_xor_sync(0xFFFFFFFFu, (uint32_t)v, off);
        const uint32_t hi = __shfl_xor_sync(0xFFFFFFFFu, (uint32_t)(v >> 32), off);
        v += ((uint64_t)hi << 32) | lo;
    }
    return v;
}
__device__ __forceinline__ int64_t warp_max_i64(int64_t v) {
    for (int off = 16; off > 0; off >>= 1) {
        const uint32_t lo = __shfl_xor_sync(0xFFFFFFFFu, (uint32_t)v, off);
        const uint32_t hi = __shfl_xor_sync(0xFFFFFFFFu, (uint32_t)((uint64_t)v >> 32), off);
        v = max(v, (int64_t)(((uint64_t)hi << 32) | lo));
    }
    return v;
}

template <int W>
__global__ void __launch_bounds__(BlockCfg<W>::kThreads)
eval_block_kernel(const EvalParams P, const int tile_recs, const int bucket) {
    using C = BlockCfg<W>;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    unsigned char* base = smem_raw;
    uint4* const tiles = reinterpret_cast<uint4*>(base);        base += (size_t)kBStages * tile_recs * 16;
    Payload* const spay = reinterpret_cast<Payload*>(base);     base += (size_t)C::kSmemPay * MAASO_WMAX * sizeof(Payload);
    int64_t* const classes = reinterpret_cast<int64_t*>(base);  base += (size_t)P.n_classes * 24;
    uint64_t* const full_bar = reinterpret_cast<uint64_t*>(base); base += kBStages * 8;
    int64_t* const sT = reinterpret_cast<int64_t*>(base);       base += (size_t)C::kMaxInst * 8;
    uint64_t* const smask = reinterpret_cast<uint64_t*>(base);  base += (size_t)C::kMaxInst * 8;
    uint64_t* const dk = reinterpret_cast<uint64_t*>(base);     base += (size_t)C::kMaxInst * 16;
    int64_t* const dt0 = reinterpret_cast<int64_t*>(base);      base += (size_t)C::kMaxInst * 16;
    uint64_t* const red = reinterpret_cast<uint64_t*>(base);    base += (size_t)W * 9 * 8;
    int32_t* const steps = reinterpret_cast<int32_t*>(base);    base += (size_t)P.n_rows * 64 * 4;
    uint32_t* const sK = reinterpret_cast<uint32_t*>(base);     base += (size_t)C::kMaxInst * 4;
    uint32_t* const sw = reinterpret_cast<uint32_t*>(base);     base += (size_t)C::kMaxInst * 4;
    InstMeta* const meta = reinterpret_cast<InstMeta*>(base);   base += (size_t)C::kMaxInst * sizeof(InstMeta);
    uint16_t* const keys = reinterpret_cast<uint16_t*>(base);   base += (size_t)C::kMaxInst * MAASO_WMAX * 2;
    uint32_t* const empty_cnt = reinterpret_cast<uint32_t*>(base); base += kBStages * 4;
    uint32_t* const hbc = reinterpret_cast<uint32_t*>(base);    base += 8 * 4;
    uint32_t* const work = reinterpret_cast<uint32_t*>(base);

    const uint32_t tid = threadIdx.x, lane = tid & 31u, warp = tid >> 5;
    for (uint32_t i = tid; i < P.n_rows * 64u; i += C::kThreads)
        steps[i] = P.rows[(i >> 6) * kRowStride + 2 + (i & 63u)];
    for (uint32_t i = tid; i < P.n_classes * 3u; i += C::kThreads) classes[i] = P.classes[i];
    if (tid == 0) {
        for (int s = 0; s < kBStages; s++) { mbar_init(&full_bar[s], 1); empty_cnt[s] = 0; }
        work[1] = 0;
        fence_barrier_init();
    }
    __syncthreads();

    // running requests of instances beyond the shared-memory payload area live in global scratch
    Payload* const gpay = P.payload + (size_t)blockIdx.x * (MAASO_MAX_INSTANCES - C::kSmemPay) * MAASO_WMAX;
    const bool optimistic = (P.flags & MAASO_FLAG_PRED_OPTIMISTIC) != 0;
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
        const uint32_t n_i = P.offsets[cand + 1] - lo;
        for (uint32_t i = tid; i < n_i; i += C::kThreads) {
            const uint32_t word = P.inst[lo + i];
            InstMeta m;
            m.model = word & 0xFu;
            m.B = (word >> 12) & 0xFFu;
            m.row = m.model * P.n_strategies + ((word >> 4) & 0xFFu);
            m.stepB = (uint32_t)P.rows[m.row * kRowStride + 2 + m.B - 1];
            m.pre_base = (uint32_t)P.rows[m.row * kRowStride + 0];
            m.pre_q16 = (uint32_t)P.rows[m.row * kRowStride + 1];
            meta[i] = m;
            sT[i] = 0; sK[i] = 0; sw[i] = 0; smask[i] = 0;
        }
        if (tid < 8) hbc[tid] = 0;
        const uint32_t cmask = use_mask ? P.class_mask[cand] : 0xFFFFFFFFu;
        const Dump dump = dump_for(P, cand);
        Stats st; st.clear();
        int64_t now = 0;
        uint32_t n_counted = 0, n_rejected = 0, status = 0, buf = 0;
        uint64_t attempts = 0;
        if (tid == 0 && !P.stall_test) {
            for (uint32_t j = 0; j < (uint32_t)kBStages && j < n_tiles; j++) {
                const uint32_t s = (tile_seq + j) % kBStages;
                const uint32_t recs = min((uint32_t)tile_recs, P.n_req - j * tile_recs);
                mbar_expect_tx(&full_bar[s], recs * 16u);
                bulk_load(tiles + (size_t)s * tile_recs, P.reqs + (size_t)j * tile_recs, recs * 16u, &full_bar[s]);
            }
        }
        __syncthreads();

        // Advance instance i to `now` (drain: until empty); all 32 lanes cooperate, lane l
        // holds slots l and l+32.  Returns steps to the next completion (0x10000 if none).
        auto advance = [&](uint32_t i, int64_t t_now, bool drain) -> uint32_t {
            int64_t T = sT[i];
            uint32_t K = sK[i], w = sw[i];
            uint64_t mask = smask[i];
            const InstMeta m = meta[i];
            const uint16_t* krow = keys + i * MAASO_WMAX;
            const Payload* pay = i < (uint32_t)C::kSmemPay ? spay + i * MAASO_WMAX
                                                           : gpay + (size_t)(i - C::kSmemPay) * MAASO_WMAX;
            bool have0 = (mask >> lane) & 1ull, have1 = (mask >> (lane + 32)) & 1ull;
            const uint32_t key0 = krow[lane], key1 = krow[lane + 32];
            auto next_completion = [&]() -> uint32_t {
                const uint32_t d0 = have0 ? ((key0 - K) & 0xFFFFu) : 0x10000u;
                const uint32_t d1 = have1 ? ((key1 - K) & 0xFFFFu) : 0x10000u;
                return __reduce_min_sync(0xFFFFFFFFu, min(d0, d1));
            };
            uint32_t kfin = next_completion();
            bool changed = false;
            while (w > 0 && (drain || T < t_now)) {
                changed = true;
                const uint32_t s = (uint32_t)steps[m.row * 64u + w - 1];
                if (!drain && t_now - T <= (int64_t)(kfin - 1) * (int64_t)s) {
                    const uint32_t k = ceil_div_steps(t_now - T, s);
                    T += (int64_t)k * (int64_t)s;
                    K += k;
                    kfin -= k;
                    break;
                }
                T += (int64_t)kfin * (int64_t)s;
                K += kfin;
                const bool done0 = have0 && ((key0 - K) & 0xFFFFu) == 0;
                const bool done1 = have1 && ((key1 - K) & 0xFFFFu) == 0;
                if (done0 || done1) {
                    const Payload* p = pay + (done0 ? lane : lane + 32);
                    for (int rep = 0; rep < 2; rep++) {
                        if (rep == 0 ? done0 : done1) {
                            p = pay + (rep == 0 ? lane : lane + 32);
                            const uint4 a = reinterpret_cast<const uint4*>(p)[0];
                            const uint4 b = reinterpret_cast<const uint4*>(p)[1];
                            const int64_t first_tok = (int64_t)(((uint64_t)a.y << 32) | a.x);
                            const int64_t arrival = (int64_t)(((uint64_t)a.w << 32) | a.z);
                            const uint32_t cls = b.y >> 16;
                            if (account_completion(st, classes, i, b.x, arrival, first_tok, T, b.y & 0xFFFFu,
                                                   cls, dump))
                                atomicAdd(&hbc[cls < 7 ? cls : 7], 1u);
                        }
                    }
                }
                if (done0) have0 = false;
                if (done1) have1 = false;
                const uint32_t b0 = __ballot_sync(0xFFFFFFFFu, done0), b1 = __ballot_sync(0xFFFFFFFFu, done1);
                mask &= ~((uint64_t)b0 | ((uint64_t)b1 << 32));
                w -= __popc(b0) + __popc(b1);
                kfin = next_completion();
            }
            if (!drain && w == 0 && T < t_now) { T = t_now; changed = true; }
            if (changed && lane == 0) { sT[i] = T; sK[i] = K; sw[i] = w; smask[i] = mask; }
            __syncwarp();
            return kfin;
        };

        for (uint32_t t = 0; t < n_tiles; t++) {
            const uint32_t s = tile_seq % kBStages, parity = (tile_seq / kBStages) & 1u;
            bool ok = mbar_wait_bounded(&full_bar[s], parity, P.wait_cycles);
            if (!__all_sync(0xFFFFFFFFu, ok)) {
                mbar_wait_bounded(&full_bar[s], parity, P.wait_cycles);
                status = MAASO_CAND_ETIMEOUT;
                work[1] = 1;  // the block stops taking work
            }
            // a timeout anywhere in the block ends this candidate for every warp at the same tile
            if (__syncthreads_or(status != 0 && status != MAASO_CAND_ELOOP)) { status = MAASO_CAND_ETIMEOUT; break; }
            const uint4* tile = tiles + (size_t)s * tile_recs;
            const uint32_t recs = min((uint32_t)tile_recs, P.n_req - t * tile_recs);
            for (uint32_t ri = 0; ri < recs; ri++) {
                const Request q = decode_request(tile[ri]);
                const uint32_t req = t * tile_recs + ri;
                if (status != 0 || !((cmask >> (q.cls & 31u)) & 1u)) continue;  // uniform in the block
                n_counted++;
                now = max(now, q.arrival);
                const int64_t lim_ttft = classes[q.cls * 3 + 0];
                const int64_t lim_tbt = classes[q.cls * 3 + 1];
                const int64_t lim_e2e = classes[q.cls * 3 + 2];
                for (uint32_t tries = 1;; tries++) {
                    attempts++;
                    uint64_t* const dkb = dk + buf * C::kMaxInst;
                    int64_t* const dtb = dt0 + buf * C::kMaxInst;
                    for (uint32_t i = warp; i < n_i; i += W) {
                        const InstMeta m = meta[i];
                        uint64_t key = kKeyInf;
                        int64_t t0 = 0;
                        if (m.model == q.model) {
                            const uint32_t kfin = advance(i, now, false);
                            const int64_t T = sT[i];
                            const uint32_t w = sw[i];
                            const int64_t pre = prefill_us(m.pre_base, m.pre_q16, q.in_tokens);
                            uint64_t tier;
                            int64_t sB = (int64_t)m.stepB;
                            if (w < m.B) {
                                tier = 0; t0 = T;
                                if (optimistic) sB = (int64_t)steps[m.row * 64u + min(w + 1, m.B) - 1];
                            } else {
                                tier = 1; t0 = T + (int64_t)kfin * (int64_t)m.stepB;
                            }
                            const int64_t first = t0 + pre;
                            const int64_t fin = first + (int64_t)(q.S - 1) * sB;
                            const bool feas = (lim_ttft < 0 || first - q.arrival <= lim_ttft) &&
                                              (lim_tbt < 0 || q.S == 1 || sB <= lim_tbt) &&
                                              (lim_e2e < 0 || fin - q.arrival <= lim_e2e);
                            if (feas) key = (tier << 63) | (uint64_t)first;
                        }
                        if (lane == 0) { dkb[i] = key; dtb[i] = t0; }
                    }
                    __syncthreads();
                    // every warp finds the winner itself
                    uint64_t mine = kKeyInf;
                    for (uint32_t j = lane; j < n_i; j += 32) mine = min(mine, dkb[j]);
                    const uint64_t best = warp_min_u64(mine);
                    if (best == kKeyInf) {
                        if (tid == 0) {
                            n_rejected++;
                            st.checksum += rejected_hash(req);
                            if (P.rej_by_model)
                                atomicAdd(&P.rej_by_model[(size_t)cand * MAASO_MAX_MODELS + q.model], 1u);
                            if (dump.finish) dump.finish[req] = -1;
                            if (dump.first) dump.first[req] = -1;
                            if (dump.inst) dump.inst[req] = -1;
                        }
                        break;
                    }
                    uint32_t jm = 0xFFFFFFFFu;
                    for (uint32_t j = lane; j < n_i; j += 32)
                        if (dkb[j] == best) { jm = j; break; }
                    const uint32_t win = __reduce_min_sync(0xFFFFFFFFu, jm);  // lowest index wins ties
                    if ((best >> 63) == 0) {
                        if (win % W == warp) {
                            // "map": prefill at the boundary, then occupy the lowest free slot
                            const InstMeta m = meta[win];
                            if (lane == 0) {
                                const int64_t pre = prefill_us(m.pre_base, m.pre_q16, q.in_tokens);
                                const int64_t T = sT[win] + pre;
                                sT[win] = T;
                                if (q.S == 1) {
                                    if (account_completion(st, classes, win, req, q.arrival, T, T, 1, q.cls, dump))
                                        atomicAdd(&hbc[q.cls < 7 ? q.cls : 7], 1u);
                                } else {
                                    const uint64_t mask = smask[win];
                                    const int slot = __ffsll((long long)~mask) - 1;
                                    Payload* pay = win < (uint32_t)C::kSmemPay
                                                       ? spay + win * MAASO_WMAX
                                                       : gpay + (size_t)(win - C::kSmemPay) * MAASO_WMAX;
                                    keys[win * MAASO_WMAX + slot] = (uint16_t)((sK[win] + q.S - 1) & 0xFFFFu);
                                    store_payload(pay + slot, T, q.arrival, req, q.S, q.cls);
                                    smask[win] = mask | (1ull << slot);
                                    sw[win] = sw[win] + 1;
                                }
                            }
                            __syncwarp();
                        }
                        break;
                    }
                    now = dtb[win];  // wait until that slot frees
                    buf ^= 1u;
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
                    const uint32_t nt = t + kBStages;
                    if (nt < n_tiles) {
                        const uint32_t nrecs = min((uint32_t)tile_recs, P.n_req - nt * tile_recs);
                        fence_proxy_async();
                        mbar_expect_tx(&full_bar[s], nrecs * 16u);
                        bulk_load(tiles + (size_t)s * tile_recs, P.reqs + (size_t)nt * tile_recs, nrecs * 16u,
                                  &full_bar[s]);
                    }
                }
            }
            tile_seq++;
        }

        if (status == 0)
            for (uint32_t i = warp; i < n_i; i += W) advance(i, 0, true);
        // block reduction of the per-lane statistics
        const uint64_t r_served = warp_sum_u64(st.served), r_hit = warp_sum_u64(st.hit);
        const uint64_t r_sttft = warp_sum_u64((uint64_t)st.sum_ttft), r_se2e = warp_sum_u64((uint64_t)st.sum_e2e);
        const uint64_t r_tok = warp_sum_u64(st.tokens), r_chk = warp_sum_u64(st.checksum);
        const int64_t r_mttft = warp_max_i64(st.max_ttft), r_me2e = warp_max_i64(st.max_e2e);
        const int64_t r_mk = warp_max_i64(st.makespan);
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
static cudaError_t launch_one(const EvalParams& P, int grid, int tile_recs, int bucket, cudaStream_t stream) {
    const size_t smem = block_smem_bytes<W>(P.n_rows, P.n_classes, tile_recs);
    cudaError_t e = cudaFuncSetAttribute(eval_block_kernel<W>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    eval_block_kernel<W><<<grid, BlockCfg<W>::kThreads, smem, stream>>>(P, tile_recs, bucket);
    return cudaGetLastError();
}

template <int W>
static int occupancy_one(const EvalParams& P, int tile_recs) {
    const size_t smem = block_smem_bytes<W>(P.n_rows, P.n_classes, tile_recs);
    cudaFuncSetAttribute(eval_block_kernel<W>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    int n = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, eval_block_kernel<W>, BlockCfg<W>::kThreads, smem) !=
        cudaSuccess)
        return 1;
    return n < 1 ? 1 : n;
}

// the generic kernel: 16 warps striding over up to 128 instances (buckets with at most 8 instances
// use the register-resident kernel of eval_block_reg.cu)
cudaError_t launch_eval_block(const EvalParams& P, int bucket, int grid, int tile_recs, cudaStream_t stream) {
    return launch_one<16>(P, grid, tile_recs, bucket, stream);
}
int occupancy_eval_block(const EvalParams& P, int, int tile_recs) { return occupancy_one<16>(P, tile_recs); }
size_t block_payload_per_cta(int) {
    return (size_t)(MAASO_MAX_INSTANCES - BlockCfg<16>::kSmemPay) * MAASO_WMAX;  // Payload entries
}

}  // namespace maaso
