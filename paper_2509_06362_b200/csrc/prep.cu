// Candidate decode + validation (constraints (c) and (d) of Sec. IV-C, table ranges) and
// sorting of valid candidates into launch buckets; helpers for the per-request dump buffers.
#include "common.cuh"

namespace maaso {

// Where a valid candidate can be scored.  `code` = its bucket among the lane-group / block buckets
// (0..9) and its cost bin, `code2` = its bucket among the thread-mapping buckets (10..18) and the
// bin; 0xFFFFFFFF = it has no such place.  A candidate with both is placed by the batch-wide choice
// plan_kernel makes (MAASO_MAP_AUTO).
__global__ void prep_kernel(const EvalParams P) {
    const uint32_t c = blockIdx.x * blockDim.x + threadIdx.x;
    if (c >= P.n_cand) return;
    const uint32_t lo = P.offsets[c], hi = P.offsets[c + 1];
    uint32_t status = 0, n = 0, sum_b = 0;
    uint32_t units = 0;  // thread mapping: 16-byte units of cold instance state (per instance 2 + key blocks + minima)
    uint64_t supply = 0; // decode tokens per second the placement can produce with every slot busy
    const bool variant = (P.flags & (MAASO_FLAG_ENGINE_FROZEN | MAASO_FLAG_TBT_MAXGAP | MAASO_FLAG_INSTANCE_QUEUES)) != 0;
    const bool threads_ok = !variant && (P.mapping == MAASO_MAP_THREAD || P.mapping == MAASO_MAP_AUTO);
    const bool groups_ok = P.mapping != MAASO_MAP_THREAD;
    if (hi < lo || hi > P.n_inst) {
        status = MAASO_CAND_EBADINST;  // malformed CSR row
    } else {
        n = hi - lo;
        if (n > MAASO_MAX_INSTANCES) {
            status = MAASO_CAND_ETOOMANY;
        } else {
            uint64_t devsum = 0;
            for (uint32_t i = 0; i < n; i++) {
                const uint32_t word = P.inst[lo + i];
                const uint32_t m = word & 0xFu, s = (word >> 4) & 0xFFu, b = (word >> 12) & 0xFFu;
                if ((word >> 20) != 0 || m >= P.n_models || s >= P.n_strategies || b < 1 || b > MAASO_WMAX) {
                    status |= MAASO_CAND_EBADINST;
                    continue;
                }
                sum_b += b;
                units += 2u + 2u * ((b + 7u) >> 3) + 2u;
                supply += (uint64_t)b * 1000000ull / (uint64_t)P.rows[(m * P.n_strategies + s) * kRowStride + 1 + b];
                devsum += (uint64_t)P.devices[s];
                if (P.devices[s] < P.min_devices[m]) status |= MAASO_CAND_EMEMFIT;
            }
            if (devsum > P.budget) status |= MAASO_CAND_EBUDGET;
        }
    }
    // where it can go
    int bg = -1, bt = -1;
    if (!status) {
        if (threads_ok) {
            // as many lanes per item as placements of this size fit the warp's pools
            const uint32_t fit = n ? min(P.thread_pool_units / units, P.thread_hot_units / (2u * n)) : 32u;
            const uint32_t lanes[9] = {32, 24, 16, 12, 8, 6, 4, 2, 1};
            for (int i = 0; i < 9; i++)
                if (fit >= lanes[i]) { bt = kThreadBucket0 + i; break; }
        }
        if (P.mapping == MAASO_MAP_BLOCK) bg = n <= 2 ? 6 : (n <= 4 ? 7 : (n <= 8 ? 8 : kGenericBlockBucket));
        else if (groups_ok && n <= 32) bg = n <= 1 ? 0 : 32 - __clz((int)(n - 1));
        // More than 32 instances: one warp per placement with the lane-group code (every engine), or the thread
        // mapping where that exists and can hold the placement; the batch-wide choice of plan_kernel decides
        // between the two.  (One block per placement only when the block mapping is asked for.)
        if (bg < 0 && (groups_ok || bt < 0)) bg = kWideBucket;
    }
    if (P.dump_row) P.dump_row[c] = -1;
    const uint32_t n_traces = P.n_traces > 1 ? P.n_traces : 1u;
    for (uint32_t t = 0; t < n_traces; t++) {
        const size_t oc = (size_t)t * P.n_cand + c;  // the candidate's record in trace t's block
        if (P.rej_by_model)
            for (int m = 0; m < MAASO_MAX_MODELS; m++) P.rej_by_model[oc * MAASO_MAX_MODELS + m] = 0;
        // Invalid candidates get their final record here.  Valid ones are pre-marked "not scored"
        // (ETIMEOUT); the scoring kernel overwrites the record when it finishes the candidate, so a
        // kernel that gave up on a bounded wait leaves no record undefined.
        uint4* o = reinterpret_cast<uint4*>(P.out + oc);
        o[0] = make_uint4(status ? status : MAASO_CAND_ETIMEOUT, 0, 0, 0);
        for (int i = 1; i < 8; i++) o[i] = make_uint4(0, 0, 0, 0);
    }
    if (status) {
        P.code[c] = 0xFFFFFFFFu;
        P.code2[c] = 0xFFFFFFFFu;
        return;
    }
    // Cost estimate: the total batch cap (how many requests the placement can have in flight;
    // it tracks the number of served requests and so the number of simulation events).
    const uint32_t bin = (kCostBins - 1) - min((uint32_t)(kCostBins - 1), sum_b / 8u);
    P.code[c] = bg >= 0 ? (((uint32_t)bg << 8) | bin) : 0xFFFFFFFFu;
    P.code2[c] = bt >= 0 ? (((uint32_t)bt << 8) | bin) : 0xFFFFFFFFu;
    if (bg >= 0 && bt >= 0) {
        atomicAdd(&P.hist[(bg == kWideBucket ? kHistBothW : kHistBothG + bg) * kCostBins + bin], 1u);
        atomicAdd(&P.hist[(kHistBothT + bt - kThreadBucket0) * kCostBins + bin], 1u);
        // loaded beyond what it can decode: most of its requests will be turned away, which the
        // thread mapping does for next to nothing
        atomicAdd(&P.bucket_count[kCtrBoth], 1u);
        if ((uint64_t)P.demand_tok_s >= 2ull * supply) atomicAdd(&P.bucket_count[kCtrLoaded], 1u);
    } else if (bg == kWideBucket) {
        atomicAdd(&P.hist[kHistWide * kCostBins + bin], 1u);
    } else if (bg >= 0) {
        atomicAdd(&P.hist[(kHistOnlyG + bg) * kCostBins + bin], 1u);
    } else {
        atomicAdd(&P.hist[(kHistOnlyT + bt - kThreadBucket0) * kCostBins + bin], 1u);
    }
}

// One block, one thread per cost bin: (0) the batch-wide choice between lane groups and threads for
// the candidates that can go either way (MAASO_MAP_AUTO): threads if most of them are loaded beyond
// their decode capacity and there are enough of them to fill the GPU one placement per lane; (1) if the
// resident lane-group grid has warps to spare, promote the most expensive candidates of the narrower
// lane-group buckets to a warp of their own (bucket 5) so that their event handling is not
// serialised with other candidates' in the same warp; (2) turn the per-bin histograms into write
// cursors (bins in decreasing cost order).
__device__ __forceinline__ uint32_t block_inclusive_scan(uint32_t v, uint32_t* buf) {
    const int t = threadIdx.x;
    buf[t] = v;
    __syncthreads();
    for (int off = 1; off < kCostBins; off <<= 1) {
        const uint32_t add = t >= off ? buf[t - off] : 0u;
        __syncthreads();
        buf[t] += add;
        __syncthreads();
    }
    const uint32_t r = buf[t];
    __syncthreads();
    return r;
}

__global__ void __launch_bounds__(kCostBins) plan_kernel(const EvalParams P) {
    __shared__ uint32_t buf[kCostBins];
    __shared__ uint32_t tot[6];
    const int bin = threadIdx.x;
    const uint32_t n_both = P.bucket_count[kCtrBoth], n_loaded = P.bucket_count[kCtrLoaded];
    const bool use_threads = n_loaded >= P.thread_min_cand && 2u * n_loaded >= n_both;
    // final counts of this bin per bucket
    uint32_t cnt[kNumBuckets];
    for (int b = 0; b < kThreadBucket0; b++)
        cnt[b] = P.hist[(kHistOnlyG + b) * kCostBins + bin] + (use_threads ? 0u : P.hist[(kHistBothG + b) * kCostBins + bin]);
    for (int b = kThreadBucket0; b < kThreadBucket0 + kThreadBuckets; b++)
        cnt[b] = P.hist[(kHistOnlyT + b - kThreadBucket0) * kCostBins + bin] +
                 (use_threads ? P.hist[(kHistBothT + b - kThreadBucket0) * kCostBins + bin] : 0u);
    cnt[kWideBucket] = P.hist[kHistWide * kCostBins + bin] + (use_threads ? 0u : P.hist[kHistBothW * kCostBins + bin]);
    uint32_t cut = 0;  // bins below `cut` are promoted
    uint32_t narrow = 0;
    for (int b = 0; b < 5; b++) narrow += cnt[b];
    if (P.mapping != MAASO_MAP_BLOCK && P.mapping != MAASO_MAP_THREAD) {
        // warps the lane-group buckets need: bucket totals = sums over the bins
        uint32_t need = 0;
        for (int b = 0; b <= 5; b++) {
            const uint32_t incl = block_inclusive_scan(cnt[b], buf);
            if (bin == kCostBins - 1) tot[b] = incl;
        }
        __syncthreads();
        for (int b = 0; b <= 5; b++) need += (tot[b] + (32u >> b) - 1) / (32u >> b);
        // every work item exists once per trace, and a promoted candidate takes a warp in each of them
        const uint32_t n_tr = P.n_traces > 1 ? P.n_traces : 1u;
        const uint64_t need_all = (uint64_t)need * n_tr;
        const uint32_t spare = P.group_warps > need_all
                                   ? (uint32_t)((P.group_warps - need_all) / n_tr * P.promote_pct / 100) : 0;
        const uint32_t incl = block_inclusive_scan(narrow, buf);
        cut = (uint32_t)__syncthreads_count(incl <= spare);  // prefix sums are monotone
    }
    __syncthreads();
    for (int b = 0; b < kNumBuckets; b++) {
        uint32_t v = cnt[b];
        if (b < 5 && (uint32_t)bin < cut) v = 0;
        if (b == 5 && (uint32_t)bin < cut) v += narrow;
        const uint32_t incl = block_inclusive_scan(v, buf);
        P.hist[(kHistCursor + b) * kCostBins + bin] = incl - v;
        if (bin == kCostBins - 1) P.bucket_count[b] = incl;
    }
    if (bin == 0) {
        P.bucket_count[kCtrCut] = cut;
        P.bucket_count[kCtrUseThreads] = use_threads ? 1u : 0u;
    }
}

__global__ void scatter_kernel(const EvalParams P) {
    const uint32_t c = blockIdx.x * blockDim.x + threadIdx.x;
    if (c >= P.n_cand) return;
    const uint32_t cg = P.code[c], ct = P.code2[c];
    if (cg == 0xFFFFFFFFu && ct == 0xFFFFFFFFu) return;
    const uint32_t code = (cg != 0xFFFFFFFFu && ct != 0xFFFFFFFFu) ? (P.bucket_count[kCtrUseThreads] ? ct : cg)
                                                                    : (cg != 0xFFFFFFFFu ? cg : ct);
    uint32_t b = code >> 8;
    const uint32_t bin = code & 0xFFu;
    if (b < 5 && bin < P.bucket_count[kCtrCut]) b = 5;
    const uint32_t pos = atomicAdd(&P.hist[(kHistCursor + b) * kCostBins + bin], 1u);
    P.bucket_list[(size_t)b * P.n_cand + pos] = c;
}

__global__ void dump_map_kernel(const EvalParams P, const uint32_t* dump_idx) {
    const uint32_t d = blockIdx.x * blockDim.x + threadIdx.x;
    if (d >= P.dump_n) return;
    const uint32_t c = dump_idx[d];
    if (c < P.n_cand) P.dump_row[c] = (int32_t)d;
}

__global__ void dump_fill_kernel(int64_t* finish, int64_t* first, int32_t* inst, size_t n) {
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
        if (finish) finish[i] = -2;
        if (first) first[i] = -2;
        if (inst) inst[i] = -2;
    }
}

// The checksum term of a rejected request depends on the request alone: computed once per trace.
__global__ void rej_hash_kernel(uint64_t* out, uint32_t n) {
    const uint32_t r = blockIdx.x * blockDim.x + threadIdx.x;
    if (r < n) out[r] = rejected_hash(r);
}
// Prepared trace records for the lane-group kernel (layout: common.cuh).
__global__ void cook_trace_kernel(const uint4* reqs, const int64_t* classes, uint4* out, uint32_t n) {
    const uint32_t r = blockIdx.x * blockDim.x + threadIdx.x;
    if (r >= n) return;
    const Request q = decode_request(reqs[r]);
    const int64_t l_ttft = classes[q.cls * 3 + 0], l_tbt = classes[q.cls * 3 + 1], l_e2e = classes[q.cls * 3 + 2];
    const int64_t dl_ttft = l_ttft < 0 ? INT64_MAX : q.arrival + l_ttft;
    const int64_t dl_e2e = l_e2e < 0 ? INT64_MAX : q.arrival + l_e2e;
    const uint32_t tbt32 = (l_tbt < 0 || l_tbt > 0xFFFFFFFFll) ? 0xFFFFFFFFu : (uint32_t)l_tbt;
    const uint64_t h = rejected_hash(r);
    auto lo = [](uint64_t v) { return (uint32_t)v; };
    auto hi = [](uint64_t v) { return (uint32_t)(v >> 32); };
    uint4* o = out + (size_t)r * kCookedWords;
    o[0] = make_uint4(lo((uint64_t)q.arrival), hi((uint64_t)q.arrival), lo((uint64_t)dl_ttft), hi((uint64_t)dl_ttft));
    o[1] = make_uint4(lo((uint64_t)dl_e2e), hi((uint64_t)dl_e2e), q.in_tokens, tbt32);
    o[2] = make_uint4(lo(h), hi(h), (q.S - 1u) | (q.cls << 16) | (q.model << 24), 0u);
}

// Scan tiles of the thread mapping.  Tile t (kScanTile requests) is a header followed by one
// 16-byte record per request.
//   record: {arrival - the tile's base arrival (all ones: does not fit 32 bits, look at the full record),
//            TTFT limit, end-to-end limit (each clamped to 32 bits; all ones = none, or too large to
//            matter here), model | cls << 8 | (output tokens - 1) << 16}.  Once the dispatcher's clock has
//            passed arrival + limit, no instance can serve the request in time.
//   header units 0..3: eight int64, entry k (classes 7 and up share entry 7) = the largest arrival +
//            min(TTFT, end-to-end limit) over the tile's requests of that class: INT64_MAX if one of
//            them has no limit, INT64_MIN if the tile has none, so "clock beyond the entries of the
//            classes I count" means the whole tile is late;
//   unit 4: base arrival (int64) = arrival of the tile's first request;
//   units 5..20: per class slot a 256-bit map of the tile's requests of that class;
//   units 21..36: the same per model (models 7 and up share slot 7).
__global__ void scan_trace_kernel(const uint4* reqs, const int64_t* classes, uint4* scan, uint32_t n) {
    const uint32_t tile = blockIdx.x, t = threadIdx.x;  // kScanTile threads
    __shared__ int64_t thr[8];
    if (t < 8) thr[t] = INT64_MIN;
    __syncthreads();
    const uint32_t r = tile * kScanTile + t;
    uint4* const base = scan + (size_t)tile * (kScanTile + kScanHdrUnits);
    const int64_t base_arrival = decode_request(reqs[tile * kScanTile]).arrival;
    uint32_t cslot = 0xFFu, mslot = 0xFFu;
    if (r < n) {
        const Request q = decode_request(reqs[r]);
        const int64_t l_ttft = classes[q.cls * 3 + 0], l_e2e = classes[q.cls * 3 + 2];
        const uint32_t t32 = (l_ttft < 0 || l_ttft >= 0xFFFFFFFFll) ? 0xFFFFFFFFu : (uint32_t)l_ttft;
        const uint32_t e32 = (l_e2e < 0 || l_e2e >= 0xFFFFFFFFll) ? 0xFFFFFFFFu : (uint32_t)l_e2e;
        const int64_t rel = q.arrival - base_arrival;
        const uint32_t rel32 = rel >= 0xFFFFFFFFll ? 0xFFFFFFFFu : (uint32_t)rel;
        base[kScanHdrUnits + t] = make_uint4(rel32, t32, e32, q.model | (q.cls << 8) | ((q.S - 1u) << 16));
        const uint32_t lim32 = min(t32, e32);
        const int64_t v = lim32 == 0xFFFFFFFFu ? INT64_MAX : q.arrival + (int64_t)lim32;
        cslot = q.cls < 7 ? q.cls : 7;
        mslot = q.model < 7 ? q.model : 7;
        atomicMax(reinterpret_cast<long long*>(&thr[cslot]), (long long)v);
    }
    uint32_t* const words = reinterpret_cast<uint32_t*>(base);
    for (uint32_t k = 0; k < 8; k++) {
        const uint32_t cb = __ballot_sync(0xFFFFFFFFu, cslot == k), mb = __ballot_sync(0xFFFFFFFFu, mslot == k);
        if ((t & 31u) == 0) {
            words[(kScanHdrClassBits + 2 * k) * 4 + (t >> 5)] = cb;
            words[(kScanHdrModelBits + 2 * k) * 4 + (t >> 5)] = mb;
        }
    }
    __syncthreads();
    if (t < 4) {
        const uint64_t a = (uint64_t)thr[2 * t], b = (uint64_t)thr[2 * t + 1];
        base[t] = make_uint4((uint32_t)a, (uint32_t)(a >> 32), (uint32_t)b, (uint32_t)(b >> 32));
    }
    if (t == 4) base[kScanHdrBase] = make_uint4((uint32_t)base_arrival, (uint32_t)((uint64_t)base_arrival >> 32), 0u, 0u);
    if (t >= 5 && t < 8) base[kScanHdrUnits - 3 + (t - 5)] = make_uint4(0u, 0u, 0u, 0u);  // padding units 37..39
}
size_t scan_trace_units(uint32_t n) {
    const size_t tiles = ((size_t)n + kScanTile - 1) / kScanTile;
    return (tiles ? tiles : 1) * (kScanTile + kScanHdrUnits);
}
cudaError_t launch_scan_trace(const uint4* reqs, const int64_t* classes, uint4* scan, uint32_t n) {
    if (n) scan_trace_kernel<<<(n + kScanTile - 1) / kScanTile, kScanTile>>>(reqs, classes, scan, n);
    return cudaGetLastError();
}
cudaError_t launch_cook_trace(const uint4* reqs, const int64_t* classes, uint4* out, uint32_t n) {
    if (n) cook_trace_kernel<<<(n + 255) / 256, 256>>>(reqs, classes, out, n);
    return cudaGetLastError();
}

cudaError_t launch_rej_hash(uint64_t* out, uint32_t n) {
    if (n) rej_hash_kernel<<<(n + 255) / 256, 256>>>(out, n);
    return cudaGetLastError();
}

cudaError_t launch_prep(const EvalParams& P, const uint32_t* dump_idx, cudaStream_t stream, int* launches) {
    if (P.dump_n) {
        const size_t n = (size_t)P.dump_n * P.n_req;
        if (n) {
            dump_fill_kernel<<<(unsigned)min((size_t)4096, (n + 255) / 256), 256, 0, stream>>>(
                P.dump_finish, P.dump_first, P.dump_inst, n);
            (*launches)++;
        }
    }
    prep_kernel<<<(P.n_cand + 255) / 256, 256, 0, stream>>>(P);
    plan_kernel<<<1, kCostBins, 0, stream>>>(P);
    scatter_kernel<<<(P.n_cand + 255) / 256, 256, 0, stream>>>(P);
    (*launches) += 3;
    if (P.dump_n) {
        dump_map_kernel<<<(P.dump_n + 255) / 256, 256, 0, stream>>>(P, dump_idx);
        (*launches)++;
    }
    return cudaGetLastError();
}

}  // namespace maaso
