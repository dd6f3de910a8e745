// Scoring kernel, thread mapping: ONE THREAD replays one candidate and walks over the instances
// that can serve the request's model; the 32 candidates of a warp share the staged trace.
//
// Why: a request concerns only the instances of its model, and under load most instances are
// full and far from their next completion, so the work per (candidate, request) is a few
// loads and compares per capable instance.  With a lane per instance (lane-group mapping)
// every warp instruction serves one to four candidates and most lanes idle; here it serves 32.
//
// Where the state lives.  All instance state is in shared memory, in 16-byte units laid out
// unit-major: unit u of lane l sits at (u * lanes + l) * 16 bytes, so whatever unit each lane
// touches, the eight lanes of a quarter warp hit eight different 16-byte bank groups and a
// 128-bit access never conflicts.  A lane needs 2 units for its per-model instance ranges, 4
// per instance (clock and next completion; level, step and prefill terms; step counter and
// smallest key; slot mask and offsets) and, per instance, one 32-byte block per 8 virtual slots
// for the slot keys plus one block for the block minima.  A warp takes candidates of similar
// size (sorted by the validation kernels); how many lanes work on an item is what fits the
// block's pool: large placements run with fewer lanes instead of not at all.
//
// Slot keys: `end index << 7 | generation << 6 | slot` (an empty slot keeps its generation and
// slot bits under an all-ones end index).  The generation bit says which of the slot's two
// scratch entries in global memory holds the data of the running request (first-token time,
// arrival, request index, length, class, instance); entries are written at admission and come
// back through asynchronous copies into a per-lane queue when the request completes, so no
// load from global memory sits on the replay path.  The queue is accounted by all lanes
// together every few requests (or by a lane alone when its queue is full).
//
// Clocks are lazy: an instance that nothing happens to is not written back; its clock is
// recomputed from the last stored step boundary when it is looked at, which lands on the same
// boundaries as long as its level (and so its step time) has not changed.
//
// Each thread block is one warp with its own two-stage trace pipeline (1-D bulk copies + mbarrier,
// no multicast) and takes work items from one global counter; there is no block barrier.
#include "lane_sim.cuh"

namespace maaso {

constexpr uint32_t kFullMaskT = 0xFFFFFFFFu;
constexpr int kTTile = kScanTile;               // requests per scan tile
constexpr uint32_t kTEndEmpty = 0x1FFFFFFu;    // end-index field of an empty key
constexpr uint32_t kTRelMax = (1u << 25) - 2u; // largest end index a key can hold
#ifndef MAASO_TQUEUE
#define MAASO_TQUEUE 4
#endif
constexpr int kTQueue = MAASO_TQUEUE;           // queued completions per lane
#ifndef MAASO_THREAD_BPS
#define MAASO_THREAD_BPS 12
#endif
constexpr int kTDoneLanes = 2;                     // finished lanes that are handled together
constexpr int kTScanSteps = 2;                     // scan iterations between two looks at the waiting lanes
constexpr int kTBlocksPerSM = MAASO_THREAD_BPS;    // one-warp blocks per SM the register budget allows (3 per scheduler)

// Lanes that work on one item, by launch bucket (bucket 9 = placements the pool cannot hold at all).
__host__ __device__ inline uint32_t thread_lanes_of(int bucket) {
    const uint32_t l[9] = {32, 24, 16, 12, 8, 6, 4, 2, 1};
    return l[bucket];
}

// Pool units one placement needs: ranges + per instance 4 state units, 2 per block of 8 slots, 2 for the minima.
__host__ __device__ inline uint32_t thread_units_of_instance(uint32_t B) { return 4u + 2u * ((B + 7u) >> 3) + 2u; }

struct TPool {
    unsigned char* base;  // pool + lane * 16
    uint32_t stride;      // bytes from one unit of this lane to the next (= lanes * 16)
    __device__ __forceinline__ uint4* unit(uint32_t u) const {
        return reinterpret_cast<uint4*>(base + (size_t)u * stride);
    }
    __device__ __forceinline__ uint32_t* word(uint32_t u, uint32_t w) const {
        return reinterpret_cast<uint32_t*>(base + (size_t)u * stride) + w;
    }
};

// Working copy of one instance (units 0..2 of its state).
struct TInst {
    int64_t T;    // clock at the last stored step boundary
    int64_t tc;   // time of the next completion if nobody is admitted (valid while w > 0)
    uint32_t w, B, model, row;
    uint32_t sw;  // one decode step at the current level (valid while w > 0)
    uint32_t pre_base, pre_q16;
    uint32_t K;     // decode steps done at T since the counter last restarted
    uint32_t kmin;  // smallest slot key
    uint32_t stepB; // step at the batch cap: the worst case F(M,P,B_I)
    uint32_t swn;   // step at the level right after one more admission (optimistic estimate)
};

// The hot part (what a prediction reads): unit 2j = clock and next completion, unit 2j+1 = level, batch cap,
// model, table row | current step | step at the batch cap | step after one more admission.  The prefill
// terms of the row come from the warp's row table.  K and kmin belong to the cold part (t_load_keys).
__device__ __forceinline__ void t_load(const TPool& hp, const uint2* rowtab, uint32_t j, TInst& in) {
    const uint4 a = *hp.unit(2u * j), b = *hp.unit(2u * j + 1u);
    in.T = (int64_t)(((uint64_t)a.y << 32) | a.x);
    in.tc = (int64_t)(((uint64_t)a.w << 32) | a.z);
    in.w = b.x & 0xFFu; in.B = (b.x >> 8) & 0xFFu; in.model = (b.x >> 16) & 0xFFu; in.row = b.x >> 24;
    in.sw = b.y; in.stepB = b.z; in.swn = b.w;
    const uint2 pr = rowtab[in.row];
    in.pre_base = pr.x; in.pre_q16 = pr.y;
    in.K = 0; in.kmin = 0;
}
__device__ __forceinline__ void t_store(const TPool& hp, uint32_t j, const TInst& in) {
    *hp.unit(2u * j) = make_uint4((uint32_t)in.T, (uint32_t)((uint64_t)in.T >> 32), (uint32_t)in.tc,
                                  (uint32_t)((uint64_t)in.tc >> 32));
    *hp.unit(2u * j + 1u) = make_uint4(in.w | (in.B << 8) | (in.model << 16) | (in.row << 24), in.sw, in.stepB, in.swn);
}

struct TStats {
    Stats st;
    uint32_t hbc[8];
};

// What a thread needs besides the instance at hand.
struct TEnv {
    TPool hp;             // hot part of the instances (2 units each: what a prediction reads), shared memory
    const uint2* rowtab;  // per table row: prefill base, prefill slope (shared memory, one copy per warp)
    TPool pl;             // cold part: one unit per instance (slot mask, offsets), then the slot keys; shared or global memory
    int64_t* qf;          // this lane's queue column: entry j at qf[j * 32] = finish time
    uint4* qa;            // entry j at qa[j * 32] = first-token time, arrival time
    uint2* qb;            // entry j at qb[j * 32] = request index, S | cls << 16 | instance << 24
    uint4* pay_a;         // global scratch of this lane, entry 2 * slot number + generation
    uint2* pay_b;
    const int32_t* rows;  // latency tables (global, read through the read-only path at events only)
    TStats* ls;
    const EvalParams* P;
    int64_t oc;           // index of the candidate's record, negative for a lane without one
    uint32_t qn;          // completions waiting in the queue
};

// Statistics of this lane's queued completions (Phi_S indicator, latency and throughput sums).
static __device__ __noinline__ void t_flush(TStats* ls, const int64_t* qf, const uint4* qa, const uint2* qb, uint32_t n,
                                     const int64_t* classes, int64_t* dump_finish, int64_t* dump_first,
                                     int32_t* dump_inst, uint32_t* hist) {
    async_copies_done();
    Stats st = ls->st;
    const Dump no_dump{nullptr, nullptr, nullptr, nullptr};
    const bool dumping = dump_finish || dump_first || dump_inst || hist;
    for (uint32_t j = 0; j < n; j++) {
        const int64_t t_fin = qf[j * 32];
        const uint4 a = qa[j * 32];
        const uint2 b = qb[j * 32];
        const int64_t first = (int64_t)(((uint64_t)a.y << 32) | a.x);
        const int64_t arrival = (int64_t)(((uint64_t)a.w << 32) | a.z);
        const uint32_t cls = (b.y >> 16) & 0xFFu, inst = b.y >> 24;
        const bool hit = account_completion(st, classes, inst, b.x, arrival, first, t_fin, b.y & 0xFFFFu, cls, no_dump);
        if (hit) ls->hbc[cls < 7 ? cls : 7]++;
        if (dumping) {
            if (dump_finish) dump_finish[b.x] = t_fin;
            if (dump_first) dump_first[b.x] = first;
            if (dump_inst) dump_inst[b.x] = (int32_t)inst;
            if (hist) atomicAdd(hist + ttft_bin(first - arrival), 1u);
        }
    }
    ls->st = st;
}

__device__ __forceinline__ void t_flush_now(TEnv& e) {
    Dump dump{nullptr, nullptr, nullptr, nullptr};
    if (e.oc >= 0) dump = dump_for(*e.P, (uint32_t)e.oc);
    t_flush(e.ls, e.qf, e.qa, e.qb, e.qn, e.P->classes, dump.finish, dump.first, dump.inst, dump.hist);
    e.qn = 0;
}

// A running request has left its instance at t_fin: queue the finish time and start the copies
// of what it remembered.  A full queue is accounted by this lane alone first.
// Nothing waits for the copies here, so the retirements of one visit overlap their reads.  No entry
// is overwritten under a copy: a lane has no copy in flight when it starts a distributor round (it
// waits for them there, long after they were issued), the only write of a round is the admission
// at its end, and that goes to the other entry of its slot than the previous occupant's, the only
// one of that slot a copy of the same round can read.
__device__ __forceinline__ void t_push_slot(TEnv& e, int64_t t_fin, uint32_t pidx) {
    if (e.qn == (uint32_t)kTQueue) t_flush_now(e);
    const uint32_t j = e.qn;
    e.qf[j * 32] = t_fin;
    async_copy16(e.qa + j * 32, e.pay_a + pidx);
    async_copy8(e.qb + j * 32, e.pay_b + pidx);
    e.qn = j + 1;
}
// Same for a request of one output token, which completes at admission: everything is in registers.
__device__ __forceinline__ void t_push_now(TEnv& e, int64_t t_fin, uint4 a, uint2 b) {
    if (e.qn == (uint32_t)kTQueue) t_flush_now(e);
    const uint32_t j = e.qn;
    e.qf[j * 32] = t_fin;
    e.qa[j * 32] = a;
    e.qb[j * 32] = b;
    e.qn = j + 1;
}

__device__ __forceinline__ uint32_t t_step(const TEnv& e, uint32_t row, uint32_t level) {  // level >= 1
    return (uint32_t)__ldg(e.rows + row * kRowStride + 1u + level);
}

// Key storage of instance j: blocks of 8 keys from unit ko, then the 8 block minima.
struct TKeys {
    uint32_t ko;    // first key unit
    uint32_t so;    // number of this instance's slot 0 among the lane's slots (scratch entries)
    uint64_t mask;  // occupied slots; bits at and above B are always set
};
// The cold part of instance j: unit 2j = slot mask, key offset | slot offset; unit 2j+1 = step counter K,
// smallest key.  Read and written at events only.
__device__ __forceinline__ TKeys t_load_keys(const TPool& pl, uint32_t j, TInst& in) {
    const uint4 d = *pl.unit(2u * j);
    const uint2 c = *reinterpret_cast<const uint2*>(pl.unit(2u * j + 1u));
    TKeys k;
    k.mask = ((uint64_t)d.y << 32) | d.x;
    k.ko = d.z & 0xFFFFu;
    k.so = d.z >> 16;
    in.K = c.x;
    in.kmin = c.y;
    return k;
}
__device__ __forceinline__ void t_store_cold(const TPool& pl, uint32_t j, uint64_t mask, const TInst& in) {
    *reinterpret_cast<uint2*>(pl.unit(2u * j)) = make_uint2((uint32_t)mask, (uint32_t)(mask >> 32));
    *reinterpret_cast<uint2*>(pl.unit(2u * j + 1u)) = make_uint2(in.K, in.kmin);
}

// The counter has just reached the smallest end index (clock = in.T): retire every request that
// ends here, one per round, fix the block minima, the level and the cached next completion.
__device__ __forceinline__ void t_retire(TInst& in, TKeys& ks, TEnv& e) {
    const uint32_t Kc = in.K, nblk = (in.B + 7u) >> 3;
    uint4* const bm_lo = e.pl.unit(ks.ko + 2u * nblk);
    uint4* const bm_hi = e.pl.unit(ks.ko + 2u * nblk + 1u);
    do {
        const uint32_t slot = in.kmin & 63u, b = slot >> 3, sj = slot & 7u, gen = (in.kmin >> 6) & 1u;
        const uint4 k0 = *e.pl.unit(ks.ko + 2u * b), k1 = *e.pl.unit(ks.ko + 2u * b + 1u);
        const uint4 m0 = *bm_lo, m1 = *bm_hi;
        const uint32_t cleared = (kTEndEmpty << 7) | (in.kmin & 127u);
        *e.pl.word(ks.ko + 2u * b + (sj >> 2), sj & 3u) = cleared;
        uint32_t kv[8] = {k0.x, k0.y, k0.z, k0.w, k1.x, k1.y, k1.z, k1.w};
#pragma unroll
        for (int i = 0; i < 8; i++) kv[i] = (uint32_t)i == sj ? cleared : kv[i];
        const uint32_t bmin = min8(kv);
        *(reinterpret_cast<uint32_t*>(b < 4u ? bm_lo : bm_hi) + (b & 3u)) = bmin;
        uint32_t mv[8] = {m0.x, m0.y, m0.z, m0.w, m1.x, m1.y, m1.z, m1.w};
#pragma unroll
        for (int i = 0; i < 8; i++) mv[i] = (uint32_t)i == b ? bmin : mv[i];
        in.kmin = min8(mv);
        ks.mask &= ~(1ull << slot);
        in.w--;
        t_push_slot(e, in.T, 2u * (ks.so + slot) + gen);
    } while ((in.kmin >> 7) == Kc);
    if (in.w > 0) {
        in.sw = t_step(e, in.row, in.w);
        in.tc = in.T + (int64_t)((in.kmin >> 7) - Kc) * (int64_t)in.sw;
    }
    in.swn = t_step(e, in.row, min(in.w + 1u, in.B));
}

// "reduce" with events: run whole decode steps until the clock reaches `now` (drain: until the
// instance is empty), retiring what completes on the way.  `ks`: the instance's cold part, loaded by the caller.
__device__ __forceinline__ void t_events(TInst& in, TKeys& ks, int64_t now, bool drain, TEnv& e) {
    while (in.w > 0 && (drain || in.T < now)) {
        if (!drain && now <= in.tc - (int64_t)in.sw) {
            // the clock reaches `now` before anything completes (fewer steps than the longest request has tokens)
            const uint32_t k = ceil_div_small(now - in.T, in.sw, rcp_approx((float)in.sw));
            in.T += (int64_t)k * (int64_t)in.sw;
            in.K += k;
            break;
        }
        in.K = in.kmin >> 7;
        in.T = in.tc;
        t_retire(in, ks, e);
    }
    if (!drain && in.w == 0 && in.T < now) in.T = now;  // an idle instance starts at once
}
// The same with the cold part read and everything written back.
__device__ __forceinline__ void t_advance_events(TInst& in, uint32_t j, int64_t now, bool drain, TEnv& e) {
    TKeys ks = t_load_keys(e.pl, j, in);
    t_events(in, ks, now, drain, e);
    t_store(e.hp, j, in);
    t_store_cold(e.pl, j, ks.mask, in);
}

// All live end indices move down by the counter value K (which restarts at 0).  Rare.
static __device__ __noinline__ uint32_t t_rebase(unsigned char* base, uint32_t stride, uint32_t ko, uint32_t nblk, uint32_t K,
                                         uint32_t kmin) {
    const TPool pl{base, stride};
    const uint32_t d = K << 7;
    for (uint32_t u = 0; u < 2u * nblk + 2u; u++)
        for (uint32_t w = 0; w < 4u; w++) {
            uint32_t* p = pl.word(ko + u, w);
            if ((*p >> 7) != kTEndEmpty) *p -= d;
        }
    return (kmin >> 7) != kTEndEmpty ? kmin - d : kmin;
}

// "map": prefill at the step boundary in.T (running decodes stall), then occupy a free slot.
// `kadd`: decode steps the clock in.T is ahead of the stored step counter (a clock that was advanced lazily).
// `ks`: the instance's cold part, loaded by the caller; everything is written back here.
__device__ __forceinline__ void t_admit(TInst& in, TKeys& ks, uint32_t j, const CookedReq& q, uint32_t req, int64_t pre,
                                        uint32_t kadd, TEnv& e) {
    in.K += kadd;
    in.T += pre;
    const uint4 pa = make_uint4((uint32_t)in.T, (uint32_t)((uint64_t)in.T >> 32), (uint32_t)q.arrival,
                                (uint32_t)((uint64_t)q.arrival >> 32));
    const uint2 pb = make_uint2(req, (q.Sm1 + 1u) | (q.cls << 16) | (j << 24));
    if (q.Sm1 == 0) {  // done at the end of its prefill, never occupies a slot
        in.tc += pre;
        t_push_now(e, in.T, pa, pb);
        t_store(e.hp, j, in);
        t_store_cold(e.pl, j, ks.mask, in);
        return;
    }
    const uint32_t nblk = (in.B + 7u) >> 3;
    if (in.w == 0) in.K = 0;  // no live end index: the counter restarts
    if (in.K + q.Sm1 > kTRelMax) {
        in.kmin = t_rebase(e.pl.base, e.pl.stride, ks.ko, nblk, in.K, in.kmin);
        in.K = 0;
    }
    const uint32_t slot = (uint32_t)(__ffsll((long long)~ks.mask) - 1);
    uint32_t* const kw = e.pl.word(ks.ko + (slot >> 2), slot & 3u);
    const uint32_t gen = ((*kw >> 6) & 1u) ^ 1u;  // the other scratch entry than the previous occupant's
    const uint32_t key = ((in.K + q.Sm1) << 7) | (gen << 6) | slot;
    *kw = key;
    const uint32_t pidx = 2u * (ks.so + slot) + gen;
    // read once, much later, through an asynchronous copy: written past the caches' working set
    __stcs(e.pay_a + pidx, pa);
    __stcs(e.pay_b + pidx, pb);
    const uint32_t b = slot >> 3;
    uint32_t* const bm = e.pl.word(ks.ko + 2u * nblk + (b >> 2), b & 3u);
    *bm = min(*bm, key);
    in.kmin = min(in.kmin, key);
    ks.mask |= 1ull << slot;
    in.w++;
    in.sw = t_step(e, in.row, in.w);
    in.swn = t_step(e, in.row, min(in.w + 1u, in.B));
    in.tc = in.T + (int64_t)((in.kmin >> 7) - in.K) * (int64_t)in.sw;
    t_store(e.hp, j, in);
    t_store_cold(e.pl, j, ks.mask, in);
}

// Per-request side outputs of a rejection (dump rows, per-model counts); rare.
__device__ __forceinline__ void t_reject_side(const EvalParams& P, uint32_t oc, uint32_t req, uint32_t model) {
    const Dump dump = dump_for(P, oc);
    if (P.rej_by_model) atomicAdd(&P.rej_by_model[(size_t)oc * MAASO_MAX_MODELS + model], 1u);
    if (dump.finish) dump.finish[req] = -1;
    if (dump.first) dump.first[req] = -1;
    if (dump.inst) dump.inst[req] = -1;
}

struct ThreadSmem {
    unsigned char* hot;  // per lane: model ranges, one entry per model, the live map of the lane's current tile
    uint4* qa;           // [kTQueue][32]
    uint2* qb;
    int64_t* qf;
    uint2* rowtab;        // [n_rows] prefill base, prefill slope
    unsigned char* hpool; // hot part of the instances
    unsigned char* pool;  // cold part (shared-memory mode)
};
// per lane: model ranges (8 models per unit), one entry per model, the classes each model can serve at all
// (one word per model), the live map of the current tile (2 units)
__host__ __device__ inline uint32_t t_hot_units(uint32_t n_models) {
    return ((n_models + 7u) >> 3) + n_models + ((n_models + 3u) >> 2) + 2u;
}
__host__ __device__ inline size_t t_fixed_smem(uint32_t n_models, uint32_t n_rows) {
    return (size_t)t_hot_units(n_models) * 512u + (size_t)kTQueue * 32 * (16 + 8 + 8) + (((size_t)n_rows * 8u + 15u) & ~(size_t)15u);
}
__device__ __forceinline__ ThreadSmem t_carve(unsigned char* base, uint32_t n_models, uint32_t n_rows, uint32_t hot_bytes) {
    ThreadSmem s;
    s.hot = base;
    base += (size_t)t_hot_units(n_models) * 512u;
    s.qa = reinterpret_cast<uint4*>(base);
    base += (size_t)kTQueue * 32 * 16;
    s.qb = reinterpret_cast<uint2*>(base);
    base += (size_t)kTQueue * 32 * 8;
    s.qf = reinterpret_cast<int64_t*>(base);
    base += (size_t)kTQueue * 32 * 8;
    s.rowtab = reinterpret_cast<uint2*>(base);
    base += ((size_t)n_rows * 8u + 15u) & ~(size_t)15u;
    s.hpool = base;
    base += hot_bytes;
    s.pool = base;
    return s;
}

__device__ __forceinline__ uint4 ldg_nc(const uint4* p) { return __ldg(p); }
__device__ __forceinline__ void prefetch_l1(const void* p) { asm volatile("prefetch.global.L1 [%0];" ::"l"(p)); }

enum : uint32_t { kLaneIdle = 0, kLaneScan = 1, kLaneWait = 2, kLaneDone = 3 };

// OPT: the distributor predicts with the step time right after admission (optimistic estimate);
// a wait is then followed by a new choice.  Under the worst-case estimate the choice after a
// wait is known beforehand (same argument as in the lane-group kernel) and is only counted.
//
// How a lane walks its trace.  Most requests of a loaded placement are rejected for a reason that
// needs no look at the instances' state: the placement has no instance of the model, or the
// dispatcher's clock (and the earliest time any instance of the model could start a prefill) has
// passed the request's first-token or end-to-end deadline.  The trace is therefore kept as scan
// tiles (prep.cu): 256 requests with, per class, the latest deadline in the tile and a bit map of
// the class's requests, and per model a bit map.  A lane entering a tile builds its live map:
// requests of classes that are not late as a whole and of models the placement serves.  A tile
// without live requests costs five loads; a live request costs a 16-byte record and a compare
// against the model's lower bound; only what survives goes to the distributor.  Nothing is counted
// per request on the way: a placement's request count and the checksum of "all of them rejected"
// come from per-class totals of the trace, and an admission takes its request out again.
//
// The lanes of a warp are independent: each has its own placement and its own position in the
// trace, and takes the next placement of the bucket when it is through.  What they share is the
// instruction stream, so the warp alternates between scan iterations (for the lanes that can go
// on) and distributor rounds (for the lanes that stand at a request which needs one), and starts a
// round when `theta` lanes wait or nobody can scan.
template <bool OPT>
__global__ void __launch_bounds__(32, kTBlocksPerSM)
eval_thread_kernel(const __grid_constant__ EvalParams P, const uint32_t pool_bytes, const uint32_t hot_bytes,
                   const uint32_t theta, unsigned char* const arena) {
    // arena: the instances' state lives in global memory (one region of pool_bytes per warp, kept hot by
    // L1/L2) instead of shared memory, which leaves room for many more resident warps; null = shared memory
    extern __shared__ __align__(128) unsigned char smem_raw[];
    const ThreadSmem sm = t_carve(smem_raw, P.n_models, P.n_rows, hot_bytes);
    unsigned char* const pool = arena ? arena + (size_t)blockIdx.x * pool_bytes : sm.pool;
    const uint32_t lane = threadIdx.x;
    if (P.stall_test) return;  // test hook: nothing is scored, every valid candidate keeps its "not scored" mark
    for (uint32_t r = lane; r < P.n_rows; r += 32u)
        sm.rowtab[r] = make_uint2((uint32_t)P.rows[r * kRowStride + 0], (uint32_t)P.rows[r * kRowStride + 1]);
    __syncwarp();

    const uint32_t pool_units = pool_bytes / 16u;
    const bool use_mask = P.class_mask != nullptr && P.n_classes <= 32;
    const uint32_t n_traces = P.n_traces > 1 ? P.n_traces : 1u;
    // a lane's hot units: [0, rr) per-model instance ranges, [rr, rr + M) one entry per model (lower bound
    // of any predicted first token, smallest prefill base, smallest prediction step), then the live map
    const uint32_t rr = (P.n_models + 7u) >> 3;
    const uint32_t cfu = rr + P.n_models;                  // per model: the classes whose TBT limit some instance can meet
    const uint32_t lm = cfu + ((P.n_models + 3u) >> 2);    // first unit of the live map
    const TPool hot{sm.hot + lane * 16u, 512u};

    TStats ls;
    TEnv e;
    e.qf = sm.qf + lane;
    e.qa = sm.qa + lane;
    e.qb = sm.qb + lane;
    e.rows = P.rows;
    e.rowtab = sm.rowtab;
    e.ls = &ls;
    e.P = &P;
    e.qn = 0;
    e.oc = -1;

    // buckets with the fewest lanes per warp (the largest placements) first
    for (int b = 8; b >= 0; b--) {
        const uint32_t L = thread_lanes_of(b);
        const uint32_t cnt = P.bucket_count[kThreadBucket0 + b];
        const uint64_t total = (uint64_t)cnt * n_traces;
        if (total == 0 || *(volatile uint32_t*)&P.work_ctr[5 + b] >= total) continue;
        const uint32_t cap_units = pool_units / L;  // what one lane may use
        const uint32_t hot_cap = hot_bytes / 16u / L;
        // The cold part: unit-major like the hot part in shared memory; in the arena every lane has a region
        // of its own, so that an instance's mask, counters, keys and block minima share one or two cache lines.
        e.pl.base = arena ? pool + (size_t)lane * cap_units * 16u : pool + lane * 16u;
        e.pl.stride = arena ? 16u : L * 16u;
        e.hp.base = sm.hpool + lane * 16u;
        e.hp.stride = L * 16u;
        {   // scratch entries of this lane: two per slot, at most 4 slots per pool unit
            unsigned char* const wbase = reinterpret_cast<unsigned char*>(P.payload) + (size_t)blockIdx.x * pool_units * 8u * 24u;
            e.pay_a = reinterpret_cast<uint4*>(wbase) + (size_t)lane * cap_units * 8u;
            e.pay_b = reinterpret_cast<uint2*>(wbase + (size_t)pool_units * 8u * 16u) + (size_t)lane * cap_units * 8u;
        }
        bool open = lane < L;         // this lane may still find a placement in the bucket
        uint32_t state = kLaneIdle;
        // the lane's placement and where it stands
        uint32_t cand = 0, n_i = 0, status = 0, hasmodel = 0, cmask = 0, hmask = 0, mmask = 0, n_counted = 0;
        uint32_t n_req = 0, pos = 0, cur_tile = 0xFFFFFFFFu, out_base = 0;
        const uint4* cooked = nullptr;
        const uint4* scan = nullptr;
        uint64_t rej_sum = 0, extra = 0;
        int64_t now = 0, tile_base = 0;
        bool side = false;

        for (;;) {
            // ---- lanes without a placement take the next one of the bucket --------------------------------
            if (open && state == kLaneIdle) {
                const uint64_t idx = atomicAdd(&P.work_ctr[5 + b], 1u);
                if (idx >= total) {
                    open = false;
                } else {
                    const uint32_t tr = (uint32_t)(idx % n_traces);
                    cand = P.bucket_list[(size_t)(kThreadBucket0 + b) * P.n_cand + (uint32_t)(idx / n_traces)];
                    cooked = P.trace_cooked[tr];
                    scan = P.trace_scan[tr];
                    n_req = P.trace_n[tr];
                    out_base = tr * P.n_cand;
                    e.oc = (int64_t)(out_base + cand);
                    e.qn = 0;
                    ls.st.clear();
                    for (int i = 0; i < 8; i++) ls.hbc[i] = 0;
                    status = 0;
                    hasmodel = 0;
                    const uint32_t lo = P.offsets[cand];
                    n_i = P.offsets[cand + 1] - lo;
                    uint32_t rng_lo[MAASO_MAX_MODELS], rng_hi[MAASO_MAX_MODELS], min_pre[MAASO_MAX_MODELS], min_step[MAASO_MAX_MODELS];
                    for (int m = 0; m < MAASO_MAX_MODELS; m++) { rng_lo[m] = 0xFFu; rng_hi[m] = 0u; min_pre[m] = 0xFFFFFFFFu; min_step[m] = 0xFFFFFFFFu; }
                    uint32_t ko = 2u * n_i, so = 0;  // cold units: two per instance, then the key blocks
                    for (uint32_t j = 0; j < n_i; j++) {
                        const uint32_t word = P.inst[lo + j];
                        const uint32_t m = word & 0xFu, B = (word >> 12) & 0xFFu;
                        const uint32_t row = m * P.n_strategies + ((word >> 4) & 0xFFu);
                        const uint32_t nblk = (B + 7u) >> 3;
                        TInst in;
                        in.T = 0; in.tc = 0; in.w = 0; in.B = B; in.model = m; in.row = row; in.sw = 1;
                        in.pre_base = (uint32_t)P.rows[row * kRowStride + 0];
                        in.pre_q16 = (uint32_t)P.rows[row * kRowStride + 1];
                        in.K = 0; in.kmin = 0xFFFFFFFFu;
                        in.stepB = (uint32_t)P.rows[row * kRowStride + 1 + B];
                        in.swn = (uint32_t)P.rows[row * kRowStride + 2];
                        if (ko + 2u * nblk + 2u > cap_units || 2u * (j + 1u) > hot_cap) { status = MAASO_CAND_ETIMEOUT; break; }  // cannot happen: sized by the validation kernel
                        t_store(e.hp, j, in);
                        const uint64_t mask = B >= 64u ? 0ull : (~0ull << B);
                        *e.pl.unit(2u * j) = make_uint4((uint32_t)mask, (uint32_t)(mask >> 32), ko | (so << 16), 0u);
                        *e.pl.unit(2u * j + 1u) = make_uint4(0u, 0xFFFFFFFFu, 0u, 0u);
                        for (uint32_t u = 0; u < 2u * nblk; u++) {
                            const uint32_t s0 = (kTEndEmpty << 7) | (4u * u);
                            *e.pl.unit(ko + u) = make_uint4(s0, s0 + 1u, s0 + 2u, s0 + 3u);
                        }
                        const uint4 ones = make_uint4(0xFFFFFFFFu, 0xFFFFFFFFu, 0xFFFFFFFFu, 0xFFFFFFFFu);
                        *e.pl.unit(ko + 2u * nblk) = ones;
                        *e.pl.unit(ko + 2u * nblk + 1u) = ones;
                        ko += 2u * nblk + 2u;
                        so += 8u * nblk;
                        rng_lo[m] = min(rng_lo[m], j);
                        rng_hi[m] = j + 1u;
                        hasmodel |= 1u << m;
                        // the smallest step a prediction for this model can use: the step at the batch cap, or
                        // (optimistic estimate) at any level up to it
                        uint32_t ms = in.stepB;
                        if (OPT)
                            for (uint32_t w = 1; w < B; w++) ms = min(ms, (uint32_t)P.rows[row * kRowStride + 1 + w]);
                        min_step[m] = min(min_step[m], ms);
                        min_pre[m] = min(min_pre[m], in.pre_base);
                    }
                    // per-model instance ranges: halfword m = first index | (last index + 1) << 8
                    for (uint32_t u = 0; u < rr; u++) {
                        uint32_t rw[4];
                        for (int i = 0; i < 4; i++) {
                            const uint32_t m0 = 8u * u + 2u * i, m1 = m0 + 1u;
                            const uint32_t a = rng_lo[m0] >= rng_hi[m0] ? 0u : (rng_lo[m0] | (rng_hi[m0] << 8));
                            const uint32_t c = rng_lo[m1] >= rng_hi[m1] ? 0u : (rng_lo[m1] | (rng_hi[m1] << 8));
                            rw[i] = a | (c << 16);
                        }
                        *hot.unit(u) = make_uint4(rw[0], rw[1], rw[2], rw[3]);
                    }
                    // nothing runs yet: every predicted first token lies at or after the smallest prefill base
                    for (uint32_t m = 0; m < P.n_models; m++) *hot.unit(rr + m) = make_uint4(min_pre[m], 0u, min_pre[m], min_step[m]);
                    // A request of more than one token is served only by an instance whose prediction step meets
                    // the class's TBT limit (Sec. IV-F step 3).  Which classes a model's instances can serve at all
                    // is fixed for the placement: bit c of the model's word (classes 32 and up are not filtered).
                    for (uint32_t m = 0; m < P.n_models; m++) *hot.word(cfu + (m >> 2), m & 3u) = 0u;
                    for (uint32_t c = 0; c < P.n_classes && c < 32u; c++) {
                        const int64_t l_tbt = P.classes[c * 3u + 1u];
                        const uint32_t t32 = (l_tbt < 0 || l_tbt > 0xFFFFFFFFll) ? 0xFFFFFFFFu : (uint32_t)l_tbt;
                        for (uint32_t m = 0; m < P.n_models; m++)
                            if (t32 == 0xFFFFFFFFu || min_step[m] <= t32) *hot.word(cfu + (m >> 2), m & 3u) |= 1u << c;
                    }
                    cmask = use_mask ? P.class_mask[cand] : 0xFFFFFFFFu;
                    // header entries of a scan tile this lane has to look at (classes 7 and up share entry 7)
                    hmask = (cmask & 0x7Fu) | ((cmask >> 7) ? 0x80u : 0u);
                    mmask = (hasmodel & 0x7Fu) | ((hasmodel >> 7) ? 0x80u : 0u);  // the same for the per-model maps
                    side = P.rej_by_model != nullptr;
                    if (P.dump_row) side = side || P.dump_row[cand] >= 0;
                    // every request of the subset counted as rejected; admissions take theirs out
                    n_counted = 0;
                    rej_sum = 0;
                    const uint64_t* ct = P.trace_class_tot[tr];
                    for (uint32_t c = 0; c < P.n_classes; c++)
                        if (!use_mask || ((cmask >> c) & 1u)) {
                            n_counted += (uint32_t)ct[2u * c];
                            rej_sum += ct[2u * c + 1u];
                        }
                    now = 0;
                    extra = 0;
                    pos = 0;
                    cur_tile = 0xFFFFFFFFu;
                    state = (status == 0 && n_req > 0) ? kLaneScan : kLaneDone;
                }
            }
            if (!__any_sync(kFullMaskT, state != kLaneIdle)) break;  // the bucket is done as far as this warp goes

            // ---- scan iterations -------------------------------------------------------------------------------
            // Two per pass (measured: 1, 2, 3, 4, 6): a lane that has found its request idles through the rest
            // of them, a lane that still scans idles through the round that follows.
#pragma unroll 1
            for (int c = 0; c < kTScanSteps; c++) {
                if (state != kLaneScan) continue;
                const uint32_t tile = pos / (uint32_t)kTTile;
                const uint4* const th = scan + (size_t)tile * (kScanTile + kScanHdrUnits);
                const uint32_t recs = min((uint32_t)kTTile, n_req - tile * kTTile);
                if (tile != cur_tile) {
                    // A new tile: its live map for this lane = requests of a class that is not late as a whole
                    // (the dispatcher's clock has not passed the class's header entry) and of a model the
                    // placement has an instance of.  Everything else in the tile is rejected without a look.
                    cur_tile = tile;
                    uint4 lo = make_uint4(0u, 0u, 0u, 0u), hi = lo, hb = lo;
                    if (side) {
                        lo = hi = make_uint4(0xFFFFFFFFu, 0xFFFFFFFFu, 0xFFFFFFFFu, 0xFFFFFFFFu);  // every rejection is written out
                        hb = ldg_nc(th + kScanHdrBase);
                    } else {
                        // One round trip for the whole header: the eight class entries, the base arrival, and the
                        // maps of class slots 0..3 and model slots 0..3 as far as this placement can need them
                        // (which of the class maps count is known once the entries are here).  Slots 4..7 follow
                        // in a second step for the placements that use them.
                        const uint4 z4 = make_uint4(0u, 0u, 0u, 0u);
                        const uint4 h0 = ldg_nc(th), h1 = ldg_nc(th + 1), h2 = ldg_nc(th + 2), h3 = ldg_nc(th + 3);
                        hb = ldg_nc(th + kScanHdrBase);
                        uint4 ca[4], cx[4], ma[4], mx[4];
#pragma unroll
                        for (uint32_t k = 0; k < 4u; k++) {
                            const bool hc = (hmask >> k) & 1u, hm = (mmask >> k) & 1u;
                            ca[k] = hc ? ldg_nc(th + kScanHdrClassBits + 2u * k) : z4;
                            cx[k] = hc ? ldg_nc(th + kScanHdrClassBits + 2u * k + 1u) : z4;
                            ma[k] = hm ? ldg_nc(th + kScanHdrModelBits + 2u * k) : z4;
                            mx[k] = hm ? ldg_nc(th + kScanHdrModelBits + 2u * k + 1u) : z4;
                        }
                        const uint32_t hw[16] = {h0.x, h0.y, h0.z, h0.w, h1.x, h1.y, h1.z, h1.w, h2.x, h2.y, h2.z, h2.w, h3.x, h3.y, h3.z, h3.w};
                        uint32_t livec = 0;
#pragma unroll
                        for (int k = 0; k < 8; k++) {
                            const int64_t thr = (int64_t)(((uint64_t)hw[2 * k + 1] << 32) | hw[2 * k]);
                            if (((hmask >> k) & 1u) && thr >= now) livec |= 1u << k;
                        }
                        uint4 mlo = z4, mhi = z4;
#pragma unroll
                        for (uint32_t k = 0; k < 4u; k++) {
                            const uint32_t s = 0u - ((livec >> k) & 1u);  // all ones for a live class
                            lo.x |= ca[k].x & s; lo.y |= ca[k].y & s; lo.z |= ca[k].z & s; lo.w |= ca[k].w & s;
                            hi.x |= cx[k].x & s; hi.y |= cx[k].y & s; hi.z |= cx[k].z & s; hi.w |= cx[k].w & s;
                            mlo.x |= ma[k].x; mlo.y |= ma[k].y; mlo.z |= ma[k].z; mlo.w |= ma[k].w;
                            mhi.x |= mx[k].x; mhi.y |= mx[k].y; mhi.z |= mx[k].z; mhi.w |= mx[k].w;
                        }
                        if (((livec | mmask) >> 4) != 0u) {
#pragma unroll 1
                            for (uint32_t k = 4; k < 8u; k++) {
                                if ((livec >> k) & 1u) {
                                    const uint4 a = ldg_nc(th + kScanHdrClassBits + 2u * k), x = ldg_nc(th + kScanHdrClassBits + 2u * k + 1u);
                                    lo.x |= a.x; lo.y |= a.y; lo.z |= a.z; lo.w |= a.w;
                                    hi.x |= x.x; hi.y |= x.y; hi.z |= x.z; hi.w |= x.w;
                                }
                                if ((mmask >> k) & 1u) {
                                    const uint4 a = ldg_nc(th + kScanHdrModelBits + 2u * k), x = ldg_nc(th + kScanHdrModelBits + 2u * k + 1u);
                                    mlo.x |= a.x; mlo.y |= a.y; mlo.z |= a.z; mlo.w |= a.w;
                                    mhi.x |= x.x; mhi.y |= x.y; mhi.z |= x.z; mhi.w |= x.w;
                                }
                            }
                        }
                        lo.x &= mlo.x; lo.y &= mlo.y; lo.z &= mlo.z; lo.w &= mlo.w;
                        hi.x &= mhi.x; hi.y &= mhi.y; hi.z &= mhi.z; hi.w &= mhi.w;
                    }
                    if ((lo.x | lo.y | lo.z | lo.w | hi.x | hi.y | hi.z | hi.w) == 0u) {
                        pos = tile * kTTile + recs;  // nothing to look at in this tile
                    } else {
                        *hot.unit(lm) = lo;
                        *hot.unit(lm + 1u) = hi;
                        tile_base = (int64_t)(((uint64_t)hb.y << 32) | hb.x);
                    }
                } else {
                    // the next live requests at or after pos: up to four of one 32-request word of the map
                    uint32_t ri = pos - tile * kTTile;
                    uint32_t bits = *hot.word(lm + (ri >> 7), (ri >> 5) & 3u) >> (ri & 31u);
                    while (bits == 0u) {
                        ri = (ri | 31u) + 1u;
                        if (ri >= recs) break;
                        bits = *hot.word(lm + (ri >> 7), (ri >> 5) & 3u);
                    }
                    if (ri >= recs) {
                        pos = tile * kTTile + recs;
                    } else {
                        const uint4* const rp = th + kScanHdrUnits;  // the tile's scan records
                        uint32_t at[4];
                        uint4 sr[4];
                        bool have[4], real[4];
#pragma unroll
                        for (int k = 0; k < 4; k++) {
                            have[k] = bits != 0u;
                            at[k] = ri + (uint32_t)__ffs((int)bits) - 1u;
                            bits &= bits - 1u;
                            have[k] = have[k] && at[k] < recs;
                            sr[k] = ldg_nc(rp + (have[k] ? at[k] : ri));
                        }
#pragma unroll
                        for (int k = 0; k < 4; k++) {
                            const uint32_t model = sr[k].w & 0xFFu;
                            // in the request subset, and a model the placement serves
                            const uint32_t cls = (sr[k].w >> 8) & 0xFFu;
                            bool r = have[k] && ((cmask >> (cls & 31u)) & 1u) && ((hasmodel >> model) & 1u);
                            if (r) {
                                // Too late whatever the instance?  Every predicted first token of this model lies at
                                // or after flb: the dispatcher's clock plus the smallest prefill base, and the lower
                                // bound kept from the latest look at the model's instances (times only move forward).
                                // And no instance of the model may meet the class's TBT limit at all.  (One guarded block
                                // with all its loads at the top: branches in this loop cost more than the work they skip.)
                                const uint4 me = *hot.unit(rr + model);
                                const uint32_t cf = *hot.word(cfu + (model >> 2), model & 3u);
                                const uint32_t Sm1 = sr[k].w >> 16;
                                const bool tbt_dead = Sm1 != 0u && cls < 32u && !((cf >> cls) & 1u);
                                const int64_t arrival = tile_base + (int64_t)sr[k].x;
                                const int64_t flb = max(max(now, arrival) + (int64_t)me.z, (int64_t)(((uint64_t)me.y << 32) | me.x));
                                const bool late_first = sr[k].y != 0xFFFFFFFFu && arrival + (int64_t)sr[k].y < flb;
                                const bool late_end = sr[k].z != 0xFFFFFFFFu && arrival + (int64_t)sr[k].z < flb + (int64_t)((uint64_t)Sm1 * me.w);
                                // an arrival offset of all ones does not fit 32 bits: the distributor looks at the full record
                                r = !(tbt_dead || (sr[k].x != 0xFFFFFFFFu && (late_first || late_end)));
                            }
                            real[k] = r;
                        }
                        // the first of them that needs the distributor stops the lane; the ones before it are
                        // rejected (overflow protection, the plain case: nobody can meet the deadline)
                        uint32_t next = recs;
                        bool stop = false;
#pragma unroll
                        for (int k = 0; k < 4; k++) {
                            if (stop || !have[k]) continue;
                            if (real[k]) {
                                stop = true;
                                next = at[k];
                            } else {
                                if (side && ((cmask >> ((sr[k].w >> 8) & 31u)) & 1u))
                                    t_reject_side(P, out_base + cand, tile * kTTile + at[k], sr[k].w & 0xFFu);
                                next = at[k] + 1u;
                            }
                        }
                        pos = tile * kTTile + next;
                        if (stop) {
                            // the request's full record is read when the waiting lanes are served; a load into
                            // registers here would make the next iteration wait for it
                            state = kLaneWait;
                            const uint4* full = cooked + (size_t)pos * kCookedWords;
                            prefetch_l1(full);
                            prefetch_l1(full + 2);
                        }
                    }
                }
                if (state == kLaneScan && pos >= n_req) state = kLaneDone;
            }

            // ---- a distributor round for the waiting lanes, once enough of them wait --------------------------
            const uint32_t wl = __ballot_sync(kFullMaskT, state == kLaneWait);
            const uint32_t act = __ballot_sync(kFullMaskT, state == kLaneScan);
            // Once the bucket has run out of placements nothing is gained by collecting lanes for a round: what
            // is left is a tail of placements whose own chains of rounds bound the launch, so a waiting lane
            // is served at once.
            const bool tail = __any_sync(kFullMaskT, lane < L && !open);
            if (wl != 0u && ((uint32_t)__popc(wl) >= (tail ? 1u : theta) || act == 0u)) {
                // statistics of completed requests, all lanes together
                if (__any_sync(kFullMaskT, e.qn >= (uint32_t)(kTQueue - 1))) t_flush_now(e);
                if (state == kLaneWait) {
                    async_copies_done();  // of earlier rounds: none in flight while this round admits
                    const uint32_t req = pos;
                    const uint4* const full = cooked + (size_t)req * kCookedWords;
                    const CookedReq q = decode_cooked(ldg_nc(full), ldg_nc(full + 1), ldg_nc(full + 2));
                    pos++;
                    now = max(now, q.arrival);  // pending time: the dispatcher never goes back
                    // instances of the request's model
                    const uint4 rg = *hot.unit(q.model >> 3);
                    const uint32_t rgw = (q.model & 4u) ? ((q.model & 2u) ? rg.w : rg.z) : ((q.model & 2u) ? rg.y : rg.x);
                    const uint32_t rh = (q.model & 1u) ? (rgw >> 16) : (rgw & 0xFFFFu);
                    const uint32_t j_lo = rh & 0xFFu, j_hi = rh >> 8;
                    bool pending = true;
                    uint32_t tries = 0;
                    do {
                        tries++;
                        uint64_t best = kKeyInf;
                        uint32_t bj = 0, bk = 0;
                        int64_t bT = 0, bpre = 0;
                        // smallest and second smallest (start time + prefill base) over the model's instances
                        int64_t lb1 = INT64_MAX, lb2 = INT64_MAX;
                        uint32_t lb1j = 0xFFFFFFFFu;
                        for (uint32_t j = j_lo; j < j_hi; j++) {
                            TInst in;
                            t_load(e.hp, e.rowtab, j, in);
                            if (in.model != q.model) continue;
                            // "reduce": where the instance's clock stands once it has reached `now`
                            int64_t T = in.T;
                            uint32_t kadd = 0;
                            if (in.w > 0) {
                                if (T < now) {
                                    if (now > in.tc - (int64_t)in.sw) {  // something completes on the way
                                        t_advance_events(in, j, now, false, e);
                                        T = in.T;
                                    } else if (in.w < in.B) {
                                        kadd = ceil_div_small(now - T, in.sw, rcp_approx((float)in.sw));
                                        T += (int64_t)kadd * (int64_t)in.sw;
                                    }
                                }
                            } else if (T < now) {
                                T = now;
                            }
                            // distributor prediction (Sec. IV-F steps 2-3)
                            const int64_t pre = prefill_us(in.pre_base, in.pre_q16, q.in_tokens);
                            const bool free_slot = in.w < in.B;
                            const int64_t t0 = free_slot ? T : in.tc;
                            const uint32_t sB = (OPT && free_slot) ? in.swn : in.stepB;
                            const int64_t first = t0 + pre;
                            const int64_t fin = first + (int64_t)((uint64_t)q.Sm1 * sB);
                            {
                                const int64_t lb = t0 + (int64_t)in.pre_base;
                                if (lb < lb1) { lb2 = lb1; lb1 = lb; lb1j = j; }
                                else if (lb < lb2) lb2 = lb;
                            }
                            const bool ok = first <= q.dl_ttft && (q.Sm1 == 0 || sB <= q.tbt32) && fin <= q.dl_e2e;
                            const uint64_t key = ((uint64_t)(free_slot ? 0u : 1u) << 63) | (uint64_t)first;
                            if (ok && key < best) { best = key; bj = j; bk = kadd; bT = T; bpre = pre; }
                        }
                        int64_t lb_new = lb1;  // the model's lower bound as this look at its instances leaves it
                        if (best == kKeyInf) {
                            // overflow protection: nobody can meet the deadline -> rejected
                            if (side) t_reject_side(P, out_base + cand, req, q.model);
                            pending = false;
                        } else {
                            TInst in;
                            t_load(e.hp, e.rowtab, bj, in);
                            TKeys ks{0u, 0u, 0ull};
                            bool admit = true;
                            uint32_t kadd = 0;
                            if ((best >> 63) == 0) {
                                ks = t_load_keys(e.pl, bj, in);
                                in.T = bT;  // the clock as the prediction saw it
                                kadd = bk;
                            } else {
                                // every capable instance is full: wait until the chosen slot frees
                                now = in.tc;
                                if (!OPT) {
                                    tries++;  // the second round, counted only
                                    ks = t_load_keys(e.pl, bj, in);
                                    t_events(in, ks, now, false, e);
                                } else {
                                    admit = false;
                                    if (tries >= kAttemptCap) {
                                        status = MAASO_CAND_ELOOP;
                                        pending = false;
                                    }
                                }
                            }
                            if (admit) {
                                t_admit(in, ks, bj, q, req, bpre, kadd, e);
                                rej_sum -= q.rej;
                                pending = false;
                                lb_new = min(lb1j == bj ? lb2 : lb1, (in.w < in.B ? in.T : in.tc) + (int64_t)in.pre_base);
                            }
                        }
                        if (lb1 != INT64_MAX)
                            *reinterpret_cast<uint2*>(hot.unit(rr + q.model)) = make_uint2((uint32_t)lb_new, (uint32_t)((uint64_t)lb_new >> 32));
                    } while (OPT && pending);
                    extra += tries - 1u;
                    state = (status != 0u || pos >= n_req) ? kLaneDone : kLaneScan;  // a flagged candidate is given up
                }
            }

            // ---- lanes that are through their trace: drain, account what is still queued, write the record -----
            // Two of them together where it can be had (the drain, the record and the set-up of the next placement are long paths
            // that a lane alone would walk with the other 31 idle), unless nobody else is at work or the bucket
            // has run out.
            const uint32_t dn = __ballot_sync(kFullMaskT, state == kLaneDone);
            if (dn != 0u && ((uint32_t)__popc(dn) >= (uint32_t)kTDoneLanes || tail ||
                             !__any_sync(kFullMaskT, state == kLaneScan || state == kLaneWait))) {
                if (state == kLaneDone) {
                    if (status == 0) {
                        for (uint32_t j = 0; j < n_i; j++) {
                            TInst in;
                            t_load(e.hp, e.rowtab, j, in);
                            if (in.w > 0) t_advance_events(in, j, 0, true, e);
                        }
                    }
                    t_flush_now(e);
                    Stats st = ls.st;
                    st.checksum += rej_sum;
                    write_result(P.out + out_base + cand, status, n_counted, n_counted - st.served, (uint64_t)n_counted + extra, st,
                                 ls.hbc);
                    state = kLaneIdle;
                    e.oc = -1;
                }
            }
        }
        __syncwarp();
    }
}

cudaError_t launch_eval_thread(const EvalParams& P, int grid, uint32_t pool_bytes, uint32_t hot_bytes, uint32_t theta,
                               void* arena, cudaStream_t stream) {
    auto kernel = (P.flags & MAASO_FLAG_PRED_OPTIMISTIC) ? eval_thread_kernel<true> : eval_thread_kernel<false>;
    const size_t smem = (arena ? 0 : (size_t)pool_bytes) + hot_bytes + t_fixed_smem(P.n_models, P.n_rows);
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(kernel, cudaFuncAttributePreferredSharedMemoryCarveout, 100);
    if (e != cudaSuccess) return e;
    kernel<<<grid, 32, smem, stream>>>(P, pool_bytes, hot_bytes, theta, static_cast<unsigned char*>(arena));
    return cudaGetLastError();
}

int occupancy_eval_thread(const EvalParams& P, uint32_t pool_bytes, uint32_t hot_bytes, bool in_smem) {
    auto kernel = (P.flags & MAASO_FLAG_PRED_OPTIMISTIC) ? eval_thread_kernel<true> : eval_thread_kernel<false>;
    const size_t smem = (in_smem ? (size_t)pool_bytes : 0) + hot_bytes + t_fixed_smem(P.n_models, P.n_rows);
    cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    cudaFuncSetAttribute(kernel, cudaFuncAttributePreferredSharedMemoryCarveout, 100);
    int n = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, kernel, 32, smem) != cudaSuccess) return 1;
    return n < 1 ? 1 : n;
}

uint32_t thread_fixed_smem(uint32_t n_models, uint32_t n_rows) { return (uint32_t)t_fixed_smem(n_models, n_rows); }

// Global scratch one warp of the thread mapping needs: two entries of 24 bytes per slot, 4 slots per pool unit.
size_t thread_scratch_per_warp(uint32_t pool_bytes) { return (size_t)(pool_bytes / 16u) * 8u * 24u; }

}  // namespace maaso
