// One simulated instance owned by one lane: continuous batching with at most B virtual
// slots (simulator of Sec. V-A), clock advanced in whole decode steps whose length comes
// from the latency table row of the instance (Eq. 1 as a table).
//
// Slot bookkeeping.  A running request is identified by the value of the instance's step
// counter at which it ends.  Its slot key is one 32-bit word, `end index << 6 | slot`, so
// the minimum over keys names the next completion and the slot that holds it at once; an
// empty slot is all ones.  The keys of a lane sit in shared memory in blocks of 8 (one
// 32-byte read) followed by one minimum per block, so a completion re-reads one block and
// the 8 block minima; a lane takes as many blocks from its thread block's key pool as its
// batch cap needs (lanes the pool cannot hold use global scratch through the same pointers).
// The step counter is relative: it restarts at 0 whenever the instance is idle, and all
// live keys are rebased when an end index would not fit 26 bits.
//
// No load from global memory sits on the per-request path (an L2 hit costs several hundred
// cycles, and every step of a candidate's replay depends on the previous one).  What a
// running request must remember (first-token time, arrival, request index, length, class:
// 24 bytes) is written to global scratch at admission and never read back by a load: when
// the request completes, asynchronous copies (cp.async) move it into a small per-lane queue
// in shared memory together with the finish time.  The statistics are accumulated later,
// by all lanes of the warp together (flush_queue), into per-lane sums that live in local
// memory so that they cost no registers in the replay loop.  Each slot has two scratch entries used
// alternately, and a lane lets at most one group of copies be in flight, so an entry is
// never overwritten while a copy may still read it.
#pragma once
#include "common.cuh"

namespace maaso {

constexpr uint32_t kKeyEmpty = 0xFFFFFFFFu;
constexpr uint32_t kRelMax = (1u << 26) - 2u;  // largest end index a key can hold
constexpr int kKeyUnitBytes = 32;              // pool unit: one block of 8 keys (or the 8 block minima)
#ifndef MAASO_QUEUE
#define MAASO_QUEUE 4
#endif
#ifndef MAASO_FLUSH_AT
#define MAASO_FLUSH_AT 3
#endif
constexpr int kQueue = MAASO_QUEUE;            // queued completions per lane in shared memory
constexpr int kFlushAt = MAASO_FLUSH_AT;       // the warp accounts its queues once some lane holds this many
constexpr int kQueueOvf = 72;                  // further entries per lane in global scratch
constexpr int kOvfEntryBytes = 48;             // overflow entry: finish, req, S|cls; first token, arrival; largest gap
// Per-lane global scratch: payload A [64 slots][2] x 16 B, payload B [64][2] x 8 B, queue
// overflow x 48 B, and room for a lane's pool slice if the shared-memory pool is full (at most
// 64 keys + 8 block minima of 8 bytes, or 64 keys + 8 minima of 4 bytes + 64 x 16 bytes of gap data).
constexpr size_t kLaneScratchA = 0;
constexpr size_t kLaneScratchB = 64 * 2 * 16;
constexpr size_t kLaneScratchOvf = kLaneScratchB + 64 * 2 * 8;
constexpr size_t kLaneScratchKeys = kLaneScratchOvf + (size_t)kQueueOvf * kOvfEntryBytes;
constexpr size_t kLaneScratchBytes = kLaneScratchKeys + (9 + 5 * 8 + 8) * kKeyUnitBytes + 32;
static_assert(kLaneScratchBytes % 32 == 0 && kLaneScratchKeys % 16 == 0, "lane scratch layout");

struct LaneInst {
    static constexpr bool kAlwaysLoop = false;
    static constexpr bool kQueues = false;  // a wait is resolved in one round under the worst-case estimate
    static constexpr uint32_t kKeyWords = 1;    // 32-bit words per slot key
    static constexpr uint32_t kGapWords = 5;    // 32-bit words per slot of gap data (largest-gap mode only)
    static constexpr uint32_t kGapListUnits = 8; // 32-byte units of the lane's list of stretch gaps (16 entries)
    int64_t T;        // clock, always a decode-step boundary (may lag `now` while the instance is full)
    int64_t tc;       // time of the next completion if nobody is admitted (valid while w > 0)
    uint32_t K;       // decode steps done at T since the counter last restarted
    uint32_t w;       // running requests
    uint32_t B;       // batch cap = number of virtual slots
    uint32_t kmin;    // smallest slot key (next completion), kKeyEmpty when idle
    uint32_t sw;      // step[w-1]: length of one decode step at the current level (valid while w > 0)
    float rsw;        // 1 / sw
    uint32_t qn;      // completions waiting in this lane's queue
    uint64_t mask;    // occupied slots; bits at and above B are always set
    uint64_t gen;     // per slot: which of its two scratch entries the current occupant uses
    uint64_t stall;   // largest-gap mode: prefill time since the instance's latest decode-step end
    bool dirty;       // largest-gap mode: an admission or a retirement happened since the latest stretch was recorded
    uint32_t sidx;    // largest-gap mode: index of the next stretch (decode steps at one level, after one stall);
                      // at most two per request of the lane, so 32 bits outlast any trace that fits the device
    uint32_t sdepth;  // largest-gap mode: entries in the lane's list of stretch gaps
    const int32_t* step;  // shared-memory row: step[w-1] = one decode step with w running
    uint32_t stepB;   // step[B-1]
    uint32_t pre_base, pre_q16;
    uint32_t model;
};

struct LaneEnv {
    uint32_t* keys;          // this lane's slot keys, 8 per block of its batch cap (pool or global scratch)
    uint4* bm_lo;            // this lane's block minima, blocks 0..3 (right after the keys)
    uint4* bm_hi;            // blocks 4..7
    bool keys_shared;        // keys and block minima are in the shared-memory pool (the usual case)
    int64_t* qf;             // this lane's queue column: entry j at qf[j * kGroupThreads] = finish time
    uint4* qa;               // entry j at qa[j * kGroupThreads] = first-token time, arrival time
    uint2* qb;               // entry j at qb[j * kGroupThreads] = request index, S | cls << 16
    uint4* pay_a;            // global scratch [64][2]: first-token time, arrival time
    uint2* pay_b;            // global scratch [64][2]: request index, S | cls << 16
    unsigned char* ovf;      // this lane's queue overflow (global scratch, kOvfEntryBytes each)
    int64_t* qg;             // largest-gap mode: entry j at qg[j * kGroupThreads] = largest token gap; else null
    uint64_t* mg;            // largest-gap mode: per slot, largest gap among stretches that left the list (after the minima)
    uint64_t* dl;            // largest-gap mode: per slot, part of its first stretch's stall that ended with its first token
    uint32_t* first;         // largest-gap mode: per slot, index of the first stretch its request takes part in
    uint4* stk;              // largest-gap mode: list of stretch gaps {gap lo, gap hi, stretch index, -}, decreasing gaps
};

// Per-lane sums of completed requests; only flush_queue touches them.
struct LaneStats {
    Stats st;
    uint32_t hbc[8];    // hits by class
    const int64_t* qg;  // the lane's queue column of largest token gaps, null outside the largest-gap mode
};

// Asynchronous copies global -> shared: no register, nothing waits for them until a wait.
__device__ __forceinline__ void async_copy16(void* dst_smem, const void* src_gmem) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_addr(dst_smem)), "l"(src_gmem) : "memory");
}
__device__ __forceinline__ void async_copy8(void* dst_smem, const void* src_gmem) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"(smem_addr(dst_smem)), "l"(src_gmem) : "memory");
}
// Close the group of copies just issued and wait until only that group may still be in flight.
__device__ __forceinline__ void async_commit_keep_one() {
    asm volatile("cp.async.commit_group;\n\tcp.async.wait_group 1;" ::: "memory");
}
__device__ __forceinline__ void async_copies_done() {
    asm volatile("cp.async.wait_all;" ::: "memory");
}

__device__ __forceinline__ uint32_t min8(const uint32_t (&v)[8]) {
    return min(min(__vimin3_u32(v[0], v[1], v[2]), __vimin3_u32(v[3], v[4], v[5])), min(v[6], v[7]));
}

// *p = min(*p, v).  In shared memory as a reduction (nothing waits for the old value).  A lane
// whose keys live in global scratch reads and writes them with plain loads and stores only: a
// reduction would be carried out in L2 and a later load of the same lane could still be served
// a stale line from L1.
__device__ __forceinline__ void block_min_update(uint32_t* p, uint32_t v, bool shared) {
    if (shared)
        asm volatile("red.shared.min.u32 [%0], %1;" ::"r"(smem_addr(p)), "r"(v) : "memory");
    else
        *p = min(*p, v);
}

__device__ __forceinline__ uint32_t* bm_entry(const LaneEnv& env, uint32_t b) {
    return reinterpret_cast<uint32_t*>(b < 4u ? env.bm_lo : env.bm_hi) + (b & 3u);
}

// A running request has left the instance at t_fin: queue the finish time and start the
// copies of what it remembered (scratch entry `idx` = 2 * slot + generation).
template <bool MAXGAP>
__device__ __forceinline__ void lane_push_slot(LaneInst& in, const LaneEnv& env, int64_t t_fin, uint32_t idx,
                                               int64_t gap, uint32_t& status) {
    const uint32_t j = in.qn;
    if (j < (uint32_t)kQueue) {
        env.qf[j * kGroupThreads] = t_fin;
        if (MAXGAP) env.qg[j * kGroupThreads] = gap;
        async_copy16(env.qa + j * kGroupThreads, env.pay_a + idx);
        async_copy8(env.qb + j * kGroupThreads, env.pay_b + idx);
        async_commit_keep_one();
    } else if (j < (uint32_t)(kQueue + kQueueOvf)) {
        const uint4 a = env.pay_a[idx];
        const uint2 b = env.pay_b[idx];
        uint4* o = reinterpret_cast<uint4*>(env.ovf + (size_t)(j - kQueue) * kOvfEntryBytes);
        o[0] = make_uint4((uint32_t)t_fin, (uint32_t)((uint64_t)t_fin >> 32), b.x, b.y);
        o[1] = a;
        if (MAXGAP) o[2] = make_uint4((uint32_t)gap, (uint32_t)((uint64_t)gap >> 32), 0u, 0u);
    } else {
        status = MAASO_CAND_ELOOP;  // cannot happen: at most 64 completions per lane between flushes
        return;
    }
    in.qn = j + 1;
}

// Same for a request that completes at admission (one output token): everything is in registers.
template <bool MAXGAP, class Inst>
__device__ __forceinline__ void lane_push_now(Inst& in, const LaneEnv& env, int64_t t_fin, uint4 a, uint2 b,
                                              int64_t gap, uint32_t& status) {
    const uint32_t j = in.qn;
    if (j < (uint32_t)kQueue) {
        env.qf[j * kGroupThreads] = t_fin;
        if (MAXGAP) env.qg[j * kGroupThreads] = gap;
        env.qa[j * kGroupThreads] = a;
        env.qb[j * kGroupThreads] = b;
    } else if (j < (uint32_t)(kQueue + kQueueOvf)) {
        uint4* o = reinterpret_cast<uint4*>(env.ovf + (size_t)(j - kQueue) * kOvfEntryBytes);
        o[0] = make_uint4((uint32_t)t_fin, (uint32_t)((uint64_t)t_fin >> 32), b.x, b.y);
        o[1] = a;
        if (MAXGAP) o[2] = make_uint4((uint32_t)gap, (uint32_t)((uint64_t)gap >> 32), 0u, 0u);
    } else {
        status = MAASO_CAND_ELOOP;
        return;
    }
    in.qn = j + 1;
}

// Statistics of the queued completions (Phi_S indicator, latency and throughput sums), by
// all lanes of the warp together; every lane handles its own `n` entries.
template <bool MAXGAP>
__device__ __forceinline__ void flush_queue_body(LaneStats* ls, const int64_t* qf, const uint4* qa, const uint2* qb,
                                                 const unsigned char* ovf, uint32_t n, const int64_t* classes,
                                                 uint32_t inst_idx, int64_t* dump_finish, int64_t* dump_first,
                                                 int32_t* dump_inst, uint32_t* hist) {
    async_copies_done();
    Stats st = ls->st;
    const Dump no_dump{nullptr, nullptr, nullptr, nullptr};
    const bool dumping = dump_finish || dump_first || dump_inst || hist;
    for (uint32_t j = 0; j < n; j++) {
        int64_t t_fin, gap = -1;  // gap stays negative unless the TBT term is checked on the largest gap
        uint4 a;
        uint2 b;
        if (j < (uint32_t)kQueue) {
            t_fin = qf[j * kGroupThreads];
            a = qa[j * kGroupThreads];
            b = qb[j * kGroupThreads];
            if (MAXGAP) gap = ls->qg[j * kGroupThreads];
        } else {
            const uint4* o = reinterpret_cast<const uint4*>(ovf + (size_t)(j - kQueue) * kOvfEntryBytes);
            const uint4 h = o[0];
            t_fin = (int64_t)(((uint64_t)h.y << 32) | h.x);
            a = o[1];
            b = make_uint2(h.z, h.w);
            if (MAXGAP) { const uint4 x = o[2]; gap = (int64_t)(((uint64_t)x.y << 32) | x.x); }
        }
        const int64_t first = (int64_t)(((uint64_t)a.y << 32) | a.x);
        const int64_t arrival = (int64_t)(((uint64_t)a.w << 32) | a.z);
        const uint32_t cls = b.y >> 16;
        bool hit;
        if (MAXGAP) hit = account_completion(st, classes, inst_idx, b.x, arrival, first, t_fin, b.y & 0xFFFFu, cls, no_dump, gap);
        else hit = account_completion(st, classes, inst_idx, b.x, arrival, first, t_fin, b.y & 0xFFFFu, cls, no_dump);
        if (hit) ls->hbc[cls < 7 ? cls : 7]++;
        if (dumping) {
            if (dump_finish) dump_finish[b.x] = t_fin;
            if (dump_first) dump_first[b.x] = first;
            if (dump_inst) dump_inst[b.x] = (int32_t)inst_idx;
            if (hist) atomicAdd(hist + ttft_bin(first - arrival), 1u);
        }
    }
    ls->st = st;
}

// Out of line on purpose: the sums stay in local memory and the replay loop stays small.  One
// copy per form of the TBT term, so that the usual one carries nothing of the other.
static __device__ __noinline__ void flush_queue(LaneStats* ls, const int64_t* qf, const uint4* qa, const uint2* qb,
                                         const unsigned char* ovf, uint32_t n, const int64_t* classes,
                                         uint32_t inst_idx, int64_t* dump_finish, int64_t* dump_first,
                                         int32_t* dump_inst, uint32_t* hist) {
    flush_queue_body<false>(ls, qf, qa, qb, ovf, n, classes, inst_idx, dump_finish, dump_first, dump_inst, hist);
}
static __device__ __noinline__ void flush_queue_maxgap(LaneStats* ls, const int64_t* qf, const uint4* qa, const uint2* qb,
                                                const unsigned char* ovf, uint32_t n, const int64_t* classes,
                                                uint32_t inst_idx, int64_t* dump_finish, int64_t* dump_first,
                                                int32_t* dump_inst, uint32_t* hist) {
    flush_queue_body<true>(ls, qf, qa, qb, ovf, n, classes, inst_idx, dump_finish, dump_first, dump_inst, hist);
}

__device__ __forceinline__ void lane_reset(LaneInst& in, const int32_t* steps) {
    in.T = 0; in.tc = 0; in.K = 0; in.w = 0; in.kmin = kKeyEmpty; in.sw = 1; in.rsw = 1.0f; in.qn = 0;
    in.mask = ~0ull; in.gen = 0; in.stall = 0; in.dirty = false; in.sidx = 0; in.sdepth = 0;
    in.B = 1; in.model = 0xFFFFFFFFu; in.step = steps; in.stepB = 1; in.pre_base = 0; in.pre_q16 = 0;
}

// The counter K has just reached the smallest end index (clock = in.T).  Retire every
// request that ends here, one per round (the smallest key names its slot), fix the block
// minima, the level and the cached next completion.
// Largest-gap mode.  The instance is about to take its first decode step(s) since an admission or a
// retirement: a new stretch.  Every running request's next token comes `stall` (prefills since the
// latest step end) plus one step after that step end; a request admitted at this boundary got its
// first token part-way through the stall and waits that much less.  Further steps of the stretch
// are not longer.  A request's largest gap is therefore the maximum of the stretch gaps over the
// stretches it lives through, minus its own part of the stall in the first one.  The lane keeps
// the suffix maxima of the stretch gaps (a list with decreasing gaps and increasing stretch
// indices: the largest gap of stretches a..now is the oldest entry with index >= a), so a new
// stretch costs a few pops and one push and a completion one look-up.
constexpr uint32_t kGapList = 16;

__device__ __forceinline__ uint64_t gap_of(const uint4& e) { return ((uint64_t)e.y << 32) | e.x; }

// The list is full of strictly decreasing gaps: fold its oldest entry into the slots it concerns
// (exactly what the look-up would have found there) and drop it.  Rare, kept out of line.
static __device__ __noinline__ void gaps_drop_oldest(uint64_t* mg, uint64_t* dl, uint32_t* first, uint4* stk, uint32_t nslots) {
    const uint4 e = stk[0];
    const uint64_t v = gap_of(e);
    for (uint32_t i = 0; i < nslots; i++) {
        const uint32_t f = first[i];
        if (f > e.z) continue;
        mg[i] = max(mg[i], f == e.z ? v - dl[i] : v);
        first[i] = e.z + 1u;  // later stretches are still in the list, without a share of a stall
        dl[i] = 0;
    }
    for (uint32_t j = 0; j + 1u < kGapList; j++) stk[j] = stk[j + 1u];
}

__device__ __forceinline__ void gaps_fold(LaneInst& in, const LaneEnv& env) {
    const uint64_t g = in.stall + in.sw;
    uint32_t d = in.sdepth;
    while (d > 0 && gap_of(env.stk[d - 1u]) <= g) d--;  // dominated by this stretch from now on
    if (d == kGapList) {
        gaps_drop_oldest(env.mg, env.dl, env.first, env.stk, 8u * ((in.B + 7u) >> 3));
        d--;
    }
    env.stk[d] = make_uint4((uint32_t)g, (uint32_t)(g >> 32), in.sidx, 0u);
    in.sdepth = d + 1u;
    in.sidx++;
    in.stall = 0;
    in.dirty = false;
}

// Largest token gap of the request in `slot`, which completes now (its last stretch is in the list).
__device__ __forceinline__ uint64_t gaps_of_slot(const LaneInst& in, const LaneEnv& env, uint32_t slot) {
    const uint32_t a = env.first[slot];
    uint64_t r = env.mg[slot];
    for (uint32_t j = 0; j < in.sdepth; j++) {
        const uint4 e = env.stk[j];
        if (e.z < a) continue;
        uint64_t v = gap_of(e);
        if (e.z == a) {  // its first stretch: it had waited part of the stall already
            v -= env.dl[slot];
            if (j + 1u < in.sdepth) v = max(v, gap_of(env.stk[j + 1u]));
        }
        r = max(r, v);
        break;
    }
    return r;
}

template <bool MAXGAP>
__device__ __forceinline__ void lane_retire(LaneInst& in, const LaneEnv& env, uint32_t& status) {
    const uint32_t Kc = in.K;
    do {
        const uint32_t slot = in.kmin & 63u, b = slot >> 3, sj = slot & 7u;
        const uint4* kp = reinterpret_cast<const uint4*>(env.keys + 8u * b);
        const uint4 k0 = kp[0], k1 = kp[1];
        const uint4 m0 = *env.bm_lo, m1 = *env.bm_hi;
        env.keys[slot] = kKeyEmpty;
        uint32_t kv[8] = {k0.x, k0.y, k0.z, k0.w, k1.x, k1.y, k1.z, k1.w};
#pragma unroll
        for (int j = 0; j < 8; j++) kv[j] = (uint32_t)j == sj ? kKeyEmpty : kv[j];
        const uint32_t bmin = min8(kv);
        *bm_entry(env, b) = bmin;
        uint32_t mv[8] = {m0.x, m0.y, m0.z, m0.w, m1.x, m1.y, m1.z, m1.w};
#pragma unroll
        for (int i = 0; i < 8; i++) mv[i] = (uint32_t)i == b ? bmin : mv[i];
        in.kmin = min8(mv);
        in.mask &= ~(1ull << slot);
        in.w--;
        lane_push_slot<MAXGAP>(in, env, in.T, 2u * slot + (uint32_t)((in.gen >> slot) & 1ull),
                               MAXGAP ? (int64_t)gaps_of_slot(in, env, slot) : -1, status);
    } while ((in.kmin >> 6) == Kc);
    if (MAXGAP) in.dirty = true;  // the level changes: the next step has another length
    if (in.w > 0) {
        in.sw = (uint32_t)in.step[in.w - 1];
        in.rsw = rcp_approx((float)in.sw);
        in.tc = in.T + (int64_t)((in.kmin >> 6) - Kc) * (int64_t)in.sw;
    }
}

// "reduce": run whole decode steps until the clock reaches `now` (drain: until empty).
// A full instance whose next completion lies beyond `now` is left untouched: nothing
// observable depends on its clock until a slot frees, and later updates land on the same
// step boundaries.
template <bool MAXGAP>
__device__ __forceinline__ void lane_advance(LaneInst& in, int64_t now, bool drain, const LaneEnv& env,
                                             uint32_t& status) {
    while (in.w > 0 && (drain || in.T < now)) {
        if (!drain && now <= in.tc - (int64_t)in.sw) {
            // the clock reaches `now` before anything completes
            if (in.w < in.B) {
                if (MAXGAP && in.dirty) gaps_fold(in, env);
                // fewer steps than the longest request has tokens: the quotient fits the fast exact division
                const uint32_t k = ceil_div_small(now - in.T, in.sw, in.rsw);
                in.T += (int64_t)k * (int64_t)in.sw;
                in.K += k;
            }
            break;
        }
        if (MAXGAP && in.dirty) gaps_fold(in, env);
        in.K = in.kmin >> 6;
        in.T = in.tc;
        lane_retire<MAXGAP>(in, env, status);
    }
    if (!drain && in.w == 0 && in.T < now) {  // an idle instance starts at once
        in.T = now;
        if (MAXGAP) in.stall = 0;
    }
}

// One request as the replay loop sees it (decoded from a prepared trace record).
struct CookedReq {
    int64_t arrival;
    int64_t dl_ttft;   // latest first-token time that meets the TTFT limit
    int64_t dl_e2e;    // latest finish time that meets the end-to-end limit
    uint64_t rej;      // checksum term if it is rejected
    uint32_t in_tokens;
    uint32_t tbt32;    // TBT limit, 0xFFFFFFFF = none
    uint32_t Sm1;      // output tokens - 1
    uint32_t cls, model;
};

__device__ __forceinline__ CookedReq decode_cooked(const uint4& a, const uint4& b, const uint4& c) {
    CookedReq q;
    q.arrival = (int64_t)(((uint64_t)a.y << 32) | a.x);
    q.dl_ttft = (int64_t)(((uint64_t)a.w << 32) | a.z);
    q.dl_e2e = (int64_t)(((uint64_t)b.y << 32) | b.x);
    q.in_tokens = b.z;
    q.tbt32 = b.w;
    q.rej = ((uint64_t)c.y << 32) | c.x;
    q.Sm1 = c.z & 0xFFFFu;
    q.cls = (c.z >> 16) & 0xFFu;
    q.model = c.z >> 24;
    return q;
}

constexpr uint32_t kOffSat = 0x7FFFFFFEu;  // predicted first token this far after `now` or further
constexpr uint32_t kKey32Inf = 0xFFFFFFFFu;

// Distributor prediction for one instance (Sec. IV-F steps 2-3).  Returns the 32-bit choice
// key, tier << 31 | (predicted first-token time - now) clamped to kOffSat, or kKey32Inf if the
// request cannot meet its SLO there; t0 = time the request could start its prefill, first =
// predicted first-token time (never before `now`).
__device__ __forceinline__ uint32_t lane_predict(const LaneInst& in, const CookedReq& q, int64_t pre, int64_t now,
                                                 bool optimistic, int64_t& t0, int64_t& first) {
    uint32_t tier;
    uint32_t sB = in.stepB;  // worst case F(M,P,B_I)
    if (in.w < in.B) {
        tier = 0;
        t0 = in.T;
        if (optimistic) sB = (uint32_t)in.step[min(in.w + 1, in.B) - 1];
    } else {
        tier = 1;
        t0 = in.tc;  // exact time its next slot frees
    }
    first = t0 + pre;
    const int64_t fin = first + (int64_t)((uint64_t)q.Sm1 * sB);
    const bool ok = first <= q.dl_ttft && (q.Sm1 == 0 || sB <= q.tbt32) && fin <= q.dl_e2e;
    const uint64_t off = (uint64_t)(first - now);
    const uint32_t o31 = off >= (uint64_t)kOffSat ? kOffSat : (uint32_t)off;
    return ok ? ((tier << 31) | o31) : kKey32Inf;
}

// All live end indices move down by the current counter value `K` (the caller restarts the
// counter at 0).  Returns the rebased smallest key.  Rare: kept out of line, arguments by value.
static __device__ __noinline__ uint32_t lane_rebase(uint32_t* keys, uint32_t nslots, uint4* bm_lo, uint4* bm_hi,
                                             uint32_t K, uint32_t kmin) {
    const uint32_t d = K << 6;
    for (uint32_t s = 0; s < nslots; s++) {
        const uint32_t k = keys[s];
        if (k != kKeyEmpty) keys[s] = k - d;
    }
    for (uint32_t b = 0; b < 8; b++) {
        uint32_t* e = reinterpret_cast<uint32_t*>(b < 4u ? bm_lo : bm_hi) + (b & 3u);
        if (*e != kKeyEmpty) *e -= d;
    }
    return kmin != kKeyEmpty ? kmin - d : kmin;
}

// "map": prefill at the step boundary (running decodes stall), then occupy a free slot.
template <bool MAXGAP>
__device__ __forceinline__ void lane_admit(LaneInst& in, const CookedReq& q, uint32_t req, int64_t pre, int64_t now,
                                           const LaneEnv& env, uint32_t& status) {
    (void)now;  // the instance's own clock is at or after `now`
    in.T += pre;
    if (MAXGAP) {  // the prefill delays the next token of everybody who is running here
        in.stall += (uint64_t)pre;
        in.dirty = true;
    }
    const uint4 pa = make_uint4((uint32_t)in.T, (uint32_t)((uint64_t)in.T >> 32), (uint32_t)q.arrival,
                                (uint32_t)((uint64_t)q.arrival >> 32));
    const uint2 pb = make_uint2(req, (q.Sm1 + 1u) | (q.cls << 16));
    if (q.Sm1 == 0) {  // done at the end of its prefill, never occupies a slot
        in.tc += pre;
        lane_push_now<MAXGAP>(in, env, in.T, pa, pb, MAXGAP ? 0 : -1, status);
        return;
    }
    if (in.w == 0) in.K = 0;  // no live end index: the counter restarts
    if (in.K + q.Sm1 > kRelMax) {
        in.kmin = lane_rebase(env.keys, 8u * ((in.B + 7u) >> 3), env.bm_lo, env.bm_hi, in.K, in.kmin);
        in.K = 0;
    }
    const uint32_t slot = (uint32_t)(__ffsll((long long)~in.mask) - 1);
    const uint32_t key = ((in.K + q.Sm1) << 6) | slot;
    env.keys[slot] = key;
    if (MAXGAP) {  // no gap yet; its first token came `stall` after the latest step end
        env.mg[slot] = 0;
        env.dl[slot] = in.stall;
        env.first[slot] = in.sidx;  // the stretch that the next clock movement opens
    }
    in.gen ^= 1ull << slot;
    const uint32_t idx = 2u * slot + (uint32_t)((in.gen >> slot) & 1ull);
    env.pay_a[idx] = pa;
    env.pay_b[idx] = pb;
    block_min_update(bm_entry(env, slot >> 3), key, env.keys_shared);
    in.kmin = min(in.kmin, key);
    in.mask |= 1ull << slot;
    in.w++;
    in.sw = (uint32_t)in.step[in.w - 1];
    in.rsw = rcp_approx((float)in.sw);
    in.tc = in.T + (int64_t)((in.kmin >> 6) - in.K) * (int64_t)in.sw;
}

}  // namespace maaso
