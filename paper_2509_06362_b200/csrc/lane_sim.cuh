// One simulated instance owned by one lane: continuous batching with at most B virtual
// slots (simulator of Sec. V-A), clock advanced in whole decode steps whose length comes
// from the latency table row of the instance (Eq. 1 as a table).
//
// Slot bookkeeping.  A running request is identified by the value of the instance's step
// counter at which it ends; only the low 16 bits are kept (a request has at most 65535
// output tokens, so distances to the counter are below 2^16 and order is preserved).
// The 64 slot keys of a lane sit in shared memory in 8 blocks of 8, followed by the key of
// each block's nearest completion, so a completion re-scans one block of 8 keys instead of
// all 64.  The time of the instance's next completion is cached (`tc`): between events it
// does not change, which lets a full instance skip its clock update entirely.
#pragma once
#include "common.cuh"

namespace maaso {

constexpr int kKeyStride = 72;  // uint16 per lane: 64 slot keys + 8 block minima (144 bytes)

struct LaneInst {
    int64_t T;        // clock, always a decode-step boundary (may lag `now` while the instance is full)
    int64_t tc;       // time of the next completion if nobody is admitted (valid while w > 0)
    uint32_t K;       // decode steps done at T (only differences modulo 2^16 are used)
    uint32_t w;       // running requests
    uint32_t B;       // batch cap = number of virtual slots
    uint32_t kmin;    // low 16 bits of the smallest completion index among running requests
    uint32_t sw;      // step[w-1]: length of one decode step at the current level (valid while w > 0)
    float rsw;        // 1 / sw
    uint32_t bslots;  // 3 bits per block: which of its 8 slots holds the block minimum
    uint64_t mask;    // occupied slots
    const int32_t* step;  // shared-memory row: step[w-1] = one decode step with w running
    uint32_t stepB;   // step[B-1]
    uint32_t pre_base, pre_q16;
    uint32_t model;
};

struct LaneEnv {
    uint16_t* keys;          // this lane's kKeyStride shared-memory halfwords
    Payload* pay;            // this lane's 64 payload entries (global scratch)
    uint32_t* hbc;           // this lane's 8 hit-by-class counters (shared memory)
    const int64_t* classes;  // shared memory
    uint32_t inst_idx;
    Dump dump;
};

// Bring the payload of the request that will complete next into L1 ahead of its use.
__device__ __forceinline__ void prefetch_l1(const void* p) {
    asm volatile("prefetch.global.L1 [%0];" ::"l"(p));
}

__device__ __forceinline__ uint32_t half_of(const uint4& v, int j) {  // j static after unrolling
    const uint32_t word = (j >> 1) == 0 ? v.x : ((j >> 1) == 1 ? v.y : ((j >> 1) == 2 ? v.z : v.w));
    return (j & 1) ? (word >> 16) : (word & 0xFFFFu);
}

// The counter K has just reached the smallest completion index (clock = in.T).  Retire every
// request that ends here, fix the block minima, the level and the cached next completion.
__device__ __forceinline__ void lane_retire(LaneInst& in, const LaneEnv& env, Stats& st) {
    const uint32_t K16 = in.K & 0xFFFFu;
    const uint4 bm = *reinterpret_cast<const uint4*>(env.keys + 64);
    uint32_t hit_blocks = 0, nd = 0x10000u, nb = 0;
#pragma unroll
    for (int b = 0; b < 8; b++) {  // branch-free per block: empty blocks count as infinitely far
        if (b > 0 && 8u * b >= in.B) break;  // blocks beyond the batch cap are never used
        const bool occ = ((uint32_t)(in.mask >> (8 * b)) & 0xFFu) != 0;
        const uint32_t d = occ ? ((half_of(bm, b) - K16) & 0xFFFFu) : 0x10000u;
        hit_blocks |= (d == 0 ? 1u : 0u) << b;
        const uint32_t dd = d == 0 ? 0x10000u : d;
        nb = dd < nd ? (uint32_t)b : nb;
        nd = min(nd, dd);
    }
    while (hit_blocks) {
        const int b = __ffs((int)hit_blocks) - 1;
        hit_blocks &= hit_blocks - 1;
        const uint32_t occ = (uint32_t)(in.mask >> (8 * b)) & 0xFFu;
        const uint4 kv = *reinterpret_cast<const uint4*>(env.keys + 8 * b);
        uint32_t done = 0, bd = 0x10000u, bj = 0;
#pragma unroll
        for (int j = 0; j < 8; j++) {
            const uint32_t d = ((occ >> j) & 1u) ? ((half_of(kv, j) - K16) & 0xFFFFu) : 0x10000u;
            done |= (d == 0 ? 1u : 0u) << j;
            const uint32_t dd = d == 0 ? 0x10000u : d;
            bj = dd < bd ? (uint32_t)j : bj;
            bd = min(bd, dd);
        }
        in.bslots = (in.bslots & ~(7u << (3 * b))) | (bj << (3 * b));
        nb = bd < nd ? (uint32_t)b : nb;
        in.mask &= ~((uint64_t)done << (8 * b));
        in.w -= __popc(done);
        env.keys[64 + b] = (uint16_t)(K16 + bd);
        nd = min(nd, bd);
        while (done) {
            const int j = __ffs((int)done) - 1;
            done &= done - 1;
            const Payload* p = env.pay + 8 * b + j;
            const uint4 a = reinterpret_cast<const uint4*>(p)[0];
            const uint4 c = reinterpret_cast<const uint4*>(p)[1];
            const int64_t first_tok = (int64_t)(((uint64_t)a.y << 32) | a.x);
            const int64_t arrival = (int64_t)(((uint64_t)a.w << 32) | a.z);
            const uint32_t cls = c.y >> 16;
            if (account_completion(st, env.classes, env.inst_idx, c.x, arrival, first_tok, in.T, c.y & 0xFFFFu,
                                   cls, env.dump))
                env.hbc[cls < 7 ? cls : 7]++;
        }
    }
    in.kmin = (K16 + nd) & 0xFFFFu;
    if (in.w > 0) {
        in.sw = (uint32_t)in.step[in.w - 1];
        in.rsw = __frcp_rn((float)in.sw);
        in.tc = in.T + (int64_t)nd * (int64_t)in.sw;
        prefetch_l1(env.pay + 8 * nb + ((in.bslots >> (3 * nb)) & 7u));
    }
}

// "reduce": run whole decode steps until the clock reaches `now` (drain: until empty).
// A full instance whose next completion lies beyond `now` is left untouched: nothing
// observable depends on its clock until a slot frees, and later updates land on the same
// step boundaries.
__device__ __forceinline__ void lane_advance(LaneInst& in, int64_t now, bool drain, const LaneEnv& env,
                                             Stats& st) {
    while (in.w > 0 && (drain || in.T < now)) {
        if (!drain && now <= in.tc - (int64_t)in.sw) {
            // the clock reaches `now` before anything completes
            if (in.w < in.B) {
                // fewer than kfin <= 65535 steps: the quotient fits the fast exact division
                const uint32_t k = ceil_div_small(now - in.T, in.sw, in.rsw);
                in.T += (int64_t)k * (int64_t)in.sw;
                in.K += k;
            }
            break;
        }
        in.K += (in.kmin - in.K) & 0xFFFFu;
        in.T = in.tc;
        lane_retire(in, env, st);
    }
    if (!drain && in.w == 0 && in.T < now) in.T = now;  // an idle instance starts at once
}

// Distributor prediction for one instance (Sec. IV-F steps 2-3).  Returns the 64-bit
// choice key (tier << 63 | predicted first-token time) or kKeyInf if the request cannot
// meet its SLO there; t0 = time the request could start its prefill.  Limits: "no limit" is
// passed as INT64_MAX here (all compared quantities are far below it).
__device__ __forceinline__ uint64_t lane_predict(const LaneInst& in, const Request& q, int64_t pre,
                                                 int64_t lim_ttft, int64_t lim_tbt, int64_t lim_e2e,
                                                 bool optimistic, int64_t& t0) {
    uint64_t tier;
    int64_t sB = (int64_t)in.stepB;  // worst case F(M,P,B_I)
    if (in.w < in.B) {
        tier = 0;
        t0 = in.T;
        if (optimistic) sB = (int64_t)in.step[min(in.w + 1, in.B) - 1];
    } else {
        tier = 1;
        t0 = in.tc;  // exact time its next slot frees
    }
    const int64_t first = t0 + pre;
    const int64_t fin = first + (int64_t)(q.S - 1) * sB;
    const bool ok = first - q.arrival <= lim_ttft && (q.S == 1 || sB <= lim_tbt) && fin - q.arrival <= lim_e2e;
    return ok ? ((tier << 63) | (uint64_t)first) : kKeyInf;
}

// "map": prefill at the step boundary (running decodes stall), then occupy a free slot.
__device__ __forceinline__ void lane_admit(LaneInst& in, const Request& q, uint32_t req, int64_t pre,
                                           const LaneEnv& env, Stats& st) {
    in.T += pre;
    if (q.S == 1) {  // done at the end of its prefill, never occupies a slot
        in.tc += pre;
        if (account_completion(st, env.classes, env.inst_idx, req, q.arrival, in.T, in.T, 1, q.cls, env.dump))
            env.hbc[q.cls < 7 ? q.cls : 7]++;
        return;
    }
    const int slot = __ffsll((long long)~in.mask) - 1;
    const int b = slot >> 3;
    const uint32_t key = (in.K + q.S - 1) & 0xFFFFu;
    const uint32_t dist = (key - in.K) & 0xFFFFu;
    env.keys[slot] = (uint16_t)key;
    store_payload(env.pay + slot, in.T, q.arrival, req, q.S, q.cls);
    const uint32_t occ = (uint32_t)(in.mask >> (8 * b)) & 0xFFu;
    if (occ == 0 || dist < (((uint32_t)env.keys[64 + b] - in.K) & 0xFFFFu)) {
        env.keys[64 + b] = (uint16_t)key;
        in.bslots = (in.bslots & ~(7u << (3 * b))) | ((uint32_t)(slot & 7) << (3 * b));
    }
    if (in.w == 0 || dist < ((in.kmin - in.K) & 0xFFFFu)) {
        in.kmin = key;
        prefetch_l1(env.pay + slot);
    }
    in.mask |= 1ull << slot;
    in.w++;
    in.sw = (uint32_t)in.step[in.w - 1];
    in.rsw = __frcp_rn((float)in.sw);
    in.tc = in.T + (int64_t)((in.kmin - in.K) & 0xFFFFu) * (int64_t)in.sw;
}

}  // namespace maaso
