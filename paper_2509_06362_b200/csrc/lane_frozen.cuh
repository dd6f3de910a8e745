// One simulated instance owned by one lane, for the engine that fixes a request's decode
// speed at its admission (Sec. IV-C read literally: the decode latency is S_r / F(M,P,B,W_i)
// with W_i the concurrency "when request r arrives"; the simulator of Sec. V-A keeps B
// virtual slots per instance).  A slot is busy from the admission of its request until the
// request's finish time; later admissions do not slow a running request down and prefills
// stall nobody, so the finish time is known at admission and the request is accounted there.
//
// Slot bookkeeping mirrors lane_sim.cuh with 64-bit keys: `finish time << 6 | slot`, empty =
// all ones, 8 keys per block plus one minimum per block in the thread block's key pool, so
// the minimum over keys names the next slot to free.  Times must stay below 2^57 us.
#pragma once
#include "lane_sim.cuh"

namespace maaso {

constexpr uint64_t kKey64Empty = ~0ull;

struct FrozenInst {
    static constexpr bool kAlwaysLoop = true;   // the single-round shortcut of the default engine does not hold here
    static constexpr bool kQueues = false;      // a request that finds every instance full waits at the dispatcher
    static constexpr uint32_t kKeyWords = 2;    // 32-bit words per slot key
    static constexpr uint32_t kGapWords = 0;    // every gap of a request is its fixed speed: nothing to track
    static constexpr uint32_t kGapListUnits = 0;
    uint64_t kmin;    // smallest slot key (the slot that frees next), kKey64Empty when idle
    uint64_t mask;    // busy slots; bits at and above B are always set
    uint32_t w;       // busy slots (requests running at the time of the last release)
    uint32_t B;       // batch cap = number of virtual slots
    uint32_t qn;      // admitted requests waiting in this lane's queue for their accounting
    const int32_t* step;  // shared-memory row: step[w-1] = one decode step with w running
    uint32_t stepB;   // step[B-1]
    uint32_t pre_base, pre_q16;
    uint32_t model;
};

__device__ __forceinline__ void lane_reset(FrozenInst& in, const int32_t* steps) {
    in.kmin = kKey64Empty; in.mask = ~0ull; in.w = 0; in.B = 1; in.qn = 0;
    in.step = steps; in.stepB = 1; in.pre_base = 0; in.pre_q16 = 0; in.model = 0xFFFFFFFFu;
}

__device__ __forceinline__ uint64_t min8_u64(const uint64_t (&v)[8]) {
    return min(min(min(v[0], v[1]), min(v[2], v[3])), min(min(v[4], v[5]), min(v[6], v[7])));
}

// The slot named by the smallest key has reached its finish time: free it.
__device__ __forceinline__ void frozen_release(FrozenInst& in, const LaneEnv& env) {
    uint64_t* keys = reinterpret_cast<uint64_t*>(env.keys);
    uint64_t* bm = reinterpret_cast<uint64_t*>(env.bm_lo);
    const uint32_t slot = (uint32_t)in.kmin & 63u, b = slot >> 3, sj = slot & 7u;
    uint64_t kv[8], mv[8];
#pragma unroll
    for (int j = 0; j < 8; j++) kv[j] = keys[8u * b + j];
#pragma unroll
    for (int j = 0; j < 8; j++) mv[j] = bm[j];
    keys[slot] = kKey64Empty;
#pragma unroll
    for (int j = 0; j < 8; j++) kv[j] = (uint32_t)j == sj ? kKey64Empty : kv[j];
    const uint64_t bmin = min8_u64(kv);
    bm[b] = bmin;
#pragma unroll
    for (int j = 0; j < 8; j++) mv[j] = (uint32_t)j == b ? bmin : mv[j];
    in.kmin = min8_u64(mv);
    in.mask &= ~(1ull << slot);
    in.w--;
}

// Free every slot whose request has finished by `now`.  Nothing to drain at the end of the
// trace: every admitted request was accounted at its admission.
template <bool MAXGAP>
__device__ __forceinline__ void lane_advance(FrozenInst& in, int64_t now, bool drain, const LaneEnv& env,
                                             uint32_t& status) {
    (void)status;
    if (drain) return;
    while (in.w > 0 && (int64_t)(in.kmin >> 6) <= now) frozen_release(in, env);
}

// Distributor prediction (Sec. IV-F steps 2-3), same key as the default engine's.  A free slot
// starts now; otherwise the request could start when the earliest slot frees.  The worst case is
// the step at the batch cap; the optimistic estimate, with a free slot, is the step the request
// will really get (level = running + 1).
__device__ __forceinline__ uint32_t lane_predict(const FrozenInst& in, const CookedReq& q, int64_t pre, int64_t now,
                                                 bool optimistic, int64_t& t0, int64_t& first) {
    uint32_t tier;
    uint32_t sB = in.stepB;
    if (in.w < in.B) {
        tier = 0;
        t0 = now;
        if (optimistic) sB = (uint32_t)in.step[in.w];
    } else {
        tier = 1;
        t0 = (int64_t)(in.kmin >> 6);
    }
    first = t0 + pre;
    const int64_t fin = first + (int64_t)((uint64_t)q.Sm1 * sB);
    const bool ok = first <= q.dl_ttft && (q.Sm1 == 0 || sB <= q.tbt32) && fin <= q.dl_e2e;
    const uint64_t off = (uint64_t)(first - now);
    const uint32_t o31 = off >= (uint64_t)kOffSat ? kOffSat : (uint32_t)off;
    return ok ? ((tier << 31) | o31) : kKey32Inf;
}

// Admission at `now` into a free slot: the speed is the table step of the level running + 1 and
// stays; the slot is held until the finish time (also for a request of one token).
template <bool MAXGAP>
__device__ __forceinline__ void lane_admit(FrozenInst& in, const CookedReq& q, uint32_t req, int64_t pre, int64_t now,
                                           const LaneEnv& env, uint32_t& status) {
    const int64_t first_tok = now + pre;
    const uint32_t speed = (uint32_t)in.step[in.w];
    const int64_t t_end = first_tok + (int64_t)((uint64_t)q.Sm1 * speed);
    if (((uint64_t)t_end >> 57) != 0) {  // beyond what a slot key can hold
        status = MAASO_CAND_ELOOP;
        return;
    }
    uint64_t* keys = reinterpret_cast<uint64_t*>(env.keys);
    uint64_t* bm = reinterpret_cast<uint64_t*>(env.bm_lo);
    const uint32_t slot = (uint32_t)(__ffsll((long long)~in.mask) - 1);
    const uint64_t key = ((uint64_t)t_end << 6) | slot;
    keys[slot] = key;
    // plain read-modify-write: a 64-bit `red.shared.min` here gave results that changed from run to
    // run (it is not one hardware operation on shared memory), and the lane owns these words anyway
    bm[slot >> 3] = min(bm[slot >> 3], key);
    in.kmin = min(in.kmin, key);
    in.mask |= 1ull << slot;
    in.w++;
    const uint4 pa = make_uint4((uint32_t)first_tok, (uint32_t)((uint64_t)first_tok >> 32), (uint32_t)q.arrival,
                                (uint32_t)((uint64_t)q.arrival >> 32));
    const uint2 pb = make_uint2(req, (q.Sm1 + 1u) | (q.cls << 16));
    lane_push_now<MAXGAP>(in, env, t_end, pa, pb, MAXGAP ? (q.Sm1 ? (int64_t)speed : 0) : -1, status);
}

// The same engine with a queue in front of every instance (Sec. II-A: requests beyond the batch
// cap wait in the instance's queue): a request whose chosen instance is full is handed over at
// once and starts when the slot that frees first frees; the dispatcher does not wait.
struct QueueInst : FrozenInst {
    static constexpr bool kQueues = true;
};

// Queued admission: the request takes over the slot with the smallest key (earliest finish,
// lowest slot among equals) at that slot's finish time.  Its level counts the other slots still
// busy at that moment, i.e. all of them except those that end at exactly the same time.
template <bool MAXGAP>
__device__ __forceinline__ void lane_admit_queued(FrozenInst& in, const CookedReq& q, uint32_t req, int64_t pre,
                                                  const LaneEnv& env, uint32_t& status) {
    uint64_t* keys = reinterpret_cast<uint64_t*>(env.keys);
    uint64_t* bm = reinterpret_cast<uint64_t*>(env.bm_lo);
    const uint32_t slot = (uint32_t)in.kmin & 63u, b = slot >> 3, sj = slot & 7u;
    const int64_t start = (int64_t)(in.kmin >> 6);
    uint64_t kv[8], mv[8];
#pragma unroll
    for (int j = 0; j < 8; j++) kv[j] = keys[8u * b + j];
#pragma unroll
    for (int j = 0; j < 8; j++) mv[j] = bm[j];
#pragma unroll
    for (int j = 0; j < 8; j++) kv[j] = (uint32_t)j == sj ? kKey64Empty : kv[j];
    uint64_t bmin = min8_u64(kv);
#pragma unroll
    for (int j = 0; j < 8; j++) mv[j] = (uint32_t)j == b ? bmin : mv[j];
    uint32_t same = 0;
    if ((int64_t)(min8_u64(mv) >> 6) == start) {  // rare: some other slot ends at the same time
        for (uint32_t x = 0; x < in.B; x++) same += (x != slot && (int64_t)(keys[x] >> 6) == start) ? 1u : 0u;
    }
    const uint32_t speed = (uint32_t)in.step[in.B - 1u - same];
    const int64_t first_tok = start + pre;
    const int64_t t_end = first_tok + (int64_t)((uint64_t)q.Sm1 * speed);
    if (((uint64_t)t_end >> 57) != 0) {
        status = MAASO_CAND_ELOOP;
        return;
    }
    const uint64_t key = ((uint64_t)t_end << 6) | slot;
    keys[slot] = key;
    bmin = min(bmin, key);
    bm[b] = bmin;
#pragma unroll
    for (int j = 0; j < 8; j++) mv[j] = (uint32_t)j == b ? bmin : mv[j];
    in.kmin = min8_u64(mv);
    const uint4 pa = make_uint4((uint32_t)first_tok, (uint32_t)((uint64_t)first_tok >> 32), (uint32_t)q.arrival,
                                (uint32_t)((uint64_t)q.arrival >> 32));
    const uint2 pb = make_uint2(req, (q.Sm1 + 1u) | (q.cls << 16));
    lane_push_now<MAXGAP>(in, env, t_end, pa, pb, MAXGAP ? (q.Sm1 ? (int64_t)speed : 0) : -1, status);
}

}  // namespace maaso
