// One simulated instance owned by one lane: continuous batching with at most B virtual
// slots (simulator of Sec. V-A), clock advanced in whole decode steps whose length comes
// from the latency table row of the instance (Eq. 1 as a table).
#pragma once
#include "common.cuh"

namespace maaso {

struct LaneInst {
    int64_t T;        // clock, always a decode-step boundary
    uint32_t K;       // decode steps done (only differences modulo 2^16 are used)
    uint32_t w;       // running requests
    uint32_t B;       // batch cap = number of virtual slots
    uint32_t kmin;    // low 16 bits of the smallest completion index among running requests
    uint64_t mask;    // occupied slots
    const int32_t* step;  // shared-memory row: step[w-1] = one decode step with w running
    uint32_t stepB;   // step[B-1]
    uint32_t pre_base, pre_q16;
    uint32_t model;
};

// Slot keys of one lane: low 16 bits of the completion index, in shared memory.
// Completion distances are below 2^16 because a request has at most 65535 output tokens.

// "reduce": run whole decode steps until the clock reaches `now` (drain: until empty).
// Completed requests are accounted into st / hbc.
__device__ __forceinline__ void lane_advance(LaneInst& in, int64_t now, bool drain, uint16_t* keys,
                                             const Payload* pay, Stats& st, uint32_t* hbc,
                                             const int64_t* classes, uint32_t inst_idx,
                                             const Dump& dump) {
    while (in.w > 0 && (drain || in.T < now)) {
        const uint32_t s = (uint32_t)in.step[in.w - 1];
        const uint32_t kfin = (in.kmin - in.K) & 0xFFFFu;  // steps until the next completion, >= 1
        if (!drain && now - in.T <= (int64_t)(kfin - 1) * (int64_t)s) {
            // the clock reaches `now` before anything completes: k = ceil((now - T) / s) < kfin
            const uint32_t k = ceil_div_steps(now - in.T, s);
            in.T += (int64_t)k * (int64_t)s;
            in.K += k;
            break;
        }
        in.T += (int64_t)kfin * (int64_t)s;
        in.K += kfin;
        const uint32_t K16 = in.K & 0xFFFFu;
        uint32_t nd = 0x10000u;
        uint64_t m = in.mask;
        while (m) {
            const int i = __ffsll((long long)m) - 1;
            m &= m - 1;
            const uint32_t d = ((uint32_t)keys[i] - K16) & 0xFFFFu;
            if (d == 0) {
                const uint4 a = reinterpret_cast<const uint4*>(pay + i)[0];
                const uint4 b = reinterpret_cast<const uint4*>(pay + i)[1];
                const int64_t first_tok = (int64_t)(((uint64_t)a.y << 32) | a.x);
                const int64_t arrival = (int64_t)(((uint64_t)a.w << 32) | a.z);
                const uint32_t cls = b.y >> 16;
                if (account_completion(st, classes, inst_idx, b.x, arrival, first_tok, in.T,
                                       b.y & 0xFFFFu, cls, dump))
                    hbc[cls < 7 ? cls : 7]++;
                in.mask &= ~(1ull << i);
                in.w--;
            } else {
                nd = min(nd, d);
            }
        }
        in.kmin = (K16 + nd) & 0xFFFFu;
    }
    if (!drain && in.w == 0 && in.T < now) in.T = now;  // an idle instance starts at once
}

// Distributor prediction for one instance (Sec. IV-F steps 2-3).  Returns the 64-bit
// choice key (tier << 63 | predicted first-token time) or kKeyInf if the request cannot
// meet its SLO there; t0 = time the request could start its prefill.
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
        t0 = in.T + (int64_t)((in.kmin - in.K) & 0xFFFFu) * (int64_t)in.stepB;  // w == B
    }
    const int64_t first = t0 + pre;
    const int64_t fin = first + (int64_t)(q.S - 1) * sB;
    const bool ok = (lim_ttft < 0 || first - q.arrival <= lim_ttft) &&
                    (lim_tbt < 0 || q.S == 1 || sB <= lim_tbt) &&
                    (lim_e2e < 0 || fin - q.arrival <= lim_e2e);
    return ok ? ((tier << 63) | (uint64_t)first) : kKeyInf;
}

// "map": prefill at the step boundary (running decodes stall), then occupy a free slot.
__device__ __forceinline__ void lane_admit(LaneInst& in, const Request& q, uint32_t req, int64_t pre,
                                           uint16_t* keys, Payload* pay, Stats& st, uint32_t* hbc,
                                           const int64_t* classes, uint32_t inst_idx,
                                           const Dump& dump) {
    in.T += pre;
    if (q.S == 1) {  // done at the end of its prefill, never occupies a slot
        if (account_completion(st, classes, inst_idx, req, q.arrival, in.T, in.T, 1, q.cls, dump))
            hbc[q.cls < 7 ? q.cls : 7]++;
        return;
    }
    const int slot = __ffsll((long long)~in.mask) - 1;
    const uint32_t key = (in.K + q.S - 1) & 0xFFFFu;
    keys[slot] = (uint16_t)key;
    store_payload(pay + slot, in.T, q.arrival, req, q.S, q.cls);
    if (in.w == 0 || ((key - in.K) & 0xFFFFu) < ((in.kmin - in.K) & 0xFFFFu)) in.kmin = key;
    in.mask |= 1ull << slot;
    in.w++;
}

}  // namespace maaso
