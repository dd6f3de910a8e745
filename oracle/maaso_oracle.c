/*
 * CPU oracle for placement scoring by trace replay.  TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, single-threaded discrete-event simulation of what the placer's
 * simulator computes for ONE candidate placement: requests are taken in trace
 * order, the SLO-aware distributor picks an instance (or blocks, or rejects), every
 * instance runs continuous batching with at most B virtual slots, and decode-step
 * times come from the profiler's latency tables.  Nothing here is tuned; nothing
 * here is shared with the CUDA library (own structs, own constants, own helpers).
 * Only the tests, the smoke check and the benchmark's CPU-baseline leg call it.
 *
 * Passages followed (paper section / equation):
 *   - "Simulator Implementation" (Sec. V-A): virtual slots = inference batch size;
 *     "map" puts a request into a free slot, "reduce" advances instance clocks when
 *     no slot is free and retries, until the request is accommodated or rejected.
 *   - Distributor, Sec. IV-F steps 1-3: sub-cluster mapping (class mask), capability
 *     check + choice among capable instances, overflow protection with the
 *     worst-case throughput F(M,P,B_I).
 *   - Profiler, Sec. IV-B Eq. 1: decode rate depends on min(B, W); here as a table
 *     step_us[w] = time of one decode step with w running requests, w <= B.
 *   - Sec. II-A "Inference Batch Size": at most B running requests, others wait.
 *   - Sec. IV-C: L_r = L_q + L_d, SLO indicator [L_q + L_d <= tau_r] (objective
 *     Phi_S), constraints (b)-(d).
 *   - Sec. V-A "Evaluation Metrics": SLO attainment, decoding throughput, response
 *     latency = time to first token.
 *
 * Readings taken where the paper is silent or ambiguous (all integer microseconds):
 *   - Prefill of a request runs alone at a decode-step boundary of its instance and
 *     stalls the running decodes; the first token appears when it ends.
 *       prefill = base + ((q16 * in_tokens + 32768) >> 16)
 *   - Decode speed is dynamic: one step for all w running requests takes step_us[w];
 *     admissions and completions happen only at step boundaries.
 *   - One FIFO at the dispatcher (head-of-line): a blocked request holds back later
 *     ones; `now` only moves forward.
 *   - Choice among feasible instances: free slot first, then earliest predicted first
 *     token, then lowest instance index.
 *   - "Block" = defer while some full instance is still predicted feasible at the exact
 *     time its next slot frees; reject once none is.
 *   - A request with one output token completes at the end of its prefill and never
 *     occupies a slot.
 *   - TBT limit is on the mean gap: finish - first_token <= (S-1) * tbt.
 *
 * Parity pins (tests/, marker "not gpu"): hand-worked timelines under tests/golden/,
 * the single-server FIFO (Lindley) closed form for B = 1, the no-contention closed
 * form, a token-by-token re-formulation, conservation / monotonicity invariants,
 * mask algebra, the no-cascade special case with zero prefill, and brute-force
 * ranking.  Agreement with the paper's figures is "parity unpinned": the figures,
 * measured profiles and traces are not available.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORC_WMAX 64
#define ORC_MAX_INST 128
#define ORC_ATTEMPT_CAP (2u + ORC_MAX_INST * ORC_WMAX)

/* candidate status bits */
#define ORC_EBUDGET 1u   /* devices used exceed the budget: constraint (c) */
#define ORC_EMEMFIT 2u   /* an instance has fewer devices than its model needs: (d) */
#define ORC_ETOOMANY 4u  /* more than ORC_MAX_INST instances */
#define ORC_EBADINST 8u  /* unknown model / strategy, batch cap outside 1..64, reserved bits */
#define ORC_ETIMEOUT 16u /* never set by the oracle */
#define ORC_ELOOP 32u    /* attempt cap hit (cannot happen if the termination argument holds) */
#define ORC_EINVARIANT 0x80000000u /* an internal invariant failed: the oracle is wrong */

#define ORC_FLAG_PRED_OPTIMISTIC 1u
#define ORC_FLAG_TBT_MAXGAP 4u    /* the TBT term of the hit test looks at the largest gap between two
                                     consecutive tokens of the request instead of the mean gap */
#define ORC_FLAG_INSTANCE_QUEUES 8u /* requests wait at the instance they were given, not at the dispatcher
                                       (implies the engine that fixes the decode speed at admission) */
#define ORC_FLAG_ENGINE_FROZEN 2u /* the paper-literal engine: decode speed fixed at admission (below) */

typedef struct {
    int64_t arrival_us;
    uint32_t in_tokens;
    uint16_t out_tokens;
    uint8_t cls;
    uint8_t model;
} orc_request;

typedef struct {
    int64_t ttft_us, tbt_us, e2e_us; /* negative = no limit */
} orc_slo;

typedef struct {
    uint32_t n_models, n_strategies, wmax;
    const int32_t *devices;         /* [S] */
    const int32_t *min_devices;     /* [M] */
    const int32_t *prefill_base_us; /* [M][S] */
    const int32_t *prefill_q16;     /* [M][S] */
    const int32_t *step_us;         /* [M][S][wmax], entry w-1 = step time at running count w */
} orc_profile;

typedef struct {
    uint32_t status, n_counted, n_served, n_hit, n_rejected, n_cascade;
    uint32_t hit_by_class[8];
    int64_t sum_ttft_us, max_ttft_us, sum_e2e_us, max_e2e_us, makespan_us;
    uint64_t tokens_out, checksum, attempts, reserved;
} orc_result;

typedef struct {
    int used;
    uint32_t req;
    int64_t arrival, first_tok;
    int64_t fin_idx; /* value of the instance's step counter at which this request ends */
    int64_t last_tok; /* time of its latest token */
    int64_t max_gap;  /* largest gap between two consecutive tokens so far */
    uint32_t S;
    uint32_t cls;
} slot_t;

typedef struct {
    uint32_t model, strat, B;
    const int32_t *step; /* step[w-1] */
    int64_t pre_base;
    int64_t pre_q16;
    int64_t T; /* clock; always a step boundary */
    int64_t K; /* decode steps done so far */
    uint32_t w; /* running requests */
    slot_t slots[ORC_WMAX];
} inst_t;

typedef struct {
    const orc_slo *classes;
    orc_result *res;
    int64_t *dump_finish; /* [n] or NULL */
    int64_t *dump_first;
    int32_t *dump_inst;
    int bad; /* invariant violated */
    int tbt_maxgap; /* hit test on the largest token gap (ORC_FLAG_TBT_MAXGAP) */
} ctx_t;

/* SplitMix64 output mixer (public domain, Steele/Lea/Flood) */
static uint64_t mix64(uint64_t z) {
    z ^= z >> 30; z *= 0xBF58476D1CE4E5B9ull;
    z ^= z >> 27; z *= 0x94D049BB133111EBull;
    z ^= z >> 31;
    return z;
}
static uint64_t rotl64(uint64_t x, int r) { return (x << r) | (x >> (64 - r)); }

/* A request leaves the system served: Phi_S indicator, latency and throughput sums. */
static void complete(ctx_t *c, uint32_t inst_idx, uint32_t req, int64_t arrival, int64_t first_tok,
                     int64_t t_fin, uint32_t S, uint32_t cls, int64_t max_gap) {
    const orc_slo *k = &c->classes[cls];
    int64_t ttft = first_tok - arrival, e2e = t_fin - arrival, span = t_fin - first_tok;
    /* TBT term: mean gap (the normalised deadline of Sec. III-C as a per-token budget), or, as an
     * option, the largest single gap (a request of one token has no gap) */
    int tbt_ok = k->tbt_us < 0 || (c->tbt_maxgap ? max_gap <= k->tbt_us : span <= (int64_t)(S - 1) * k->tbt_us);
    int hit = (k->ttft_us < 0 || ttft <= k->ttft_us) && tbt_ok &&
              (k->e2e_us < 0 || e2e <= k->e2e_us);
    orc_result *r = c->res;
    if (ttft < 0 || span < 0) c->bad = 1;
    r->n_served++;
    if (hit) { r->n_hit++; r->hit_by_class[cls < 7 ? cls : 7]++; } else r->n_cascade++;
    r->sum_ttft_us += ttft; if (ttft > r->max_ttft_us) r->max_ttft_us = ttft;
    r->sum_e2e_us += e2e;   if (e2e > r->max_e2e_us) r->max_e2e_us = e2e;
    r->tokens_out += S;
    if (t_fin > r->makespan_us) r->makespan_us = t_fin;
    r->checksum += mix64((uint64_t)req * 0x9E3779B97F4A7C15ull ^ (uint64_t)t_fin ^
                         rotl64((uint64_t)first_tok, 32) ^ ((uint64_t)inst_idx << 56));
    if (c->dump_finish) c->dump_finish[req] = t_fin;
    if (c->dump_first) c->dump_first[req] = first_tok;
    if (c->dump_inst) c->dump_inst[req] = (int32_t)inst_idx;
}

static int64_t min_fin(const inst_t *in) {
    int64_t m = INT64_MAX;
    for (uint32_t j = 0; j < in->B; j++)
        if (in->slots[j].used && in->slots[j].fin_idx < m) m = in->slots[j].fin_idx;
    return m;
}

/* "reduce": run whole decode steps until the clock reaches t (t < 0 means: until empty). */
static void advance(ctx_t *c, inst_t *in, uint32_t inst_idx, int64_t t) {
    int drain = t < 0;
    while (in->w > 0 && (drain || in->T < t)) {
        int64_t s = in->step[in->w - 1];
        int64_t kfin = min_fin(in) - in->K;
        int64_t k = kfin;
        if (kfin < 1) c->bad = 1;
        if (!drain) {
            int64_t need = (t - in->T + s - 1) / s; /* ceil */
            if (need < k) k = need;
        }
        for (uint32_t j = 0; j < in->B; j++) {
            /* token gaps of this jump: the first one reaches back to the request's latest token (so it
             * includes prefills that stalled the batch), the other k - 1 are s, which is not larger */
            slot_t *sl = &in->slots[j];
            if (!sl->used) continue;
            int64_t gap = in->T + s - sl->last_tok;
            if (gap > sl->max_gap) sl->max_gap = gap;
            sl->last_tok = in->T + k * s;
        }
        in->T += k * s;
        in->K += k;
        for (uint32_t j = 0; j < in->B; j++) {
            slot_t *sl = &in->slots[j];
            if (sl->used && sl->fin_idx == in->K) {
                complete(c, inst_idx, sl->req, sl->arrival, sl->first_tok, in->T, sl->S, sl->cls, sl->max_gap);
                sl->used = 0;
                in->w--;
            }
        }
    }
    if (!drain && in->w == 0 && in->T < t) in->T = t; /* an idle instance starts at once */
}

static int64_t prefill_us(const inst_t *in, uint32_t in_tokens) {
    return in->pre_base + (int64_t)(((uint64_t)in->pre_q16 * in_tokens + 32768u) >> 16);
}

/* Validate the instance list against constraints (c), (d) and the table ranges. */
static uint32_t validate(const orc_profile *p, const uint32_t *inst, uint32_t n_inst, uint32_t budget) {
    uint32_t status = 0;
    uint64_t devsum = 0;
    if (n_inst > ORC_MAX_INST) return ORC_ETOOMANY;
    for (uint32_t i = 0; i < n_inst; i++) {
        uint32_t word = inst[i];
        uint32_t m = word & 0xF, s = (word >> 4) & 0xFF, b = (word >> 12) & 0xFF;
        if ((word >> 20) != 0 || m >= p->n_models || s >= p->n_strategies || b < 1 || b > p->wmax ||
            b > ORC_WMAX) {
            status |= ORC_EBADINST;
            continue;
        }
        devsum += (uint64_t)p->devices[s];
        if (p->devices[s] < p->min_devices[m]) status |= ORC_EMEMFIT;
    }
    if (devsum > budget) status |= ORC_EBUDGET;
    return status;
}

/*
 * The paper-literal engine ("frozen virtual slots").  Sec. IV-C writes the decode latency
 * of request r as S_r / F(M, P, B, W_i) with W_i "the number of concurrent requests when
 * request r arrives", and the simulator of Sec. V-A only keeps, per instance, B virtual
 * slots and when each becomes free.  Read literally: the decode speed of a request is fixed
 * when it is admitted, later admissions do not slow it down and prefills stall nobody.
 *   - a slot is busy from the admission of its request until that request's finish time;
 *     the running count w of an instance at time `now` = slots whose finish time is > now;
 *   - admission at time t into an instance with w running: first token at t + prefill,
 *     one token every step[w + 1] afterwards, finish = first + (S - 1) * step[w + 1];
 *     the slot is held until the finish time (also when S = 1);
 *   - the distributor is the one of the default engine: free slot first (start now), else the
 *     time the earliest slot frees; feasibility with the worst case step[B], or, with the
 *     optimistic flag and a free slot, with the step the request will really get; a wait moves
 *     `now` to that time and the choice is made again;
 *   - everything about a request is known at admission, so it is accounted there.
 * With B = 1 everywhere the two engines coincide (nobody runs beside anybody).
 *
 * Per-instance queues (ORC_FLAG_INSTANCE_QUEUES).  Sec. II-A lets requests beyond the batch cap
 * wait "in a waiting queue" of the instance, and Sec. IV-F step 2 sends a request to the instance
 * with the shortest queue.  In this engine every finish time is known, so the queue of an
 * instance can be measured in time: a request that finds every slot busy is given, at its
 * arrival, to the feasible instance where it would get its first token earliest, takes the slot
 * that frees first there (lowest index among equals), starts when that slot frees and runs at
 * the step of the level it finds then (1 + the other slots still busy at that moment).  The
 * dispatcher does not wait: the next request is handled at its own arrival time, so requests
 * queue per instance, first come first served, and a request for another instance can overtake.
 */
typedef struct {
    uint32_t model, B;
    const int32_t *step;
    int64_t pre_base, pre_q16;
    int busy[ORC_WMAX];
    int64_t until[ORC_WMAX]; /* finish time of the request in the slot */
} frozen_inst_t;

static void frozen_replay(ctx_t *c, const orc_profile *p, const uint32_t *inst, uint32_t n_inst,
                          const orc_request *reqs, uint64_t n, const orc_slo *classes, int has_mask,
                          uint32_t class_mask, uint32_t flags, orc_result *out) {
    frozen_inst_t *F = (frozen_inst_t *)calloc(n_inst ? n_inst : 1, sizeof(frozen_inst_t));
    if (!F) { c->bad = 1; return; }
    for (uint32_t i = 0; i < n_inst; i++) {
        uint32_t word = inst[i];
        F[i].model = word & 0xF; F[i].B = (word >> 12) & 0xFF;
        size_t row = (size_t)F[i].model * p->n_strategies + ((word >> 4) & 0xFF);
        F[i].step = p->step_us + row * p->wmax;
        F[i].pre_base = p->prefill_base_us[row];
        F[i].pre_q16 = (int64_t)(uint32_t)p->prefill_q16[row];
    }
    int64_t clock = 0;
    for (uint64_t r = 0; r < n && !out->status; r++) {
        const orc_request *q = &reqs[r];
        if (has_mask && ((class_mask >> q->cls) & 1u) == 0) continue; /* not in R_x */
        const orc_slo *k = &classes[q->cls];
        int64_t len = q->out_tokens;
        out->n_counted++;
        if (q->arrival_us > clock) clock = q->arrival_us;
        for (uint32_t round = 0;; round++) {
            if (round >= ORC_ATTEMPT_CAP) { out->status = ORC_ELOOP; break; }
            out->attempts++;
            int found = 0, pick_tier = 0; int64_t pick_first = 0, pick_start = 0; uint32_t pick = 0;
            for (uint32_t i = 0; i < n_inst; i++) {
                frozen_inst_t *f = &F[i];
                if (f->model != q->model) continue;
                uint32_t running = 0; int64_t earliest = INT64_MAX;
                for (uint32_t j = 0; j < f->B; j++) {
                    if (f->busy[j] && f->until[j] <= clock) f->busy[j] = 0; /* the slot is free again */
                    if (f->busy[j]) { running++; if (f->until[j] < earliest) earliest = f->until[j]; }
                }
                int tier_i = running < f->B ? 0 : 1;
                int64_t start = tier_i == 0 ? clock : earliest;
                int64_t prefill = f->pre_base + (int64_t)(((uint64_t)f->pre_q16 * q->in_tokens + 32768u) >> 16);
                int64_t s_pred = f->step[f->B - 1];
                if ((flags & ORC_FLAG_PRED_OPTIMISTIC) && tier_i == 0) s_pred = f->step[running];
                int64_t p_first = start + prefill, p_fin = p_first + (len - 1) * s_pred;
                int ok = (k->ttft_us < 0 || p_first - q->arrival_us <= k->ttft_us) &&
                         (k->tbt_us < 0 || len == 1 || s_pred <= k->tbt_us) &&
                         (k->e2e_us < 0 || p_fin - q->arrival_us <= k->e2e_us);
                if (!ok) continue;
                if (!found || tier_i < pick_tier || (tier_i == pick_tier && p_first < pick_first)) {
                    found = 1; pick_tier = tier_i; pick_first = p_first; pick_start = start; pick = i;
                }
            }
            if (!found) {
                out->n_rejected++;
                out->checksum += mix64((uint64_t)r * 0x9E3779B97F4A7C15ull ^ ~0ull);
                if (c->dump_finish) c->dump_finish[r] = -1;
                if (c->dump_first) c->dump_first[r] = -1;
                if (c->dump_inst) c->dump_inst[r] = -1;
                break;
            }
            if (pick_tier == 0) {
                frozen_inst_t *f = &F[pick];
                uint32_t running = 0, j = f->B;
                for (uint32_t x = 0; x < f->B; x++) { if (f->busy[x]) running++; else if (j == f->B) j = x; }
                if (j >= f->B) { c->bad = 1; break; }
                int64_t speed = f->step[running];        /* level running + 1, fixed from now on */
                int64_t first_tok = clock + f->pre_base + (int64_t)(((uint64_t)f->pre_q16 * q->in_tokens + 32768u) >> 16);
                int64_t t_end = first_tok + (len - 1) * speed;
                f->busy[j] = 1; f->until[j] = t_end;
                complete(c, pick, (uint32_t)r, q->arrival_us, first_tok, t_end, (uint32_t)len, q->cls,
                         len > 1 ? speed : 0); /* every gap of the request is `speed` */
                break;
            }
            if (pick_start <= clock) c->bad = 1;
            if (flags & ORC_FLAG_INSTANCE_QUEUES) { /* queue at the chosen instance; the dispatcher moves on */
                frozen_inst_t *f = &F[pick];
                uint32_t j = f->B;
                for (uint32_t x = 0; x < f->B; x++)
                    if (j == f->B || f->until[x] < f->until[j]) j = x; /* the slot that frees first */
                if (j >= f->B || !f->busy[j] || f->until[j] != pick_start) { c->bad = 1; break; }
                uint32_t still = 0; /* other slots still busy when this one frees */
                for (uint32_t x = 0; x < f->B; x++)
                    if (x != j && f->until[x] > pick_start) still++;
                int64_t q_speed = f->step[still];
                int64_t q_first = pick_start + f->pre_base + (int64_t)(((uint64_t)f->pre_q16 * q->in_tokens + 32768u) >> 16);
                int64_t q_end = q_first + (len - 1) * q_speed;
                f->until[j] = q_end;
                complete(c, pick, (uint32_t)r, q->arrival_us, q_first, q_end, (uint32_t)len, q->cls,
                         len > 1 ? q_speed : 0);
                break;
            }
            clock = pick_start; /* wait for that slot, then choose again */
        }
    }
    free(F);
}

/*
 * Score one candidate.  inst[n_inst]: packed words (model bits 0-3, strategy 4-11, batch
 * cap 12-19).  has_mask/class_mask: requests whose class bit is clear are not part of the
 * request subset R_x this placement is scored on (ignored when n_classes > 32).
 * dump_* (each [n] or NULL): per request finish time / first-token time / instance;
 * -1 = rejected, -2 = not counted.
 * Returns 0; the outcome is in out->status.
 */
int orc_eval_candidate(const orc_profile *p, const orc_request *reqs, uint64_t n,
                       const orc_slo *classes, uint32_t n_classes, const uint32_t *inst,
                       uint32_t n_inst, int has_mask, uint32_t class_mask, uint32_t budget,
                       uint32_t flags, orc_result *out, int64_t *dump_finish, int64_t *dump_first,
                       int32_t *dump_inst) {
    ctx_t c;
    memset(out, 0, sizeof(*out));
    c.classes = classes; c.res = out; c.bad = 0;
    c.tbt_maxgap = (flags & ORC_FLAG_TBT_MAXGAP) != 0;
    c.dump_finish = dump_finish; c.dump_first = dump_first; c.dump_inst = dump_inst;
    for (uint64_t r = 0; r < n; r++) {
        if (dump_finish) dump_finish[r] = -2;
        if (dump_first) dump_first[r] = -2;
        if (dump_inst) dump_inst[r] = -2;
    }
    out->status = validate(p, inst, n_inst, budget);
    if (out->status) return 0;
    if (n_classes > 32) has_mask = 0;

    inst_t *I = (inst_t *)calloc(n_inst ? n_inst : 1, sizeof(inst_t));
    if (!I) return -1;
    for (uint32_t i = 0; i < n_inst; i++) {
        uint32_t word = inst[i];
        I[i].model = word & 0xF; I[i].strat = (word >> 4) & 0xFF; I[i].B = (word >> 12) & 0xFF;
        size_t row = (size_t)I[i].model * p->n_strategies + I[i].strat;
        I[i].step = p->step_us + row * p->wmax;
        I[i].pre_base = p->prefill_base_us[row];
        I[i].pre_q16 = (int64_t)(uint32_t)p->prefill_q16[row];
    }

    if (flags & (ORC_FLAG_ENGINE_FROZEN | ORC_FLAG_INSTANCE_QUEUES)) {
        frozen_replay(&c, p, inst, n_inst, reqs, n, classes, has_mask, class_mask, flags, out);
        goto replay_done;
    }
    int64_t now = 0;
    for (uint64_t r = 0; r < n && !out->status; r++) {
        const orc_request *q = &reqs[r];
        if (has_mask && !((class_mask >> q->cls) & 1u)) continue; /* not in R_x */
        const orc_slo *k = &classes[q->cls];
        int64_t S = q->out_tokens;
        out->n_counted++;
        if (q->arrival_us > now) now = q->arrival_us; /* pending time: never back in time */
        for (uint32_t attempt = 0;; attempt++) {
            if (attempt >= ORC_ATTEMPT_CAP) { out->status = ORC_ELOOP; break; }
            out->attempts++;
            for (uint32_t i = 0; i < n_inst; i++) {
                int64_t before = I[i].T;
                advance(&c, &I[i], i, now);
                if (I[i].T < before || I[i].w > I[i].B) c.bad = 1;
            }
            int have = 0; int best_tier = 0; int64_t best_first = 0, best_t0 = 0; uint32_t best_i = 0;
            for (uint32_t i = 0; i < n_inst; i++) {
                inst_t *in = &I[i];
                if (in->model != q->model) continue;
                int tier; int64_t t0;
                if (in->w < in->B) { tier = 0; t0 = in->T; }             /* a free virtual slot */
                else { tier = 1; t0 = in->T + (min_fin(in) - in->K) * (int64_t)in->step[in->w - 1]; }
                int64_t pre = prefill_us(in, q->in_tokens);
                int64_t sB = in->step[in->B - 1];                        /* worst case F(M,P,B_I) */
                if ((flags & ORC_FLAG_PRED_OPTIMISTIC) && tier == 0) {
                    uint32_t wn = in->w + 1 < in->B ? in->w + 1 : in->B;
                    sB = in->step[wn - 1];
                }
                int64_t first = t0 + pre, fin = first + (S - 1) * sB;
                int feasible = (k->ttft_us < 0 || first - q->arrival_us <= k->ttft_us) &&
                               (k->tbt_us < 0 || S == 1 || sB <= k->tbt_us) &&
                               (k->e2e_us < 0 || fin - q->arrival_us <= k->e2e_us);
                if (!feasible) continue;
                if (!have || tier < best_tier || (tier == best_tier && first < best_first)) {
                    have = 1; best_tier = tier; best_first = first; best_t0 = t0; best_i = i;
                }
            }
            if (!have) { /* overflow protection: no instance can meet the deadline */
                out->n_rejected++;
                out->checksum += mix64((uint64_t)r * 0x9E3779B97F4A7C15ull ^ ~0ull);
                if (dump_finish) dump_finish[r] = -1;
                if (dump_first) dump_first[r] = -1;
                if (dump_inst) dump_inst[r] = -1;
                break;
            }
            if (best_tier == 0) { /* "map": prefill at the boundary, then occupy a slot */
                inst_t *in = &I[best_i];
                in->T += prefill_us(in, q->in_tokens);
                if (S == 1) {
                    complete(&c, best_i, (uint32_t)r, q->arrival_us, in->T, in->T, 1, q->cls, 0);
                } else {
                    uint32_t j = 0;
                    while (j < in->B && in->slots[j].used) j++;
                    if (j >= in->B) { c.bad = 1; break; }
                    slot_t *sl = &in->slots[j];
                    sl->used = 1; sl->req = (uint32_t)r; sl->arrival = q->arrival_us;
                    sl->first_tok = in->T; sl->fin_idx = in->K + S - 1; sl->S = (uint32_t)S;
                    sl->last_tok = in->T; sl->max_gap = 0;
                    sl->cls = q->cls;
                    in->w++;
                }
                break;
            }
            if (best_t0 <= now) c.bad = 1; /* a wait must move time strictly forward */
            now = best_t0;                 /* wait until that slot frees, then try again */
        }
    }
    if (!out->status)
        for (uint32_t i = 0; i < n_inst; i++) advance(&c, &I[i], i, -1); /* drain */
replay_done:
    free(I);

    if (!out->status) {
        if (out->n_counted != out->n_served + out->n_rejected) c.bad = 1; /* conservation */
        if (out->n_cascade != out->n_served - out->n_hit) c.bad = 1;
    }
    if (c.bad) out->status |= ORC_EINVARIANT;
    if (out->status) { /* invalid candidates carry a status and nothing else */
        uint32_t st = out->status;
        memset(out, 0, sizeof(*out));
        out->status = st;
    }
    return 0;
}

/* Score a batch: CSR offsets[n_cand+1] into inst[]; class_mask may be NULL.
 * dump_idx[dump_n] picks candidates whose per-request times are written to
 * dump_finish / dump_first / dump_inst, each [dump_n][n] (any may be NULL). */
int orc_eval_batch(const orc_profile *p, const orc_request *reqs, uint64_t n, const orc_slo *classes,
                   uint32_t n_classes, const uint32_t *offsets, const uint32_t *inst,
                   const uint32_t *class_mask, uint64_t n_cand, uint32_t budget, uint32_t flags,
                   orc_result *out, const uint32_t *dump_idx, uint32_t dump_n, int64_t *dump_finish,
                   int64_t *dump_first, int32_t *dump_inst) {
    for (uint64_t c = 0; c < n_cand; c++) {
        int64_t *df = NULL, *d1 = NULL; int32_t *di = NULL;
        for (uint32_t d = 0; d < dump_n; d++)
            if (dump_idx[d] == c) {
                if (dump_finish) df = dump_finish + (size_t)d * n;
                if (dump_first) d1 = dump_first + (size_t)d * n;
                if (dump_inst) di = dump_inst + (size_t)d * n;
            }
        int rc = orc_eval_candidate(p, reqs, n, classes, n_classes, inst + offsets[c],
                                    offsets[c + 1] - offsets[c], class_mask != NULL,
                                    class_mask ? class_mask[c] : 0, budget, flags, &out[c], df, d1, di);
        if (rc) return rc;
    }
    return 0;
}

/*
 * Composite serving score of Sec. IV-D:
 *   Phi = alpha * PhiS_n + beta * PhiT_n + (1 - beta) * PhiL_n
 *   PhiS_n = SLO satisfaction ratio            = n_hit / n_counted
 *   PhiT_n = min(PhiT, gamma_T) / gamma_T      PhiT = decoding throughput = tokens / makespan [tokens/s]
 *   PhiL_n = max(gamma_L - PhiL, 0) / gamma_L  PhiL = response latency = mean time to first token [s]
 * ("Evaluation Metrics", Sec. V-A, define throughput and response latency).
 * Readings: a placement that counted no request has PhiS_n = 0; one that served nothing has
 * PhiT_n = PhiL_n = 0; an invalid candidate scores -1.  Plain IEEE double arithmetic in the
 * order written, no fused operations.
 */
typedef struct { double alpha, beta, gamma_t, gamma_l; } orc_score_params;

int orc_score(const orc_result *res, uint64_t n, const orc_score_params *p, double *out) {
    for (uint64_t i = 0; i < n; i++) {
        const orc_result *r = &res[i];
        if (r->status != 0) { out[i] = -1.0; continue; }
        double phis = 0.0, phit = 0.0, phil = 0.0;
        if (r->n_counted > 0) phis = (double)r->n_hit / (double)r->n_counted;
        if (r->n_served > 0 && r->makespan_us > 0) {
            double thr = (double)r->tokens_out / ((double)r->makespan_us * 1e-6);
            double capped = thr < p->gamma_t ? thr : p->gamma_t;
            phit = capped / p->gamma_t;
        }
        if (r->n_served > 0) {
            double lat = ((double)r->sum_ttft_us / (double)r->n_served) * 1e-6;
            double room = p->gamma_l - lat;
            if (room < 0.0) room = 0.0;
            phil = room / p->gamma_l;
        }
        double a = p->alpha * phis;
        double b = p->beta * phit;
        double c = (1.0 - p->beta) * phil;
        out[i] = (a + b) + c;
    }
    return 0;
}

typedef struct { uint32_t strategy, batch; } orc_config;

/* Requests of each model left unserved (rejected) by every candidate: counted from the
 * per-request outcome, out[c][16]. */
int orc_rejected_by_model(const orc_profile *p, const orc_request *reqs, uint64_t n, const orc_slo *classes,
                          uint32_t n_classes, const uint32_t *offsets, const uint32_t *inst,
                          const uint32_t *class_mask, uint64_t n_cand, uint32_t budget, uint32_t flags,
                          uint32_t *out) {
    int32_t *where = (int32_t *)malloc((n ? n : 1) * sizeof(int32_t));
    if (!where) return -1;
    for (uint64_t c = 0; c < n_cand; c++) {
        orc_result r;
        int rc = orc_eval_candidate(p, reqs, n, classes, n_classes, inst + offsets[c], offsets[c + 1] - offsets[c],
                                    class_mask != NULL, class_mask ? class_mask[c] : 0, budget, flags, &r, NULL,
                                    NULL, where);
        if (rc) { free(where); return rc; }
        for (int m = 0; m < 16; m++) out[c * 16 + m] = 0;
        for (uint64_t q = 0; q < n; q++)
            if (where[q] == -1) out[c * 16 + reqs[q].model]++;
    }
    free(where);
    return 0;
}

/*
 * Histogram of the time to first token ("response latency", Sec. V-A "Evaluation Metrics")
 * of the requests a candidate served, for tail percentiles.  The paper reports the mean
 * only; the bins are this library's definition: bin 0 holds t < 1024 us; for t >= 1024,
 * with e = floor(log2 t) and h = the bit of t just below its leading one, the bin is
 * 1 + 2 (e - 10) + h, capped at 63 (two bins per octave, the last one open).
 * Computed from the per-request first-token times, out[c][64].
 */
static uint32_t orc_ttft_bin(int64_t t) {
    if (t < 1024) return 0;
    int e = 0;
    while ((t >> (e + 1)) != 0) e++;   /* floor(log2 t) */
    uint32_t h = (uint32_t)((t >> (e - 1)) & 1);
    uint32_t b = 1u + 2u * (uint32_t)(e - 10) + h;
    return b > 63u ? 63u : b;
}

int orc_ttft_hist(const orc_profile *p, const orc_request *reqs, uint64_t n, const orc_slo *classes,
                  uint32_t n_classes, const uint32_t *offsets, const uint32_t *inst,
                  const uint32_t *class_mask, uint64_t n_cand, uint32_t budget, uint32_t flags,
                  uint32_t *out) {
    int64_t *first = (int64_t *)malloc((n ? n : 1) * sizeof(int64_t));
    if (!first) return -1;
    for (uint64_t c = 0; c < n_cand; c++) {
        orc_result r;
        int rc = orc_eval_candidate(p, reqs, n, classes, n_classes, inst + offsets[c], offsets[c + 1] - offsets[c],
                                    class_mask != NULL, class_mask ? class_mask[c] : 0, budget, flags, &r, NULL,
                                    first, NULL);
        if (rc) { free(first); return rc; }
        for (int b = 0; b < 64; b++) out[c * 64 + b] = 0;
        if (r.status != 0) continue;
        for (uint64_t q = 0; q < n; q++)
            if (first[q] >= 0) out[c * 64 + orc_ttft_bin(first[q] - reqs[q].arrival_us)]++;
    }
    free(first);
    return 0;
}

/* Upper bound of the `permille`-th rank (1..1000) of one 64-bin histogram: the largest value
 * of the first bin at which the cumulative count reaches ceil(permille * total / 1000);
 * INT64_MAX in the open last bin, -1 for an empty histogram. */
int64_t orc_ttft_percentile(const uint32_t *hist, uint32_t permille) {
    uint64_t total = 0;
    for (int b = 0; b < 64; b++) total += hist[b];
    if (total == 0) return -1;
    uint64_t target = ((uint64_t)permille * total + 999) / 1000;
    if (target < 1) target = 1;
    uint64_t cum = 0;
    for (int b = 0; b < 64; b++) {
        cum += hist[b];
        if (cum >= target) {
            if (b == 0) return 1023;
            if (b == 63) return INT64_MAX;
            int e = 10 + (b - 1) / 2, h = (b - 1) & 1;
            /* bin b covers [2^e + h 2^(e-1), 2^e + (h+1) 2^(e-1) - 1] */
            return ((int64_t)1 << e) + (int64_t)(h + 1) * ((int64_t)1 << (e - 1)) - 1;
        }
    }
    return INT64_MAX;
}

/*
 * Alg. 1, "Simulator-Based Instance Configuration", taken literally.  For every configuration
 * (P, B) of the (already pruned) list: start from the empty placement; while GPUs remain and
 * some model is not saturated, add an instance (m', P, B) of the model m' with the most
 * unserved requests among the non-saturated ones (ties: lowest model index), evaluate the
 * serving score of the tentative placement on R_x with the simulator, accept it if the score
 * improved, otherwise mark m' saturated; record the best score and placement per GPU count.
 * As printed, k is the GPU count of the placement BEFORE the tentative instance is added;
 * that reading is kept.  A tentative placement that violates a constraint (budget, memory fit,
 * instance limit) scores -1 and is therefore never accepted.
 * R_x = requests whose class bit is set in class_mask (all if has_mask == 0).
 * Outputs: phi_star[gpus + 1], istar_len[gpus + 1], istar_inst[gpus + 1][128] (packed words).
 */
int orc_ins_deploy(const orc_profile *p, const orc_request *reqs, uint64_t n, const orc_slo *classes,
                   uint32_t n_classes, int has_mask, uint32_t class_mask, uint32_t gpus,
                   const orc_config *configs, uint32_t n_configs, const orc_score_params *sp, uint32_t flags,
                   double *phi_star, uint32_t *istar_len, uint32_t *istar_inst) {
    int32_t *where = (int32_t *)malloc((n ? n : 1) * sizeof(int32_t));
    if (!where) return -1;
    if (n_classes > 32) has_mask = 0;
    for (uint32_t k = 0; k <= gpus; k++) { phi_star[k] = 0.0; istar_len[k] = 0; }
    for (uint32_t c = 0; c < n_configs; c++) {
        uint32_t I[ORC_MAX_INST + 1], nI = 0;
        int sat[16] = {0};
        uint32_t unserved[16] = {0};
        double phi = 0.0;
        const uint32_t dev = (uint32_t)p->devices[configs[c].strategy];
        for (uint64_t q = 0; q < n; q++)  /* R_res = R_x: nothing is served yet */
            if (!has_mask || ((class_mask >> reqs[q].cls) & 1u)) unserved[reqs[q].model]++;
        for (;;) {
            if (nI * dev >= gpus) break;                      /* gpuCount(I) < |G_x| */
            int mp = -1;                                      /* mostUnservedModel over M \ M_sat */
            for (uint32_t m = 0; m < p->n_models; m++)
                if (!sat[m] && (mp < 0 || unserved[m] > unserved[mp])) mp = (int)m;
            if (mp < 0) break;                                /* M_sat == M */
            if (nI > ORC_MAX_INST) break;
            I[nI] = ((uint32_t)mp & 0xF) | ((configs[c].strategy & 0xFF) << 4) | ((configs[c].batch & 0xFF) << 12);
            orc_result r;
            int rc = orc_eval_candidate(p, reqs, n, classes, n_classes, I, nI + 1, has_mask, class_mask, gpus,
                                        flags, &r, NULL, NULL, where);
            if (rc) { free(where); return rc; }
            double phi2;
            orc_score(&r, 1, sp, &phi2);
            if (phi2 > phi) {                                 /* accept the new instance */
                phi = phi2;
                nI++;
                for (int m = 0; m < 16; m++) unserved[m] = 0;
                for (uint64_t q = 0; q < n; q++)
                    if (where[q] == -1) unserved[reqs[q].model]++;
            } else {
                sat[mp] = 1;                                  /* stop deploying m' */
            }
            /* Phi*[k], I*[k] hold "solutions for all possible GPU allocations k" (Sec. IV-E): k is the
             * device count of the placement that is stored, i.e. gpuCount(I) after the decision above.
             * (The listing takes k before the addition, which files an accepted placement under fewer
             * devices than it occupies; Alg. 2 then pairs placements that overrun the cluster.) */
            const uint32_t k = nI * dev;
            if (phi > phi_star[k]) {
                phi_star[k] = phi;
                istar_len[k] = nI;
                for (uint32_t i = 0; i < nI; i++) istar_inst[(size_t)k * ORC_MAX_INST + i] = I[i];
            }
        }
    }
    free(where);
    return 0;
}

/*
 * getPrunedConfigs of Alg. 1: the configuration tree of Sec. III-C with the two pruning rules
 * of Sec. IV-D.
 *  (1) Parallelism-strategy pruning, on the tables: strategy P is dropped if some other strategy Q
 *      needs no more devices, hosts every model that P hosts, and is at least as fast for those
 *      models (every decode level, prefill base and slope), i.e. P "fails to outperform" Q "while
 *      consuming" at least as many resources; identical rows on equal devices keep the lower
 *      index.  A strategy on which no model fits is dropped as well.
 *  (2) Batch-size pruning, by simulation on R_x: for each remaining strategy and each batch cap of
 *      the caller's list, a probe placement with one instance (m, P, B) of every model that fits is
 *      replayed; a batch cap is kept iff no other cap of the same strategy has at least as many SLO
 *      hits and at most the same mean response latency (time to first token, exact rational
 *      compare; nothing served = infinite latency) with one of the two strictly better: the
 *      Pareto front between latency and SLO satisfaction.  Equal outcomes keep the smaller cap.
 * Order of the result (in-order traversal of the tree = decreasing decode throughput): strategies
 * by increasing level-1 decode step of model 0 (ties: lower index), batch caps ascending.
 * out: (strategy, batch) pairs, *out_n of them; capacity n_strategies * n_batches.
 */
/* Q can stand in for S: every model that fits on S also fits on Q, and for those models Q is at
 * least as fast at every decode level and in prefill. */
static int orc_faster_or_equal(const orc_profile *p, uint32_t q, uint32_t s, int *strict) {
    for (uint32_t m = 0; m < p->n_models; m++) {
        if (p->devices[s] < p->min_devices[m]) continue;   /* S cannot host this model anyway */
        if (p->devices[q] < p->min_devices[m]) return 0;   /* Q cannot replace S for it */
        size_t rq = (size_t)m * p->n_strategies + q, rs = (size_t)m * p->n_strategies + s;
        if (p->prefill_base_us[rq] > p->prefill_base_us[rs]) return 0;
        if ((uint32_t)p->prefill_q16[rq] > (uint32_t)p->prefill_q16[rs]) return 0;
        if (p->prefill_base_us[rq] < p->prefill_base_us[rs] ||
            (uint32_t)p->prefill_q16[rq] < (uint32_t)p->prefill_q16[rs]) *strict = 1;
        for (uint32_t w = 0; w < p->wmax; w++) {
            if (p->step_us[rq * p->wmax + w] > p->step_us[rs * p->wmax + w]) return 0;
            if (p->step_us[rq * p->wmax + w] < p->step_us[rs * p->wmax + w]) *strict = 1;
        }
    }
    return 1;
}

int orc_prune_configs(const orc_profile *p, const orc_request *reqs, uint64_t n, const orc_slo *classes,
                      uint32_t n_classes, int has_mask, uint32_t class_mask, const uint32_t *batches,
                      uint32_t n_batches, uint32_t flags, orc_config *out, uint32_t *out_n) {
    uint32_t S = p->n_strategies;
    int *keep = (int *)calloc(S, sizeof(int));
    uint32_t *order = (uint32_t *)malloc(S * sizeof(uint32_t));
    orc_result *res = (orc_result *)malloc((size_t)(n_batches ? n_batches : 1) * sizeof(orc_result));
    if (!keep || !order || !res) { free(keep); free(order); free(res); return -1; }
    /* (1) strategy pruning */
    for (uint32_t s = 0; s < S; s++) {
        int fits = 0;
        for (uint32_t m = 0; m < p->n_models; m++) if (p->devices[s] >= p->min_devices[m]) fits = 1;
        keep[s] = fits;
        for (uint32_t q = 0; q < S && keep[s]; q++) {
            if (q == s || p->devices[q] > p->devices[s]) continue;
            int strict = 0;
            if (!orc_faster_or_equal(p, q, s, &strict)) continue;
            if (strict || p->devices[q] < p->devices[s] || q < s) keep[s] = 0;
        }
    }
    /* tree order: decreasing decode throughput = increasing level-1 step of model 0 */
    uint32_t ns = 0;
    for (uint32_t s = 0; s < S; s++) if (keep[s]) order[ns++] = s;
    for (uint32_t i = 1; i < ns; i++)
        for (uint32_t j = i; j > 0; j--) {
            uint32_t a = order[j - 1], b = order[j];
            int32_t sa = p->step_us[(size_t)a * p->wmax], sb = p->step_us[(size_t)b * p->wmax];
            if (sa > sb || (sa == sb && a > b)) { order[j - 1] = b; order[j] = a; } else break;
        }
    /* (2) batch pruning per strategy */
    *out_n = 0;
    int rc = 0;
    for (uint32_t i = 0; i < ns && !rc; i++) {
        uint32_t s = order[i];
        for (uint32_t b = 0; b < n_batches && !rc; b++) {
            uint32_t inst[16], ni = 0;
            for (uint32_t m = 0; m < p->n_models; m++)
                if (p->devices[s] >= p->min_devices[m]) inst[ni++] = (m & 0xF) | ((s & 0xFF) << 4) | ((batches[b] & 0xFF) << 12);
            rc = orc_eval_candidate(p, reqs, n, classes, n_classes, inst, ni, has_mask, class_mask, 0xFFFFFFFFu,
                                    flags, &res[b], NULL, NULL, NULL);
        }
        for (uint32_t b = 0; b < n_batches && !rc; b++) {
            int dominated = res[b].status != 0;
            for (uint32_t c = 0; c < n_batches && !dominated; c++) {
                if (c == b || res[c].status != 0) continue;
                /* latency compare: sum_b / served_b vs sum_c / served_c, nothing served = infinite */
                int lat_c_le, lat_c_lt;
                if (res[c].n_served == 0) { lat_c_le = res[b].n_served == 0; lat_c_lt = 0; }
                else if (res[b].n_served == 0) { lat_c_le = 1; lat_c_lt = 1; }
                else {
                    unsigned __int128 l = (unsigned __int128)(uint64_t)res[c].sum_ttft_us * res[b].n_served;
                    unsigned __int128 r = (unsigned __int128)(uint64_t)res[b].sum_ttft_us * res[c].n_served;
                    lat_c_le = l <= r; lat_c_lt = l < r;
                }
                int hit_c_ge = res[c].n_hit >= res[b].n_hit, hit_c_gt = res[c].n_hit > res[b].n_hit;
                if (hit_c_ge && lat_c_le && (hit_c_gt || lat_c_lt)) dominated = 1;
                else if (hit_c_ge && lat_c_le && !hit_c_gt && !lat_c_lt && batches[c] < batches[b]) dominated = 1;
            }
            if (!dominated) { out[*out_n].strategy = s; out[*out_n].batch = batches[b]; (*out_n)++; }
        }
    }
    free(keep); free(order); free(res);
    return rc;
}

/*
 * Alg. 2, "Dynamic Resource Partition", taken literally.  R_t / R_l = requests whose class bit
 * is set in mask_t / mask_l (byRequestSLO); G'_l = floor(|R_l| / |R| * |G|) with |R| = |R_t| + |R_l|
 * (integer arithmetic); Alg. 1 on (R_l, G'_l) and on (R_t, G); Phi_opt starts at the best
 * homogeneous score max_k Phi*[k] of Alg. 1 on (R, G) if `baseline` is set, else at 0; then for
 * g_l = 1 .. G'_l with g_t = |G| - g_l the pair maximising Phi_t*[g_t] + Phi_l*[g_l] is kept
 * (strictly better only).  Outputs: out_g[2] = (g_t, g_l), both 0 if no partition beat Phi_opt;
 * *out_phi = Phi_opt; placements of the chosen pair (lengths 0 if none).
 */
int orc_partition(const orc_profile *p, const orc_request *reqs, uint64_t n, const orc_slo *classes,
                  uint32_t n_classes, uint32_t mask_t, uint32_t mask_l, uint32_t gpus, const orc_config *configs,
                  uint32_t n_configs, const orc_score_params *sp, uint32_t flags, int baseline, uint32_t *out_g,
                  double *out_phi, uint32_t *len_t, uint32_t *inst_t, uint32_t *len_l, uint32_t *inst_l) {
    uint64_t n_t = 0, n_l = 0;
    for (uint64_t q = 0; q < n; q++) {
        if ((mask_t >> reqs[q].cls) & 1u) n_t++;
        if ((mask_l >> reqs[q].cls) & 1u) n_l++;
    }
    const uint32_t gl_max = (n_t + n_l) ? (uint32_t)((n_l * (uint64_t)gpus) / (n_t + n_l)) : 0;
    size_t cells = (size_t)gpus + 1;
    double *phi_t = (double *)malloc(cells * sizeof(double)), *phi_l = (double *)malloc(cells * sizeof(double));
    double *phi_h = (double *)malloc(cells * sizeof(double));
    uint32_t *ln_t = (uint32_t *)malloc(cells * 4), *ln_l = (uint32_t *)malloc(cells * 4), *ln_h = (uint32_t *)malloc(cells * 4);
    uint32_t *in_t = (uint32_t *)malloc(cells * ORC_MAX_INST * 4), *in_l = (uint32_t *)malloc(cells * ORC_MAX_INST * 4);
    uint32_t *in_h = (uint32_t *)malloc(cells * ORC_MAX_INST * 4);
    int rc = -1;
    if (phi_t && phi_l && phi_h && ln_t && ln_l && ln_h && in_t && in_l && in_h) {
        rc = orc_ins_deploy(p, reqs, n, classes, n_classes, 1, mask_l, gl_max, configs, n_configs, sp, flags, phi_l, ln_l, in_l);
        if (!rc) rc = orc_ins_deploy(p, reqs, n, classes, n_classes, 1, mask_t, gpus, configs, n_configs, sp, flags, phi_t, ln_t, in_t);
        double phi_opt = 0.0;
        if (!rc && baseline) {
            rc = orc_ins_deploy(p, reqs, n, classes, n_classes, 1, mask_t | mask_l, gpus, configs, n_configs, sp, flags, phi_h, ln_h, in_h);
            for (uint32_t k = 0; !rc && k <= gpus; k++) if (phi_h[k] > phi_opt) phi_opt = phi_h[k];
        }
        if (!rc) {
            out_g[0] = out_g[1] = 0; *len_t = *len_l = 0;
            for (uint32_t gl = 1; gl <= gl_max; gl++) {
                const uint32_t gt = gpus - gl;
                if (phi_t[gt] + phi_l[gl] > phi_opt) {
                    phi_opt = phi_t[gt] + phi_l[gl];
                    out_g[0] = gt; out_g[1] = gl;
                    *len_t = ln_t[gt]; *len_l = ln_l[gl];
                    memcpy(inst_t, in_t + (size_t)gt * ORC_MAX_INST, ln_t[gt] * 4);
                    memcpy(inst_l, in_l + (size_t)gl * ORC_MAX_INST, ln_l[gl] * 4);
                }
            }
            *out_phi = phi_opt;
        }
    }
    free(phi_t); free(phi_l); free(phi_h); free(ln_t); free(ln_l); free(ln_h); free(in_t); free(in_l); free(in_h);
    return rc;
}

/* Ranking by score (order 1): higher score first, then lower index; NaN scores last. */
static const double *g_score;
static int cmp_score(const void *pa, const void *pb) {
    uint32_t a = *(const uint32_t *)pa, b = *(const uint32_t *)pb;
    double x = g_score[a], y = g_score[b];
    int nx = x != x, ny = y != y;
    if (nx != ny) return nx ? 1 : -1;
    if (!nx && x != y) return x > y ? -1 : 1;
    return a < b ? -1 : (a > b ? 1 : 0);
}
int orc_topk_scores(const double *scores, uint64_t n, uint32_t k, uint32_t *out_idx) {
    uint32_t *idx = (uint32_t *)malloc((n ? n : 1) * sizeof(uint32_t));
    if (!idx) return -1;
    for (uint64_t i = 0; i < n; i++) idx[i] = (uint32_t)i;
    g_score = scores;
    qsort(idx, n, sizeof(uint32_t), cmp_score);
    for (uint64_t i = 0; i < k && i < n; i++) out_idx[i] = idx[i];
    free(idx);
    return 0;
}

/*
 * Ranking used for "keep the best placements" (order 0): valid candidates first; more SLO
 * hits first; then lower mean time-to-first-token, sum/n_served compared exactly by
 * cross-multiplication in 128 bits (a candidate that served nothing ranks after any that
 * served something); then lower candidate index.
 */
static const orc_result *g_res;
static int before(uint32_t a, uint32_t b) {
    const orc_result *x = &g_res[a], *y = &g_res[b];
    int vx = x->status == 0, vy = y->status == 0;
    if (vx != vy) return vx > vy;
    if (vx) {
        if (x->n_hit != y->n_hit) return x->n_hit > y->n_hit;
        int sx = x->n_served > 0, sy = y->n_served > 0;
        if (sx != sy) return sx > sy;
        if (sx) {
            unsigned __int128 l = (unsigned __int128)(uint64_t)x->sum_ttft_us * y->n_served;
            unsigned __int128 r = (unsigned __int128)(uint64_t)y->sum_ttft_us * x->n_served;
            if (l != r) return l < r;
        }
    }
    return a < b;
}
static int cmp(const void *pa, const void *pb) {
    uint32_t a = *(const uint32_t *)pa, b = *(const uint32_t *)pb;
    if (a == b) return 0;
    return before(a, b) ? -1 : 1;
}
/* out_idx[min(k, n)] = indices of the k best candidates, best first. */
int orc_topk(const orc_result *res, uint64_t n, uint32_t k, uint32_t order, uint32_t *out_idx) {
    if (order != 0) return -1;
    uint32_t *idx = (uint32_t *)malloc((n ? n : 1) * sizeof(uint32_t));
    if (!idx) return -1;
    for (uint64_t i = 0; i < n; i++) idx[i] = (uint32_t)i;
    g_res = res;
    qsort(idx, n, sizeof(uint32_t), cmp);
    for (uint64_t i = 0; i < k && i < n; i++) out_idx[i] = idx[i];
    free(idx);
    return 0;
}
