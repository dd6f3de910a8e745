"""A second, deliberately different formulation of the trace replay, for tiny inputs.

It decodes token by token: every instance keeps, for each running request, the number of
tokens still to produce, and its clock moves one decode step at a time.  There is no
step counter, no completion index and no multi-step jump, so a mistake in the
event-jump arithmetic of the C oracle (ceil-division, the minimum over completion
indices, the completion test) shows up as a disagreement.  Pure Python, exact integers.
Used only by the CPU tests as a pin for the oracle.
"""
from fractions import Fraction


class _Inst:
    def __init__(self, model, step, base, q16, cap):
        self.model, self.step, self.base, self.q16, self.cap = model, step, base, q16, cap
        self.clock = 0
        self.running = []  # dicts: req, arrival, first, left, S, cls

    def prefill(self, in_tokens):
        return self.base + ((self.q16 * in_tokens + 32768) >> 16)

    def one_step(self, done):
        self.clock += int(self.step[len(self.running) - 1])
        keep = []
        for r in self.running:
            r["stamps"].append(self.clock)    # every running request gets a token at the end of the step
            r["left"] -= 1
            if r["left"] == 0:
                done(r, self.clock)
            else:
                keep.append(r)
        self.running = keep

    def run_until(self, t, done):
        while self.running and self.clock < t:
            self.one_step(done)
        if not self.running and self.clock < t:
            self.clock = t

    def next_free_time(self):
        """time at which the first running request ends if nobody else is admitted"""
        left = min(r["left"] for r in self.running)
        return self.clock + left * int(self.step[len(self.running) - 1])


def simulate(profile, trace, classes, instances, class_mask=None, optimistic=False, maxgap=False):
    """instances: list of (model, strategy, batch).  Returns a dict of statistics and
    per-request lists finish / first / inst (-1 rejected, -2 not counted).
    maxgap: the TBT term looks at the largest difference between consecutive token timestamps."""
    S_ = profile["n_strategies"]
    insts = []
    for (m, s, b) in instances:
        insts.append(_Inst(m, profile["step_us"][m][s], int(profile["prefill_base_us"][m][s]),
                           int(profile["prefill_q16"][m][s]) & 0xFFFFFFFF, b))
    n = len(trace)
    finish, first, where = [-2] * n, [-2] * n, [-2] * n
    st = dict(n_counted=0, n_served=0, n_hit=0, n_rejected=0, n_cascade=0, sum_ttft_us=0,
              max_ttft_us=0, sum_e2e_us=0, max_e2e_us=0, makespan_us=0, tokens_out=0, attempts=0)

    def lim(v):
        return None if v < 0 else int(v)

    def done_on(idx):
        def done(r, t):
            c = classes[r["cls"]]
            ttft, e2e, span = r["first"] - r["arrival"], t - r["arrival"], t - r["first"]
            if maxgap:
                ts = r["stamps"]
                worst = max([b - a for a, b in zip(ts, ts[1:])], default=0)
                tbt_ok = lim(c["tbt_us"]) is None or worst <= lim(c["tbt_us"])
            else:
                tbt_ok = (lim(c["tbt_us"]) is None or r["S"] == 1 or
                          Fraction(span, r["S"] - 1) <= lim(c["tbt_us"]))
            ok = ((lim(c["ttft_us"]) is None or ttft <= lim(c["ttft_us"])) and tbt_ok and
                  (lim(c["e2e_us"]) is None or e2e <= lim(c["e2e_us"])))
            st["n_served"] += 1
            st["n_hit"] += ok
            st["n_cascade"] += (not ok)
            st["sum_ttft_us"] += ttft
            st["max_ttft_us"] = max(st["max_ttft_us"], ttft)
            st["sum_e2e_us"] += e2e
            st["max_e2e_us"] = max(st["max_e2e_us"], e2e)
            st["makespan_us"] = max(st["makespan_us"], t)
            st["tokens_out"] += r["S"]
            finish[r["req"]], first[r["req"]], where[r["req"]] = t, r["first"], idx
        return done

    now = 0
    for k in range(n):
        q = trace[k]
        cls, S, arrival = int(q["cls"]), int(q["out_tokens"]), int(q["arrival_us"])
        if class_mask is not None and len(classes) <= 32 and not (class_mask >> cls) & 1:
            continue
        st["n_counted"] += 1
        now = max(now, arrival)
        c = classes[cls]
        while True:
            st["attempts"] += 1
            for idx, ins in enumerate(insts):
                ins.run_until(now, done_on(idx))
            options = []
            for idx, ins in enumerate(insts):
                if ins.model != int(q["model"]):
                    continue
                free = len(ins.running) < ins.cap
                start = ins.clock if free else ins.next_free_time()
                level = ins.cap
                if optimistic and free:
                    level = min(ins.cap, len(ins.running) + 1)
                per_tok = int(ins.step[level - 1])
                t_first = start + ins.prefill(int(q["in_tokens"]))
                t_end = t_first + (S - 1) * per_tok
                if lim(c["ttft_us"]) is not None and t_first - arrival > lim(c["ttft_us"]):
                    continue
                if lim(c["tbt_us"]) is not None and S > 1 and per_tok > lim(c["tbt_us"]):
                    continue
                if lim(c["e2e_us"]) is not None and t_end - arrival > lim(c["e2e_us"]):
                    continue
                options.append((0 if free else 1, t_first, idx, start))
            if not options:
                st["n_rejected"] += 1
                finish[k] = first[k] = where[k] = -1
                break
            tier, t_first, idx, start = min(options)
            if tier == 0:
                ins = insts[idx]
                ins.clock += ins.prefill(int(q["in_tokens"]))
                rec = dict(req=k, arrival=arrival, first=ins.clock, left=S - 1, S=S, cls=cls, stamps=[ins.clock])
                if S == 1:
                    done_on(idx)(rec, ins.clock)
                else:
                    ins.running.append(rec)
                break
            now = start
    for idx, ins in enumerate(insts):
        while ins.running:
            ins.one_step(done_on(idx))
    st.update(finish_us=finish, first_us=first, inst=where)
    return st


def simulate_frozen(profile, trace, classes, instances, class_mask=None, optimistic=False, maxgap=False,
                    queues=False):
    """The engine that fixes a request's decode speed at admission, in a formulation that
    shares nothing with the C oracle's: no slots at all.  Every instance keeps the list of
    token timestamps of the requests admitted to it (one list per request, built token by
    token); the running count at time t is the number of lists whose last entry is after t."""
    insts = []
    for (m, s, b) in instances:
        insts.append(dict(model=m, step=[int(x) for x in profile["step_us"][m][s]],
                          base=int(profile["prefill_base_us"][m][s]),
                          q16=int(profile["prefill_q16"][m][s]) & 0xFFFFFFFF, cap=b, tokens=[]))
    n = len(trace)
    finish, first, where = [-2] * n, [-2] * n, [-2] * n
    st = dict(n_counted=0, n_served=0, n_hit=0, n_rejected=0, n_cascade=0, sum_ttft_us=0,
              max_ttft_us=0, sum_e2e_us=0, max_e2e_us=0, makespan_us=0, tokens_out=0, attempts=0)

    def lim(v):
        return None if v < 0 else int(v)

    def ends_after(ins, t):
        return [tok[-1] for tok in ins["tokens"] if tok[-1] > t]

    t_now = 0
    for k in range(n):
        q = trace[k]
        cls, S, arrival, n_in = int(q["cls"]), int(q["out_tokens"]), int(q["arrival_us"]), int(q["in_tokens"])
        if class_mask is not None and len(classes) <= 32 and not (class_mask >> cls) & 1:
            continue
        st["n_counted"] += 1
        t_now = max(t_now, arrival)
        c = classes[cls]
        while True:
            st["attempts"] += 1
            options = []
            for idx, ins in enumerate(insts):
                if ins["model"] != int(q["model"]):
                    continue
                alive = ends_after(ins, t_now)
                free = len(alive) < ins["cap"]
                # full: a place frees when fewer than cap of the requests sent here so far are unfinished
                # (first come first served; with queues some of them have not even started yet)
                start = t_now if free else sorted(alive)[-ins["cap"]]
                per_tok = ins["step"][ins["cap"] - 1]
                if optimistic and free:
                    per_tok = ins["step"][len(alive)]          # level len(alive) + 1
                t_first = start + ins["base"] + ((ins["q16"] * n_in + 32768) >> 16)
                t_end = t_first + (S - 1) * per_tok
                if lim(c["ttft_us"]) is not None and t_first - arrival > lim(c["ttft_us"]):
                    continue
                if lim(c["tbt_us"]) is not None and S > 1 and per_tok > lim(c["tbt_us"]):
                    continue
                if lim(c["e2e_us"]) is not None and t_end - arrival > lim(c["e2e_us"]):
                    continue
                options.append((0 if free else 1, t_first, idx, start))
            if not options:
                st["n_rejected"] += 1
                finish[k] = first[k] = where[k] = -1
                break
            tier, _, idx, start = min(options)
            if tier == 1 and not queues:
                t_now = start
                continue
            ins = insts[idx]
            t_adm = t_now if tier == 0 else start               # queued: starts when that request ends
            gap = ins["step"][len(ends_after(ins, t_adm))]      # fixed for the whole request
            stamps = [t_adm + ins["base"] + ((ins["q16"] * n_in + 32768) >> 16)]
            for _ in range(S - 1):
                stamps.append(stamps[-1] + gap)
            ins["tokens"].append(stamps)
            t_first, t_end = stamps[0], stamps[-1]
            ttft, e2e = t_first - arrival, t_end - arrival
            if maxgap:
                worst = max([b - a for a, b in zip(stamps, stamps[1:])], default=0)
                tbt_ok = lim(c["tbt_us"]) is None or worst <= lim(c["tbt_us"])
            else:
                tbt_ok = lim(c["tbt_us"]) is None or S == 1 or Fraction(t_end - t_first, S - 1) <= lim(c["tbt_us"])
            ok = ((lim(c["ttft_us"]) is None or ttft <= lim(c["ttft_us"])) and tbt_ok and
                  (lim(c["e2e_us"]) is None or e2e <= lim(c["e2e_us"])))
            st["n_served"] += 1
            st["n_hit"] += ok
            st["n_cascade"] += (not ok)
            st["sum_ttft_us"] += ttft
            st["max_ttft_us"] = max(st["max_ttft_us"], ttft)
            st["sum_e2e_us"] += e2e
            st["max_e2e_us"] = max(st["max_e2e_us"], e2e)
            st["makespan_us"] = max(st["makespan_us"], t_end)
            st["tokens_out"] += S
            finish[k], first[k], where[k] = t_end, t_first, idx
            break
    st.update(finish_us=finish, first_us=first, inst=where)
    return st
