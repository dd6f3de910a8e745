"""Seeded synthetic request traces.

Draw order is fixed: inter-arrival gaps, input lengths, output lengths, SLO class,
model, then the long-output redraw for the document class.
"""
import numpy as np
from .formats import REQUEST_DTYPE


def make_trace(n, rate, seed, *, cv=1.0, class_mix=(0.5, 0.3, 0.2), model_mix=(1.0,),
               in_dist=("lognormal", 6.0, 0.8, 16, 4096),
               out_dist=("lognormal", 4.5, 1.0, 1, 2048),
               doc_class=2, doc_out=(2048, 8192)):
    """n requests; gamma inter-arrival gaps with mean 1/rate seconds and the given
    coefficient of variation (cv = 1 is a Poisson process).

    in_dist / out_dist: ("lognormal", mu, sigma, lo, hi) or ("pareto", alpha, xmin, lo, hi).
    Requests of class `doc_class` (None to disable) redraw their output length
    uniformly in doc_out (inclusive)."""
    rng = np.random.default_rng(seed)
    shape = 1.0 / (cv * cv)
    gaps = rng.gamma(shape, 1.0 / (rate * shape), size=n)
    arrival = np.floor(np.cumsum(gaps) * 1e6).astype(np.int64)

    def draw(dist):
        kind = dist[0]
        if kind == "lognormal":
            _, mu, sigma, lo, hi = dist
            x = rng.lognormal(mu, sigma, size=n)
        elif kind == "pareto":
            _, alpha, xmin, lo, hi = dist
            x = xmin * (1.0 + rng.pareto(alpha, size=n))
        else:
            raise ValueError(kind)
        return np.clip(np.floor(x + 0.5), lo, hi).astype(np.int64)

    in_tok = draw(in_dist)
    out_tok = draw(out_dist)
    cls = rng.choice(len(class_mix), size=n, p=np.asarray(class_mix) / np.sum(class_mix))
    model = rng.choice(len(model_mix), size=n, p=np.asarray(model_mix) / np.sum(model_mix))
    if doc_class is not None:
        redraw = rng.integers(doc_out[0], doc_out[1] + 1, size=n)
        out_tok = np.where(cls == doc_class, redraw, out_tok)

    t = np.zeros(n, dtype=REQUEST_DTYPE)
    t["arrival_us"] = arrival
    t["in_tokens"] = in_tok
    t["out_tokens"] = out_tok
    t["cls"] = cls
    t["model"] = model
    return t


def trace_from_rows(rows):
    """rows: (arrival_us, in_tokens, out_tokens, cls, model) per request, in arrival order."""
    t = np.zeros(len(rows), dtype=REQUEST_DTYPE)
    for k, (a, n_in, n_out, c, m) in enumerate(rows):
        t[k] = (a, n_in, n_out, c, m)
    return t


def shrinking_prompts_trace(n_followers=40, spacing_us=30_000, first_prompt=90_000, prompt_step=2_000,
                            long_out=6_000, follower_out=(150, 900), n_classes=3):
    """One long-running request, then followers whose prompts shrink from one to the next while all of
    them keep running: with a prefill time that falls faster than the decode step grows, every
    admission stalls the batch for a little less than the one before."""
    rows = [(0, 100, long_out, n_classes - 1, 0)]
    for k in range(n_followers):
        rows.append(((k + 1) * spacing_us, first_prompt - k * prompt_step,
                     follower_out[0] + (k * 37) % (follower_out[1] - follower_out[0]), k % n_classes, 0))
    return trace_from_rows(rows)
