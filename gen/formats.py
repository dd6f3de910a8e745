"""Binary layouts shared by every consumer of the synthetic inputs.

Only layouts and bit packing live here; nothing in this file simulates anything.
"""
import numpy as np

WMAX = 64            # largest batch cap a latency table covers
MAX_INSTANCES = 128  # most instances one candidate placement may hold
SLO_NONE = -1        # "no limit" marker for an SLO term (any negative value)

# One request of the trace: 16 bytes, sorted by (arrival, index).
REQUEST_DTYPE = np.dtype([
    ("arrival_us", "<i8"),
    ("in_tokens", "<u4"),
    ("out_tokens", "<u2"),
    ("cls", "u1"),
    ("model", "u1"),
])
assert REQUEST_DTYPE.itemsize == 16

# One SLO class: limits in microseconds, negative = no limit.
SLO_DTYPE = np.dtype([("ttft_us", "<i8"), ("tbt_us", "<i8"), ("e2e_us", "<i8")])
assert SLO_DTYPE.itemsize == 24

# Per-candidate result record: 128 bytes, all integer.
RESULT_DTYPE = np.dtype([
    ("status", "<u4"),
    ("n_counted", "<u4"),
    ("n_served", "<u4"),
    ("n_hit", "<u4"),
    ("n_rejected", "<u4"),
    ("n_cascade", "<u4"),
    ("hit_by_class", "<u4", (8,)),
    ("sum_ttft_us", "<i8"),
    ("max_ttft_us", "<i8"),
    ("sum_e2e_us", "<i8"),
    ("max_e2e_us", "<i8"),
    ("makespan_us", "<i8"),
    ("tokens_out", "<u8"),
    ("checksum", "<u8"),
    ("attempts", "<u8"),
    ("reserved", "<u8"),
])
assert RESULT_DTYPE.itemsize == 128


def pack_inst(model, strategy, batch):
    """Pack (model, strategy, batch cap) into the 32-bit instance word.

    bits 0-3 model, bits 4-11 strategy, bits 12-19 batch cap, bits 20-31 zero.
    """
    model = np.asarray(model, dtype=np.uint32)
    strategy = np.asarray(strategy, dtype=np.uint32)
    batch = np.asarray(batch, dtype=np.uint32)
    return (model & 0xF) | ((strategy & 0xFF) << 4) | ((batch & 0xFF) << 12)


def unpack_inst(word):
    word = np.asarray(word, dtype=np.uint32)
    return word & 0xF, (word >> 4) & 0xFF, (word >> 12) & 0xFF


def make_classes(rows):
    """rows: iterable of (ttft_us, tbt_us, e2e_us); None means no limit."""
    out = np.zeros(len(rows), dtype=SLO_DTYPE)
    for k, (a, b, c) in enumerate(rows):
        out[k] = (SLO_NONE if a is None else a,
                  SLO_NONE if b is None else b,
                  SLO_NONE if c is None else c)
    return out
