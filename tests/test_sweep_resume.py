"""Resumable chunked sweeps: bookkeeping only, scoring injected (the CPU oracle here)."""
import os

import numpy as np
import pytest

import gen


def test_chunked_sweep_resumes_where_it_stopped(tmp_path, oracle_mod):
    from paper_2509_06362_b200.sweep import chunked_sweep, chunk_ranges
    cfg = gen.make_config("tiny", n_req=120)
    mask = np.random.default_rng(2).integers(1, 8, size=143).astype(np.uint32)
    calls = []

    def score(off, inst, m):
        calls.append(len(off) - 1)
        if len(calls) == 3 and fail[0]:
            raise RuntimeError("interrupted")          # the run dies in its third range
        return oracle_mod.eval_placements(cfg["profile"], cfg["traces"][0], cfg["classes"], off, inst, cfg["budget"], m)

    fail = [True]
    with pytest.raises(RuntimeError):
        chunked_sweep(score, cfg["offsets"], cfg["inst"], 40, str(tmp_path), mask)
    assert calls == [40, 40, 40]
    assert sorted(os.listdir(tmp_path)) == ["chunk_000000000_000000040.npy", "chunk_000000040_000000080.npy"]
    # a truncated file of a later range must not be taken for a finished one
    (tmp_path / "chunk_000000120_000000143.npy").write_bytes(b"\x93NUMPY garbage")
    fail[0] = False
    calls.clear()
    seen = []
    rec, scored, resumed = chunked_sweep(score, cfg["offsets"], cfg["inst"], 40, str(tmp_path), mask,
                                         on_chunk=lambda lo, hi, r: seen.append((lo, hi, r)))
    assert calls == [40, 23] and (scored, resumed) == (2, 2)
    assert seen == [(0, 40, True), (40, 80, True), (80, 120, False), (120, 143, False)]
    want = oracle_mod.eval_placements(cfg["profile"], cfg["traces"][0], cfg["classes"], cfg["offsets"], cfg["inst"],
                                      cfg["budget"], mask)
    assert rec.tobytes() == want.tobytes()
    # a third run scores nothing
    calls.clear()
    rec2, scored, resumed = chunked_sweep(score, cfg["offsets"], cfg["inst"], 40, str(tmp_path), mask)
    assert calls == [] and (scored, resumed) == (0, 4) and rec2.tobytes() == want.tobytes()
    assert chunk_ranges(0, 5) == [] and chunk_ranges(5, 5) == [(0, 5)] and chunk_ranges(6, 5) == [(0, 5), (5, 6)]
