"""The profiled constants of bench.py: they are printed only for the kernel sources they were taken
from (a hash of csrc/ stored beside them), and they must be the figures of the committed ncu summary."""
import os
import re
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def test_profiled_constants_match_the_committed_summary():
    import bench
    p = bench.PROFILED
    if p is None:
        return
    assert set(p) >= {"workload", "mapping", "kernel", "warp_inst_per_launch", "dram_bytes_per_launch", "csrc_sha256"}
    assert re.fullmatch(r"[0-9a-f]{64}", p["csrc_sha256"])
    text = open(os.path.join(ROOT, "profiles", "eval_thread_kernel_multimodel_sweep_counters.md")).read()
    num = lambda key: int(re.search(re.escape(key) + r" \| ([0-9,]+)", text).group(1).replace(",", ""))
    assert num("smsp__inst_executed.sum") == p["warp_inst_per_launch"]
    assert num("dram__bytes_read.sum") + num("dram__bytes_write.sum") == p["dram_bytes_per_launch"]


def test_source_hash_sees_every_kernel_file(tmp_path, monkeypatch):
    import bench
    h0 = bench.csrc_sha256()
    assert re.fullmatch(r"[0-9a-f]{64}", h0) and h0 == bench.csrc_sha256()
    # the hash covers names and contents of all .cu / .cuh files: a copy with one byte more differs
    src = os.path.join(ROOT, "paper_2509_06362_b200", "csrc")
    dst = tmp_path / "paper_2509_06362_b200" / "csrc"
    dst.mkdir(parents=True)
    for name in os.listdir(src):
        if name.endswith((".cu", ".cuh")):
            (dst / name).write_bytes(open(os.path.join(src, name), "rb").read())
    monkeypatch.setattr(bench, "ROOT", str(tmp_path))
    assert bench.csrc_sha256() == h0
    with open(dst / "eval_thread.cu", "ab") as f:
        f.write(b"\n")
    assert bench.csrc_sha256() != h0
