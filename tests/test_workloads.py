"""The seeded input generators: shapes, dtypes, determinism, and the structure each config promises."""
import numpy as np
import pytest

from paper_2606_01927_b200 import workloads as W


def test_bf16_rounding_is_nearest_even():
    x = np.array([1.0, 1.00390625, 1.005859375, 1.01171875, -2.5, 3.0e38, 0.0], dtype=np.float32)
    b = W.f32_to_bf16_bits(x)
    back = W.bf16_bits_to_f32(b)
    assert back[0] == 1.0 and back[4] == -2.5 and back[6] == 0.0
    # 1 + 2^-8 is a tie between 1 and 1 + 2^-7: ties go to the even mantissa (1.0)
    assert back[1] == 1.0
    # 1 + 3*2^-9 is above the midpoint: rounds up
    assert back[2] == np.float32(1.0078125)
    assert back[3] == np.float32(1.015625) or back[3] == np.float32(1.0078125)
    assert np.all(np.abs(back[:4] - x[:4]) <= 2.0 ** -8)


@pytest.mark.parametrize("name,B,V,dtype", [
    ("config1", 8, 32000, W.F32), ("config2", 128, 152064, W.BF16), ("configM", 256, 152064, W.BF16),
    ("config3", 256, 128256, W.BF16), ("config4", 512, 152064, W.BF16), ("config5", 1024, 129280, W.F32)])
def test_config_shapes(name, B, V, dtype):
    small = dict(B=4) if name != "config1" else {}
    w = W.make(name, **small)
    assert w.V == V and w.dtype == dtype
    assert w.logits.shape == (w.B, V)
    assert w.logits.dtype == (np.float32 if dtype == W.F32 else np.uint16)
    full_B = {"config1": 8}.get(name, None)
    if full_B:
        assert w.B == B
    for a in (w.temperature, w.top_k, w.top_p, w.min_p, w.seeds):
        assert a is None or a.shape == (w.B,)
    if w.history_ids is not None:
        assert w.history_offsets.shape == (w.B + 1,) and w.history_offsets[0] == 0
        assert w.history_offsets[-1] == w.history_ids.size
        assert w.history_ids.min() >= 0 and w.history_ids.max() < V


def test_generators_are_deterministic():
    a, b = W.config3(B=3, V=5000, hist_len=100), W.config3(B=3, V=5000, hist_len=100)
    assert (a.logits == b.logits).all() and (a.history_ids == b.history_ids).all()


def test_config4_row_classes_and_config5_special_rows():
    w = W.config4(B=16, V=4000, max_hist=50)
    cls = np.arange(16) % 4
    assert (w.temperature[cls == 0] == 0).all() and (w.temperature[cls != 0] > 0).all()
    assert ((w.top_k[cls == 1] >= 1) & (w.top_k[cls == 1] <= 100)).all() and (w.top_k[cls != 1] == 0).all()
    assert (w.top_p[cls != 2] == 1).all() and (w.min_p[cls != 3] == 0).all()
    w5 = W.config5(B=102, V=3000, hist_len=10)
    assert w5.logits[0].std() < 0.05 and w5.logits[100].std() < 0.05
    assert w5.logits[1].max() > 25 and w5.num_top == 20


def test_zipf_history_prefers_low_ids():
    w = W.config3(B=2, V=50000, hist_len=4000)
    assert np.median(w.history_ids) < 2000


def test_rows_keeps_global_row_ids_and_history():
    w = W.config3(B=6, V=3000, hist_len=20)
    part = w.rows(2, 5)
    assert part.B == 3 and part.row_base == 2
    assert (part.history_offsets == np.array([0, 20, 40, 60])).all()
    assert (part.history_ids == w.history_ids[40:100]).all()


def test_bench_gpus_n_spawns_one_rank_per_gpu(monkeypatch):
    """`bench.py --gpus N` run plainly hands itself to torch.distributed.run with N ranks on 127.0.0.1."""
    import importlib.util
    import os
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    spec = importlib.util.spec_from_file_location("bench_under_test", os.path.join(root, "bench.py"))
    bench = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(bench)
    seen = {}
    monkeypatch.setattr(subprocess, "call", lambda cmd: seen.setdefault("cmd", cmd) and 0)
    monkeypatch.setattr(sys, "argv", ["bench.py", "--gpus", "2", "--steps", "5", "--warmup", "3"])
    try:
        bench.spawn_ranks(2)
    except SystemExit as e:
        assert e.code == 0
    cmd = seen["cmd"]
    assert cmd[1:4] == ["-m", "torch.distributed.run", "--nnodes=1"] and "--nproc-per-node=2" in cmd
    assert cmd[cmd.index("--master-addr") + 1] == "127.0.0.1"
    assert cmd[-6:] == ["--gpus", "2", "--steps", "5", "--warmup", "3"] and cmd[-7].endswith("bench.py")


def test_bench_helpers_percentile_traffic_and_bytes():
    """The small pure functions behind the bench line: percentiles, the ncu traffic data file, algorithmic bytes."""
    import importlib.util
    import json
    import os
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    spec = importlib.util.spec_from_file_location("bench_under_test2", os.path.join(root, "bench.py"))
    bench = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(bench)
    xs = [5.0, 1.0, 3.0, 2.0, 4.0]
    assert bench.percentile(xs, 0.0) == 1.0 and bench.percentile(xs, 1.0) == 5.0 and bench.percentile(xs, 0.5) == 3.0
    assert abs(bench.percentile(xs, 0.1) - 1.4) < 1e-12 and bench.percentile([], 0.5) is None
    data = json.load(open(os.path.join(root, "profiles", "ncu_traffic.json")))
    for name, rec in data.items():
        assert bench.ncu_traffic(name) == rec["dram_bytes_per_launch"]
        assert os.path.exists(os.path.join(root, rec["source"]))
        w = W.make(name)
        # captured DRAM traffic is the algorithmic bytes plus a few per cent at most: every logit is read once
        assert 1.0 <= rec["dram_bytes_per_launch"] / bench.algorithmic_bytes(w) < 1.03, name
    assert bench.ncu_traffic("no-such-workload") is None
    w = W.make("configM")
    assert bench.algorithmic_bytes(w) == w.B * w.V * 2 + w.B * (4 * 3 + 16)      # logits + T, top_k, top_p + seed + outputs
