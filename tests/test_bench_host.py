"""Host-side logic of bench.py that needs no GPU: region statistics, byte accounting, the config object
both arms print, the clock sampler's parsing and windowing."""
import datetime
import importlib.util
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
spec = importlib.util.spec_from_file_location("bench_module", os.path.join(ROOT, "bench.py"))
bench = importlib.util.module_from_spec(spec)
sys.modules["bench_module"] = bench
spec.loader.exec_module(bench)

from paper_2604_02292_b200 import workloads  # noqa: E402


def test_region_stats_take_the_median_region():
    st = bench.region_stats([2.0, 1.0, 9.0, 1.2, 1.1], steps=10)
    assert st["ms_per_step"] == 0.12 and st["ms_per_step_min"] == 0.1 and st["ms_per_step_max"] == 0.9
    assert st["repeats"] == 5


def test_algorithmic_bytes_of_a_causal_workload():
    wl = workloads.make_config(3, batch=2)
    Bt, H, Lq, Lk = wl.shape
    n = Bt * H * Lq * Lk
    assert bench.algorithmic_bytes(wl, True) == 2 * n                      # the metric's flat 2 B/element
    valid = Bt * H * (Lq * (Lq + 1) // 2)                                   # square causal head: i + 1 keys in row i
    assert bench.algorithmic_bytes(wl, False) == valid + n
    plain = workloads.make_config(2, batch=2)
    assert bench.algorithmic_bytes(plain, False) == 2 * plain.elements


def test_both_arms_print_the_same_config_object():
    wl = workloads.make_config(2, batch=3)
    a = bench.config_dict(wl, "u8div")
    b = bench.config_dict(workloads.make_config(2, batch=3), "u8div")
    assert a == b and a["workload"] == "config2" and a["flags"] == 0 and a["mode"] == "u8div"
    assert bench.config_dict(wl, "u16clb")["flags"] == 3
    c3 = bench.config_dict(workloads.make_config(3, batch=1), "u8clb")
    assert c3["flags"] == 4 | 2


def test_buffer_sets_exceed_l2():
    for c, batch in ((1, None), (2, 4096), (3, 256)):
        wl = workloads.make_config(c, batch=batch) if c == 1 else None
        if wl is None:
            # the full-size workloads are too slow to draw here; only their sizes matter
            shape = {2: (4096, 4, 64, 64), 3: (256, 8, 128, 128)}[c]

            class W:
                elements = int(np.prod(shape))
            wl = W()
        n = bench.buffer_sets(wl, 1)
        assert 4 <= n <= 64
        assert n == 64 or 2 * wl.elements * n >= 4 * bench.L2_BYTES


def test_clock_sampler_windows_its_samples():
    s = bench.ClockSampler(0)
    s.proc = object()                                   # pretend nvidia-smi ran

    def line(t, mhz, cap):
        stamp = datetime.datetime.fromtimestamp(t).strftime("%Y/%m/%d %H:%M:%S.%f")[:-3]
        return f"{stamp}, {mhz}, 1965, 800.5, 0x4, Not Active, Not Active, Not Active, {cap}"

    class FakeProc:
        def __init__(self, lines):
            self.stdout = lines

    lines = [line(1000.0, 300, "Not Active"), line(1001.0, 1900, "Active"), line(1001.5, 1800, "Active"),
             line(1002.0, 1965, "Not Active"), "garbage line", line(1010.0, 210, "Not Active")]
    s.proc = FakeProc(lines)
    s._read()
    assert len(s.samples) == 5
    inside = s.summary([(1000.9, 1002.1)])
    assert inside["samples"] == 3 and inside["sm_mhz"] == 1900.0 and inside["sm_min_mhz"] == 1800.0
    assert inside["sm_max_mhz"] == 1965.0 and inside["reasons"] == ["sw_power_cap"]
    assert s.summary([(2000.0, 2001.0)])["samples"] == 0
