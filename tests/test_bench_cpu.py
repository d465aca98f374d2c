"""Host-side checks of bench.py that need no GPU: the recorded DRAM traffic of the two headline kernels
belongs to the sources in the tree, and the algorithmic byte counts are the ones the documents state."""
import importlib.util
import os

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _bench():
    spec = importlib.util.spec_from_file_location("bench_module", os.path.join(ROOT, "bench.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    return mod


def test_recorded_traffic_belongs_to_the_kernels_in_the_tree():
    """bench.py reports `roofline.traffic` only while the sources of the captured kernel are unchanged (their hash
    is stored beside the byte count).  A change to those sources must come with a new capture: this fails until
    the stored hash and byte count have been brought up to date."""
    bench = _bench()
    for name, rec in bench.TRAFFIC.items():
        assert os.path.exists(os.path.join(ROOT, rec["profile"])), rec["profile"]
        assert bench.recorded_traffic(name) == rec["bytes"], (
            "sources of %s changed since its ncu capture: re-capture and update TRAFFIC in bench.py" % rec["kernel"])


def test_algorithmic_bytes_of_the_two_long_workloads():
    bench = _bench()
    from paper_2106_09236_b200 import workloads as wl
    from oracle import psattn_oracle as orc

    def count(c, L):
        return orc.count(c, L)
    for name, want in (("large_bf16", 69420608), ("long_bf16", 140252944)):
        w = wl.WORKLOADS[name]
        got = bench.algorithmic_bytes(w, np.full(w.B, w.T), count, 2)
        assert got == want, (name, got)
