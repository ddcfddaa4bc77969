"""CPU-side checks of the boundary: the library builds for sm_100a, loads without a GPU, exports every function the
header declares, reports (not faults) when no device is present, and its host-side scalar rules agree with the paper's
cases and with the CPU checker."""
import ctypes
import math
import os
import re

import pytest

from oracle import dblp_oracle as orc
from paper_2605_01989_b200 import build as dblp_build
from paper_2605_01989_b200 import workloads as wl

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def binding():
    dblp_build.build()
    from paper_2605_01989_b200 import binding as b
    b.lib()
    return b


def declared_functions():
    text = open(os.path.join(ROOT, "include", "dblp.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(dblp_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_function_is_exported(binding):
    names = declared_functions()
    assert {"dblp_packetize", "dblp_apply_loss", "dblp_aggregate", "dblp_check_bound"} <= set(names)
    lib = ctypes.CDLL(binding.LIB_PATH)
    for n in names:
        assert hasattr(lib, n), n
    assert set(names) == set(binding.EXPORTS)


def test_structs_have_the_declared_sizes(binding):
    assert ctypes.sizeof(binding.dblp_loss_model_t) == 80
    assert ctypes.sizeof(binding.dblp_counters_t) == 56
    assert ctypes.sizeof(binding.dblp_device_buffers_t) == 17 * 8


def test_host_rules_match_the_paper_and_the_checker(binding):
    for prev, cur in [(1.0, 0.5), (1.0, 0.6), (1.0, 1.6), (1.0, 1.5), (1.0, 1.4), (0.0, 1.0), (2.0, 0.0), (3.0, 3.0),
                      (7.25, 3.625), (1e-30, 2e-30), (5.0, 2.5000001)]:
        assert binding.dblp_clr(prev, cur, 0.5) == orc.clr(prev, cur, 0.5)
    lo, hi = 24000, 424000
    for prev, cur in [(1.0, 0.9), (1.0, 0.4), (1.0, 2.0), (0.0, 0.0)]:
        for epoch in (0, 1):
            for first in (0, 1):
                for current in (lo, hi):
                    a = binding.dblp_select_bound(prev, cur, 0.5, lo, hi, epoch, first, current)
                    assert a == orc.select_bound(prev, cur, 0.5, lo, hi, epoch, first, current)
    assert binding.dblp_select_bound(1.0, 0.9, 0.5, lo, hi, 1, 0, lo) == hi
    assert binding.dblp_select_bound(1.0, 0.4, 0.5, lo, hi, 1, 0, hi) == lo
    assert binding.dblp_select_bound(0.0, 0.0, 0.5, lo, hi, 0, 1, hi) == lo


def test_rates_helper_gives_the_thresholds_the_workloads_use(binding):
    for i in range(5):
        c = wl.config(i)
        th = c.loss.thresholds(c.C)
        m = binding.dblp_loss_model_from_rates(c.loss.kind, c.loss.mean_loss, c.loss.mean_burst, c.loss.window_frac,
                                               c.loss.p_in, c.loss.p_out, c.C)
        for k, v in th.items():
            assert getattr(m, k) == v, (c.name, k)
    m = binding.dblp_loss_model_from_rates("iid", 1.0)
    assert m.t_drop == 1 << 32
    assert binding.dblp_loss_model_from_rates("microburst", window_frac=0.05, C_=72672).window_len == math.ceil(0.05 * 72672)


def test_without_a_device_calls_fail_loudly(binding):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    with pytest.raises(binding.DblpError) as e:
        binding.Plan([1000], "f32", 1024, 2)
    assert e.value.status == -4 and "CUDA" in str(e.value)


def test_product_sources_never_reach_for_the_oracle():
    pkg = os.path.join(ROOT, "paper_2605_01989_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                assert "oracle" not in open(os.path.join(dirpath, f)).read().lower(), f
