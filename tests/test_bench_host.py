"""Host logic of bench.py that needs no GPU: the byte models of the kernels, the clock sampler's
per-window statistics, the bounded sample of the CPU leg."""
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import bench  # noqa: E402
from paper_1909_04823_b200 import synth  # noqa: E402


def _stats():
    return dict(nnz=1000, B=10, F=5, k=8, S=4, H=0, U=300, ops=synth.OP_LR | synth.OP_FM | synth.OP_POOL, adagrad=True,
                rep_rows=0, super=False, shift=0, new_keys=True)


def test_kernel_byte_models_are_what_the_comments_say():
    st = _stats()
    row = 4 * st["k"] + 16
    # gradient scatter: offsets, one index word per occurrence, gE once, A, gL / gF, each key's gradient once
    want = 4 * (10 * 5 + 1) + 4 * 1000 + 4 * 10 * 5 * 8 + 4 * 10 * 12 + 8 * 10 + row * 300
    assert bench.kernel_bytes("grad_scatter_kernel", st) == want
    # update: gradient row read + cleared, weights and state read + written, the row number
    assert bench.kernel_bytes("update_rows_kernel", st) == 300 * (2 * row + 4 * row + 8)
    assert bench.kernel_bytes("pool_kernel", st) == 4 * 51 + 4 * 1000 + 4 * 8 * 300 + 4 * 10 * 5 * 8
    assert bench.kernel_bytes("no_such_kernel", st) is None
    assert bench.occurrence_bytes("pool_kernel", st) == 4 * 8 * 1000
    assert bench.kernel_flops("tc_gemm_fwd", dict(st, H=16)) == 2 * 10 * 5 * 8 * 16
    # every kernel with a traffic constant has a byte model
    for (_, name) in bench.NCU_DRAM_TRAFFIC:
        assert bench.kernel_bytes(name, dict(st, super=True)) is not None, name


def test_clock_sampler_windows_without_nvml():
    s = bench.ClockSampler.__new__(bench.ClockSampler)       # no thread, no NVML: fill the samples by hand
    import threading
    s.samples = [(t, 1000.0 + 10 * i, (0x4 if i == 3 else 0), 500.0 + i) for i, t in enumerate(np.arange(0.0, 1.0, 0.1))]
    s.max_mhz = 1965.0
    s._stop = threading.Event(); s._thread = None
    w = s.window(0.25, 0.55)
    assert w["samples"] == 3 and w["sm_mhz"] == 1040.0 and w["reasons"] == ["sw_power_cap"]
    assert s.window(0.31, 0.32)["samples"] == 1               # shorter than the sampling period: nearest sample
    out = s.stop([(0.0, 0.25), (0.75, 1.0)])
    assert out["samples"] == 5 and out["sm_max_mhz"] == 1965.0 and out["reasons"] == [] and out["scope"] == "timed windows only"


def test_cpu_leg_takes_a_prefix_of_the_batch():
    w = synth.config(1)
    b = synth.Stream(w).next_batch()
    sb = bench.sub_batch(b, 7)
    assert sb.batch == 7 and sb.offsets[0] == 0 and sb.offsets[-1] == sb.ids.shape[0] == b.offsets[7 * w.fields]
    assert np.array_equal(sb.ids, b.ids[:sb.nnz])
    assert bench.shift_of(1 << 20) == 0 and bench.shift_of((1 << 20) + 1) == 1 and bench.shift_of(1 << 40) == 6
