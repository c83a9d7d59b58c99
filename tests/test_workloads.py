"""The shape tables and seeded generators (no GPU)."""
import numpy as np

from paper_1603_05279_b200 import workloads as wl


def test_mac_counts_of_the_named_workloads():
    assert abs(sum(wl.macs(s) for s in wl.ALEXNET) / 1e9 - 248.63) < 0.01
    assert abs(wl.macs(wl.RESNET18[0]) / 1e9 - 29.60) < 0.01
    assert abs(wl.macs(wl.RESNET18[1]) / 1e9 - 14.80) < 0.01
    assert abs(sum(wl.macs(s) for s in wl.chain_shapes()) / 1e9 - 429.13) < 0.01
    assert len(wl.SWEEP) == 24 and len(wl.chain_shapes()) == 16


def test_generators_are_seeded_and_counter_based():
    s = wl.SINGLE[0]
    a, b = wl.make_input(s, 1000), wl.make_input(s, 1000)
    assert a.dtype == np.float32 and a.shape == (1, 64, 14, 14) and np.array_equal(a, b)
    assert not np.array_equal(a, wl.make_input(s, 1001))
    w = wl.make_weights(wl.ALEXNET[0], 2000)
    assert w.shape == (256, 96, 5, 5) and abs(float(w.std()) - 0.01) < 5e-4
    assert abs(float(a.mean())) < 0.05 and abs(float(a.std()) - 1) < 0.05
