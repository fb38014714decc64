"""Pins for the Algorithm 1 oracle: the paper's worked example (Table II in,
Table III out), the layer-granular baseline row, Table IV's internal
arithmetic, and structural invariants of the allocation."""
import json
import os

import numpy as np
import pytest

from oracle import partition_oracle as P
from paper_2108_06629_b200 import inputs as I

G = os.path.join(os.path.dirname(__file__), "golden")


def load(name):
    with open(os.path.join(G, name)) as f:
        return json.load(f)


def test_worked_example_reproduces_table3():
    g = load("sample_network_tables.json")
    t2, t3 = g["table2_cycles"], g["table3"]
    fix = [int(a + b) for a, b in zip(t2["FP"], t2["BP_G"])]
    flex = [int(x) for x in t2["BP_delta"]]
    r = P.partition(fix, flex, t3["processors"])
    assert r["used"] == 3 and r["relax_rounds"] == 0
    assert r["stage"] == [0, 1, 2, 2]
    assert r["delay"] == [2, 1, 0, 0]
    tol = 0.01
    # every processor ends at the same total (the paper prints 3.22e7 three times)
    for s in range(3):
        assert abs(r["loads"][s] - t3["layerpipe_total"][s]) <= tol * t3["layerpipe_total"][s]
    # borrowed = delta'' placed beside the *next* layer; assigned = the rest
    borrowed = [0, 0, 0]
    for l in range(4):
        for (s, amt, tag) in r["dgrad"][l]:
            if tag == "delta''":
                borrowed[s] += amt
    for s in range(3):
        want_b = t3["layerpipe_borrowed"][s]
        assert abs(borrowed[s] - want_b) <= tol * max(want_b, 1.0)
        want_a = t3["layerpipe_assigned"][s]
        assert abs((r["loads"][s] - borrowed[s]) - want_a) <= tol * want_a
    gain = (max(t3["pipedream"]) - max(r["loads"])) / max(t3["pipedream"])
    assert round(100 * gain) == g["throughput_gain_percent"]


def test_layer_granular_baseline_row():
    g = load("sample_network_tables.json")
    t2, t3 = g["table2_cycles"], g["table3"]
    tot = [a + b + c for a, b, c in zip(t2["FP"], t2["BP_G"], t2["BP_delta"])]
    edges, loads = P.layer_granular_partition(tot, 3)
    assert edges == (0, 1, 2, 4)                       # {1}, {2}, {3, 4}
    for got, want in zip(loads, t3["pipedream"]):
        assert abs(got - want) <= 0.01 * want


def test_table4_internal_arithmetic():
    g = load("vgg16_speedup_table.json")
    imp = [100 * (a / b - 1) for a, b in zip(g["layerpipe"], g["pipedream"])]
    for got, want in zip(imp, g["improvement_percent"]):
        assert abs(got - want) < 0.6                  # printed speedups carry two decimals
    assert abs(np.mean(g["improvement_percent"]) - g["average_improvement_percent"]) < 1.0


@pytest.mark.parametrize("name", list(I.WORKLOADS))
def test_allocation_invariants_on_the_workloads(name):
    wl = I.WORKLOADS[name]
    fix, flex = P.mac_costs(wl["layers"], wl["batch"])
    r = P.partition(fix, flex, wl["stages"])
    L = len(fix)
    assert r["used"] <= wl["stages"]
    assert sum(r["loads"]) == sum(fix) + sum(flex)                 # nothing lost or duplicated
    assert all(r["stage"][l] <= r["stage"][l + 1] for l in range(L - 1))   # stages are contiguous
    assert r["delay"] == [r["used"] - 1 - s for s in r["stage"]]
    for l in range(L):
        assert sum(a for (_, a, _) in r["dgrad"][l]) == flex[l]
        for (s, _, _) in r["dgrad"][l]:
            # delta of layer l only ever sits with layer l or layer l+1's processor range
            hi = r["stage"][l + 1] if l + 1 < L else r["stage"][l]
            assert r["stage"][l] <= s <= hi
    if wl["delays"] is not None:
        assert r["delay"] == wl["delays"]                           # explicit delays = the planner's
