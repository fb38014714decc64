"""Host-side checks that need no GPU: the shared library loads and exports every symbol
the header declares, the planner behind the C ABI agrees bit-exactly with the oracle's
Algorithm 1, and argument validation rejects bad input without side effects."""
import ctypes as C
import json
import os
import re

import pytest

from oracle import partition_oracle as P
from paper_2108_06629_b200 import binding as lpb
from paper_2108_06629_b200 import build as lpbuild
from paper_2108_06629_b200 import inputs as I

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def built():
    lpbuild.build()


def test_library_exports_every_declared_symbol():
    hdr = open(os.path.join(ROOT, "include", "layerpipe.h")).read()
    hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
    declared = set(re.findall(r"\b(lp_[a-z0-9_]+)\s*\(", hdr))
    assert declared == set(lpb.EXPORTS)
    lib = lpb.lib()
    for name in declared:
        assert getattr(lib, name) is not None


@pytest.mark.parametrize("name", list(I.WORKLOADS))
def test_planner_matches_oracle_bit_exactly(name):
    wl = I.WORKLOADS[name]
    fix, flex = P.mac_costs(wl["layers"], wl["batch"])
    want = P.partition(fix, flex, wl["stages"])
    got = lpb.lp_plan(wl["layers"], wl["batch"], wl["stages"])
    assert got["stage"] == want["stage"]
    assert got["delay"] == want["delay"]
    assert got["used"] == want["used"]
    assert got["T_p"] == want["T_p"]
    assert got["relax_rounds"] == want["relax_rounds"]
    for l, pieces in enumerate(want["dgrad"]):
        exp_s = [s for (s, _, _) in pieces] + [-1] * (2 - len(pieces))
        exp_a = [a for (_, a, _) in pieces] + [0] * (2 - len(pieces))
        assert got["piece_stage"][2 * l:2 * l + 2] == exp_s
        assert got["piece_amount"][2 * l:2 * l + 2] == exp_a


def test_planner_on_the_papers_worked_example():
    g = json.load(open(os.path.join(ROOT, "tests", "golden", "sample_network_tables.json")))
    t2 = g["table2_cycles"]
    fix = [int(a + b) for a, b in zip(t2["FP"], t2["BP_G"])]
    flex = [int(x) for x in t2["BP_delta"]]
    for n_proc in (1, 2, 3, 4, 6):
        want = P.partition(fix, flex, n_proc)
        got = lpb.lp_plan_costs(fix, flex, n_proc)
        assert (got["stage"], got["delay"], got["used"], got["T_p"], got["relax_rounds"]) == \
            (want["stage"], want["delay"], want["used"], want["T_p"], want["relax_rounds"])
    assert lpb.lp_plan_costs(fix, flex, 3)["stage"] == [0, 1, 2, 2]


def test_workspace_size_is_pure_host_arithmetic():
    wl = I.WORKLOADS["mlp8_4096"]
    a = lpb.lp_workspace_size(wl["layers"], wl["stages"], None, wl["delays"], wl["batch"], momentum=0.9)
    b = lpb.lp_workspace_size(wl["layers"], wl["stages"], None, wl["delays"], wl["batch"], momentum=0.0)
    params = sum(l["n_in"] * l["n_out"] for l in wl["layers"])
    ring = sum(l["n_in"] * l["n_out"] * (d + 1) for l, d in zip(wl["layers"], wl["delays"]))
    assert a - b >= 4 * params                     # momentum adds one fp32 copy
    assert b >= 4 * params + 2 * ring              # fp32 master + bf16 ring
    assert b < 4 * params + 2 * ring + (1 << 29)   # stashes and split-K partials are small beside them
    c = lpb.lp_workspace_size(wl["layers"], wl["stages"], None, wl["delays"], wl["batch"],
                              flags=lpb.LP_CAPTURE_GRADS)
    assert c - b >= 4 * params                     # keeping G costs one more fp32 copy


def test_bad_arguments_are_rejected():
    wl = I.WORKLOADS["mlp4_784"]
    with pytest.raises(lpb.LayerPipeError) as e:
        lpb.lp_workspace_size(wl["layers"], 0, None, None, wl["batch"])
    assert e.value.code == lpb.LP_ERR_INVALID_ARG
    bad = [dict(l) for l in wl["layers"]]
    bad[1]["n_in"] = 255
    with pytest.raises(lpb.LayerPipeError) as e:
        lpb.lp_workspace_size(bad, 4, None, None, wl["batch"])
    assert e.value.code == lpb.LP_ERR_INVALID_ARG
    with pytest.raises(lpb.LayerPipeError) as e:
        lpb.lp_workspace_size(wl["layers"], 4, None, [3, 2, 1, -1], wl["batch"])
    assert e.value.code == lpb.LP_ERR_INVALID_ARG
    with pytest.raises(lpb.LayerPipeError) as e:      # an empty minibatch is refused, not run
        lpb.lp_workspace_size(wl["layers"], 4, None, None, 0)
    assert e.value.code == lpb.LP_ERR_INVALID_ARG
    # pixel rows are indexed with 32 bits: batch x image size beyond that is refused, not wrapped
    big = I.vgg(2048, [64, "P"], [10])
    with pytest.raises(lpb.LayerPipeError) as e:
        lpb.lp_workspace_size(big, 1, None, None, 16)
    assert e.value.code == lpb.LP_ERR_UNSUPPORTED
    # a first convolution layer with three channels keeps 3x3 patch rows of 32 bf16 per pixel
    small = I.vgg(16, [16, 32], [10])
    sz = lpb.lp_workspace_size(small, 1, None, None, 8)
    assert sz >= 2 * 8 * 16 * 16 * 32
    # timeline access without a handle
    n = __import__("ctypes").c_int()
    assert lpb.lib().lp_get_task_timeline(None, 0, 0, None, None, n) == lpb.LP_ERR_INVALID_ARG
    lib = lpb.lib()
    assert lib.lp_step(None, None, None, None) == lpb.LP_ERR_INVALID_ARG
    assert lib.lp_destroy(None) == lpb.LP_ERR_INVALID_ARG
    assert lib.lp_gemm_bf16(3, 1, 1, 1, None, 8, None, 8, None, 4, None) == lpb.LP_ERR_INVALID_ARG
    assert lib.lp_set_tuning(100, 0, 0) == lpb.LP_ERR_INVALID_ARG
