"""Writes tests/golden/chaos_levels.json: how far two correct executions of the SAME
delayed-gradient recursion drift apart when only the accumulation arithmetic differs.

Calls nothing but the CPU oracle.  For each configuration the mirror-mode oracle (bf16
rounding at the documented points) is run twice on the same seeded inputs, once accumulating
in float32 and once in float64.  Both are faithful executions of Eqs. 1-6; they differ the way
a GPU run differs from either of them: the last bits of the fp32 values handed to each bf16
rounding.  A differently rounded element perturbs the next layer, ReLU gates and pooling
winners flip, and the trajectories separate.  The recorded separation is the level below which
a free-running comparison between two implementations carries no information; the GPU
free-running tests bound their GPU-vs-oracle errors by a small multiple of it.

Usage:  python tests/golden/make_chaos_levels.py        (about five minutes of CPU)
"""
import json
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

from oracle import layerpipe_oracle as O          # noqa: E402
from oracle import partition_oracle as P          # noqa: E402
from paper_2108_06629_b200 import inputs as I     # noqa: E402  (seeded generators only)


def rel(a, b):
    a = np.asarray(a, dtype=np.float64).ravel()
    b = np.asarray(b, dtype=np.float64).ravel()
    return float(np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300))


def level(layers, batch, delays, lr, mu, steps):
    W0, b0 = I.initial_weights(layers, 0)
    a = O.DelayedGradientTrainer(layers, delays, lr, mu, W0, b0, mirror=True, dtype=np.float32)
    b = O.DelayedGradientTrainer(layers, delays, lr, mu, W0, b0, mirror=True, dtype=np.float64)
    g0 = g_later = loss = 0.0
    for n in range(steps):
        x, y = I.minibatch(layers, batch, n)
        ra, rb = a.step(x, y), b.step(x, y)
        loss = max(loss, abs(ra["loss"] - rb["loss"]) / abs(rb["loss"]))
        g = max(rel(ra["dW"][l], rb["dW"][l]) for l in range(len(layers)))
        if n == 0:
            g0 = g
        else:
            g_later = max(g_later, g)
    Wa, _ = a.weights()
    Wb, _ = b.weights()
    w = max(rel(Wa[l], Wb[l]) for l in range(len(layers)))
    dw = max(rel(Wa[l] - W0[l], Wb[l] - W0[l]) for l in range(len(layers)))
    return dict(steps=steps, grad_step0=g0, grad_later=g_later, loss=loss, weights=w, weight_change=dw)


def planned(layers, batch, stages):
    fix, flex = P.mac_costs(layers, batch)
    return P.partition(fix, flex, stages)["delay"]


def main():
    out = {}
    for name, steps in (("mlp4_784", 10), ("mlp8_4096", 12), ("vgg_small_32", 10)):
        wl = I.WORKLOADS[name]
        delays = wl["delays"] or planned(wl["layers"], wl["batch"], wl["stages"])
        out[name] = level(wl["layers"], wl["batch"], delays, wl["lr"], wl["momentum"], steps)
        print(name, out[name], flush=True)
    # the two smaller free-running cases of the GPU suite
    layers = I.mlp([384] * 6 + [100], "gelu")
    out["gelu6"] = level(layers, 96, planned(layers, 96, 4), 0.02, 0.9, 12)
    layers = I.vgg(16, [16, 32, "P", 64, "P"], [48, 10])
    out["cnn16"] = level(layers, 32, planned(layers, 32, 3), 0.02, 0.9, 8)
    with open(os.path.join(ROOT, "tests", "golden", "chaos_levels.json"), "w") as f:
        json.dump(out, f, indent=1, sort_keys=True)
        f.write("\n")


if __name__ == "__main__":
    main()
