"""Writes tests/golden/chaos_levels.json: how far correct executions of the SAME
delayed-gradient recursion drift apart when only the accumulation arithmetic differs.

Calls nothing but the CPU oracle.  For each configuration the mirror-mode oracle (bf16
rounding at the documented points) is run three times on the same seeded inputs: accumulating
in float32, in float64, and in float32 on the same network with its hidden units renumbered
(a symmetry of the equations that changes the order of every sum).  All are faithful
executions of Eqs. 1-6; they differ the way a GPU run differs from any of them: the last bits
of the fp32 values handed to each bf16 rounding.  The largest pairwise separation is recorded.  A differently rounded element perturbs the next layer, ReLU gates and pooling
winners flip, and the trajectories separate.  The recorded separation is the level below which
a free-running comparison between two implementations carries no information; the GPU
free-running tests bound their GPU-vs-oracle errors by a small multiple of it.

Usage:  python tests/golden/make_chaos_levels.py        (about ten minutes of CPU)
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


def permuted_network(layers, W0, b0, seed):
    """The same network with its hidden units (channels) renumbered: a symmetry of Eqs. 1-6, so
    every quantity is the same up to the renumbering -- but every contraction adds its terms in a
    different order, which makes it a third correct execution with different rounding.
    Returns (W0', b0', perms) with perms[l] = permutation of layer l's outputs (identity for the
    last layer) such that W'[l] = W[l][perms[l]] with its input index permuted by perms[l-1]."""
    rng = np.random.default_rng(seed)
    L = len(layers)
    perms = [rng.permutation(l["n_out"]) if i < L - 1 else np.arange(l["n_out"]) for i, l in enumerate(layers)]
    Wp, bp = [], []
    for i, lay in enumerate(layers):
        W = np.asarray(W0[i])[perms[i]]
        if i > 0:
            pin = perms[i - 1]
            if lay["kind"] == "conv":
                W = W[..., pin]
            elif layers[i - 1]["kind"] == "conv":          # flattened (h, w, c) input: channels are the fastest index
                C = layers[i - 1]["n_out"]
                W = W.reshape(W.shape[0], -1, C)[:, :, pin].reshape(W.shape[0], -1)
            else:
                W = W[:, pin]
        Wp.append(np.ascontiguousarray(W))
        bp.append(np.asarray(b0[i])[perms[i]])
    return Wp, bp, perms


def unpermute(layers, Wlist, perms):
    """Weights (or gradients) of the renumbered network in the original numbering."""
    out = []
    for i, lay in enumerate(layers):
        W = np.asarray(Wlist[i])
        if i > 0:
            inv = np.argsort(perms[i - 1])
            if lay["kind"] == "conv":
                W = W[..., inv]
            elif layers[i - 1]["kind"] == "conv":
                C = layers[i - 1]["n_out"]
                W = W.reshape(W.shape[0], -1, C)[:, :, inv].reshape(W.shape[0], -1)
            else:
                W = W[:, inv]
        out.append(W[np.argsort(perms[i])])
    return out


def level(layers, batch, delays, lr, mu, steps):
    """Largest separation, over the three pairs of (float32, float64, float32 with renumbered units)."""
    W0, b0 = I.initial_weights(layers, 0)
    Wp, bp, perms = permuted_network(layers, W0, b0, 7)
    runs = [O.DelayedGradientTrainer(layers, delays, lr, mu, W0, b0, mirror=True, dtype=np.float32),
            O.DelayedGradientTrainer(layers, delays, lr, mu, W0, b0, mirror=True, dtype=np.float64),
            O.DelayedGradientTrainer(layers, delays, lr, mu, Wp, bp, mirror=True, dtype=np.float32)]
    pairs = ((0, 1), (0, 2), (1, 2))
    g0 = g_later = loss = 0.0
    for n in range(steps):
        x, y = I.minibatch(layers, batch, n)
        recs = [r.step(x, y) for r in runs]
        dWs = [recs[0]["dW"], recs[1]["dW"], unpermute(layers, recs[2]["dW"], perms)]
        for a, b in pairs:
            loss = max(loss, abs(recs[a]["loss"] - recs[b]["loss"]) / abs(recs[b]["loss"]))
            g = max(rel(dWs[a][l], dWs[b][l]) for l in range(len(layers)))
            if n == 0:
                g0 = max(g0, g)
            else:
                g_later = max(g_later, g)
    Ws = [runs[0].weights()[0], runs[1].weights()[0], unpermute(layers, runs[2].weights()[0], perms)]
    w = dw = 0.0
    for a, b in pairs:
        w = max(w, max(rel(Ws[a][l], Ws[b][l]) for l in range(len(layers))))
        dw = max(dw, max(rel(Ws[a][l] - W0[l], Ws[b][l] - W0[l]) for l in range(len(layers))))
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
