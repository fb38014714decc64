"""Activation recomputation instead of stashing (Section III-A: the delays between a and the
backward pass stand for either).  With LP_RECOMPUTE a layer whose input is produced inside its
own stage keeps that input only briefly and the backward pass re-runs the producing forward
task on the stashed weight version.  The re-run is the same kernel on the same operands, so
everything the run produces must be BIT-IDENTICAL to the stashing run -- with minibatches in
flight, under both schedules -- while the workspace shrinks and the launch count grows by one
forward task per recomputed layer and minibatch."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu


def _run(layers, batch, n_stages, stage, delays, lr, mu, steps, schedule, mode, flags):
    import torch
    from paper_2108_06629_b200 import binding as lpb
    from paper_2108_06629_b200 import inputs as I
    W0, b0 = I.initial_weights(layers, 0)
    tr = lpb.Trainer(layers, batch, n_stages, stage=stage, delays=delays, lr=lr, momentum=mu, schedule=schedule,
                     flags=flags, W0=W0, b0=b0)
    xs, ys = [], []
    for n in range(steps):
        x, y = I.minibatch(layers, batch, n)
        xs.append(torch.from_numpy(x).cuda())
        ys.append(torch.from_numpy(y).cuda())
    torch.cuda.synchronize()
    if mode == "gated":
        torch.cuda._sleep(300_000_000)
    for n in range(steps):
        tr.step(xs[n], ys[n])
        if mode == "sync":
            torch.cuda.synchronize()
    tr.flush()
    torch.cuda.synchronize()
    out = dict(loss=[tr.get_loss(n) for n in range(steps)], W=[tr.get_weights(l) for l in range(len(layers))],
               launches=tr.kernel_launches(), bytes=tr.workspace_bytes)
    assert tr.device_status() == (0, 0)
    tr.close()
    return out


def _check(layers, batch, n_stages, stage, delays, lr, mu, steps, n_recomputed, extra_per_layer=1):
    from paper_2108_06629_b200 import binding as lpb
    ref = _run(layers, batch, n_stages, stage, delays, lr, mu, steps, lpb.LP_SCHED_LAYERPIPE, "sync", 0)
    assert all(np.isfinite(ref["loss"]))
    for sched in (lpb.LP_SCHED_LAYERPIPE, lpb.LP_SCHED_FUSED_B):
        for mode in ("sync", "natural", "gated"):
            got = _run(layers, batch, n_stages, stage, delays, lr, mu, steps, sched, mode, lpb.LP_RECOMPUTE)
            assert got["loss"] == ref["loss"], (sched, mode)
            for a, b in zip(got["W"], ref["W"]):
                assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])
            assert got["bytes"] < ref["bytes"]
            assert got["launches"] == ref["launches"] + steps * n_recomputed * extra_per_layer, (got["launches"], ref["launches"])
    return ref["bytes"], got["bytes"]


def test_recompute_gelu_mlp_three_stages():
    """Stages {0,1,2 | 3,4 | 5}, delays 6 / 3 / 0: the inputs of layers 1, 2 (stash of 8) and 4 (stash
    of 5) are recomputed, with the stored z their GELU' needs; layer 3 opens its stage and keeps its stash."""
    from paper_2108_06629_b200 import inputs as I
    layers = I.mlp([264, 192, 320, 136, 200, 72, 40], "gelu")
    a, b = _check(layers, 56, 3, [0, 0, 0, 1, 1, 2], [6, 6, 6, 3, 3, 0], 0.02, 0.9, 16, n_recomputed=3)
    print("workspace %d -> %d bytes" % (a, b))


def test_recompute_convnet_with_pooling():
    """One long-delay stage of four convolution layers, two of them pooled: the recomputed inputs come
    with their pooling positions (and the pool kernel runs again: two launches for those layers)."""
    import torch
    from paper_2108_06629_b200 import binding as lpb
    from paper_2108_06629_b200 import inputs as I
    layers = I.vgg(16, [16, 16, "P", 32, 32, "P"], [10])
    stage, delays = [0, 0, 0, 0, 1], [4, 4, 4, 4, 0]
    ref = _run(layers, 8, 2, stage, delays, 0.0005, 0.9, 12, lpb.LP_SCHED_LAYERPIPE, "sync", 0)
    for sched in (lpb.LP_SCHED_LAYERPIPE, lpb.LP_SCHED_FUSED_B):
        for mode in ("natural", "gated"):
            got = _run(layers, 8, 2, stage, delays, 0.0005, 0.9, 12, sched, mode, lpb.LP_RECOMPUTE)
            assert got["loss"] == ref["loss"], (sched, mode)
            for a, b in zip(got["W"], ref["W"]):
                assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])
            assert got["bytes"] < ref["bytes"] and got["launches"] > ref["launches"]


def test_recompute_changes_nothing_where_it_cannot_pay():
    """One layer per stage, or short delays: no layer qualifies, the flag is inert."""
    from paper_2108_06629_b200 import binding as lpb
    from paper_2108_06629_b200 import inputs as I
    wl = I.WORKLOADS["mlp4_784"]
    a = _run(wl["layers"], wl["batch"], 4, None, wl["delays"], wl["lr"], 0.0, 6, lpb.LP_SCHED_LAYERPIPE, "natural", 0)
    b = _run(wl["layers"], wl["batch"], 4, None, wl["delays"], wl["lr"], 0.0, 6, lpb.LP_SCHED_LAYERPIPE, "natural", lpb.LP_RECOMPUTE)
    assert a["loss"] == b["loss"] and a["bytes"] == b["bytes"] and a["launches"] == b["launches"]
