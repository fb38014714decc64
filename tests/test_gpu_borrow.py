"""Operational parallelism executed (Section III-B, Fig. 5(c)-(d)): the delta contraction of a
layer divided by output channels into delta'' (borrowed by the stage that holds layer l+1) and
delta' (the layer's own stage), as two concurrent kernels.

Asserted: the split launch produces delta^{l-1} BIT-IDENTICAL to the unsplit one; each piece
matches the oracle's channel split (dgrad_partial on the corresponding slice of W, then f' and
one rounding) on identical operands; and whole training runs with the planner's pieces, with
minibatches in flight, are bit-identical to runs without the split, under both schedules."""
import numpy as np
import pytest

from gpu_common import assert_bf16_close

pytestmark = pytest.mark.gpu


def _pieces_from_ratio(L, ratios, stage):
    """piece arrays in the planner's layout from {layer: (amount'', amount')}."""
    ps, pa = [-1] * (2 * L), [0] * (2 * L)
    for l in range(1, L):
        a0, a1 = ratios.get(l, (1, 0))
        ps[2 * l], pa[2 * l] = min(stage[l] + 1, max(stage)), a0
        if a1:
            ps[2 * l + 1], pa[2 * l + 1] = stage[l], a1
    return ps, pa


def _split_delta_case(layers, batch, stages, ratios, tile_n=0, expect_cols=None):
    from oracle import layerpipe_oracle as O
    from oracle.bf16 import rn_bf16
    from paper_2108_06629_b200 import binding as lpb
    from paper_2108_06629_b200 import inputs as I
    L = len(layers)
    W0, b0 = I.initial_weights(layers, 0)
    lpb.lp_set_tuning(tile_n, 0, 0)
    try:
        whole = lpb.Trainer(layers, batch, stages, lr=0.05, momentum=0.0, W0=W0, b0=b0)
        split = lpb.Trainer(layers, batch, stages, lr=0.05, momentum=0.0, W0=W0, b0=b0)
    finally:
        lpb.lp_set_tuning(0, 0, 0)
    stage, delays, _ = whole.get_schedule()
    ps, pa = _pieces_from_ratio(L, ratios, stage)
    cols = split.set_delta_split(ps, pa)
    if expect_cols is not None:
        assert cols == expect_cols, cols
    assert any(c > 0 for c in cols)
    orc = O.DelayedGradientTrainer(layers, delays, 0.05, 0.0, W0, b0, mirror=True, dtype=np.float32)
    x, y = I.minibatch(layers, batch, 0)
    Wv = [orc.stash[l][0][0] for l in range(L)]
    rec = orc.step(x, y, capture=True)
    for l in range(1, L):
        outs = []
        for tr in (whole, split):
            tr.debug_write("ring_w", l, 0, Wv[l])
            tr.debug_write("delta", l, 0, rec["delta"][l])
            tr.debug_write("input", l, 0, rec["a"][l])
            if layers[l - 1]["act"] == "gelu":
                tr.debug_write("z", l - 1, 0, rec["zs"][l - 1])
            if layers[l - 1].get("pool", 0):
                tr.debug_write("pool_idx", l - 1, 0, rec["amax"][l - 1].astype(np.float32))
            tr.debug_run_task("delta", l, 0)
            outs.append(tr.debug_read("delta", l - 1, 0))
        assert np.array_equal(outs[0], outs[1]), ("split delta differs from the unsplit one", l)
        if cols[l] == 0 or layers[l - 1].get("pool", 0):
            continue
        # the oracle's channel split: each piece from its own slice of W (input channels = columns of
        # the product), f' of the matching slice of z, one rounding
        lay = layers[l]
        c = cols[l]
        want = np.asarray(rec["delta"][l - 1])
        got = outs[1].reshape(want.shape)
        for lo, hi in ((0, c), (c, lay["n_in"])):
            sub = dict(lay, n_in=hi - lo)
            part = O.dgrad_partial(sub, rec["delta"][l], Wv[l][..., lo:hi])
            zs = np.asarray(rec["zs"][l - 1])
            assert zs.ndim == part.ndim                     # (an FC layer on a flattened image is not split here)
            piece = rn_bf16(O.apply_act_grad(layers[l - 1]["act"], part, zs[..., lo:hi]))
            # the oracle's pieces concatenate to its whole (two BLAS calls: the last fp32 bit may differ before the rounding)
            assert_bf16_close(piece, want[..., lo:hi], "oracle piece against oracle whole", min_equal=0.999)
            assert_bf16_close(got[..., lo:hi], piece, "delta piece [%d, %d) of layer %d" % (lo, hi, l),
                              k_terms=lay["n_out"] * lay.get("R", 1) * lay.get("S", 1))
    for tr in (whole, split):
        assert tr.device_status() == (0, 0)
        tr.close()


def test_split_delta_fc_single_cta_tiles():
    from paper_2108_06629_b200 import inputs as I
    layers = I.mlp([520, 600, 328, 75], "gelu")
    # delta of layer 1 writes 600 columns = 5 tiles of 128, ratio 2 : 3 -> 2 tiles; layer 2: 328 columns = 3 tiles, 1 : 2 -> 1 tile
    _split_delta_case(layers, 72, 3, {1: (2, 3), 2: (1, 2)}, expect_cols=[0, 256, 128])


def test_split_delta_fc_sm_pair_tiles():
    from paper_2108_06629_b200 import inputs as I
    layers = I.mlp([700, 1100, 520, 75], "gelu")
    # forced 256 x 256 pair tiles: layer 1 writes 1100 columns = 5 tiles (1 : 1 -> 3 tiles), layer 2 520 columns = 3 tiles (3 : 1 -> 2)
    _split_delta_case(layers, 300, 3, {1: (1, 1), 2: (3, 1)}, tile_n=512, expect_cols=[0, 768, 512])


def test_split_delta_fc_persistent_pair_kernel():
    """Batch 2048, 4864 -> 2048: the delta contraction takes 224-column pair tiles (176 of them, 32 k-blocks) and runs
    as the persistent pair kernel with two accumulators; its two pieces start at column 0 and at a tile boundary."""
    from paper_2108_06629_b200 import inputs as I
    layers = I.mlp([1024, 4864, 2048, 75], "gelu")
    _split_delta_case(layers, 2048, 3, {1: (1, 1), 2: (1, 2)})


def test_split_delta_convolution_single_cta_and_pair_tiles(conv_pair_tiles):
    from paper_2108_06629_b200 import inputs as I
    layers = I.vgg(8, [384, 384, 384], [10])
    # batch 6: three 128-pixel boxes (odd) -> single-CTA 128-wide tiles, 384 input channels = 3 tiles
    _split_delta_case(layers, 6, 3, {1: (1, 2), 2: (2, 1)}, expect_cols=[0, 128, 256, 0])
    # batch 8: four boxes -> 256-pixel x 256-column pair tiles, 384 channels = 2 tiles
    _split_delta_case(layers, 8, 3, {1: (1, 1), 2: (1, 3)}, expect_cols=[0, 256, 256, 0])


def test_narrow_split_k_and_halo_layers_keep_one_piece():
    from paper_2108_06629_b200 import binding as lpb
    from paper_2108_06629_b200 import inputs as I
    layers = I.vgg(16, [16, 32, "P"], [40, 10])
    W0, b0 = I.initial_weights(layers, 0)
    tr = lpb.Trainer(layers, 8, 2, W0=W0, b0=b0)
    L = len(layers)
    cols = tr.set_delta_split([1] * (2 * L), [5] * (2 * L))
    assert cols[1] == 0 and cols[3] == 0    # halo-tile delta; a single column tile
    lib = lpb.lib()
    assert lib.lp_set_delta_split(tr.h, None, None, None) == lpb.LP_ERR_INVALID_ARG
    with pytest.raises(lpb.LayerPipeError):
        tr.set_delta_split([9] * (2 * L), [5] * (2 * L))       # stage out of range
    import torch
    x, y = I.minibatch(layers, 8, 0)
    tr.step(torch.from_numpy(x).cuda(), torch.from_numpy(y).cuda())
    with pytest.raises(lpb.LayerPipeError) as e:
        tr.set_delta_split([1] * (2 * L), [5] * (2 * L))       # too late
    assert e.value.code == lpb.LP_ERR_NOT_READY
    tr.close()


def _train(layers, batch, stages, lr, mu, steps, schedule, mode, split, tile_n=0):
    import torch
    from paper_2108_06629_b200 import binding as lpb
    from paper_2108_06629_b200 import inputs as I
    W0, b0 = I.initial_weights(layers, 0)
    lpb.lp_set_tuning(tile_n, 0, 0)
    try:
        tr = lpb.Trainer(layers, batch, stages, lr=lr, momentum=mu, schedule=schedule, W0=W0, b0=b0)
    finally:
        lpb.lp_set_tuning(0, 0, 0)
    cols = None
    if split:
        plan = lpb.lp_plan(layers, batch, stages)
        cols = tr.set_delta_split(plan["piece_stage"], plan["piece_amount"])
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
    tr.flush()
    torch.cuda.synchronize()
    out = dict(loss=[tr.get_loss(n) for n in range(steps)], W=[tr.get_weights(l) for l in range(len(layers))], cols=cols)
    assert tr.device_status() == (0, 0)
    tr.close()
    return out


@pytest.mark.parametrize("case", ["mlp", "mlp_pair", "cnn"])
def test_training_with_the_planners_pieces_is_bit_identical(case):
    """Algorithm 1's pieces (lp_plan) executed: free-running and gated, LayerPipe and fused-B."""
    from paper_2108_06629_b200 import binding as lpb
    from paper_2108_06629_b200 import inputs as I
    if case == "mlp":
        args, tile = (I.mlp([520, 600, 328, 456, 392, 75], "gelu"), 72, 4, 0.02, 0.9, 10), 0
    elif case == "mlp_pair":
        args, tile = (I.mlp([1100, 1300, 1100, 900, 75], "gelu"), 300, 4, 0.02, 0.0, 8), 512
    else:
        args, tile = (I.vgg(8, [384, 384, 384], [10]), 6, 3, 0.0005, 0.0, 8), 0
    ref = _train(*args, lpb.LP_SCHED_LAYERPIPE, "natural", False, tile)
    n_split = 0
    for sched in (lpb.LP_SCHED_LAYERPIPE, lpb.LP_SCHED_FUSED_B):
        for mode in ("natural", "gated"):
            got = _train(*args, sched, mode, True, tile)
            n_split = sum(1 for c in got["cols"] if c > 0)
            assert got["loss"] == ref["loss"], (case, sched, mode)
            for a, b in zip(got["W"], ref["W"]):
                assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])
    assert n_split >= 1, "the plan split no layer of this case"
