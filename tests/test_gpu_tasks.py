"""Per-task parity with the SAME operands on both sides.

The oracle walks the delayed-gradient recursion on seeded inputs and records every
operand and result of every task.  For each task the operands it recorded are written
into the library's buffers (lp_debug_write), the one CUDA task is run
(lp_debug_run_task) and its outputs are read back and compared.  Nothing the oracle
consumes comes from the GPU.  With identical operands the only freedom left is the
summation order inside a contraction, so bf16 results may differ by one bf16 spacing on
the rare elements that sat next to a rounding boundary and fp32 results by fp32
round-off; the stated tolerance (relative L2 <= 2e-3 per tensor) holds with a wide
margin and much sharper bounds are asserted."""
import numpy as np
import pytest

from gpu_common import assert_bf16_close, rel_l2

pytestmark = pytest.mark.gpu


def run_teacher_forced(layers, batch, stages, delays, lr, mu, steps, check_steps=None, fused=True, bias=True, check_layers=None):
    from oracle import layerpipe_oracle as O
    from paper_2108_06629_b200 import binding as lpb
    from paper_2108_06629_b200 import inputs as I
    W0, b0 = I.initial_weights(layers, 0)
    rng = np.random.default_rng(5)
    b0 = [rng.standard_normal(b.shape).astype(np.float32) * 0.1 if bias else None for b in b0]   # exercise the bias path
    flags = lpb.LP_CAPTURE_GRADS | (0 if fused else lpb.LP_UNFUSED_UPDATE)
    tr = lpb.Trainer(layers, batch, stages, delays=delays, lr=lr, momentum=mu, flags=flags, W0=W0, b0=b0)
    delays = tr.get_schedule()[1]
    orc = O.DelayedGradientTrainer(layers, delays, lr, mu, W0, b0, mirror=True, dtype=np.float32)
    L = len(layers)
    worst = {}

    def k_fwd(l):       # terms of layer l's forward contraction (its delta contraction has k_bwd terms)
        return layers[l]["n_in"] * (layers[l].get("R", 1) * layers[l].get("S", 1))

    def k_bwd(l):
        return layers[l]["n_out"] * (layers[l].get("R", 1) * layers[l].get("S", 1))

    def note(k, v):
        worst[k] = max(worst.get(k, 0.0), v)

    for n in range(steps):
        x, y = I.minibatch(layers, batch, n)
        pre_W = [w.copy() for w in orc.W]
        pre_b = [None if b is None else b.copy() for b in orc.b]
        pre_mW = [m.copy() for m in orc.mW]
        pre_mb = [None if m is None else m.copy() for m in orc.mb]
        stash = [dict(s) for s in orc.stash]
        rec = orc.step(x, y, capture=True)
        if check_steps is not None and n not in check_steps:
            continue
        slot = rec["slot"]
        todo = range(L) if check_layers is None else sorted(check_layers)     # layers whose tasks are run and compared
        # weight versions this minibatch reads
        for l in todo:
            Wv, bv = stash[l][rec["v"][l]]
            tr.debug_write("ring_w", l, slot[l], Wv)
            if bias:
                tr.debug_write("ring_b", l, slot[l], bv)
        tr.debug_write("labels", 0, n, y.astype(np.float32))
        # forward tasks
        for l in todo:
            tr.debug_write("input", l, n, rec["a"][l])
            tr.debug_run_task("forward", l, n)
            if l < L - 1:
                note("a", assert_bf16_close(tr.debug_read("input", l + 1, n), rec["a"][l + 1], "a^%d step %d" % (l + 1, n), k_terms=k_fwd(l)))
                if layers[l].get("pool", 0):
                    # which window element wins may legitimately differ where two candidates are within
                    # a rounding of each other; everywhere else the recorded position must agree
                    same = float((tr.debug_read("pool_idx", l, n) == rec["amax"][l]).mean())
                    assert same > 0.995, ("pool argmax", l, n, same)
                if layers[l]["act"] == "gelu":
                    note("z", assert_bf16_close(tr.debug_read("z", l, n), rec["zs"][l], "z^%d step %d" % (l, n), k_terms=k_fwd(l)))
            else:
                got_zL = tr.debug_read("logits", 0, n)
                r = rel_l2(got_zL, rec["zL"])
                if r >= 1e-5 + 1e-7 * np.sqrt(k_fwd(l)):      # fp32 accumulation over k_fwd terms on both sides
                    # A very long contraction with few outputs (one 224 x 224 image: 200704 terms, 10 logits): the
                    # outputs are small against the sum of the magnitudes of their terms, and the fp32 oracle's own
                    # accumulation error shows.  Judge both against float64 on the same operands, with the
                    # bound of an accumulator that is truncated once per 16-term tensor-core step (the running sum
                    # of the MMA is not rounded to nearest: its error grows with K, not with sqrt(K)).
                    a64 = np.asarray(rec["a"][l], dtype=np.float64).reshape(batch, -1)
                    Wv, bv = stash[l][rec["v"][l]]
                    W64 = np.asarray(Wv, dtype=np.float64).reshape(layers[l]["n_out"], -1)
                    ref = a64 @ W64.T + (0.0 if bv is None else np.asarray(bv, dtype=np.float64))
                    bound = (k_fwd(l) / 16.0) * 2.0 ** -23 * np.linalg.norm(np.abs(a64) @ np.abs(W64).T)
                    err_gpu = np.linalg.norm(got_zL.reshape(ref.shape) - ref)
                    err_orc = np.linalg.norm(np.asarray(rec["zL"], dtype=np.float64).reshape(ref.shape) - ref)
                    assert err_gpu <= bound, ("logits against float64", n, err_gpu, bound, err_orc)
                    r = err_gpu / np.linalg.norm(ref)
                note("logits", r)
        # loss task
        tr.debug_write("logits", 0, n, rec["zL"])
        tr.debug_run_task("loss", 0, n)
        note("deltaL", assert_bf16_close(tr.debug_read("delta", L - 1, n), rec["delta"][L - 1], "delta^L step %d" % n))
        loss = float(tr.debug_read("loss", 0, n)[0])
        assert abs(loss - rec["loss"]) <= 2e-6 * max(1.0, abs(rec["loss"])), (loss, rec["loss"])
        # backward tasks
        for l in reversed(todo):
            tr.debug_write("delta", l, n, rec["delta"][l])
            tr.debug_write("input", l, n, rec["a"][l])
            if l > 0:
                if layers[l - 1]["act"] == "gelu":
                    tr.debug_write("z", l - 1, n, rec["zs"][l - 1])
                if layers[l - 1].get("pool", 0):
                    tr.debug_write("pool_idx", l - 1, n, rec["amax"][l - 1].astype(np.float32))
                tr.debug_run_task("delta", l, n)
                note("delta", assert_bf16_close(tr.debug_read("delta", l - 1, n), rec["delta"][l - 1],
                                                "delta^%d step %d" % (l - 1, n), k_terms=k_bwd(l)))
            # pre-update state of the oracle; with the fused update the G kernel itself applies Eq. 6
            tr.debug_write("master_w", l, 0, pre_W[l])
            if bias:
                tr.debug_write("master_b", l, 0, pre_b[l])
            if mu != 0.0:
                tr.debug_write("mom_w", l, 0, pre_mW[l])
                if bias:
                    tr.debug_write("mom_b", l, 0, pre_mb[l])
            tr.debug_run_task("G", l, n)
            r = rel_l2(tr.debug_read("grad_w", l, 0), rec["dW"][l])
            k_g = int(np.prod(rec["delta"][l].shape[:-1]))        # terms of the G contraction: samples (x pixels)
            assert r < 2e-5 + 1e-7 * np.sqrt(k_g), ("G", l, n, r)   # fp32 accumulation over k_g terms on both sides
            note("G", r)
            if not fused:
                tr.debug_write("grad_w", l, 0, rec["dW"][l])      # Eq. 6 from the oracle's gradient
            tr.debug_run_task("update", l, n)
            if bias:
                r = rel_l2(tr.debug_read("grad_b", l, 0), rec["db"][l])
                assert r < 2e-5, ("db", l, n, r)
                note("db", r)
            dWn = np.linalg.norm(rec["dW"][l])
            step_err = np.linalg.norm(tr.debug_read("master_w", l, 0) - orc.W[l]) / max(lr * dWn, 1e-30)
            assert step_err < 1e-3, ("update of W relative to the step taken", l, n, step_err)
            if bias:
                assert rel_l2(tr.debug_read("master_b", l, 0), orc.b[l]) < 1e-5
            if mu != 0.0:
                assert rel_l2(tr.debug_read("mom_w", l, 0), orc.mW[l]) < 1e-6 + 1e-7 * np.sqrt(k_g)   # m = mu m + G carries G's accumulation error
            new_slot = (n + 1) % (delays[l] + 1)
            Wq, bq = orc.stash[l][n + 1]
            note("ring", assert_bf16_close(tr.debug_read("ring_w", l, new_slot), Wq, "ring W^%d step %d" % (l, n),
                                           min_equal=0.995))
            if bias:
                assert rel_l2(tr.debug_read("ring_b", l, new_slot), bq) < 1e-5
    rc, detail = tr.device_status()
    assert rc == 0, detail
    tr.close()
    return worst


def test_tasks_mlp4_784_full_config():
    from paper_2108_06629_b200 import inputs as I
    wl = I.WORKLOADS["mlp4_784"]
    w = run_teacher_forced(wl["layers"], wl["batch"], wl["stages"], wl["delays"], wl["lr"], wl["momentum"], wl["steps"])
    print("worst per-task errors", w)


def test_tasks_gelu_momentum_ragged_sizes():
    """GELU + momentum, feature sizes that are not multiples of the 128 x 128 tile nor of 8
    (padded pitches), batch 72 (ragged M)."""
    from paper_2108_06629_b200 import inputs as I
    layers = I.mlp([200, 328, 130, 257, 75], "gelu")
    w = run_teacher_forced(layers, 72, 4, [3, 2, 1, 0], 0.05, 0.9, 6)
    print("worst per-task errors", w)


def test_tasks_unfused_update_path():
    """LP_UNFUSED_UPDATE: G is written to memory and Eq. 6 runs as its own kernel."""
    from paper_2108_06629_b200 import inputs as I
    layers = I.mlp([200, 328, 130, 75], "gelu")
    run_teacher_forced(layers, 72, 3, [2, 1, 0], 0.05, 0.9, 5, fused=False)
    run_teacher_forced(I.mlp([96, 160, 24], "relu"), 40, 2, [1, 0], 0.05, 0.0, 4, fused=False)
    # convolution layers (patch-matrix first layer, halo-tile G, split-K G) with the separate update kernel
    run_teacher_forced(I.vgg(16, [16, 32, "P", 72], [10]), 8, 2, None, 0.05, 0.9, 3, fused=False)


def test_tasks_split_k_forward_and_delta():
    """Forced split-K (3 and 8 splits, more splits than k-blocks in some layers): partial tiles
    reduced in split order by the last CTA of each tile."""
    from paper_2108_06629_b200 import binding as lpb
    from paper_2108_06629_b200 import inputs as I
    layers = I.mlp([520, 328, 200, 75], "gelu")
    for sk in (3, 8):
        lpb.lp_set_tuning(0, 0, sk)
        try:
            run_teacher_forced(layers, 72, 3, [2, 1, 0], 0.05, 0.9, 4)
        finally:
            lpb.lp_set_tuning(0, 0, 0)


def test_tasks_persistent_tile_loop():
    """Forced persistent CTAs on a layer with more tiles (21 x 18) than resident CTAs: every CTA
    walks several tiles, so the pipeline, the double-buffered accumulator and the streamed
    update tiles (Eq. 6 in the G epilogue) run across tile boundaries.  With and without momentum."""
    from paper_2108_06629_b200 import binding as lpb
    from paper_2108_06629_b200 import inputs as I
    layers = I.mlp([2200, 2600, 520, 75], "gelu")
    lpb.lp_set_tuning(0, 0, 512)
    try:
        run_teacher_forced(layers, 72, 3, [2, 1, 0], 0.05, 0.9, 3)
        run_teacher_forced(layers, 72, 3, [2, 1, 0], 0.05, 0.0, 3)
    finally:
        lpb.lp_set_tuning(0, 0, 0)


def test_tasks_small_convnet():
    """Conv 3x3 + ReLU (+ 2x2 max pool) layers followed by FC layers: implicit-GEMM forward, delta
    with the un-pooling epilogue (conv -> conv and conv -> FC), split-K G with the fused update,
    two-pass bias gradient.  Image sizes 16 / 8 / 4 exercise pixel boxes that span several rows
    and several images; 3 input channels exercise the padded first layer."""
    from paper_2108_06629_b200 import inputs as I
    layers = I.vgg(16, [16, 32, "P", 64, "P", 72, "P"], [40, 10])
    run_teacher_forced(layers, 16, 4, None, 0.05, 0.9, 4)
    # 32 x 32 and 16 x 16 images with at most 64 channels: the halo-tile kernel (one fetch of the
    # activation box per 8 x 16 pixel tile) for forward and delta, the latter also behind a pool
    layers = I.vgg(32, [16, "P", 32, 24, "P"], [10])
    run_teacher_forced(layers, 4, 3, None, 0.05, 0.9, 3)


def test_tasks_vgg_small_32_full_config():
    from paper_2108_06629_b200 import inputs as I
    wl = I.WORKLOADS["vgg_small_32"]
    w = run_teacher_forced(wl["layers"], wl["batch"], wl["stages"], wl["delays"], wl["lr"], wl["momentum"], 8,
                           check_steps={0, 7})
    print("worst per-task errors", w)


def test_tasks_sm_pair_tiles():
    """All three contractions and the fused update through the two-CTA (cta_group::2) kernel,
    forced onto shapes with ragged 256 x 256 tiles."""
    from paper_2108_06629_b200 import binding as lpb
    from paper_2108_06629_b200 import inputs as I
    layers = I.mlp([520, 328, 600, 75], "gelu")
    for code in (512, 448):          # 256-column tiles; 224-column tiles for forward and delta (G keeps 256)
        lpb.lp_set_tuning(code, 0, 0)
        try:
            run_teacher_forced(layers, 300, 3, [2, 1, 0], 0.05, 0.9, 4)
        finally:
            lpb.lp_set_tuning(0, 0, 0)


def test_tasks_wide_network_runs_its_narrow_classifier_on_sm_pairs():
    """A fully connected network whose layers are mostly wide keeps to one kind of tensor-memory
    allocation: the 10-unit classifier runs on SM-pair tiles too -- forward with N = 10, delta with
    K = 10 (one zero-filled k-block), G with M = 10 and the streamed update clipped to ten rows.
    With and without momentum (the persistent and the one-tile G kernel)."""
    from paper_2108_06629_b200 import inputs as I
    layers = I.mlp([1024, 1280, 1024, 10], "gelu")
    run_teacher_forced(layers, 1024, 3, [2, 1, 0], 0.02, 0.9, 3)
    run_teacher_forced(layers, 1024, 3, [2, 1, 0], 0.02, 0.0, 2)


def test_tasks_degenerate_shapes():
    """The paper's bias-free Eq. 1; a single layer (no delta task at all); batch 1; one stage with
    all delays zero (plain backpropagation); a delay larger than the number of steps run."""
    from paper_2108_06629_b200 import inputs as I
    nobias = [dict(l, bias=False) for l in I.mlp([72, 40, 24], "relu")]
    run_teacher_forced(nobias, 24, 2, [1, 0], 0.05, 0.9, 4, bias=False)
    run_teacher_forced(I.mlp([40, 16], "relu"), 8, 1, [0], 0.05, 0.0, 3)
    run_teacher_forced(I.mlp([24, 16, 8], "gelu"), 1, 2, [1, 0], 0.05, 0.0, 3)
    run_teacher_forced(I.mlp([64, 48, 32, 8], "gelu"), 16, 1, [0, 0, 0], 0.05, 0.9, 3)
    run_teacher_forced(I.mlp([64, 48, 8], "relu"), 16, 2, [9, 0], 0.05, 0.0, 3)


def test_tasks_papers_double_delay_convention():
    """Delays = 2 x (stages after the layer), the count Section III-A gives for the retimed graph."""
    from paper_2108_06629_b200 import inputs as I
    layers = I.mlp([96, 160, 64, 24], "relu")
    run_teacher_forced(layers, 40, 3, [4, 2, 0], 0.05, 0.0, 7)


def test_tasks_mlp8_4096_full_size():
    """The benchmark configuration at full size; three minibatches (first, one inside the
    warm-up, one after every ring has wrapped) are checked task by task."""
    from paper_2108_06629_b200 import inputs as I
    wl = I.WORKLOADS["mlp8_4096"]
    w = run_teacher_forced(wl["layers"], wl["batch"], wl["stages"], wl["delays"], wl["lr"], wl["momentum"], 10,
                           check_steps={0, 4, 9})
    print("worst per-task errors", w)


def test_tasks_mlp16_8192_full_size_one_minibatch():
    """The tensor-bound workload at full size (2048 x 8192 x 8192, sixteen layers): every task of
    one minibatch on the oracle's operands -- 256 x 256 SM-pair tiles with 64 tiles per dimension
    for all three contractions, the update of 67 M weights per layer in the G kernel."""
    from paper_2108_06629_b200 import inputs as I
    wl = I.WORKLOADS["mlp16_8192"]
    # (the sixteen layers have one shape: first, second, one in the middle and the last are run)
    w = run_teacher_forced(wl["layers"], wl["batch"], wl["stages"], wl["delays"], wl["lr"], wl["momentum"], 1,
                           check_layers={0, 1, 9, 15})
    print("mlp16_8192 worst per-task errors", w)


@pytest.mark.parametrize("pair_tiles", [False, True])
def test_tasks_vgg16_224_full_size_one_minibatch(pair_tiles, monkeypatch):
    """VGG-16 shapes at 224 x 224, batch 64, planned stages: pixel boxes with seven tiles per row
    (224 / 112 / 56 / 28 pixels), the 2 x 2 x 32 box at 14 x 14, split-K G over 3.2 M pixel rows,
    the patch-matrix first layer, the halo-tile 64 -> 64 layer, the automatic split-K and the
    persistent streamed update of the 25088 -> 4096 layer; with pair_tiles the layers of 256 and 512
    channels as persistent SM-pair tiles."""
    from paper_2108_06629_b200 import inputs as I
    if pair_tiles:
        monkeypatch.setenv("LP_CONV_PAIR", "1")
    wl = I.WORKLOADS["vgg16_224"]
    w = run_teacher_forced(wl["layers"], wl["batch"], wl["stages"], wl["delays"], wl["lr"], wl["momentum"], 1)
    print("vgg16_224 worst per-task errors", w)


def test_tasks_pixel_boxes_with_seven_tiles_per_row():
    """56 / 28 / 14 pixel images: boxes of 8 x 8 x 2, 4 x 4 x 8 and 2 x 2 x 32 pixels, seven boxes
    per image row, none of them served by the halo-tile kernels (56 is not a multiple of 16)."""
    from paper_2108_06629_b200 import inputs as I
    layers = I.vgg(56, [16, 16, "P", 32, 32, "P", 64], [10])
    run_teacher_forced(layers, 32, 4, None, 0.05, 0.9, 3)


def test_tasks_sm_pair_convolution_tiles_at_28_and_14_pixels(conv_pair_tiles):
    """256 -> 256 channels at 28 x 28 and (behind a pool) at 14 x 14, batch 64: an even number of
    128-pixel boxes, so forward and delta run as 256-pixel x 256-column tiles on SM pairs."""
    from paper_2108_06629_b200 import inputs as I
    layers = I.vgg(28, [256, 256, "P", 256], [10])
    run_teacher_forced(layers, 64, 3, None, 0.02, 0.0, 2)


def test_tasks_single_image_224_patch_layer_and_automatic_split_k():
    """One 224 x 224 RGB image: the patch-matrix first layer (forward through the halo pipeline, G as
    one tile split 148 ways over 50 k pixel rows) and a fully connected layer with 3136 k-blocks and
    a single tile, which takes the automatic four-way split-K."""
    from paper_2108_06629_b200 import inputs as I
    layers = I.vgg(224, [16, "P"], [10])
    run_teacher_forced(layers, 1, 2, None, 0.05, 0.9, 3)
    run_teacher_forced(layers, 2, 2, None, 0.05, 0.0, 2)


def test_tasks_persistent_update_walk_of_three_tiles_per_cta():
    """G of a 4500 -> 3000 layer: 24 x 36 = 864 tiles on 296 CTA slots, forced persistent, so every
    CTA streams the update of about three tiles back to back through its stage ring."""
    from paper_2108_06629_b200 import binding as lpb
    from paper_2108_06629_b200 import inputs as I
    layers = I.mlp([4500, 3000, 75], "gelu")
    lpb.lp_set_tuning(0, 0, 512)
    try:
        run_teacher_forced(layers, 72, 2, [1, 0], 0.05, 0.9, 2)
    finally:
        lpb.lp_set_tuning(0, 0, 0)


def _general_net(hw, specs, fc_out=10):
    """specs: (filter, c_out, pad, stride, pool) per convolution layer, 3 input channels."""
    from paper_2108_06629_b200 import inputs as I
    layers, c, h = [], 3, hw
    for k, cout, pad, stride, pool in specs:
        layers.append(I.conv(c, cout, h, h, "relu", pool, True, R=k, S=k, pad=pad, stride=stride))
        h = (h + 2 * pad - k) // stride + 1
        if pool:
            h //= 2
        c = cout
    layers.append(I.fc(c * h * h, fc_out, "none"))
    return layers


def test_tasks_general_filters_and_strides():
    """Filters other than 3x3 and stride 2 (the shapes of the paper's sample network, Table I, at 32
    pixels): forward and G fetch every second input pixel through a stepping tensor map, delta runs
    once per residue class of the input pixel with the taps of that class.  Every task against the
    oracle on identical operands, three minibatches with momentum."""
    # 5x5 s2, 5x5 s2, 3x3 s2, 3x3 s1: 32 -> 16 -> 8 -> 4 -> 4 pixels
    layers = _general_net(32, [(5, 16, 2, 2, 0), (5, 32, 2, 2, 0), (3, 64, 1, 2, 0), (3, 64, 1, 1, 0)])
    run_teacher_forced(layers, 16, 3, None, 0.05, 0.9, 3)
    # 7x7 s1 p3; pointwise 1x1 s1 and 1x1 s2 (three of the four residue classes of its delta have no tap);
    # a strided layer followed by a pool; wide channels (two 64-channel chunks per tap)
    layers = _general_net(16, [(7, 16, 3, 1, 0), (1, 32, 0, 1, 0), (1, 40, 0, 2, 0), (5, 136, 2, 1, 2)])
    run_teacher_forced(layers, 8, 3, None, 0.05, 0.0, 2)
    # stride 2 straight into a pool, and a 5x5 layer that receives its delta through that pool
    layers = _general_net(32, [(3, 24, 1, 2, 2), (5, 32, 2, 1, 0)])
    run_teacher_forced(layers, 16, 2, None, 0.05, 0.9, 2)


def test_tasks_sample_network_of_table1_full_size():
    """The paper's sample network (Table I) at the size of its worked example (Section IV-B): 224 x 224 x 3 input,
    batch 32, three stages; two minibatches, every task on the oracle's operands."""
    from paper_2108_06629_b200 import inputs as I
    wl = I.WORKLOADS["sample4_224"]
    w = run_teacher_forced(wl["layers"], wl["batch"], wl["stages"], wl["delays"], wl["lr"], wl["momentum"], 2)
    print("sample4_224 worst per-task errors", w)


def test_tasks_sm_pair_persistent_g_update():
    """The persistent SM-pair G kernel (one CTA pair per SM pair walks several 256 x 256 tiles, the
    update of one tile streaming under the main loop of the next): forced onto ragged shapes with
    fewer tiles than SM pairs and with more (99 tiles: a second tile for 25 pairs), with and without
    momentum (two or four chunk slots)."""
    from paper_2108_06629_b200 import binding as lpb
    from paper_2108_06629_b200 import inputs as I
    lpb.lp_set_tuning(512, 0, 512)
    try:
        run_teacher_forced(I.mlp([520, 328, 600, 75], "gelu"), 300, 3, [2, 1, 0], 0.05, 0.9, 3)
        run_teacher_forced(I.mlp([2600, 2200, 75], "gelu"), 300, 2, [1, 0], 0.05, 0.9, 2)
        run_teacher_forced(I.mlp([2600, 2200, 75], "gelu"), 300, 2, [1, 0], 0.05, 0.0, 2)
        # (the forced persistent mode also sends forward and delta through the persistent pair kernel with two
        # accumulators; here with 224-column tiles: 2600 columns = 12 tiles, the last one 136 wide)
        lpb.lp_set_tuning(448, 0, 512)
        run_teacher_forced(I.mlp([2600, 2200, 75], "gelu"), 300, 2, [1, 0], 0.05, 0.0, 2)
    finally:
        lpb.lp_set_tuning(0, 0, 0)
