"""Small, self-contained runs of single kernels on shapes of the benchmark workloads: ordinary
tests (the step must finish with a clear status word and a finite loss), sized so that a profiler
can capture one or two launches of the kernel in question without holding more than a few GB on
the device.  The ncu summaries under profiles/ name these tests in their command lines."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu


def _steps(layers, batch, n_stages, steps=3, mu=0.0, flags=0, tile=0, delays=None, lr=0.001):
    import torch
    from paper_2108_06629_b200 import binding as lpb
    from paper_2108_06629_b200 import inputs as I
    rng = np.random.default_rng(0)
    W0 = [(rng.standard_normal(I.weight_shape(l), dtype=np.float32) * np.float32(np.sqrt(2.0 / np.prod(I.weight_shape(l)[1:]))))
          for l in layers]
    b0 = [np.zeros(l["n_out"], np.float32) for l in layers]
    lpb.lp_set_tuning(tile, 0, 0)
    try:
        tr = lpb.Trainer(layers, batch, n_stages, delays=delays, lr=lr, momentum=mu,
                         flags=flags | lpb.LP_SERIAL_TASKS, W0=W0, b0=b0)
    finally:
        lpb.lp_set_tuning(0, 0, 0)
    x, y = I.minibatch(layers, batch, 0)
    xd, yd = torch.from_numpy(x).cuda(), torch.from_numpy(y).cuda()
    for _ in range(steps):
        tr.step(xd, yd)
    tr.flush()
    torch.cuda.synchronize()
    assert np.isfinite(tr.get_loss(steps - 1))
    assert tr.device_status() == (0, 0)
    tr.close()


def test_case_mlp16_layer_shapes_sm_pair_kernels():
    """Three 8192 x 8192 layers at batch 2048 (the layer shape of mlp16_8192): forward, delta and G +
    update through the SM-pair kernel, every task alone on the GPU.  About 1.3 GB on the device."""
    from paper_2108_06629_b200 import inputs as I
    _steps(I.mlp([8192] * 4, "gelu"), 2048, 3, delays=[0, 0, 0])


def test_case_mlp8_layer_shapes_weight_streaming():
    """Three 4096 x 4096 layers at batch 256 with momentum (the layer shape of mlp8_4096): the
    HBM-bound forward / delta kernels and the G kernel with the streamed update."""
    from paper_2108_06629_b200 import inputs as I
    _steps(I.mlp([4096] * 4, "gelu"), 256, 3, mu=0.9, delays=[0, 0, 0])


def test_case_vgg_block_shapes():
    """Convolution layers of the VGG workloads at reduced batch: 64 -> 64 at 112 x 112 (halo-tile kernels),
    128 -> 128 at 56 x 56, 256 -> 256 and 512 -> 512 at 28 x 28 (general kernel; SM-pair tiles with LP_CONV_PAIR=1)."""
    from paper_2108_06629_b200 import inputs as I
    _steps(I.vgg(112, [64, 64, "P", 128, 128, "P", 256, 256, 512, 512], [10]), 8, 4)


def test_case_sample_network_general_filters():
    """Table I's strided 5x5 / 3x3 layers at 224 x 224, batch 8."""
    from paper_2108_06629_b200 import inputs as I
    _steps(I.sample_net(224), 8, 3, lr=0.0005)
