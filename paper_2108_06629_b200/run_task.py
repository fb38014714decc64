"""Run one task kind of one layer a few times on a workload, device otherwise idle.

    python -m paper_2108_06629_b200.run_task WORKLOAD TASK LAYER REPS

TASK is forward | delta | G | update | loss.  Meant to be wrapped by a profiler: the handle
is created once, operands are filled with seeded random values through the verification
access of the library, then the task's kernel(s) run REPS times through lp_debug_run_task.
"""
import sys

import numpy as np


def main(argv):
    import torch
    from . import binding as lpb
    from . import inputs as I
    name, task, layer, reps = argv[0], argv[1], int(argv[2]), int(argv[3])
    wl = I.WORKLOADS[name]
    layers, B = wl["layers"], wl["batch"]
    rng = np.random.default_rng(0)
    W0 = [(rng.standard_normal(I.weight_shape(l), dtype=np.float32) *
           np.float32(np.sqrt(2.0 / np.prod(I.weight_shape(l)[1:])))) for l in layers]
    b0 = [np.zeros(l["n_out"], np.float32) for l in layers]
    tr = lpb.Trainer(layers, B, wl["stages"], delays=wl["delays"], lr=wl["lr"], momentum=wl["momentum"], W0=W0, b0=b0)
    step = 3
    tr.debug_write("input", layer, step, rng.standard_normal(tr._buf_shape("input", layer), dtype=np.float32))
    tr.debug_write("delta", layer, step, rng.standard_normal(tr._buf_shape("delta", layer), dtype=np.float32) * 1e-3)
    tr.debug_write("labels", 0, step, rng.integers(0, layers[-1]["n_out"], size=B).astype(np.float32))
    for _ in range(reps):
        tr.debug_run_task(task, layer, step)
    torch.cuda.synchronize()
    print("done", tr.device_status())
    tr.close()


if __name__ == "__main__":
    main(sys.argv[1:])
