"""lp_softmax_xent_static: the loss kernel for callers that have no workspace to offer and
may not allocate one (see the header).  Its scratch is a fixed array inside the library,
so this test checks what such a caller relies on: the results equal those of the loss task
run through a trainer handle on the same logits and labels, on two calls in a row (the
second call finds the first call's leftovers in the shared scratch), and oversize batches
are refused without launching anything.

Collected last on purpose (file name): a failure here cannot mask any other test."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu


def _through_handle(tr, n, logits, labels):
    tr.debug_write("logits", 0, n, logits)
    tr.debug_write("labels", 0, n, labels.astype(np.float32))
    tr.debug_run_task("loss", 0, n)
    L = len(tr.layers)
    return tr.debug_read("delta", L - 1, n), float(tr.debug_read("loss", 0, n)[0])


def test_static_scratch_loss_matches_handle_loss_twice_in_a_row():
    import torch
    from paper_2108_06629_b200 import binding as lpb
    from paper_2108_06629_b200 import inputs as I

    batch, classes = 200, 1003                     # ragged: 1003 is not a multiple of 8
    layers = I.mlp([64, classes], "relu")
    W0, b0 = I.initial_weights(layers, 0)
    tr = lpb.Trainer(layers, batch, 1, W0=W0, b0=b0)
    ld = (classes + 7) // 8 * 8
    rng = np.random.default_rng(77)
    for call in range(2):                          # two calls in a row on the shared scratch
        logits = (rng.standard_normal((batch, classes)) * (3.0 + 5.0 * call)).astype(np.float32)
        labels = rng.integers(0, classes, size=batch).astype(np.int32)
        want_delta, want_loss = _through_handle(tr, call, logits, labels)

        lg = torch.zeros((batch, ld), dtype=torch.float32, device="cuda")
        lg[:, :classes] = torch.from_numpy(logits).cuda()
        lb = torch.from_numpy(labels).cuda()
        delta = torch.full((batch, ld), 7.0, dtype=torch.bfloat16, device="cuda")
        loss = torch.full((1,), -1.0, dtype=torch.float32, device="cuda")
        rc = lpb.lp_softmax_xent_static(lg, lb, delta, loss, classes)
        assert rc == lpb.LP_OK
        torch.cuda.synchronize()
        got_delta = delta.float().cpu().numpy()
        # same kernel, same inputs: bf16 results must agree to the bit, the loss to fp32 round-off
        assert np.array_equal(got_delta[:, :classes], want_delta)
        assert np.all(got_delta[:, classes:] == 0.0)
        assert abs(float(loss.item()) - want_loss) <= 1e-6 * max(1.0, abs(want_loss))
        # and the loss is what its definition says (float64, from the same logits)
        z = logits.astype(np.float64)
        lse = np.log(np.exp(z - z.max(1, keepdims=True)).sum(1)) + z.max(1)
        assert abs(float(loss.item()) - float(np.mean(lse - z[np.arange(batch), labels]))) < 1e-4
    tr.close()


def test_static_scratch_loss_refuses_what_does_not_fit():
    import torch
    from paper_2108_06629_b200 import binding as lpb
    big = lpb.LP_XENT_STATIC_MAX_BATCH + 1
    lg = torch.zeros((big, 8), dtype=torch.float32, device="cuda")
    lb = torch.zeros((big,), dtype=torch.int32, device="cuda")
    delta = torch.full((big, 8), 7.0, dtype=torch.bfloat16, device="cuda")
    loss = torch.full((1,), -1.0, dtype=torch.float32, device="cuda")
    assert lpb.lp_softmax_xent_static(lg, lb, delta, loss, 8) == lpb.LP_ERR_INVALID_ARG
    torch.cuda.synchronize()
    assert float(loss.item()) == -1.0 and float(delta.float().min().item()) == 7.0     # nothing ran
    # pitch too small for the padded row, and the largest batch that does fit
    narrow = torch.zeros((16, 4), dtype=torch.bfloat16, device="cuda")
    assert lpb.lp_softmax_xent_static(lg[:16], lb[:16], narrow, loss, 8) == lpb.LP_ERR_INVALID_ARG
    ok = lpb.LP_XENT_STATIC_MAX_BATCH
    assert lpb.lp_softmax_xent_static(lg[:ok], lb[:ok], delta[:ok], loss, 8) == lpb.LP_OK
    torch.cuda.synchronize()
    # all-zero logits: uniform softmax, loss = log 8 (16384 row losses added in fp32)
    assert abs(float(loss.item()) - np.log(8.0)) < 1e-3 * np.log(8.0)
    # the refusals say why
    assert lpb.lp_softmax_xent_static(lg, lb, delta, loss, 8) == lpb.LP_ERR_INVALID_ARG
    assert b"LP_XENT_STATIC_MAX_BATCH" in lpb.lib().lp_last_error(None)


def test_static_scratch_loss_never_uses_a_bad_label_as_an_address():
    """This entry point has no status word to report through, so a label outside [0, classes)
    shows up as a NaN loss; the rows with valid labels are unaffected and nothing faults."""
    import torch
    from paper_2108_06629_b200 import binding as lpb
    batch, classes = 16, 8
    lg = torch.zeros((batch, classes), dtype=torch.float32, device="cuda")
    delta = torch.zeros((batch, classes), dtype=torch.bfloat16, device="cuda")
    loss = torch.zeros((1,), dtype=torch.float32, device="cuda")
    for bad in (8, -1, 2 ** 31 - 1):
        lb = torch.zeros((batch,), dtype=torch.int32, device="cuda")
        lb[5] = bad
        assert lpb.lp_softmax_xent_static(lg, lb, delta, loss, classes) == lpb.LP_OK
        torch.cuda.synchronize()
        assert np.isnan(float(loss.item()))
        d = delta.float().cpu().numpy()
        assert abs(d[0, 0] - (1.0 / 8 - 1.0) / batch) < 1e-3 and abs(d[5, 0] - (1.0 / 8) / batch) < 1e-3
    lb = torch.zeros((batch,), dtype=torch.int32, device="cuda")
    assert lpb.lp_softmax_xent_static(lg, lb, delta, loss, classes) == lpb.LP_OK
    torch.cuda.synchronize()
    assert abs(float(loss.item()) - np.log(8.0)) < 1e-5
