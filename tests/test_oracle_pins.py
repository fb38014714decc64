"""Pins for the CPU oracle: each test checks it against something other than
itself (torch's autograd as the textbook special case, finite differences,
closed forms that the delayed-gradient recursion must satisfy, torch's own
bf16 cast).  None of these needs a GPU."""
import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import layerpipe_oracle as O
from oracle.bf16 import rn_bf16
from paper_2108_06629_b200 import inputs as I

torch.set_num_threads(4)


# ----------------------------------------------------------------------------
# an independent statement of the same network in torch (autograd does the
# backward pass); weights are handed in, so any mix of versions can be probed
# ----------------------------------------------------------------------------
def torch_loss_and_grads(layers, Ws, bs, x, y):
    Wt = [torch.tensor(w, dtype=torch.float64, requires_grad=True) for w in Ws]
    bt = [torch.tensor(b, dtype=torch.float64, requires_grad=True) for b in bs]
    h = torch.tensor(x, dtype=torch.float64)
    if layers[0]["kind"] == "conv":
        h = h.permute(0, 3, 1, 2)                      # NHWC -> NCHW
    for l, lay in enumerate(layers):
        if lay["kind"] == "fc":
            if h.dim() == 4:
                h = h.permute(0, 2, 3, 1).reshape(h.shape[0], -1)   # flatten in (h, w, c) order
            h = F.linear(h, Wt[l], bt[l] if lay["bias"] else None)
        else:
            h = F.conv2d(h, Wt[l].permute(0, 3, 1, 2), bt[l] if lay["bias"] else None,
                         stride=lay["stride"], padding=lay["pad"])
        if lay["act"] == "relu":
            h = F.relu(h)
        elif lay["act"] == "gelu":
            h = F.gelu(h)
        if lay["pool"]:
            h = F.max_pool2d(h, 2, 2)
    loss = F.cross_entropy(h, torch.tensor(y, dtype=torch.long))
    loss.backward()
    return float(loss.detach()), [w.grad.numpy() for w in Wt], [b.grad.numpy() for b in bt]


def rel(a, b):
    return np.linalg.norm((a - b).ravel()) / max(np.linalg.norm(b.ravel()), 1e-300)


def tiny_mlp(act):
    return I.mlp([12, 9, 7, 5], act)


def tiny_cnn():
    return I.vgg(8, [4, 6, "P", 5, "P"], [7, 3])


def make(layers, batch, steps, seed=3):
    rng = np.random.default_rng(seed)
    W0 = [rng.standard_normal(I.weight_shape(l)) * np.sqrt(2.0 / np.prod(I.weight_shape(l)[1:]))
          for l in layers]
    b0 = [rng.standard_normal(l["n_out"]) * 0.1 for l in layers]
    xs = [rng.standard_normal(I.input_shape(layers, batch)) for _ in range(steps)]
    ys = [rng.integers(0, layers[-1]["n_out"], size=batch) for _ in range(steps)]
    return W0, b0, xs, ys


# ----------------------------------------------------------------------------
def test_bf16_rounding_matches_torch_cast_exhaustively():
    hi = np.arange(1 << 16, dtype=np.uint32) << np.uint32(16)
    for low in (0x0000, 0x0001, 0x7FFF, 0x8000, 0x8001, 0xFFFF, 0x1234, 0xC000):
        bits = (hi | np.uint32(low)).astype(np.uint32)
        x = bits.view(np.float32)
        want = torch.from_numpy(x.copy()).to(torch.bfloat16).to(torch.float32).numpy()
        got = rn_bf16(x)
        nan = np.isnan(want)
        assert np.array_equal(np.isnan(got), nan)
        assert np.array_equal(got[~nan].view(np.uint32), want[~nan].view(np.uint32))


@pytest.mark.parametrize("net,mu", [("relu", 0.0), ("gelu", 0.9), ("cnn", 0.5)])
def test_zero_delay_is_textbook_backprop_with_sgd(net, mu):
    layers = tiny_cnn() if net == "cnn" else tiny_mlp(net)
    B, N, lr = 6, 4, 0.05
    W0, b0, xs, ys = make(layers, B, N)
    tr = O.DelayedGradientTrainer(layers, [0] * len(layers), lr, mu, W0, b0, mirror=False,
                                  dtype=np.float64)
    Wt = [w.copy() for w in W0]
    bt = [b.copy() for b in b0]
    mW = [np.zeros_like(w) for w in W0]
    mb = [np.zeros_like(b) for b in b0]
    for n in range(N):
        rec = tr.step(xs[n], ys[n])
        loss, gW, gb = torch_loss_and_grads(layers, Wt, bt, xs[n], ys[n])
        assert abs(rec["loss"] - loss) < 1e-10
        for l in range(len(layers)):
            assert rel(rec["dW"][l], gW[l]) < 1e-10
            assert rel(rec["db"][l], gb[l]) < 1e-10
            mW[l] = mu * mW[l] + gW[l]
            Wt[l] = Wt[l] - lr * mW[l]
            mb[l] = mu * mb[l] + gb[l]
            bt[l] = bt[l] - lr * mb[l]
    Wf, bf = tr.weights()
    for l in range(len(layers)):
        assert rel(Wf[l], Wt[l]) < 1e-10 and rel(bf[l], bt[l]) < 1e-10


def test_gradients_match_central_finite_differences():
    layers = I.mlp([5, 4, 3], "gelu")
    B = 3
    W0, b0, xs, ys = make(layers, B, 1, seed=11)
    rec = O.DelayedGradientTrainer(layers, [0, 0], 0.0, 0.0, W0, b0, mirror=False,
                                   dtype=np.float64).step(xs[0], ys[0])

    def loss_at(Ws, bs):
        return O.DelayedGradientTrainer(layers, [0, 0], 0.0, 0.0, Ws, bs, mirror=False,
                                        dtype=np.float64).step(xs[0], ys[0])["loss"]
    eps = 1e-6
    for l in range(2):
        num = np.zeros_like(W0[l])
        for idx in np.ndindex(*W0[l].shape):
            Wp = [w.copy() for w in W0]
            Wm = [w.copy() for w in W0]
            Wp[l][idx] += eps
            Wm[l][idx] -= eps
            num[idx] = (loss_at(Wp, b0) - loss_at(Wm, b0)) / (2 * eps)
        assert rel(rec["dW"][l], num) < 1e-6
        numb = np.zeros_like(b0[l])
        for i in range(len(b0[l])):
            bp = [b.copy() for b in b0]
            bm = [b.copy() for b in b0]
            bp[l][i] += eps
            bm[l][i] -= eps
            numb[i] = (loss_at(W0, bp) - loss_at(W0, bm)) / (2 * eps)
        assert rel(rec["db"][l], numb) < 1e-6


@pytest.mark.parametrize("net,delays", [("relu", [2, 1, 0]), ("gelu", [4, 2, 0]),
                                        ("gelu", [1, 3, 2]), ("cnn", [3, 2, 1, 0, 0])])
def test_delayed_gradients_follow_the_stashed_weight_recursion(net, delays):
    """Eq. 6 with weight stashing, restated with torch: keep the history of all
    weight versions; minibatch n's gradient is autograd's gradient at the mixed
    point {W_l^{[max(0,n-d_l)]}}; version n+1 = version n - lr * that gradient."""
    layers = tiny_cnn() if net == "cnn" else tiny_mlp(net)
    L = len(layers)
    B, N, lr, mu = 5, 8, 0.1, 0.0
    W0, b0, xs, ys = make(layers, B, N, seed=5)
    tr = O.DelayedGradientTrainer(layers, delays, lr, mu, W0, b0, mirror=False, dtype=np.float64)
    histW = [[w.copy()] for w in W0]
    histb = [[b.copy()] for b in b0]
    for n in range(N):
        v = [max(0, n - d) for d in delays]
        rec = tr.step(xs[n], ys[n])
        assert rec["v"] == v
        loss, gW, gb = torch_loss_and_grads(layers, [histW[l][v[l]] for l in range(L)],
                                            [histb[l][v[l]] for l in range(L)], xs[n], ys[n])
        assert abs(rec["loss"] - loss) < 1e-10
        for l in range(L):
            assert rel(rec["dW"][l], gW[l]) < 1e-9
            histW[l].append(histW[l][n] - lr * gW[l])
            histb[l].append(histb[l][n] - lr * gb[l])
    Wf, bf = tr.weights()
    for l in range(L):
        assert rel(Wf[l], histW[l][N]) < 1e-10 and rel(bf[l], histb[l][N]) < 1e-10


def test_zero_step_size_makes_every_delay_setting_agree():
    layers = tiny_mlp("gelu")
    W0, b0, xs, ys = make(layers, 4, 5)
    runs = []
    for delays in ([0, 0, 0], [2, 1, 0], [4, 2, 0]):
        tr = O.DelayedGradientTrainer(layers, delays, 0.0, 0.9, W0, b0, mirror=False, dtype=np.float64)
        runs.append([tr.step(xs[n], ys[n])["dW"] for n in range(5)])
    for other in runs[1:]:
        for n in range(5):
            for l in range(3):
                assert np.array_equal(other[n][l], runs[0][n][l])


def test_warm_up_closed_form():
    """While n <= min_l d_l every minibatch still reads version 0, so
    W^{[k]} = W^{[0]} - lr * sum_{n<k} grad E_n(W^{[0]}) for k <= min d + 1."""
    layers = tiny_mlp("relu")
    delays = [4, 3, 2]
    lr = 0.2
    W0, b0, xs, ys = make(layers, 4, 3)
    tr = O.DelayedGradientTrainer(layers, delays, lr, 0.0, W0, b0, mirror=False, dtype=np.float64)
    acc = [np.zeros_like(w) for w in W0]
    for n in range(3):
        tr.step(xs[n], ys[n])
        _, gW, _ = torch_loss_and_grads(layers, W0, b0, xs[n], ys[n])
        for l in range(3):
            acc[l] += gW[l]
    Wf, _ = tr.weights()
    for l in range(3):
        assert rel(Wf[l], W0[l] - lr * acc[l]) < 1e-12


def test_version_and_slot_log():
    layers = tiny_mlp("relu")
    W0, b0, xs, ys = make(layers, 2, 9)
    for delays in ([2, 1, 0], [4, 2, 0]):          # one per stage after, and the paper's 2 x count
        tr = O.DelayedGradientTrainer(layers, delays, 0.01, 0.0, W0, b0)
        for n in range(9):
            rec = tr.step(xs[n], ys[n])
            assert rec["v"] == [max(0, n - d) for d in delays]
            assert rec["slot"] == [max(0, n - d) % (d + 1) for d in delays]
            # the stash never holds more than d_l + 1 versions (+ the one just produced)
            assert all(len(tr.stash[l]) <= delays[l] + 1 for l in range(3))


def test_split_delta_recombines():
    """Section III-B: delta is parallel over its output channels (delta', delta''
    concatenate) and over the contraction (partial sums add); applying f' after
    the product equals the fused form."""
    rng = np.random.default_rng(2)
    lay = O.fc(24, 18)
    delta = rng.standard_normal((7, 18))
    W = rng.standard_normal((18, 24))
    z = rng.standard_normal((7, 24))
    whole = O.dgrad_partial(lay, delta, W)
    cut = 16                                          # two thirds / one third of dX's channels
    d1 = O.dgrad_partial(O.fc(cut, 18), delta, W[:, :cut])
    d2 = O.dgrad_partial(O.fc(24 - cut, 18), delta, W[:, cut:])
    assert np.array_equal(np.concatenate([d1, d2], axis=1), whole)
    k = 11
    s1 = O.dgrad_partial(O.fc(24, k), delta[:, :k], W[:k])
    s2 = O.dgrad_partial(O.fc(24, 18 - k), delta[:, k:], W[k:])
    assert rel(s1 + s2, whole) < 1e-14
    fused = whole * O.act_grad("gelu", z)
    assert np.array_equal(O.apply_act_grad("gelu", whole, z), fused)
    # conv: split over the input channels of the layer (= channels of dX)
    cl = O.conv(6, 5, 4, 4)
    dc = rng.standard_normal((2, 4, 4, 5))
    Wc = rng.standard_normal((5, 3, 3, 6))
    wc = O.dgrad_partial(cl, dc, Wc)
    c1 = O.dgrad_partial(O.conv(4, 5, 4, 4), dc, Wc[..., :4])
    c2 = O.dgrad_partial(O.conv(2, 5, 4, 4), dc, Wc[..., 4:])
    assert np.array_equal(np.concatenate([c1, c2], axis=-1), wc)


def test_conv_adjoint_identity():
    """<conv(x, W), d> = <x, dgrad(d, W)> = <W, wgrad(d, x)> for the same W, x, d."""
    rng = np.random.default_rng(4)
    for stride, R, pad in ((1, 3, 1), (2, 3, 1), (2, 5, 2)):
        lay = O.conv(3, 4, 9, 9, R=R, S=R, pad=pad, stride=stride)
        x = rng.standard_normal((2, 9, 9, 3))
        W = rng.standard_normal(O.weight_shape(lay))
        z = O.linear_forward(lay, x, W)
        d = rng.standard_normal(z.shape)
        lhs = float((z * d).sum())
        assert abs(lhs - float((x * O.dgrad_partial(lay, d, W)).sum())) < 1e-9 * abs(lhs)
        assert abs(lhs - float((W * O.wgrad(lay, d, x)).sum())) < 1e-9 * abs(lhs)


def test_pool_routes_to_first_maximum():
    a = np.zeros((1, 2, 2, 1))
    out, idx = O.maxpool2(a)                        # four-way tie
    assert idx[0, 0, 0, 0] == 0
    up = O.unpool2(np.ones((1, 1, 1, 1)), idx)
    assert up[0, :, :, 0].tolist() == [[1, 0], [0, 0]]
    a[0, 1, 0, 0] = 3.0
    a[0, 1, 1, 0] = 3.0
    _, idx = O.maxpool2(a)
    assert idx[0, 0, 0, 0] == 2


def test_mirror_mode_stays_close_to_exact_and_rounds_operands():
    wl = I.WORKLOADS["mlp4_784"]
    layers = wl["layers"]
    W0, b0 = I.initial_weights(layers, 0)
    pure = O.DelayedGradientTrainer(layers, wl["delays"], wl["lr"], 0.0, W0, b0, mirror=False,
                                    dtype=np.float64)
    mir = O.DelayedGradientTrainer(layers, wl["delays"], wl["lr"], 0.0, W0, b0, mirror=True,
                                   dtype=np.float32)
    for n in range(3):
        x, y = I.minibatch(layers, wl["batch"], n)
        rp = pure.step(x, y)
        rm = mir.step(x, y, capture=True)
        for l in range(4):
            assert rel(rm["dW"][l].astype(np.float64), rp["dW"][l]) < 0.15   # sanity bound only: bf16 operands, ReLU gates may flip
        for t in rm["a"][:4] + rm["delta"]:
            assert np.array_equal(rn_bf16(t), t)      # operands really are bf16 values
        assert rm["dW"][0].dtype == np.float32


# ----------------------------------------------------------------------------
# where mirror mode rounds: an independent restatement with torch's own bf16 cast
# ----------------------------------------------------------------------------
def _tq(t):
    """Round a float64 torch tensor to bf16 the way a bf16 store does (via binary32)."""
    return t.float().bfloat16().double()


def test_mirror_mode_rounding_points_are_where_a_bf16_store_happens():
    """Mirror mode must round the weight VERSION handed to the contractions (not the master), the
    STORED z (not the z the activation is computed from), each activation, delta^L and each
    delta^{l-1} once, after the product with f'.  Restated here for a two-layer GELU net with
    torch's bf16 cast; a dropped or misplaced rounding in the oracle changes thousands of elements
    by a bf16 spacing (4e-3 relative), the comparison is exact."""
    rng = np.random.default_rng(3)
    B, n0, n1, n2, lr = 12, 40, 56, 10, 0.37
    layers = [O.fc(n0, n1, "gelu"), O.fc(n1, n2, "none")]
    W = [rng.standard_normal((n1, n0)) * 0.2, rng.standard_normal((n2, n1)) * 0.2]     # not bf16 values
    b = [rng.standard_normal(n1) * 0.1, rng.standard_normal(n2) * 0.1]
    orc = O.DelayedGradientTrainer(layers, [0, 0], lr, 0.0, W, b, mirror=True, dtype=np.float64)
    Wt = [torch.tensor(w) for w in W]
    bt = [torch.tensor(v) for v in b]
    assert not np.array_equal(rn_bf16(W[0]), W[0].astype(np.float32))
    for n in range(2):
        x = rng.standard_normal((B, n0))
        y = rng.integers(0, n2, size=B)
        rec = orc.step(x, y, capture=True)
        # the version in the stash is the rounded one, the master is not
        assert np.array_equal(orc.stash[0][n + 1][0], rn_bf16(orc.W[0]).astype(np.float64))
        assert not np.array_equal(orc.W[0], rn_bf16(orc.W[0]).astype(np.float64))
        x0 = _tq(torch.tensor(x))
        W1q, W2q = _tq(Wt[0]), _tq(Wt[1])
        z1 = x0 @ W1q.T + bt[0]                                   # bias stays fp32/fp64: not rounded
        zs1 = _tq(z1)
        a1 = _tq(F.gelu(z1))                                      # f of the UNROUNDED z
        zL = a1 @ W2q.T + bt[1]
        p = torch.softmax(zL, dim=1)
        p[torch.arange(B), torch.tensor(y)] -= 1.0
        dL = _tq(p / B)
        Phi = 0.5 * (1 + torch.erf(zs1 / np.sqrt(2.0)))
        fprime = Phi + zs1 * torch.exp(-0.5 * zs1 * zs1) / np.sqrt(2 * np.pi)   # f' on the STORED z
        d1 = _tq((dL @ W2q) * fprime)                             # one rounding, after the product
        G2, G1 = dL.T @ a1, d1.T @ x0
        assert np.array_equal(rec["a"][0], x0.numpy())
        assert np.array_equal(rec["zs"][0], zs1.numpy())
        assert np.array_equal(rec["a"][1], a1.numpy())
        assert np.array_equal(rec["delta"][1], dL.numpy())
        assert np.array_equal(rec["delta"][0], d1.numpy())
        assert np.allclose(rec["zL"], zL.numpy(), rtol=0, atol=1e-12)
        assert np.allclose(rec["dW"][1], G2.numpy(), rtol=0, atol=1e-12)
        assert np.allclose(rec["dW"][0], G1.numpy(), rtol=0, atol=1e-12)
        # sensitivity of this very test: each alternative placement is visibly different
        assert not np.array_equal(_tq(F.gelu(zs1)).numpy(), a1.numpy())            # f of the rounded z
        assert not np.array_equal(_tq(x0 @ Wt[0].T + bt[0]).numpy(), zs1.numpy())  # unrounded weights
        assert not np.array_equal(_tq(_tq(dL @ W2q) * fprime).numpy(), d1.numpy())  # two roundings
        Wt = [Wt[0] - lr * G1, Wt[1] - lr * G2]                   # Eq. 6 on the master
        bt = [bt[0] - lr * d1.sum(0), bt[1] - lr * dL.sum(0)]
        assert np.allclose(orc.W[0], Wt[0].numpy(), rtol=0, atol=1e-12)


def test_mac_costs_count_the_multiply_accumulates_of_the_direct_loops():
    """The planner's cost model says a layer costs B*Ho*Wo*Cout*R*S*Cin multiply-accumulates (FC:
    B*in*out).  Counted here by running the direct loops of Eq. 1 over the zero-padded input, one
    increment per multiply-accumulate; the loops' result is also the oracle's forward."""
    from oracle import partition_oracle as P
    rng = np.random.default_rng(4)
    B = 2
    lay = O.conv(3, 4, 7, 6, act="none", R=5, S=3, pad=2, stride=2)
    x = rng.standard_normal((B, 7, 6, 3))
    W = rng.standard_normal(O.weight_shape(lay))
    Ho, Wo = O.conv_out_hw(lay)
    xp = np.pad(x, ((0, 0), (2, 2), (2, 2), (0, 0)))
    z = np.zeros((B, Ho, Wo, 4))
    macs = 0
    for n in range(B):
        for ho in range(Ho):
            for wo in range(Wo):
                for co in range(4):
                    for r in range(5):
                        for s in range(3):
                            for ci in range(3):
                                z[n, ho, wo, co] += xp[n, 2 * ho + r, 2 * wo + s, ci] * W[co, r, s, ci]
                                macs += 1
    assert np.allclose(z, O.linear_forward(lay, x, W), atol=1e-12)
    fcl = O.fc(11, 5, "none")
    fix, flex = P.mac_costs([lay, fcl], B)
    assert fix[0] == 2 * macs and flex[0] == 0              # forward + G; the first layer has no delta
    assert fix[1] == 2 * (B * 11 * 5) and flex[1] == B * 11 * 5
    fix, flex = P.mac_costs([fcl, lay], B)
    assert flex[1] == macs                                  # delta costs one contraction
