"""Plain CPU statement of LayerPipe's delayed-gradient training step.

TEST INFRASTRUCTURE ONLY (see the package docstring): tests, the smoke check
and the benchmark's CPU-baseline leg are the only callers.

What it computes, per minibatch ``n`` and layer ``l = 1..L`` (paper notation):

  forward      z^l = W^l a^{l-1} (+ b^l),  a^l = f(z^l)              Eqs. 1, 2
  backward     dE/da^{l-1} = W^{l T} delta^l                          Eq. 4
               delta^{l-1} = dE/da^{l-1} (.) f'(z^{l-1})              Eq. 3
               G^l = delta^l a^{(l-1) T}                              Eq. 5
  update       W(n) = W(n-1) - eta G(n-M)                             Eq. 6

with the retimed pipeline of Section III-A: the delays that retiming leaves
between W and delta are a *weight stash*, so the forward and the backward pass
of minibatch ``n`` in layer ``l`` both read version ``v_l(n) = max(0, n - d_l)``
of that layer's weights (``d_l`` = the layer's delay, i.e. the staleness M of
Eq. 6 for that layer), and the delays between ``a`` and the backward pass are
an *activation stash*: the backward pass reuses exactly the forward values of
the same minibatch.  Written minibatch by minibatch this is a sequential loop,
which is the pipelined computation re-indexed by minibatch: the gradient of
minibatch ``n`` becomes visible to forward passes ``d_l`` minibatches later.

The split of the backward pass (Section III-B) changes nothing numerically:
G (task "G") and dE/da (task "delta") only share delta^l as input, and the
Hadamard product with f'(z^{l-1}) may be taken in either of the two
neighbouring stages.  ``dgrad_partial`` / ``apply_act_grad`` expose the two
halves so that tests can check the recombinations the paper relies on.

Readings where the paper is silent (each is listed again in the design notes):
bias is optional and treated like W; the loss is softmax cross-entropy averaged
over the minibatch, the last layer has no activation; ReLU'(0) = 0; GELU is the
exact erf form; momentum is ``m <- mu m + G, W <- W - eta m``; before the first
delayed gradient arrives (n < d_l) version 0 is used; max-pooling is 2x2
stride 2 after the activation and routes the gradient to the first maximum in
row-major scan order.

Modes.  ``mirror=False``: no rounding anywhere (used with float64 for the pins).
``mirror=True``: values are rounded to bfloat16 at exactly the places where a
bf16 tensor-core implementation stores a bf16 tensor: the input batch, each
weight version (from the fp32 master), each activation a^l (and its pooled
form), the stored z^l used for GELU', delta^L and every delta^{l-1}.  G, the
bias gradient, master weights, momentum and the loss stay in ``dtype``.
"""
import numpy as np
from scipy.special import erf  # library primitive (error function)

from .bf16 import rn_bf16

SQRT1_2 = 0.7071067811865476
INV_SQRT_2PI = 0.3989422804014327


# ----------------------------------------------------------------------------
# layer description (plain dicts so neither side shares code with the other)
# ----------------------------------------------------------------------------
def fc(n_in, n_out, act="relu", bias=True):
    return dict(kind="fc", n_in=n_in, n_out=n_out, act=act, pool=0, bias=bias)


def conv(c_in, c_out, H, W, act="relu", pool=0, bias=True, R=3, S=3, pad=1, stride=1):
    return dict(kind="conv", n_in=c_in, n_out=c_out, H=H, W=W, R=R, S=S, pad=pad,
                stride=stride, act=act, pool=pool, bias=bias)


def weight_shape(layer):
    if layer["kind"] == "fc":
        return (layer["n_out"], layer["n_in"])
    return (layer["n_out"], layer["R"], layer["S"], layer["n_in"])


def conv_out_hw(layer):
    Ho = (layer["H"] + 2 * layer["pad"] - layer["R"]) // layer["stride"] + 1
    Wo = (layer["W"] + 2 * layer["pad"] - layer["S"]) // layer["stride"] + 1
    return Ho, Wo


# ----------------------------------------------------------------------------
# Eq. 1: the linear / convolution operation and its two adjoints (Eqs. 4, 5)
# ----------------------------------------------------------------------------
def linear_forward(layer, a_prev, W):
    """z = W a (Eq. 1).  FC: a_prev [B,in], W [out,in].  Conv: NHWC input,
    W [Cout,R,S,Cin], cross-correlation with zero padding."""
    if layer["kind"] == "fc":
        return a_prev.reshape(a_prev.shape[0], -1) @ W.T
    p, st, R, S = layer["pad"], layer["stride"], layer["R"], layer["S"]
    Ho, Wo = conv_out_hw(layer)
    B = a_prev.shape[0]
    ap = np.pad(a_prev, ((0, 0), (p, p), (p, p), (0, 0)))
    z = np.zeros((B, Ho, Wo, layer["n_out"]), dtype=a_prev.dtype)
    for r in range(R):
        for s in range(S):
            patch = ap[:, r:r + st * Ho:st, s:s + st * Wo:st, :]
            z += patch @ W[:, r, s, :].T
    return z


def dgrad_partial(layer, delta, W):
    """dE/da^{l-1} = W^T delta (Eq. 4), the product *before* f' is applied.
    Written as the adjoint scatter of ``linear_forward``."""
    if layer["kind"] == "fc":
        return delta @ W
    p, st, R, S = layer["pad"], layer["stride"], layer["R"], layer["S"]
    Ho, Wo = conv_out_hw(layer)
    B = delta.shape[0]
    H, Wd = layer["H"], layer["W"]
    gp = np.zeros((B, H + 2 * p, Wd + 2 * p, layer["n_in"]), dtype=delta.dtype)
    for r in range(R):
        for s in range(S):
            gp[:, r:r + st * Ho:st, s:s + st * Wo:st, :] += delta @ W[:, r, s, :]
    return gp[:, p:p + H, p:p + Wd, :]


def wgrad(layer, delta, a_prev):
    """G = delta a^T (Eq. 5), summed over the minibatch (and pixels)."""
    if layer["kind"] == "fc":
        return delta.T @ a_prev.reshape(a_prev.shape[0], -1)
    p, st, R, S = layer["pad"], layer["stride"], layer["R"], layer["S"]
    Ho, Wo = conv_out_hw(layer)
    ap = np.pad(a_prev, ((0, 0), (p, p), (p, p), (0, 0)))
    G = np.zeros(weight_shape(layer), dtype=delta.dtype)
    d2 = delta.reshape(-1, layer["n_out"])
    for r in range(R):
        for s in range(S):
            patch = ap[:, r:r + st * Ho:st, s:s + st * Wo:st, :]
            G[:, r, s, :] = d2.T @ patch.reshape(-1, layer["n_in"])
    return G


def bias_grad(layer, delta):
    return delta.reshape(-1, layer["n_out"]).sum(axis=0)


# ----------------------------------------------------------------------------
# Eq. 2 / Eq. 3: activation and its derivative
# ----------------------------------------------------------------------------
def act_forward(name, z):
    if name == "none":
        return z
    if name == "relu":
        return np.maximum(z, 0)
    if name == "gelu":
        half = z.dtype.type(0.5)
        return half * z * (1 + erf(z * z.dtype.type(SQRT1_2)))
    raise ValueError(name)


def act_grad(name, z):
    """f'(z) of Eq. 3.  ReLU'(0) is taken as 0."""
    if name == "none":
        return np.ones_like(z)
    if name == "relu":
        return (z > 0).astype(z.dtype)
    if name == "gelu":
        t = z.dtype.type
        Phi = t(0.5) * (1 + erf(z * t(SQRT1_2)))
        phi = np.exp(-t(0.5) * z * z) * t(INV_SQRT_2PI)
        return Phi + z * phi
    raise ValueError(name)


def apply_act_grad(name, partial, z):
    """delta^{l-1} = dE/da^{l-1} (.) f'(z^{l-1}) (Eq. 3); the multiply that the
    inter-layer optimisation lets the neighbouring stage perform."""
    return partial * act_grad(name, z)


# ----------------------------------------------------------------------------
# 2x2 stride-2 max pooling (not in the paper; needed by the VGG-shaped workloads)
# ----------------------------------------------------------------------------
def maxpool2(a):
    B, H, W, C = a.shape
    cand = np.stack([a[:, 0::2, 0::2, :], a[:, 0::2, 1::2, :],
                     a[:, 1::2, 0::2, :], a[:, 1::2, 1::2, :]], axis=0)
    idx = np.argmax(cand, axis=0)  # first maximum in (dh, dw) row-major order
    out = np.take_along_axis(cand, idx[None], axis=0)[0]
    return out, idx.astype(np.uint8)


def unpool2(g, idx):
    B, Ho, Wo, C = g.shape
    up = np.zeros((B, 2 * Ho, 2 * Wo, C), dtype=g.dtype)
    for k, (dh, dw) in enumerate(((0, 0), (0, 1), (1, 0), (1, 1))):
        up[:, dh::2, dw::2, :] = np.where(idx == k, g, 0)
    return up


# ----------------------------------------------------------------------------
# loss: softmax cross-entropy, mean over the minibatch
# ----------------------------------------------------------------------------
def softmax_xent(zL, labels):
    """Returns (mean loss, dE/dz^L = (softmax - onehot)/B)."""
    B = zL.shape[0]
    zmax = zL.max(axis=1, keepdims=True)
    e = np.exp(zL - zmax)
    ssum = e.sum(axis=1, keepdims=True)
    p = e / ssum
    logp_y = (zL - zmax)[np.arange(B), labels] - np.log(ssum[:, 0])
    loss = -logp_y.mean()
    d = p.copy()
    d[np.arange(B), labels] -= 1
    return loss, d / zL.dtype.type(B)


# ----------------------------------------------------------------------------
# the training recursion
# ----------------------------------------------------------------------------
class DelayedGradientTrainer:
    """State: per layer the master W, b (``dtype``), momentum, and the stash of
    the last ``d_l + 1`` weight versions (Section III-A: delays between W and
    delta).  ``step`` processes one minibatch."""

    def __init__(self, layers, delays, lr, momentum, W0, b0, mirror=True, dtype=np.float32):
        assert len(layers) == len(delays) == len(W0)
        self.layers = [dict(l) for l in layers]
        self.delays = [int(d) for d in delays]
        self.dtype = np.dtype(dtype)
        self.lr = self.dtype.type(lr)
        self.mu = self.dtype.type(momentum)
        self.mirror = bool(mirror)
        self.W = [np.array(w, dtype=self.dtype).reshape(weight_shape(l)) for w, l in zip(W0, layers)]
        self.b = [np.array(b0[i], dtype=self.dtype) if l["bias"] else None
                  for i, l in enumerate(layers)]
        self.mW = [np.zeros_like(w) for w in self.W]
        self.mb = [np.zeros_like(b) if b is not None else None for b in self.b]
        self.n = 0
        # stash[l][v] = (operand form of W^{[v]}, b^{[v]}); version 0 = initial weights
        self.stash = [{0: (self._Q(w), None if b is None else b.copy())}
                      for w, b in zip(self.W, self.b)]

    def _Q(self, x):
        return rn_bf16(x).astype(self.dtype) if self.mirror else x

    def version(self, l, n):
        """Weight version read by minibatch n in layer l (0-based l)."""
        return max(0, n - self.delays[l])

    def step(self, batch, labels, capture=False):
        L = len(self.layers)
        n = self.n
        labels = np.asarray(labels).astype(np.int64)
        rec = dict(step=n, v=[self.version(l, n) for l in range(L)])
        rec["slot"] = [rec["v"][l] % (self.delays[l] + 1) for l in range(L)]

        # ---- forward (Eqs. 1, 2) with the stashed weight version -------------
        a = [None] * (L + 1)      # a[l] = input of layer l (0-based) = output of layer l-1
        zs = [None] * L           # stored pre-activation (what f' is evaluated on)
        amax = [None] * L         # pooling argmax
        a[0] = self._Q(np.asarray(batch, dtype=self.dtype))
        for l, lay in enumerate(self.layers):
            Wv, bv = self.stash[l][rec["v"][l]]
            x = a[l]
            if lay["kind"] == "conv" and x.ndim == 2:
                x = x.reshape(x.shape[0], lay["H"], lay["W"], lay["n_in"])
            z = linear_forward(lay, x, Wv)
            if bv is not None:
                z = z + bv
            if l == L - 1:
                assert lay["act"] == "none"
                zL = z
                break
            zs[l] = self._Q(z)
            out = self._Q(act_forward(lay["act"], z))
            if lay["pool"]:
                out, amax[l] = maxpool2(out)
            a[l + 1] = out

        # ---- loss and delta^L -------------------------------------------------
        loss, dL = softmax_xent(zL, labels)
        delta = self._Q(dL)
        rec["loss"] = float(loss)

        # ---- backward: G and delta are independent given delta^l --------------
        dW = [None] * L
        db = [None] * L
        deltas = [None] * L
        for l in range(L - 1, -1, -1):
            lay = self.layers[l]
            Wv, _ = self.stash[l][rec["v"][l]]          # same version as the forward pass
            x = a[l]
            if lay["kind"] == "conv" and x.ndim == 2:
                x = x.reshape(x.shape[0], lay["H"], lay["W"], lay["n_in"])
            if lay["kind"] == "fc" and delta.ndim != 2:
                delta = delta.reshape(delta.shape[0], -1)
            deltas[l] = delta
            dW[l] = wgrad(lay, delta, x)                               # task G      (Eq. 5)
            db[l] = bias_grad(lay, delta) if lay["bias"] else None
            if l > 0:
                prev = self.layers[l - 1]
                partial = dgrad_partial(lay, delta, Wv)                # task delta  (Eq. 4)
                if prev["pool"]:
                    partial = partial.reshape(amax[l - 1].shape)
                    partial = unpool2(partial, amax[l - 1])
                partial = partial.reshape(zs[l - 1].shape)
                delta = self._Q(apply_act_grad(prev["act"], partial, zs[l - 1]))   # Eq. 3

        # ---- update (Eq. 6); the new version joins the stash -------------------
        for l in range(L):
            self.mW[l] = self.mu * self.mW[l] + dW[l]
            self.W[l] = self.W[l] - self.lr * self.mW[l]
            if self.b[l] is not None:
                self.mb[l] = self.mu * self.mb[l] + db[l]
                self.b[l] = self.b[l] - self.lr * self.mb[l]
            st = self.stash[l]
            st[n + 1] = (self._Q(self.W[l]), None if self.b[l] is None else self.b[l].copy())
            for old in [v for v in st if v < n + 1 - self.delays[l]]:
                del st[old]                            # the ring keeps d_l + 1 versions
        self.n = n + 1
        rec["dW"], rec["db"] = dW, db
        if capture:
            rec["a"], rec["zs"], rec["delta"], rec["zL"], rec["amax"] = a, zs, deltas, zL, amax
        return rec

    def weights(self):
        """Master weights after every gradient computed so far has been applied
        (version ``self.n`` in every layer)."""
        return [w.copy() for w in self.W], [None if b is None else b.copy() for b in self.b]
