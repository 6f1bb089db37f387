"""Losses and gradients f(w; xi) of the two model families, in fp64.

TEST INFRASTRUCTURE (see the package header).

The paper states the problem as finite-sum minimisation of f(w; xi) (Eq. 1)
solved by the SGD recursion w <- w - eta * grad f(w; xi) (Eq. 3) and names
logistic regression and neural networks as instances; it fixes no model
details, so these are the build's own:

* softmax cross-entropy with natural log, the row maximum subtracted first;
* a bias in every layer; parameters flattened layer by layer, W_l row-major
  [in, out] followed by b_l;
* the l2 term (lambda / 2) * |W|^2 on weight matrices only;
* ReLU hidden units with derivative 0 at 0;
* a minibatch gradient is the mean over its B samples.

precision = 1 models bf16 operands with wide accumulation: values are rounded
to the nearest bf16 (ties to even) where the low-precision path rounds them -
the inputs, each W_l read from the master copy, each hidden activation after
bias + ReLU, and each dZ_l before the two backward products - while logits,
softmax, bias gradients, the gradient itself and the master update stay wide.
"""
import numpy as np


def round_bf16(a):
    """Nearest bf16 value (ties to even) of each fp64 entry, returned as fp64.

    bf16 keeps 7 stored mantissa bits; fp64 has 52, so 45 bits are dropped.
    Values are assumed to lie in bf16's normal range (or be zero)."""
    a = np.ascontiguousarray(a, dtype=np.float64)
    bits = a.view(np.uint64)
    drop = np.uint64(45)
    one = np.uint64(1)
    lsb = (bits >> drop) & one
    rounded = bits + ((one << np.uint64(44)) - one) + lsb
    rounded &= ~((one << drop) - one)
    return rounded.view(np.float64).reshape(a.shape)


def unpack(w, dims):
    """Views (W_l [in, out], b_l [out]) into the flat parameter vector."""
    out, o = [], 0
    for l in range(len(dims) - 1):
        i, j = dims[l], dims[l + 1]
        W = w[o:o + i * j].reshape(i, j)
        o += i * j
        b = w[o:o + j]
        o += j
        out.append((W, b))
    assert o == w.size
    return out


def softmax_rows(Z):
    Z = Z - Z.max(axis=1, keepdims=True)
    E = np.exp(Z)
    return E / E.sum(axis=1, keepdims=True)


def _ce(P, y):
    return -np.log(P[np.arange(len(y)), y])


def loss_and_grad(w, X, y, dims, l2=0.0, precision=0):
    """Mean loss over the rows of X (plus the l2 term) and its gradient (flat).

    Covers softmax regression (len(dims) == 2) and ReLU MLPs alike: the
    regression is the network without hidden layers."""
    w = np.asarray(w, dtype=np.float64)
    X = np.asarray(X, dtype=np.float64)
    q = round_bf16 if precision == 1 else (lambda v: v)
    layers = unpack(w, dims)
    B = X.shape[0]
    L = len(layers)
    Wq = [q(W) for W, _ in layers]
    A = [q(X)]
    Z = []
    for l in range(L):
        z = A[l] @ Wq[l] + layers[l][1]
        Z.append(z)
        if l < L - 1:
            A.append(q(np.maximum(z, 0.0)))
    P = softmax_rows(Z[-1])
    loss = _ce(P, y).mean() + 0.5 * l2 * sum((W * W).sum() for W, _ in layers)
    g = np.empty_like(w)
    glayers = unpack(g, dims)
    dZ = P.copy()
    dZ[np.arange(B), y] -= 1.0
    dZ *= 1.0 / B
    for l in range(L - 1, -1, -1):
        gW, gb = glayers[l]
        dZq = q(dZ)
        gW[...] = A[l].T @ dZq + l2 * layers[l][0]
        gb[...] = dZ.sum(axis=0)
        if l > 0:
            dA = dZq @ Wq[l].T
            dZ = dA * (Z[l - 1] > 0.0)
    return loss, g


# ---- a small convolutional classifier (the paper trains LeNet on its 28x28 sets; Appendix,
# "Objective function") ----
# The paper names the network and no more; this is the classical LeNet shape with the details
# fixed here: dims = [side, c_in, c1, c2, f1, f2, classes];
#   conv 5x5 valid (c_in -> c1) + bias, ReLU, 2x2 average pooling,
#   conv 5x5 valid (c1 -> c2) + bias, ReLU, 2x2 average pooling, flatten [c2][y][x],
#   dense f1, ReLU, dense f2, ReLU, dense classes, softmax cross-entropy (mean over the batch).
# "conv" is the cross-correlation z[c, y, x] = sum W[c, ci, dy, dx] * in[ci, y + dy, x + dx] + b[c].
# Parameters are flattened in layer order: W1 [c1, c_in, 5, 5], b1, W2 [c2, c1, 5, 5], b2, then the
# dense layers as in the MLP (W row-major [in, out], then b).  The l2 term covers every weight
# tensor (conv and dense), no bias.  Inputs are rows of side*side*c_in values, plane by plane.
KS = 5   # kernel side of both convolutions


def cnn_shapes(dims):
    side, c_in, c1, c2, f1, f2, ncls = dims
    s1 = side - KS + 1
    p1 = s1 // 2
    s2 = p1 - KS + 1
    p2 = s2 // 2
    assert s1 > 0 and s1 % 2 == 0 and s2 > 0 and s2 % 2 == 0, "sides must stay even through both stages"
    return dict(side=side, c_in=c_in, c1=c1, c2=c2, s1=s1, p1=p1, s2=s2, p2=p2, flat=c2 * p2 * p2,
                dense=[c2 * p2 * p2, f1, f2, ncls])


def cnn_n_params(dims) -> int:
    sh = cnn_shapes(dims)
    n = sh["c1"] * sh["c_in"] * KS * KS + sh["c1"] + sh["c2"] * sh["c1"] * KS * KS + sh["c2"]
    d = sh["dense"]
    return n + sum(d[l] * d[l + 1] + d[l + 1] for l in range(3))


def cnn_unpack(w, dims):
    sh = cnn_shapes(dims)
    o = 0
    def take(shape):
        nonlocal o
        n = int(np.prod(shape))
        v = w[o:o + n].reshape(shape)
        o += n
        return v
    W1 = take((sh["c1"], sh["c_in"], KS, KS)); b1 = take((sh["c1"],))
    W2 = take((sh["c2"], sh["c1"], KS, KS)); b2 = take((sh["c2"],))
    dense = []
    d = sh["dense"]
    for l in range(3):
        Wl = take((d[l], d[l + 1])); bl = take((d[l + 1],))
        dense.append((Wl, bl))
    assert o == w.size
    return W1, b1, W2, b2, dense


def _windows(a):
    """All 5x5 windows of a [B, C, H, W] array: [B, C, H-4, W-4, 5, 5] (a view)."""
    return np.lib.stride_tricks.sliding_window_view(a, (KS, KS), axis=(2, 3))


def _pool(a):
    B, C, H, W = a.shape
    return a.reshape(B, C, H // 2, 2, W // 2, 2).mean(axis=(3, 5))


def _unpool(g):
    return np.repeat(np.repeat(g, 2, axis=2), 2, axis=3) / 4.0


def cnn_loss_and_grad(w, X, y, dims, l2=0.0):
    """Mean loss over the rows of X (plus the l2 term) and its gradient (flat), fp64."""
    w = np.asarray(w, dtype=np.float64)
    sh = cnn_shapes(dims)
    B = X.shape[0]
    x0 = np.asarray(X, dtype=np.float64).reshape(B, sh["c_in"], sh["side"], sh["side"])
    W1, b1, W2, b2, dense = cnn_unpack(w, dims)
    z1 = np.einsum("bcyxij,kcij->bkyx", _windows(x0), W1) + b1[None, :, None, None]
    a1 = np.maximum(z1, 0.0)
    q1 = _pool(a1)
    z2 = np.einsum("bcyxij,kcij->bkyx", _windows(q1), W2) + b2[None, :, None, None]
    a2 = np.maximum(z2, 0.0)
    q2 = _pool(a2)
    A = [q2.reshape(B, -1)]
    Z = []
    for l in range(3):
        z = A[l] @ dense[l][0] + dense[l][1]
        Z.append(z)
        if l < 2:
            A.append(np.maximum(z, 0.0))
    P = softmax_rows(Z[-1])
    reg = (W1 * W1).sum() + (W2 * W2).sum() + sum((Wl * Wl).sum() for Wl, _ in dense)
    loss = _ce(P, y).mean() + 0.5 * l2 * reg
    g = np.empty_like(w)
    gW1, gb1, gW2, gb2, gdense = cnn_unpack(g, dims)
    dZ = P.copy()
    dZ[np.arange(B), y] -= 1.0
    dZ *= 1.0 / B
    for l in range(2, -1, -1):
        gdense[l][0][...] = A[l].T @ dZ + l2 * dense[l][0]
        gdense[l][1][...] = dZ.sum(axis=0)
        dA = dZ @ dense[l][0].T
        if l > 0:
            dZ = dA * (Z[l - 1] > 0.0)
    dz2 = _unpool(dA.reshape(q2.shape)) * (z2 > 0.0)
    gW2[...] = np.einsum("bkyx,bcyxij->kcij", dz2, _windows(q1)) + l2 * W2
    gb2[...] = dz2.sum(axis=(0, 2, 3))
    # gradient with respect to the pooled first-stage maps: every output position hands its dz2 back
    # through the window it read
    dq1 = np.zeros_like(q1)
    for i in range(KS):
        for j in range(KS):
            dq1[:, :, i:i + sh["s2"], j:j + sh["s2"]] += np.einsum("bkyx,kc->bcyx", dz2, W2[:, :, i, j])
    dz1 = _unpool(dq1) * (z1 > 0.0)
    gW1[...] = np.einsum("bkyx,bcyxij->kcij", dz1, _windows(x0)) + l2 * W1
    gb1[...] = dz1.sum(axis=(0, 2, 3))
    return loss, g


def cnn_full_loss(w, data, dims, l2=0.0, chunk=2048):
    """F(w) over the union of all clients' data for the convolutional classifier."""
    tot, cnt = 0.0, 0
    for X, y in data:
        for s in range(0, len(y), chunk):
            n = len(y[s:s + chunk])
            l, _ = cnn_loss_and_grad(w, X[s:s + chunk], y[s:s + chunk], dims, 0.0)
            tot += l * n
            cnt += n
    w = np.asarray(w, dtype=np.float64)
    W1, _, W2, _, dense = cnn_unpack(w, dims)
    reg = (W1 * W1).sum() + (W2 * W2).sum() + sum((Wl * Wl).sum() for Wl, _ in dense)
    return tot / cnt + 0.5 * l2 * reg


def full_loss(w, data, dims, l2=0.0, precision=0, chunk=8192):
    """F(w): mean loss over the union of all clients' data plus the l2 term."""
    w = np.asarray(w, dtype=np.float64)
    q = round_bf16 if precision == 1 else (lambda v: v)
    layers = unpack(w, dims)
    Wq = [q(W) for W, _ in layers]
    tot, cnt = 0.0, 0
    for X, y in data:
        for s in range(0, len(y), chunk):
            A = q(np.asarray(X[s:s + chunk], dtype=np.float64))
            for l in range(len(layers)):
                z = A @ Wq[l] + layers[l][1]
                A = q(np.maximum(z, 0.0)) if l < len(layers) - 1 else z
            tot += _ce(softmax_rows(A), y[s:s + chunk]).sum()
            cnt += len(y[s:s + chunk])
    return tot / cnt + 0.5 * l2 * sum((W * W).sum() for W, _ in layers)
