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
