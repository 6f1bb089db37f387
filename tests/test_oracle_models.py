"""Pins for the checker's losses and gradients (CPU only)."""
import numpy as np
import pytest
import torch

from oracle import models
from paper_2112_13935_b200 import workloads


def _rand_problem(dims, B, seed):
    g = np.random.default_rng(seed)
    P = workloads.n_params(dims)
    w = g.normal(0, 0.3, size=P)
    X = g.uniform(0, 1, size=(B, dims[0]))
    y = g.integers(0, dims[-1], size=B)
    return w, X, y


@pytest.mark.parametrize("dims,B", [([7, 10], 1), ([7, 10], 5), ([9, 6, 10], 4), ([8, 7, 5, 10], 3)])
@pytest.mark.parametrize("l2", [0.0, 0.05])
def test_gradient_matches_central_differences(dims, B, l2):
    w, X, y = _rand_problem(dims, B, 11)
    _, g = models.loss_and_grad(w, X, y, dims, l2)
    h = 1e-6
    for j in np.random.default_rng(3).choice(w.size, size=min(60, w.size), replace=False):
        e = np.zeros_like(w)
        e[j] = h
        fp, _ = models.loss_and_grad(w + e, X, y, dims, l2)
        fm, _ = models.loss_and_grad(w - e, X, y, dims, l2)
        assert abs((fp - fm) / (2 * h) - g[j]) < 1e-7, j


def test_softmax_regression_gradient_at_zero_by_hand():
    # w = 0: p = 1/10 for every class, so dW = x (p - onehot)^T and db = p - onehot.
    dims = [4, 10]
    x = np.array([[0.5, 0.0, 1.0, 0.25]])
    loss, g = models.loss_and_grad(np.zeros(50), x, np.array([3]), dims)
    delta = np.full(10, 0.1)
    delta[3] -= 1.0
    assert np.isclose(loss, np.log(10.0))
    np.testing.assert_allclose(g[:40].reshape(4, 10), np.outer(x[0], delta), atol=1e-15)
    np.testing.assert_allclose(g[40:], delta, atol=1e-15)


def test_matches_torch_autograd_mlp():
    # a library's reverse-mode derivative of the same loss, written independently
    dims, B = [12, 8, 6, 10], 5
    w, X, y = _rand_problem(dims, B, 4)
    _, g = models.loss_and_grad(w, X, y, dims, 0.01)
    wt = torch.tensor(w, dtype=torch.float64, requires_grad=True)
    a, o, reg = torch.tensor(X), 0, 0.0
    for l in range(3):
        i, j = dims[l], dims[l + 1]
        W = wt[o:o + i * j].reshape(i, j)
        b = wt[o + i * j:o + i * j + j]
        o += i * j + j
        reg = reg + 0.5 * 0.01 * (W * W).sum()
        a = a @ W + b
        if l < 2:
            a = torch.relu(a)
    loss = torch.nn.functional.cross_entropy(a, torch.tensor(y)) + reg
    loss.backward()
    np.testing.assert_allclose(g, wt.grad.numpy(), rtol=1e-10, atol=1e-12)


def test_softmax_rows_sum_to_one_and_survive_large_logits():
    Z = np.array([[1000.0, 999.0, -1000.0], [0.0, 0.0, 0.0]])
    P = models.softmax_rows(Z)
    np.testing.assert_allclose(P.sum(axis=1), 1.0, atol=1e-15)
    assert np.isclose(P[0, 0], 1 / (1 + np.exp(-1.0)))


def test_bf16_rounding_matches_a_library_conversion():
    g = np.random.default_rng(0)
    v = np.concatenate([g.normal(0, 1, 5000), g.uniform(0, 1, 5000), [0.0, 1.0, -1.0, 0.1, 3.0e-5]])
    v32 = v.astype(np.float32)
    want = torch.tensor(v32).to(torch.bfloat16).to(torch.float64).numpy()
    got = models.round_bf16(v32.astype(np.float64))
    np.testing.assert_array_equal(got, want)
    # ties go to even: 1 + 2^-8 is halfway between 1 and 1 + 2^-7
    assert models.round_bf16(np.array([1.0 + 2.0 ** -8]))[0] == 1.0
    assert models.round_bf16(np.array([1.0 + 3 * 2.0 ** -8]))[0] == 1.0 + 2.0 ** -6


def test_bf16_path_uses_rounded_operands():
    dims, B = [6, 5, 10], 4
    w, X, y = _rand_problem(dims, B, 9)
    l0, g0 = models.loss_and_grad(w, X, y, dims, 0.0, precision=0)
    l1, g1 = models.loss_and_grad(w, X, y, dims, 0.0, precision=1)
    assert 0 < abs(l1 - l0) < 2e-2 and 0 < np.abs(g1 - g0).max() < 5e-2
    # rounding the inputs beforehand changes nothing: they are rounded at the same points
    wq = w.copy()
    l2_, g2 = models.loss_and_grad(wq, models.round_bf16(X), y, dims, 0.0, precision=1)
    assert l2_ == l1 and np.array_equal(g1, g2)


def test_full_loss_is_the_mean_over_all_clients():
    dims = [5, 10]
    w, X, y = _rand_problem(dims, 12, 2)
    data = [(X[:5], y[:5]), (X[5:], y[5:])]
    want, _ = models.loss_and_grad(w, X, y, dims, 0.3)
    assert np.isclose(models.full_loss(w, data, dims, 0.3, chunk=4), want, rtol=1e-13)


def _bf(v):
    """Nearest bf16 of a Python float through a library conversion (not the checker's own)."""
    return float(torch.tensor(v, dtype=torch.float32).to(torch.bfloat16))


def bf16_case():
    """Two samples through a 2-2-2 network, chosen so that every value that the low-precision
    path rounds sits off the bf16 grid: x[0][0], x[1][1], W_0[0][0], W_1[1][1], both hidden
    activations of unit 0, the logits of class 0 (which stay unrounded), and every dZ entry."""
    dims = [2, 2, 2]
    X = np.array([[1 + 2.0 ** -9, 0.5], [0.25, 1 - 2.0 ** -10]])
    y = np.array([1, 0])
    W0 = np.array([[0.5 + 2.0 ** -10, -0.25], [0.25, 0.5]])
    b0 = np.array([2.0 ** -10, 0.0])
    W1 = np.array([[1.0, -1.0], [0.5, 0.25 + 2.0 ** -11]])
    b1 = np.array([2.0 ** -10, 0.0])
    w = np.concatenate([W0.ravel(), b0, W1.ravel(), b1])
    return dims, w, X, y


def bf16_case_by_hand():
    """The same case, scalar by scalar, with the rounding points of the low-precision path
    spelled out: inputs once; each weight when read; each hidden activation after bias + ReLU;
    each dZ before the two backward products (the bias gradients take the unrounded dZ)."""
    import math
    # rounded operands (exact dyadic values)
    x = [[1.0, 0.5], [0.25, 1.0]]
    W0 = [[0.5, -0.25], [0.25, 0.5]]
    W1 = [[1.0, -1.0], [0.5, 0.25]]
    b0 = [2.0 ** -10, 0.0]
    # forward, sample 0: z = (0.625 + 2^-10, 0) -> a = (0.625, 0);  sample 1: z = (0.375 + 2^-10, 0.4375)
    z0 = [[0.625 + 2.0 ** -10, 0.0], [0.375 + 2.0 ** -10, 0.4375]]
    a0 = [[0.625, 0.0], [0.375, 0.4375]]
    for b in range(2):
        for h in range(2):
            assert z0[b][h] == x[b][0] * W0[0][h] + x[b][1] * W0[1][h] + b0[h]
            assert a0[b][h] == _bf(max(z0[b][h], 0.0))
    b1 = [2.0 ** -10, 0.0]
    logits = [[0.625 + 2.0 ** -10, -0.625], [0.59375 + 2.0 ** -10, -0.265625]]     # not rounded
    for b in range(2):
        for c in range(2):
            assert logits[b][c] == a0[b][0] * W1[0][c] + a0[b][1] * W1[1][c] + b1[c]
    p = [[1 / (1 + math.exp(-(l[0] - l[1]))), 1 / (1 + math.exp(l[0] - l[1]))] for l in logits]
    loss = -(math.log(p[0][1]) + math.log(p[1][0])) / 2
    dZ1 = [[p[0][0] / 2, (p[0][1] - 1) / 2], [(p[1][0] - 1) / 2, p[1][1] / 2]]       # (p - onehot) / B
    dZ1q = [[_bf(v) for v in r] for r in dZ1]
    gW1 = [[sum(a0[b][h] * dZ1q[b][c] for b in range(2)) for c in range(2)] for h in range(2)]
    gb1 = [dZ1[0][c] + dZ1[1][c] for c in range(2)]
    # dA = dZ1q W1^T, gated by z0 > 0 (unit 1 of sample 0 is off)
    dZ0 = [[(dZ1q[b][0] * W1[h][0] + dZ1q[b][1] * W1[h][1]) * (1.0 if z0[b][h] > 0 else 0.0) for h in range(2)]
           for b in range(2)]
    dZ0q = [[_bf(v) for v in r] for r in dZ0]
    gW0 = [[sum(x[b][i] * dZ0q[b][h] for b in range(2)) for h in range(2)] for i in range(2)]
    gb0 = [dZ0[0][h] + dZ0[1][h] for h in range(2)]
    g = np.array([v for r in gW0 for v in r] + gb0 + [v for r in gW1 for v in r] + gb1)
    return loss, g


def test_bf16_rounding_points_on_a_case_worked_by_hand():
    dims, w, X, y = bf16_case()
    loss, g = models.loss_and_grad(w, X, y, dims, 0.0, precision=1)
    want_loss, want_g = bf16_case_by_hand()
    assert abs(loss - want_loss) < 1e-15
    np.testing.assert_allclose(g, want_g, rtol=0, atol=1e-16)
    # and the case separates the two precisions everywhere it should
    _, g32 = models.loss_and_grad(w, X, y, dims, 0.0, precision=0)
    assert np.abs(g - g32).max() > 1e-4


# ---- the small convolutional classifier ----
def _cnn_problem(dims, B, seed):
    g = np.random.default_rng(seed)
    w = g.normal(0, 0.2, size=models.cnn_n_params(dims))
    X = g.uniform(0, 1, size=(B, dims[0] * dims[0] * dims[1]))
    y = g.integers(0, dims[-1], size=B)
    return w, X, y


def test_cnn_parameter_count_of_the_lenet_shape():
    # 28x28x1 -> conv 6 -> pool -> conv 16 -> pool -> 256 -> 120 -> 84 -> 10
    dims = [28, 1, 6, 16, 120, 84, 10]
    sh = models.cnn_shapes(dims)
    assert (sh["s1"], sh["p1"], sh["s2"], sh["p2"], sh["flat"]) == (24, 12, 8, 4, 256)
    assert models.cnn_n_params(dims) == 156 + 2416 + 30840 + 10164 + 850 == 44426


@pytest.mark.parametrize("l2", [0.0, 0.05])
def test_cnn_gradient_matches_central_differences(l2):
    dims = [16, 2, 3, 4, 7, 6, 5]
    w, X, y = _cnn_problem(dims, 3, 21)
    _, g = models.cnn_loss_and_grad(w, X, y, dims, l2)
    h = 1e-6
    for j in np.random.default_rng(5).choice(w.size, size=80, replace=False):
        e = np.zeros_like(w)
        e[j] = h
        fp, _ = models.cnn_loss_and_grad(w + e, X, y, dims, l2)
        fm, _ = models.cnn_loss_and_grad(w - e, X, y, dims, l2)
        assert abs((fp - fm) / (2 * h) - g[j]) < 2e-7, j


def test_cnn_matches_torch_conv_pool_autograd():
    # a library's convolution, pooling and reverse-mode derivative of the same network, written independently
    import torch.nn.functional as F
    dims = [16, 2, 3, 4, 7, 6, 5]
    w, X, y = _cnn_problem(dims, 4, 8)
    loss, g = models.cnn_loss_and_grad(w, X, y, dims, 0.01)
    wt = torch.tensor(w, dtype=torch.float64, requires_grad=True)
    o = 0
    def take(*shape):
        nonlocal o
        n = int(np.prod(shape))
        v = wt[o:o + n].reshape(*shape)
        o += n
        return v
    W1, b1, W2, b2 = take(3, 2, 5, 5), take(3), take(4, 3, 5, 5), take(4)
    a = torch.tensor(X).reshape(4, 2, 16, 16)
    a = F.avg_pool2d(torch.relu(F.conv2d(a, W1, b1)), 2)
    a = F.avg_pool2d(torch.relu(F.conv2d(a, W2, b2)), 2).reshape(4, -1)
    reg = (W1 * W1).sum() + (W2 * W2).sum()
    for l, (i, j) in enumerate([(4, 7), (7, 6), (6, 5)]):
        Wl, bl = take(i, j), take(j)
        reg = reg + (Wl * Wl).sum()
        a = a @ Wl + bl
        if l < 2:
            a = torch.relu(a)
    lt = F.cross_entropy(a, torch.tensor(y)) + 0.5 * 0.01 * reg
    lt.backward()
    assert abs(loss - float(lt)) < 1e-12
    np.testing.assert_allclose(g, wt.grad.numpy(), rtol=1e-9, atol=1e-12)


def test_cnn_one_bright_pixel_by_hand():
    # one sample, one input plane, every conv weight 0 except W1[0,0,0,0] = 1 and b1 = 0: z1 = the image cropped to
    # its top-left 12x12; the image is zero except pixel (2, 3) = 0.8, so z1 has one non-zero, a1 the same, and the
    # pooled map one entry 0.8 / 4 at (1, 1).  With W2 = 0 and b2 = 0.5 every second-stage output is 0.5 (ReLU keeps
    # it, pooling keeps it), the dense layers are zero with zero bias: logits 0, loss ln(classes).
    dims = [16, 1, 1, 1, 2, 2, 3]
    w = np.zeros(models.cnn_n_params(dims))
    W1, b1, W2, b2, dense = models.cnn_unpack(w, dims)
    W1[0, 0, 0, 0] = 1.0
    b2[0] = 0.5
    x = np.zeros((1, 256))
    x[0, 2 * 16 + 3] = 0.8
    loss, g = models.cnn_loss_and_grad(w, x, np.array([1]), dims)
    assert np.isclose(loss, np.log(3.0))
    gW1, gb1, gW2, gb2, gd = models.cnn_unpack(g, dims)
    # only the last dense layer's bias sees a gradient (its input is relu(0) = 0): p - onehot = (1/3, -2/3, 1/3)
    np.testing.assert_allclose(gd[2][1], [1 / 3, -2 / 3, 1 / 3], atol=1e-15)
    assert not gd[2][0].any() and not gW1.any() and not gW2.any() and not gd[0][0].any()
    # now let the second stage read the pooled first-stage map: W2[0,0,1,1] = 4 reads q1[y+1, x+1], which is 0.2 at
    # (1, 1), so z2[0, 0] = 4 * 0.2 + 0.5 = 1.3 and the other three entries stay 0.5; pooled: (1.3 + 1.5) / 4 = 0.7.
    # Dense chain: f1 unit 0 = 2 * 0.7 = 1.4, f2 unit 1 = 3 * 1.4 = 4.2, logit 2 = 4.2.
    W2[0, 0, 1, 1] = 4.0
    dense[0][0][0, 0] = 2.0
    dense[1][0][0, 1] = 3.0
    dense[2][0][1, 2] = 1.0
    loss2, _ = models.cnn_loss_and_grad(w, x, np.array([2]), dims)
    assert np.isclose(loss2, -np.log(np.exp(4.2) / (np.exp(4.2) + 2.0)), rtol=0, atol=1e-14)
