"""Workload table and seeded synthetic input generators.

This module holds *inputs only*: the five benchmark configurations as plain
dicts and the NumPy generators for image-shaped client data sets, client
splits and initial MLP weights.  It contains none of the method's arithmetic
(no gradients, no schedule, no delay model), so both the CUDA library's
binding and the CPU checker can be fed from it without sharing any logic.

The data stand in for the paper's 28x28 grey and 32x32x3 colour
image-classification sets (Appendix, Table 2: 10 classes, 60,000 / 50,000
training points); the public sets themselves are never used.

Recipe (all draws from ``numpy.random.default_rng``):
  * class patterns  mu[k, j] ~ U(-2.0, 0.5), k < 10, j < D: every class lights up
    its own fifth of the pixels, the rest is dark
  * a sample of class k is clip(mu[k] + 0.25 * N(0, I), 0, 1)  (about 80 % of the
    pixels clip to exactly 0, like a dark background; |x|^2 is about 15 for
    D = 784, which keeps the given step sizes stable when the server adds up
    the update sums of all clients)
  * labels are uniform over the 10 classes; one label in ten is then redrawn
    uniformly, so no model separates the data and gradients never vanish
  * IID split: seeded permutation cut evenly
  * Dirichlet(alpha) label-skew split: per class, client proportions
    ~ Dir(alpha * 1_n), cumulative cut; re-drawn with seed+1, ... until every
    client owns at least max(batch, 8) samples
  * MLP start model: every W_l and b_l ~ U(-1/sqrt(in_l), 1/sqrt(in_l))
"""
from __future__ import annotations

import copy
import math

import numpy as np

N_CLASSES = 10
LABEL_NOISE = 0.1   # fraction of labels redrawn uniformly
NEVER_WAIT = 0xFFFFFFFF

# Fields follow the C struct ``aet_config`` one to one; the extra keys
# (n_rounds, data) describe the run and the data recipe.
_COMMON = dict(
    round_base=0, max_lag_d=1, lr_beta=0.0, l2=0.0, seed=0,
    delay_dist=0, compute_delay_mean=1.0, network_delay_mean=0.5,
    compute_delay_lo=0.1, compute_delay_hi=1.0,
    network_delay_lo=0.1, network_delay_hi=1.5,
    n_stragglers=0, straggler_factor=1.0, precision=0, batch=1,
)

CONFIGS = {
    "cfg1": dict(_COMMON, n_clients=4, model=0, dims=[784, 10], lr=0.01, l2=1e-4,
                 sched_a=10, sched_b=10, n_rounds=5,
                 data=dict(kind="per_client", per_client=2000, dim=784)),
    "cfg2": dict(_COMMON, n_clients=16, model=0, dims=[784, 10], lr=0.005,
                 sched_a=20, sched_b=20, n_rounds=30, n_stragglers=2, straggler_factor=10.0,
                 data=dict(kind="dirichlet", total=60000, alpha=0.5, dim=784)),
    "cfg3": dict(_COMMON, n_clients=32, model=1, dims=[784, 128, 10], lr=0.002, batch=32,
                 sched_a=64, sched_b=64, n_rounds=40, network_delay_mean=1.0,
                 data=dict(kind="iid", total=60000, dim=784)),
    "cfg4": dict(_COMMON, n_clients=64, model=1, dims=[3072, 256, 128, 10], lr=0.0005, batch=64,
                 precision=1, sched_a=128, sched_b=128, n_rounds=30,
                 n_stragglers=8, straggler_factor=20.0,
                 data=dict(kind="dirichlet", total=50000, alpha=0.3, dim=3072)),
    # lr None: the server sums (not averages) the clients' update sums, so the step
    # size is scaled with the client count, lr = 0.02 / n_clients (see get_config).
    "cfg5": dict(_COMMON, n_clients=1024, model=0, dims=[784, 10], lr=None,
                 sched_a=8, sched_b=8, n_rounds=10,
                 data=dict(kind="per_client", per_client=1024, dim=784)),
    # The paper's own setting (Appendix Table 2 and A.2): five nodes, s_i = 10 i counted from round 1,
    # eta_0 = 0.01 diminishing with beta = 0.01, d = 1, uniform delays of 0.1-1 per SGD iteration and
    # 0.1-1.5 per message; K = 60,000 iterations per node take 110 rounds (61,050 samples).
    "cfg6": dict(_COMMON, n_clients=5, model=0, dims=[784, 10], lr=0.01, lr_beta=0.01,
                 sched_a=10, sched_b=0, round_base=1, n_rounds=110, delay_dist=1,
                 data=dict(kind="iid", total=60000, dim=784)),
    # A LeNet-shaped convolutional classifier on the 28x28 set (the paper's model for those sets; Appendix,
    # "Objective function"): 16 clients, minibatch 16, s_i = 32 i + 32 for 12 rounds.
    "cfg7": dict(_COMMON, n_clients=16, model=2, dims=[28, 1, 6, 16, 120, 84, 10], lr=0.005, batch=16,
                 sched_a=32, sched_b=32, n_rounds=12, network_delay_mean=1.0,
                 data=dict(kind="iid", total=60000, dim=784)),
}


def get_config(name: str, **overrides) -> dict:
    """A deep copy of a named configuration with fields overridden."""
    cfg = copy.deepcopy(CONFIGS[name])
    data_over = overrides.pop("data", None)
    cfg.update(overrides)
    if data_over:
        cfg["data"].update(data_over)
    if cfg["lr"] is None:
        cfg["lr"] = 0.02 / cfg["n_clients"]
    cfg["name"] = name
    return cfg


def n_params(dims) -> int:
    return sum(dims[l] * dims[l + 1] + dims[l + 1] for l in range(len(dims) - 1))


CONV_K = 5   # kernel side of the convolutional classifier's two convolutions


def cnn_layer_shapes(dims):
    """(fan_in, number of weights, number of biases) of the five layers of the convolutional classifier
    dims = [side, c_in, c1, c2, f1, f2, classes] (two 5x5 valid convolutions, each followed by 2x2 average
    pooling, then three dense layers)."""
    side, c_in, c1, c2, f1, f2, ncls = dims
    p2 = ((side - CONV_K + 1) // 2 - CONV_K + 1) // 2
    flat = c2 * p2 * p2
    k2 = CONV_K * CONV_K
    return [(c_in * k2, c1 * c_in * k2, c1), (c1 * k2, c2 * c1 * k2, c2),
            (flat, flat * f1, f1), (f1, f1 * f2, f2), (f2, f2 * ncls, ncls)]


def model_n_params(cfg) -> int:
    if cfg["model"] == 2:
        return sum(nw + nb for _, nw, nb in cnn_layer_shapes(cfg["dims"]))
    return n_params(cfg["dims"])


def make_pool(n: int, dim: int, seed: int):
    """n synthetic images (float32 in [0,1], row-major [n, dim]) and int32 labels."""
    rng = np.random.default_rng(seed)
    mu = rng.uniform(-2.0, 0.5, size=(N_CLASSES, dim)).astype(np.float32)
    y = rng.integers(0, N_CLASSES, size=n).astype(np.int32)
    x = np.empty((n, dim), dtype=np.float32)
    chunk = 65536
    for s in range(0, n, chunk):
        e = min(n, s + chunk)
        z = rng.standard_normal(size=(e - s, dim), dtype=np.float32)
        z *= np.float32(0.25)
        z += mu[y[s:e]]
        np.clip(z, 0.0, 1.0, out=z)
        x[s:e] = z
    flip = rng.random(n) < LABEL_NOISE
    y = np.where(flip, rng.integers(0, N_CLASSES, size=n), y).astype(np.int32)
    return x, y


def split_iid(n: int, n_clients: int, seed: int):
    rng = np.random.default_rng(seed)
    perm = rng.permutation(n)
    return [np.sort(p) for p in np.array_split(perm, n_clients)]


def split_dirichlet(y: np.ndarray, n_clients: int, alpha: float, seed: int, min_size: int):
    """Label-skew split; returns a list of index arrays, one per client."""
    for attempt in range(1000):
        rng = np.random.default_rng(seed + attempt)
        parts = [[] for _ in range(n_clients)]
        for k in range(N_CLASSES):
            idx = np.flatnonzero(y == k)
            rng.shuffle(idx)
            prop = rng.dirichlet(alpha * np.ones(n_clients))
            cuts = (np.cumsum(prop)[:-1] * len(idx)).astype(np.int64)
            for c, piece in enumerate(np.split(idx, cuts)):
                parts[c].append(piece)
        out = [np.sort(np.concatenate(p)) for p in parts]
        if min(len(o) for o in out) >= min_size:
            return out
    raise RuntimeError("Dirichlet split: no draw gave every client enough samples")


def make_client_data(cfg: dict):
    """Per-client (x, y) arrays for a configuration.

    Returns a list of (x float32 [n_c, D] C-contiguous, y int32 [n_c]).
    Seeds: pool = cfg['seed'], split = cfg['seed'] + 1000.
    """
    d = cfg["data"]
    n = cfg["n_clients"]
    seed = int(cfg["seed"])
    dim = d["dim"]
    assert dim == (cfg["dims"][0] * cfg["dims"][0] * cfg["dims"][1] if cfg["model"] == 2 else cfg["dims"][0])
    if d["kind"] == "per_client":
        x, y = make_pool(n * d["per_client"], dim, seed)
        m = d["per_client"]
        return [(x[c * m:(c + 1) * m], y[c * m:(c + 1) * m]) for c in range(n)]
    x, y = make_pool(d["total"], dim, seed)
    if d["kind"] == "iid":
        parts = split_iid(d["total"], n, seed + 1000)
    elif d["kind"] == "dirichlet":
        parts = split_dirichlet(y, n, d["alpha"], seed + 1000, max(cfg["batch"], 8))
    else:
        raise ValueError(d["kind"])
    return [(np.ascontiguousarray(x[p]), np.ascontiguousarray(y[p])) for p in parts]


def make_start_model(cfg: dict) -> np.ndarray:
    """Start model w_0 as a flat float32 vector (layers in order, W_l row-major
    [in, out] then b_l).  Softmax regression starts at zero; MLPs are seeded."""
    dims = cfg["dims"]
    if cfg["model"] == 2:      # every tensor ~ U(-1/sqrt(fan_in), 1/sqrt(fan_in)), weights then biases, layer by layer
        rng = np.random.default_rng(int(cfg["seed"]) + 2000)
        out = []
        for fan_in, nw, nb in cnn_layer_shapes(dims):
            bound = 1.0 / math.sqrt(fan_in)
            out.append(rng.uniform(-bound, bound, size=nw).astype(np.float32))
            out.append(rng.uniform(-bound, bound, size=nb).astype(np.float32))
        return np.concatenate(out)
    P = n_params(dims)
    if cfg["model"] == 0:
        return np.zeros(P, dtype=np.float32)
    rng = np.random.default_rng(int(cfg["seed"]) + 2000)
    out = []
    for l in range(len(dims) - 1):
        bound = 1.0 / math.sqrt(dims[l])
        out.append(rng.uniform(-bound, bound, size=dims[l] * dims[l + 1]).astype(np.float32))
        out.append(rng.uniform(-bound, bound, size=dims[l + 1]).astype(np.float32))
    return np.concatenate(out)
