"""Pins for the float64 CPU oracle: it is checked against things other than itself.

Dense brute force, finite differences of the loss, autograd on the dense-masked net,
permutation layers, pattern invariance, two closed forms (scalar recurrence, circulant
full step), a sparse-library single-layer product, adjointness, and the kink and
batch-mean conventions.  Each test names the equation of the paper's Section 3.2 it pins.
"""
import os

import numpy as np
import pytest
import scipy.sparse as sp

import gen
from oracle import OracleNet, nonzero_sets

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ------------------------------------------------------------------ helpers (independent of the oracle)
def random_net(rng, n, layers, k, scale=1.0, bias_scale=0.1):
    row_ptr, col, val, bias = [], [], [], []
    for _ in range(layers):
        counts = rng.integers(0, k + 1, size=n)          # ragged rows, some empty
        counts[rng.integers(0, n)] = k
        rp = np.zeros(n + 1, dtype=np.int32)
        rp[1:] = np.cumsum(counts)
        c = np.concatenate([np.sort(rng.choice(n, size=m, replace=False)) for m in counts]).astype(np.int32)
        v = (rng.standard_normal(rp[-1]) * scale).astype(np.float32)
        row_ptr.append(rp); col.append(c); val.append(v)
        bias.append((rng.standard_normal(n) * bias_scale).astype(np.float32))
    return row_ptr, col, val, bias


def dense_of(rp, c, v, n):
    W = np.zeros((n, n)); M = np.zeros((n, n), dtype=bool)
    for i in range(n):
        for p in range(rp[i], rp[i + 1]):
            W[i, c[p]] = v[p]; M[i, c[p]] = True
    return W, M


def dense_step(Ws, Ms, bs, x0, y, eta, clamp=32.0):
    """Minibatch SGD step on dense masked matrices, rows of x0 = inputs.  Returns everything."""
    B = x0.shape[0]
    xs, zs = [x0], [None]
    for W, b in zip(Ws, bs):
        z = xs[-1] @ W.T + b
        zs.append(z); xs.append(np.clip(z, 0.0, clamp))
    fp = lambda z: ((z > 0) & (z < clamp)).astype(float)
    loss = ((xs[-1] - y) ** 2).sum() / (2 * B)
    L = len(Ws)
    deltas = [None] * (L + 1)
    deltas[L] = (xs[L] - y) * fp(zs[L])
    grads, newW = [None] * L, [None] * L
    for k in range(L, 0, -1):
        if k > 1:
            deltas[k - 1] = (deltas[k] @ Ws[k - 1]) * fp(zs[k - 1])      # old weights
        grads[k - 1] = (deltas[k].T @ xs[k - 1]) / B * Ms[k - 1]
        newW[k - 1] = Ws[k - 1] - eta * grads[k - 1]
    return dict(loss=loss, xs=xs, zs=zs, deltas=deltas, grads=grads, newW=newW)


def csr_gather(D, rp, c, n):
    return np.concatenate([D[i, c[rp[i]:rp[i + 1]]] for i in range(n)]) if rp[-1] else np.zeros(0)


def dense_loss(Ws, bs, x0, y, clamp=32.0):
    x = x0
    for W, b in zip(Ws, bs):
        x = np.clip(x @ W.T + b, 0.0, clamp)
    return ((x - y) ** 2).sum() / (2 * x0.shape[0])


def live_case(seed, n=12, layers=3, k=4, B=3, min_margin=1e-3):
    """A tiny net whose pre-activations keep away from both kinks (needed for derivative checks)."""
    for s in range(seed, seed + 2000):
        rng = np.random.default_rng(s)
        rp, c, v, b = random_net(rng, n, layers, k, scale=0.8, bias_scale=0.3)
        x0 = rng.uniform(0.0, 1.5, size=(B, n)).astype(np.float32)
        y = rng.uniform(0.0, 1.0, size=(B, n)).astype(np.float32)
        dn = [dense_of(rp[l], c[l], v[l].astype(float), n) for l in range(layers)]
        ref = dense_step([d[0] for d in dn], [d[1] for d in dn], [bb.astype(float) for bb in b],
                         x0.astype(float), y.astype(float), 0.01)
        zall = np.concatenate([z.ravel() for z in ref["zs"][1:]])
        active = np.mean(zall > 0)
        if np.min(np.minimum(np.abs(zall), np.abs(zall - 32.0))) > min_margin and 0.3 < active < 0.9 \
                and all(np.abs(d).max() > 1e-3 for d in ref["deltas"][1:]):
            return rp, c, v, b, x0, y, dn, ref
    raise RuntimeError("no kink-free case found")


# ------------------------------------------------------------------ P1: dense brute force
@pytest.mark.parametrize("seed,n,layers,k,B", [(1, 4, 1, 2, 1), (2, 9, 2, 3, 3), (3, 33, 4, 8, 3), (4, 64, 3, 6, 1)])
def test_p1_dense_brute_force(seed, n, layers, k, B):
    """Forward equation, final-layer gradient, recursion and gradient-update rule vs dense matmul."""
    rng = np.random.default_rng(seed)
    rp, c, v, b = random_net(rng, n, layers, k, scale=0.9, bias_scale=0.3)
    x0 = rng.uniform(0, 2, size=(B, n)).astype(np.float32)
    y = rng.uniform(0, 1, size=(B, n)).astype(np.float32)
    eta = 0.05
    dn = [dense_of(rp[l], c[l], v[l].astype(float), n) for l in range(layers)]
    ref = dense_step([d[0] for d in dn], [d[1] for d in dn], [bb.astype(float) for bb in b],
                     x0.astype(float), y.astype(float), float(np.float32(eta)))
    net = OracleNet(rp, c, v, b)
    out = net.train_step(x0, y, eta)
    assert abs(out["loss"] - ref["loss"]) <= 1e-12 * max(1.0, ref["loss"])
    for l in range(layers + 1):
        np.testing.assert_allclose(out["x"][l], ref["xs"][l], rtol=0, atol=1e-12)
    for l in range(1, layers + 1):
        np.testing.assert_allclose(out["delta"][l], ref["deltas"][l], rtol=0, atol=1e-12)
    for l in range(layers):
        np.testing.assert_allclose(out["grad"][l], csr_gather(ref["grads"][l], rp[l], c[l], n), rtol=0, atol=1e-12)
        np.testing.assert_allclose(net.w[l], csr_gather(ref["newW"][l], rp[l], c[l], n), rtol=0, atol=1e-12)
    # a second step starts from the updated weights
    dn2 = ref["newW"]
    ref2 = dense_step(dn2, [d[1] for d in dn], [bb.astype(float) for bb in b], x0.astype(float), y.astype(float),
                      float(np.float32(eta)))
    out2 = net.train_step(x0, y, eta)
    for l in range(layers):
        np.testing.assert_allclose(net.w[l], csr_gather(ref2["newW"][l], rp[l], c[l], n), rtol=0, atol=1e-12)
    assert abs(out2["loss"] - ref2["loss"]) <= 1e-12


# ------------------------------------------------------------------ P2: finite differences
@pytest.mark.parametrize("seed", [10, 20, 30])
def test_p2_finite_differences(seed):
    """G is dJ/dW on every stored entry; the bias gradient is dJ/db (mean of delta)."""
    rp, c, v, b, x0, y, dn, ref = live_case(seed)
    n, layers = len(b[0]), len(c)
    net = OracleNet(rp, c, v, b)
    out = net.train_step(x0, y, 0.0)
    Ws = [d[0].copy() for d in dn]; bs = [bb.astype(float) for bb in b]
    x0d, yd = x0.astype(float), y.astype(float)
    h = 1e-6
    for l in range(layers):
        p = 0
        for i in range(n):
            for q in range(rp[l][i], rp[l][i + 1]):
                j = c[l][q]
                keep = Ws[l][i, j]
                Ws[l][i, j] = keep + h; jp = dense_loss(Ws, bs, x0d, yd)
                Ws[l][i, j] = keep - h; jm = dense_loss(Ws, bs, x0d, yd)
                Ws[l][i, j] = keep
                fd = (jp - jm) / (2 * h)
                assert abs(fd - out["grad"][l][q]) <= 1e-6 * max(1e-2, abs(fd)), (l, i, j)
                p += 1
        for i in range(n):
            keep = bs[l][i]
            bs[l][i] = keep + h; jp = dense_loss(Ws, bs, x0d, yd)
            bs[l][i] = keep - h; jm = dense_loss(Ws, bs, x0d, yd)
            bs[l][i] = keep
            fd = (jp - jm) / (2 * h)
            assert abs(fd - out["bias_grad"][l][i]) <= 1e-6 * max(1e-2, abs(fd))


# ------------------------------------------------------------------ P3: autograd
@pytest.mark.parametrize("seed", [40, 50])
def test_p3_autograd(seed):
    torch = pytest.importorskip("torch")
    rp, c, v, b, x0, y, dn, _ = live_case(seed, n=16, layers=4, k=5, B=4)
    n, layers = len(b[0]), len(c)
    Ws = [torch.tensor(d[0], dtype=torch.float64, requires_grad=True) for d in dn]
    x = torch.tensor(x0, dtype=torch.float64)
    for l in range(layers):
        x = torch.clamp(x @ Ws[l].T + torch.tensor(b[l], dtype=torch.float64), 0.0, 32.0)
    J = ((x - torch.tensor(y, dtype=torch.float64)) ** 2).sum() / (2 * x0.shape[0])
    J.backward()
    out = OracleNet(rp, c, v, b).train_step(x0, y, 0.0)
    assert abs(out["loss"] - J.item()) < 1e-12
    for l in range(layers):
        np.testing.assert_allclose(out["grad"][l], csr_gather(Ws[l].grad.numpy(), rp[l], c[l], n), rtol=0, atol=1e-12)


# ------------------------------------------------------------------ P4: permutation layers
def test_p4_permutation_layers():
    """Row j of W^k lists the incoming links of output neuron j: x^L = P_L ... P_1 x^0."""
    rng = np.random.default_rng(7)
    n, layers, B = 50, 6, 5
    perms = [rng.permutation(n) for _ in range(layers)]
    rp = [np.arange(n + 1, dtype=np.int32)] * layers
    col = [p.astype(np.int32) for p in perms]                 # out[j] = in[perm[j]]
    val = [np.ones(n, dtype=np.float32)] * layers
    bias = [np.zeros(n, dtype=np.float32)] * layers
    x0 = rng.uniform(0, 32, size=(B, n)).astype(np.float32)
    want = x0.astype(float)
    for p in perms:
        want = want[:, p]
    got = OracleNet(rp, col, val, bias).infer(x0)
    assert np.array_equal(got, want)
    sets = nonzero_sets(got)
    assert all(np.array_equal(s, np.flatnonzero(w)) for s, w in zip(sets, want))


# ------------------------------------------------------------------ P5: pattern invariance
def test_p5_update_touches_only_live_stored_entries():
    rng = np.random.default_rng(11)
    n, layers, k, B = 40, 3, 5, 4
    rp, c, v, b = random_net(rng, n, layers, k, scale=0.7, bias_scale=0.2)
    x0 = rng.uniform(0, 1, size=(B, n)).astype(np.float32)
    x0[:, ::3] = 0.0                                            # dead input columns
    y = rng.uniform(0, 1, size=(B, n)).astype(np.float32)
    net = OracleNet(rp, c, v, b)
    before = [w.copy() for w in net.w]
    out = net.train_step(x0, y, 0.1)
    for l in range(layers):
        assert net.w[l].shape == before[l].shape and np.array_equal(net.col[l], c[l]) and np.array_equal(net.row_ptr[l], rp[l])
        rows = np.repeat(np.arange(n), np.diff(rp[l]))
        dead_row = np.all(out["delta"][l + 1] == 0.0, axis=0)[rows]
        dead_col = np.all(out["x"][l] == 0.0, axis=0)[c[l]]
        untouched = dead_row | dead_col
        assert untouched.any()
        assert np.array_equal(net.w[l][untouched], before[l][untouched])
        changed = net.w[l] != before[l]
        assert changed.any() and not (changed & untouched).any()
        # delta vanishes wherever the neuron is clamped or off (f' = 0 there)
        off = (out["x"][l + 1] == 0.0) | (out["x"][l + 1] == 32.0)
        assert np.all(out["delta"][l + 1][off] == 0.0)


# ------------------------------------------------------------------ P6: scalar recurrence closed form
def test_p6_scalar_recurrence_closed_form():
    rows = [list(map(float, ln.split())) for ln in open(os.path.join(GOLDEN, "scalar_recurrence.txt"))
            if ln.strip() and not ln.startswith("#")]
    n, k, layers = 64, 8, 9
    rng = np.random.default_rng(5)
    rp = [np.arange(n + 1, dtype=np.int32) * k] * layers
    col = [np.concatenate([np.sort(rng.choice(n, size=k, replace=False)) for _ in range(n)]).astype(np.int32)
           for _ in range(layers)]
    val = [np.full(n * k, 0.25)] * layers                       # k*v = 2
    bias = [np.full(n, -0.3)] * layers                          # float64 -0.3
    net = OracleNet(rp, col, val, bias)
    x0 = np.array([[r[0]] * n for r in rows])
    xs = net.infer(x0, keep_all=True)
    for l in range(layers + 1):
        for r, row in enumerate(rows):
            np.testing.assert_allclose(xs[l][r], row[l], rtol=0, atol=1e-9)


# ------------------------------------------------------------------ P7: circulant closed form for the whole step
def test_p7_circulant_full_step_closed_form():
    n, k, stride, layers, B = 48, 6, 5, 4, 2
    v, bconst, a0, t, eta, c = 0.3, -0.1, 0.4, 0.25, 0.002, 32.0
    colp = gen.circulant_pattern(n, k, stride)
    assert np.all(np.bincount(colp, minlength=n) == k)
    rp = [np.arange(n + 1, dtype=np.int32) * k] * layers
    net = OracleNet(rp, [colp] * layers, [np.full(n * k, v)] * layers, [np.full(n, bconst)] * layers)
    eta = float(np.float32(eta))
    vl = [v] * layers
    for step in range(2):
        a = [a0]; z = [None]
        for l in range(layers):
            z.append(k * vl[l] * a[-1] + bconst); a.append(min(max(z[-1], 0.0), c))
        m = [None] + [1.0 if 0 < zz < c else 0.0 for zz in z[1:]]
        assert all(mm == 1.0 for mm in m[1:])                  # the case is chosen live
        d = [None] * (layers + 1)
        d[layers] = (a[layers] - t) * m[layers]
        for l in range(layers, 1, -1):
            d[l - 1] = k * vl[l - 1] * d[l] * m[l - 1]
        out = net.train_step(np.full((B, n), a0), np.full((B, n), t), eta)
        assert abs(out["loss"] - n * (a[layers] - t) ** 2 / 2) < 1e-12
        for l in range(1, layers + 1):
            np.testing.assert_allclose(out["x"][l], a[l], rtol=0, atol=1e-13)
            np.testing.assert_allclose(out["delta"][l], d[l], rtol=0, atol=1e-13)
        for l in range(layers):
            vl[l] = vl[l] - eta * d[l + 1] * a[l]
            np.testing.assert_allclose(net.w[l], vl[l], rtol=0, atol=1e-13)


# ------------------------------------------------------------------ P8: single layer = sparse library routine
def test_p8_single_layer_is_csr_product():
    spec = gen.CFG1_TRAIN.scaled(256, 1)
    rp, col, val, bias = gen.layer(spec, 0)
    n, B = spec.n, 7
    rng = np.random.default_rng(3)
    X = rng.uniform(0, 1, size=(B, n)).astype(np.float32)
    D = rng.standard_normal((B, n))
    A = sp.csr_matrix((val.astype(float), col, rp), shape=(n, n))
    net = OracleNet([rp], [col], [val], [bias])
    z, x, scale = net.forward_layer(0, X, want_scale=True)
    np.testing.assert_allclose(z, (A @ X.astype(float).T).T + bias.astype(float), rtol=0, atol=1e-12)
    np.testing.assert_allclose(x, np.clip(z, 0, 32), rtol=0, atol=0)
    np.testing.assert_allclose(scale, (abs(A) @ np.abs(X.astype(float)).T).T + np.abs(bias.astype(float)), atol=1e-12)
    np.testing.assert_allclose(net.transposed_product(0, D), (A.T @ D.T).T, rtol=0, atol=1e-12)
    G = net.masked_gradient(0, D, X)
    Gd = (D.T @ X.astype(float)) / B
    rows = np.repeat(np.arange(n), np.diff(rp))
    np.testing.assert_allclose(G, Gd[rows, col], rtol=0, atol=1e-12)


# ------------------------------------------------------------------ P9: adjointness
def test_p9_forward_and_backward_products_are_adjoint():
    rng = np.random.default_rng(9)
    rp, c, v, b = random_net(rng, 30, 1, 6)
    net = OracleNet(rp, c, v, [np.zeros(30, dtype=np.float32)], clamp=1e30)
    x = rng.uniform(0, 1, size=(3, 30)); d = rng.standard_normal((3, 30))
    z, _, _ = net.forward_layer(0, x)
    s = net.transposed_product(0, d)
    np.testing.assert_allclose((z * d).sum(axis=1), (x * s).sum(axis=1), rtol=1e-12)


# ------------------------------------------------------------------ conventions
def test_derivative_is_zero_on_both_kinks_and_delta0_is_not_formed():
    n = 4
    rp = [np.arange(n + 1, dtype=np.int32)]
    col = [np.arange(n, dtype=np.int32)]
    net = OracleNet(rp, col, [np.ones(n, dtype=np.float32)], [np.zeros(n, dtype=np.float32)])
    x0 = np.array([[0.0, 32.0, 5.0, 40.0]], dtype=np.float32)
    y = np.array([[1.0, 1.0, 1.0, 1.0]], dtype=np.float32)
    out = net.train_step(x0, y, 0.5)
    assert np.array_equal(out["x"][1], [[0.0, 32.0, 5.0, 32.0]])
    assert np.array_equal(out["delta"][1], [[0.0, 0.0, 4.0, 0.0]])       # z = 0 and z = 32 give f' = 0
    assert out["delta"][0] is None
    np.testing.assert_allclose(net.w[0], [1.0, 1.0, 1.0 - 0.5 * 4.0 * 5.0, 1.0])


def test_batch_gradient_is_the_mean_of_per_input_gradients():
    rp, c, v, b, x0, y, _, _ = live_case(60, B=4)
    full = OracleNet(rp, c, v, b).train_step(x0, y, 0.0)
    acc = [np.zeros_like(g) for g in full["grad"]]
    loss = 0.0
    for r in range(x0.shape[0]):
        one = OracleNet(rp, c, v, b).train_step(x0[r:r + 1], y[r:r + 1], 0.0)
        loss += one["loss"]
        for l, g in enumerate(one["grad"]):
            acc[l] += g
    assert abs(full["loss"] - loss / x0.shape[0]) < 1e-12
    for l in range(len(acc)):
        np.testing.assert_allclose(full["grad"][l], acc[l] / x0.shape[0], rtol=0, atol=1e-13)


def test_bias_update_flag():
    rp, c, v, b, x0, y, _, _ = live_case(70)
    frozen = OracleNet(rp, c, v, b); frozen.train_step(x0, y, 0.1)
    assert all(np.array_equal(fb, bb.astype(float)) for fb, bb in zip(frozen.bias, b))
    moving = OracleNet(rp, c, v, b, update_bias=True)
    out = moving.train_step(x0, y, 0.1)
    eta = float(np.float32(0.1))
    for l in range(len(b)):
        np.testing.assert_allclose(moving.bias[l], b[l].astype(float) - eta * out["bias_grad"][l], atol=1e-15)
        np.testing.assert_allclose(moving.w[l], frozen.w[l], atol=0)       # same step for the weights


def test_mask_hook_replaces_the_derivative_mask():
    rp, c, v, b, x0, y, _, _ = live_case(80)
    seen = []

    def hook(k, z, scale, m):
        seen.append(k)
        assert scale is not None and np.all(scale >= np.abs(z) - 1e-12)
        return np.zeros_like(m) if k == len(c) else m

    out = OracleNet(rp, c, v, b).train_step(x0, y, 0.1, mask_hook=hook)
    assert seen == list(range(1, len(c) + 1))
    assert all(np.all(g == 0.0) for g in out["grad"])                    # delta^L = 0 kills every gradient


# ------------------------------------------------------------------ sigmoid activation (the paper's experimental setup, Section 6)
def _sig(z):
    return 1.0 / (1.0 + np.exp(-z))


def _sig_dense_loss(Ws, bs, x0, y):
    x = x0
    for W, b in zip(Ws, bs):
        x = _sig(x @ W.T + b)
    return ((x - y) ** 2).sum() / (2 * x0.shape[0])


def _sig_case(seed, n=10, layers=3, k=4, B=3):
    rng = np.random.default_rng(seed)
    rp, c, v, b = random_net(rng, n, layers, k, scale=0.9, bias_scale=0.3)
    x0 = rng.uniform(0.0, 1.0, size=(B, n)).astype(np.float32)
    y = rng.uniform(0.0, 1.0, size=(B, n)).astype(np.float32)
    return rp, c, v, b, x0, y


@pytest.mark.parametrize("seed", [5, 6])
def test_sigmoid_gradient_matches_finite_differences_and_dense_formulas(seed):
    """With activation="sigmoid": G is dJ/dW on every stored entry (central differences on an independent dense
    evaluation of J), the forward values are the dense ones, and entries outside the pattern never appear."""
    rp, c, v, b, x0, y = _sig_case(seed)
    n, layers = len(b[0]), len(c)
    dn = [dense_of(rp[l], c[l], v[l].astype(float), n) for l in range(layers)]
    Ws, bs = [d[0] for d in dn], [bb.astype(float) for bb in b]
    net = OracleNet(rp, c, v, b, activation="sigmoid")
    out = net.train_step(x0, y, 0.01)
    x = x0.astype(float)
    for l in range(layers):
        x = _sig(x @ Ws[l].T + bs[l])
        np.testing.assert_allclose(out["x"][l + 1], x, rtol=0, atol=1e-13)
    assert abs(out["loss"] - _sig_dense_loss(Ws, bs, x0.astype(float), y.astype(float))) <= 1e-13
    h = 1e-6
    for l in range(layers):
        p = 0
        for i in range(n):
            for q in range(rp[l][i], rp[l][i + 1]):
                j = c[l][q]
                Wp = [W.copy() for W in Ws]; Wm = [W.copy() for W in Ws]
                Wp[l][i, j] += h; Wm[l][i, j] -= h
                fd = (_sig_dense_loss(Wp, bs, x0.astype(float), y.astype(float))
                      - _sig_dense_loss(Wm, bs, x0.astype(float), y.astype(float))) / (2 * h)
                assert abs(out["grad"][l][p] - fd) <= 1e-7 * max(1.0, abs(fd)), (l, i, j)
                p += 1
        bp = 0
        for i in range(n):                      # bias gradient = mean of delta = dJ/db
            bsp = [bb.copy() for bb in bs]; bsm = [bb.copy() for bb in bs]
            bsp[l][i] += h; bsm[l][i] -= h
            fd = (_sig_dense_loss(Ws, bsp, x0.astype(float), y.astype(float))
                  - _sig_dense_loss(Ws, bsm, x0.astype(float), y.astype(float))) / (2 * h)
            assert abs(out["bias_grad"][l][i] - fd) <= 1e-7 * max(1.0, abs(fd))


def test_sigmoid_autograd_and_update():
    """Same step through torch autograd (float64, dense masked weights, torch.sigmoid): gradients and new weights."""
    torch = pytest.importorskip("torch")
    rp, c, v, b, x0, y = _sig_case(11, n=14, layers=4, k=5, B=2)
    n, layers = len(b[0]), len(c)
    dn = [dense_of(rp[l], c[l], v[l].astype(float), n) for l in range(layers)]
    Ws = [torch.tensor(d[0], dtype=torch.float64, requires_grad=True) for d in dn]
    x = torch.tensor(x0.astype(float))
    for l in range(layers):
        x = torch.sigmoid(x @ Ws[l].T + torch.tensor(b[l].astype(float)))
    loss = ((x - torch.tensor(y.astype(float))) ** 2).sum() / (2 * x0.shape[0])
    loss.backward()
    eta = 0.05
    net = OracleNet(rp, c, v, b, activation="sigmoid")
    out = net.train_step(x0, y, eta)
    assert abs(out["loss"] - float(loss)) <= 1e-13
    for l in range(layers):
        g = csr_gather(Ws[l].grad.numpy(), rp[l], c[l], n)
        np.testing.assert_allclose(out["grad"][l], g, rtol=0, atol=1e-13)
        np.testing.assert_allclose(net.w[l], v[l].astype(float) - float(np.float32(eta)) * g, rtol=0, atol=1e-13)


def test_sigmoid_scalar_recurrence_and_mask_hook_refusal():
    """k equal weights v per row and a constant input: every neuron follows a_l = sigmoid(k v a_{l-1} + b)."""
    n, k, layers = 64, 8, 6
    col = gen.circulant_pattern(n, k, 3)
    rp = (np.arange(n + 1) * k).astype(np.int32)
    val = np.full(n * k, 0.25, dtype=np.float32)
    bias = np.full(n, -0.5, dtype=np.float32)
    net = OracleNet([rp] * layers, [col] * layers, [val] * layers, [bias] * layers, activation="sigmoid")
    xs = net.infer(np.full((2, n), 0.3, dtype=np.float32), keep_all=True)
    a = float(np.float32(0.3))
    for l in range(1, layers + 1):
        a = 1.0 / (1.0 + np.exp(-(k * 0.25 * a - 0.5)))
        np.testing.assert_allclose(xs[l], a, rtol=0, atol=1e-14)
    with pytest.raises(ValueError):
        net.train_step(np.zeros((1, n), np.float32), np.zeros((1, n), np.float32), 0.1, mask_hook=lambda *a: a[-1])
    with pytest.raises(ValueError):
        OracleNet([rp], [col], [val], [bias], activation="tanh")


# ------------------------------------------------------------------ averaged form of the minibatch step (Discussion of Section 5)
def _dense_averaged_step(Ws, Ms, bs, x0, y, eta, activation, clamp=32.0):
    """The averaged step on dense masked matrices, one neuron at a time (loops, no shared code with the oracle)."""
    f = _sig if activation == "sigmoid" else (lambda z: np.clip(z, 0.0, clamp))
    dx = (lambda x: x * (1.0 - x)) if activation == "sigmoid" else (lambda x: ((x > 0) & (x < clamp)).astype(float))
    B, n, L = x0.shape[0], x0.shape[1], len(Ws)
    xs = [x0]
    for W, b in zip(Ws, bs):
        xs.append(f(xs[-1] @ W.T + b))
    xbar = [v.sum(axis=0) / B for v in xs]
    d = np.zeros(n)
    for bb in range(B):                                   # average of the per-input output gradients
        d += (xs[L][bb] - y[bb]) * dx(xs[L][bb]) / B
    newW, deltas = [None] * L, [None] * (L + 1)
    for k in range(L, 0, -1):
        deltas[k] = d
        W, M = Ws[k - 1], Ms[k - 1]
        back = np.zeros(n)
        upd = W.copy()
        for i in range(n):
            for j in range(n):
                if M[i, j]:
                    back[j] += W[i, j] * d[i]                       # old weight
                    upd[i, j] = W[i, j] - eta * d[i] * xbar[k - 1][j]
        newW[k - 1] = upd
        d = back * dx(xbar[k - 1])
    return newW, deltas, ((xs[L] - y) ** 2).sum() / (2 * B)


@pytest.mark.parametrize("activation,seed", [("clamped_relu", 11), ("sigmoid", 12)])
def test_averaged_step_matches_a_dense_restatement(activation, seed):
    if activation == "sigmoid":
        rp, c, v, b, x0, y = _sig_case(seed, n=9, layers=3, k=4, B=4)
    else:
        rp, c, v, b, x0, y, _, _ = live_case(seed, n=9, layers=3, k=4, B=4)
    n, L, eta = len(b[0]), len(c), float(np.float32(0.05))
    dn = [dense_of(rp[l], c[l], v[l].astype(float), n) for l in range(L)]
    newW, deltas, loss = _dense_averaged_step([d[0] for d in dn], [d[1] for d in dn], [bb.astype(float) for bb in b],
                                              x0.astype(float), y.astype(float), eta, activation)
    net = OracleNet(rp, c, v, b, activation=activation)
    out = net.train_step_averaged(x0, y, eta)
    assert abs(out["loss"] - loss) <= 1e-13 * max(1.0, loss)
    for k in range(L):
        np.testing.assert_allclose(out["delta"][k + 1][0], deltas[k + 1], rtol=1e-12, atol=1e-15)
        np.testing.assert_allclose(net.w[k], csr_gather(newW[k], rp[k], c[k], n), rtol=1e-12, atol=1e-15)
        assert np.abs(out["delta"][k + 1]).max() > 1e-6                 # the comparison is not vacuous


@pytest.mark.parametrize("activation", ["clamped_relu", "sigmoid"])
def test_averaged_step_is_algorithm_1_where_the_two_must_agree(activation):
    """B = 1: the averaged step is the plain step.  A batch of B copies of one input: every mean is that input's
    vector, so the averaged step is the single-input step too (and so is the exact minibatch step)."""
    if activation == "sigmoid":
        rp, c, v, b, x0, y = _sig_case(21, n=11, layers=4, k=4, B=1)
    else:
        rp, c, v, b, x0, y, _, _ = live_case(21, n=11, layers=4, k=4, B=1)
    eta = 0.03
    one = OracleNet(rp, c, v, b, activation=activation)
    ref = one.train_step(x0, y, eta)
    avg = OracleNet(rp, c, v, b, activation=activation)
    out = avg.train_step_averaged(x0, y, eta)
    assert out["loss"] == ref["loss"]
    for k in range(len(c)):
        assert np.array_equal(avg.w[k], one.w[k])
        assert np.array_equal(out["delta"][k + 1], ref["delta"][k + 1])
    rep = OracleNet(rp, c, v, b, activation=activation)
    out5 = rep.train_step_averaged(np.repeat(x0, 5, axis=0), np.repeat(y, 5, axis=0), eta)
    assert abs(out5["loss"] - ref["loss"]) <= 1e-14 * max(1.0, ref["loss"])
    for k in range(len(c)):
        np.testing.assert_allclose(rep.w[k], one.w[k], rtol=1e-13, atol=1e-16)


def test_averaged_step_differs_from_the_exact_minibatch_step_and_keeps_the_pattern():
    """It is an approximation: on a batch of different inputs its update is not the mean of the per-input gradients
    (the product of the means is not the mean of the products).  Like the exact step it only touches stored entries,
    and with update_bias the bias moves by -eta * delta^k."""
    rp, c, v, b, x0, y = _sig_case(31, n=10, layers=3, k=4, B=4)
    eta = 0.1
    exact = OracleNet(rp, c, v, b, activation="sigmoid")
    exact.train_step(x0, y, eta)
    avg = OracleNet(rp, c, v, b, activation="sigmoid", update_bias=True)
    out = avg.train_step_averaged(x0, y, eta)
    assert max(np.abs(avg.w[k] - exact.w[k]).max() for k in range(3)) > 1e-6
    for k in range(3):
        assert avg.w[k].shape == v[k].shape
        np.testing.assert_allclose(avg.bias[k], b[k].astype(float) - float(np.float32(eta)) * out["delta"][k + 1][0], rtol=1e-13)
        np.testing.assert_allclose(out["grad"][k], (np.asarray(v[k], dtype=float) - avg.w[k]) / float(np.float32(eta)),
                                   rtol=1e-9, atol=1e-12)
