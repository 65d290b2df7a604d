"""Why the parity bar is normwise: the experiment behind it, reproducible without a GPU.

One SGD step of the live 1024 x 120 net (He-scaled weights, bias 0, one binary input) is evaluated twice on
the CPU: by the float64 oracle, and in plain fp32 with scipy's float32 sparse products (fp32 multiply, fp32
add, the stored order: the most ordinary single-precision evaluation there is, sharing no code with the
oracle or with the CUDA kernels).  Every entry of x^k, delta^k and G^k is a signed sum, so the fp32 result
deviates from the float64 one by an amount that scales with the sum of the magnitudes of the terms, not with
the entry.  Measured here per tensor:

  normwise                      max|g - o| / max|o|                             1.8e-6
  elementwise, floor 5e-2       max|g_i - o_i| / max(|o_i|, 0.05 max|o|)        3.7e-5
  elementwise, floor 1e-3       max|g_i - o_i| / max(|o_i|, 0.001 max|o|)       9.3e-4

An elementwise bar of 1e-4 with a floor of a thousandth of the maximum is therefore not a statement about an
implementation: plain fp32 arithmetic misses it by a factor of nine on a single step, whatever the order of
its additions.  The GPU parity tests assert the first line at 1e-4, guard the second at 1e-3 and record the
third (parity_util.WORST), so that every run reports its margin under each.
"""
import numpy as np
import scipy.sparse as sp

import gen
from oracle import OracleNet
from parity_util import FLOOR, FLOOR_FINE, TOL, TOL_ELEM, rel_err, rel_err_elem


def fp32_step(rp, col, val, bias, x0, y, clamp=np.float32(32.0)):
    """x^1..x^L, delta^1..delta^L, G^1..G^L of one per-sample step in float32 throughout (B = 1)."""
    n, L = len(bias[0]), len(col)
    mats = [sp.csr_matrix((val[k], col[k], rp[k]), shape=(n, n), dtype=np.float32) for k in range(L)]
    xs = [x0.astype(np.float32)]
    for k in range(L):
        z = mats[k] @ xs[-1] + bias[k]
        assert z.dtype == np.float32
        xs.append(np.minimum(np.maximum(z, np.float32(0.0)), clamp))
    fprime = lambda x: ((x > 0) & (x < clamp)).astype(np.float32)
    deltas, grads = [None] * (L + 1), [None] * L
    deltas[L] = (xs[L] - y.astype(np.float32)) * fprime(xs[L])
    for k in range(L, 0, -1):
        rows = np.repeat(np.arange(n), np.diff(rp[k - 1]))
        grads[k - 1] = deltas[k][rows] * xs[k - 1][col[k - 1]]
        if k > 1:
            deltas[k - 1] = (mats[k - 1].T @ deltas[k]) * fprime(xs[k - 1])
    return xs, deltas, grads


def test_plain_fp32_misses_a_fine_elementwise_bar_but_not_the_normwise_one():
    spec = gen.CFG1_TRAIN.live()
    rp, col, val, bias = gen.network(spec)
    x0, y = gen.inputs(spec, 1)[0], gen.targets(spec, 1)[0]
    xs, deltas, grads = fp32_step(rp, col, val, bias, x0, y)

    # the oracle takes the fp32 evaluation's derivative decisions where the two differ at a kink, as the parity
    # harness does for the GPU's, so that the comparison downstream is like for like
    def hook(k, z, scale, mask):
        m32 = ((xs[k] > 0) & (xs[k] < 32.0)).astype(np.float64)[None, :]
        assert np.all((m32 == mask) | (np.minimum(np.abs(z), np.abs(z - 32.0)) <= 64 * 2.0 ** -24 * scale))
        return m32

    out = OracleNet(rp, col, val, bias).train_step(x0[None, :], y[None, :], 1e-3, mask_hook=hook)
    worst = {"normwise": 0.0, "coarse": 0.0, "fine": 0.0}
    for k in range(1, spec.layers + 1):
        for got, want in ((xs[k], out["x"][k][0]), (deltas[k], out["delta"][k][0]), (grads[k - 1], out["grad"][k - 1])):
            assert np.any(want != 0.0)
            worst["normwise"] = max(worst["normwise"], rel_err(got, want))
            worst["coarse"] = max(worst["coarse"], rel_err_elem(got, want, FLOOR))
            worst["fine"] = max(worst["fine"], rel_err_elem(got, want, FLOOR_FINE))
    print("plain fp32 against the float64 oracle, worst tensor of one step:", worst)
    assert worst["normwise"] <= TOL / 10, "plain fp32 should meet the normwise bar with room to spare"
    assert worst["coarse"] <= TOL_ELEM / 10
    assert worst["fine"] > 5 * TOL, "premise gone: plain fp32 now comes close to an elementwise 1e-4 bar with a 0.1 % floor"
