"""Harness shared by the GPU parity tests: error metric, kink-ambiguity protocol, net builders.

Error metric (per tensor; a tensor that is identically zero in the oracle must be identically zero on
the GPU):
  rel_err      = max_i |g_i - o_i| / max_i |o_i|                           bar TOL = 1e-4
  rel_err_elem = max_i |g_i - o_i| / max(|o_i|, FLOOR * max|o|)             guard TOL_ELEM = 1e-3
  the same with the floor at FLOOR_FINE = 1e-3 * max|o|                     recorded, not asserted
The bar is normwise because every entry is a signed sum: its fp32 rounding error scales with the sum
of the magnitudes of its terms and of the upstream errors they carry, not with the entry itself, so an
entry that is small by cancellation cannot be held to a relative bound by any fp32 evaluation order.
tests/test_error_metric.py measures this without a GPU: on one step of the live 1024 x 120 net (B = 1,
120 forward + 119 backward layers) a plain fp32 evaluation on the CPU (scipy float32 products) deviates
from the float64 oracle by 1.8e-6 normwise, 3.7e-5 under the elementwise metric with a 5 % floor and
9.3e-4 with a floor of 1e-3 * max|o|: an elementwise 1e-4 bar with a small floor is missed by fp32
arithmetic itself.  The elementwise figure is therefore only guarded (floor 5 %, 1e-3: it still catches
any entry above 5 % of the maximum that is off by more than 0.1 %); every check_close call records the
worst figure under all three metrics in WORST (per run) and SESSION_WORST (printed at the end of a test
session), so that a GPU run reports its margin under each.

Kink protocol.  f'(z) jumps at z = 0 and z = clamp, so fp32 and float64 may legitimately disagree on
the 0/1 derivative mask (and on "x != 0") when z sits within rounding error of a kink.  An entry of
layer k is *ambiguous* when min(|z|, |z - clamp|) <= tau with tau = TAU_ULPS * 2^-24 * (|b| + sum|w x|),
the scale of the rounding error of that dot product, and that scale is not zero (with every term zero both
sides compute z = b exactly, so nothing can differ).  Outside the ambiguous set the GPU's mask must
equal the oracle's bit for bit; on ambiguous entries the oracle continues with the GPU's decision, so
that everything downstream (deltas, gradients, weights) is compared like for like.  The ambiguous set
must stay small or the exact comparison would mean nothing: z is a sum of m terms of either sign, so its
density near a kink is about 1 / (2.5 * S / sqrt(m)) with S = |b| + sum|w x|, and an entry falls within
tau = 64 * 2^-24 * S of it with probability about 2 * tau * sqrt(m) / (2.5 * S) = 3e-6 * sqrt(m), i.e. 1e-5 to
2e-5 for rows of 10 to 40 live terms.  assert_few_ambiguous holds a run to AMBIGUOUS_RATE = 1e-4 of its
entries (plus a handful for small runs).

Depth.  tau covers the rounding of ONE layer's sum.  A thousand layers down, the layer's input x^{k-1} itself
differs between the two sides by the rounding accumulated below (measured 5e-6 * max|x| at 960 layers of the
65536-neuron live net, more than the 4e-6 that tau allows), so that one entry in some 1e9 can sit outside tau
and still be decided differently for no fault of the layer.  Such an entry gets a second, exact hearing: the
float64 layer is evaluated on the GPU's OWN x^{k-1} (`relayer`), and there the two decisions may differ only
within tau again.  An entry that fails both is a hard mismatch.
"""
from __future__ import annotations

import numpy as np

TAU_ULPS = 64.0
TOL = 1e-4
TOL_ELEM = 1e-3
FLOOR = 0.05
FLOOR_FINE = 1e-3
AMBIGUOUS_RATE = 1e-4
AMBIGUOUS_SLACK = 8

# worst figures seen by check_close since the last reset_worst(), per metric
WORST = {"normwise": 0.0, "elem_floor_5e-2": 0.0, "elem_floor_1e-3": 0.0}
SESSION_WORST = dict(WORST)


def reset_worst():
    for k in WORST:
        WORST[k] = 0.0


def _pair(gpu, ora):
    gpu = np.asarray(gpu, dtype=np.float64)
    ora = np.asarray(ora, dtype=np.float64)
    assert gpu.shape == ora.shape, (gpu.shape, ora.shape)
    return gpu, ora


def rel_err(gpu: np.ndarray, ora: np.ndarray) -> float:
    """Normwise: max |g - o| / max |o| (inf if the oracle tensor is zero and the GPU's is not)."""
    gpu, ora = _pair(gpu, ora)
    if ora.size == 0:
        return 0.0
    top = np.abs(ora).max()
    if top == 0.0:
        return 0.0 if not gpu.any() else float("inf")
    return float(np.abs(gpu - ora).max() / top)


def rel_err_elem(gpu: np.ndarray, ora: np.ndarray, floor: float = FLOOR) -> float:
    """Elementwise with a floor: max |g_i - o_i| / max(|o_i|, floor * max|o|)."""
    gpu, ora = _pair(gpu, ora)
    if ora.size == 0:
        return 0.0
    top = np.abs(ora).max()
    if top == 0.0:
        return 0.0 if not gpu.any() else float("inf")
    return float(np.max(np.abs(gpu - ora) / np.maximum(np.abs(ora), floor * top)))


def check_close(gpu, ora, what=""):
    """Asserts both bars; returns the normwise error.  Records the worst figure under each metric in WORST."""
    e, ee = rel_err(gpu, ora), rel_err_elem(gpu, ora)
    WORST["normwise"] = max(WORST["normwise"], e)
    WORST["elem_floor_5e-2"] = max(WORST["elem_floor_5e-2"], ee)
    WORST["elem_floor_1e-3"] = max(WORST["elem_floor_1e-3"], rel_err_elem(gpu, ora, FLOOR_FINE))
    for k in WORST:
        SESSION_WORST[k] = max(SESSION_WORST[k], WORST[k])
    assert e <= TOL, f"{what}: max relative error {e:.3g} > {TOL}"
    assert ee <= TOL_ELEM, f"{what}: elementwise relative error {ee:.3g} > {TOL_ELEM}"
    return e


class KinkProtocol:
    """mask_hook for OracleNet.train_step; `gpu_x(k)` returns the GPU's x^k [B, n] (fp32)."""

    def __init__(self, gpu_x, clamp=32.0, tau_ulps=TAU_ULPS, relayer=None):
        """relayer(k, x_prev) -> (z, scale): float64 pre-activations of layer k (1-based) and their rounding scale
        for the input x_prev [B, n]; used only for entries that differ outside tau (see the module docstring)."""
        self.gpu_x, self.clamp, self.tau_ulps, self.relayer = gpu_x, float(clamp), tau_ulps, relayer
        self.second_hearing = 0   # entries outside tau that were settled on the GPU's own layer input
        self.ambiguous = 0
        self.flipped = 0
        self.entries = 0
        self.hard_mismatch = 0
        self.worst = 0.0          # largest margin/tau among entries where the two masks differ

    def __call__(self, k, z, scale, mask):
        xg = self.gpu_x(k).astype(np.float64)
        mg = ((xg > 0.0) & (xg < self.clamp)).astype(np.float64)
        margin = np.minimum(np.abs(z), np.abs(z - self.clamp))
        tau = self.tau_ulps * 2.0 ** -24 * scale
        amb = (margin <= tau) & (scale > 0.0)
        differ = mg != mask
        self.entries += mask.size
        self.ambiguous += int(amb.sum())
        self.flipped += int(differ.sum())
        hard = differ & ~amb
        if hard.any() and self.relayer is not None:
            z2, scale2 = self.relayer(k, self.gpu_x(k - 1).astype(np.float64))
            m2 = ((z2 > 0.0) & (z2 < self.clamp)).astype(np.float64)
            margin2 = np.minimum(np.abs(z2), np.abs(z2 - self.clamp))
            settled = hard & ((mg == m2) | ((margin2 <= self.tau_ulps * 2.0 ** -24 * scale2) & (scale2 > 0.0)))
            self.second_hearing += int(settled.sum())
            hard &= ~settled
            amb = amb | settled          # the oracle continues with the GPU's decision there too
        self.hard_mismatch += int(hard.sum())
        if differ.any():
            self.worst = max(self.worst, float((margin[differ] / np.maximum(tau[differ], 1e-300)).max()))
        return np.where(amb, mg, mask)


def assert_few_ambiguous(ambiguous: int, entries: int, what=""):
    """The kink-ambiguous set must be a vanishing part of the compared entries (see the module docstring)."""
    bound = AMBIGUOUS_SLACK + AMBIGUOUS_RATE * entries
    assert ambiguous <= bound, f"{what}: {ambiguous} ambiguous entries of {entries} (bound {bound:.0f}): tau is too generous"


def ragged_net(rng, n, layers, kmax, scale=0.6, bias_scale=0.1, align4=False):
    """Random CSR layers with rows of 0..kmax entries (or multiples of 4 when align4)."""
    rps, cols, vals, biases = [], [], [], []
    for _ in range(layers):
        counts = rng.integers(0, kmax + 1, size=n)
        if align4:
            counts = counts // 4 * 4
        counts[rng.integers(0, n)] = kmax
        rp = np.zeros(n + 1, dtype=np.int32)
        rp[1:] = np.cumsum(counts)
        c = np.concatenate([np.sort(rng.choice(n, size=m, replace=False)) for m in counts]).astype(np.int32)
        rps.append(rp); cols.append(c)
        vals.append((rng.standard_normal(rp[-1]) * scale).astype(np.float32))
        biases.append((rng.standard_normal(n) * bias_scale).astype(np.float32))
    return rps, cols, vals, biases
