"""TEST INFRASTRUCTURE ONLY: float64 CPU oracle (see the package docstring).

What it computes, in the paper's notation (Section 3.2, Algorithm 1, and the
minibatch remark in the Discussion of Section 5), for L square layers W^k
(CSR, row j = incoming links of neuron j of layer k+1), biases b^k and the
activation f(z) = min(max(z, 0), c):

    forward,  k = 1..L :  z^k = W^k x^{k-1} + b^k ;  x^k = f(z^k)                (feedforward equation)
    loss               :  J = 1/(2B) sum_b ||x^L_b - y_b||^2                      (mean squared error)
    output gradient    :  delta^L_b = (x^L_b - y_b) (.) f'(z^L_b)                 (final-layer gradient equation)
    backward, k = L..1 :  s_b = (W^k)^T delta^k_b            with W^k BEFORE its update (Algorithm 1 computes
                          G^k(j,i) = 1/B sum_b delta^k_b(j) x^{k-1}_b(i)          delta^{k-1} before updating W^k)
                          W^k(j,i) <- W^k(j,i) - eta G^k(j,i)  on stored entries  (gradient update rule)
                          delta^{k-1}_b = s_b (.) f'(z^{k-1}_b)    (k > 1)        (recursive formula)

    f'(z) = 1 for 0 < z < c and 0 otherwise (zero at both kinks).

With activation="sigmoid" (the activation of the paper's own experiments, Section 6) f(z) = 1/(1+exp(-z)) and
f'(z) = f(z) (1 - f(z)); everything else is unchanged.

Readings taken where the paper is silent: the minibatch step is exact minibatch
SGD (one delta per input, gradient averaged over the batch; B = 1 is Algorithm 1
verbatim); delta^0 is never formed (x^0 is data, no z^0 exists); the bias is
frozen unless update_bias is set, in which case b^k <- b^k - eta * mean_b delta^k_b
(the bias read as one more column of W^k whose input is the constant 1).

train_step_averaged is the other reading of the same remark (Discussion of Section 5: the output gradients of
the batch are averaged into one delta^L and only that single vector is sent backwards): delta^L = mean_b delta^L_b,
then the backward loop above for ONE vector, paired with the batch means xbar^{k-1} = mean_b x^{k-1}_b, f' being
evaluated from xbar^{k-1} as it is from a single input's x^{k-1}.  The remark does not fix that pairing:
PARITY UNPINNED for this function as far as the paper goes; the pins only hold it to Algorithm 1 where the two
must agree (B = 1, a batch of identical inputs) and to a dense restatement.

All inputs are the fp32 numbers the GPU sees, widened to float64; all arithmetic
is float64.  Heavy loops live in sdnn_oracle.c; this file only sequences them.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "sdnn_oracle.c")
_LIB = os.path.join(_HERE, "libsdnn_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the C part of the oracle next to its source (no-op when up to date)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(
            ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-ffp-contract=off", "-o", _LIB, _SRC, "-lm"]
        )
    return _LIB


def _L():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        i32, dbl, vp = ctypes.c_int32, ctypes.c_double, ctypes.c_void_p
        lib.oracle_forward_layer.argtypes = [i32, i32, vp, vp, vp, vp, vp, dbl, i32, vp, vp, vp]
        lib.oracle_transposed_product.argtypes = [i32, i32, vp, vp, vp, vp, vp]
        lib.oracle_masked_gradient.argtypes = [i32, i32, vp, vp, vp, vp, vp]
        for f in (lib.oracle_forward_layer, lib.oracle_transposed_product, lib.oracle_masked_gradient):
            f.restype = None
        _lib = lib
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _f64(a, shape=None):
    a = np.ascontiguousarray(np.asarray(a), dtype=np.float64)
    if shape is not None and a.shape != shape:
        raise ValueError(f"expected shape {shape}, got {a.shape}")
    return a


def nonzero_sets(x_last: np.ndarray):
    """Per input b, the ascending indices i with x^L_b(i) != 0."""
    return [np.flatnonzero(row != 0.0).astype(np.int32) for row in x_last]


class OracleNet:
    """L square sparse layers in CSR plus biases; weights are held (and trained) in float64."""

    def __init__(self, row_ptr, col, val, bias, clamp: float = 32.0, update_bias: bool = False,
                 activation: str = "clamped_relu"):
        if activation not in ("clamped_relu", "sigmoid"):
            raise ValueError(activation)
        self.activation = activation
        self.layers = len(col)
        self.n = len(bias[0])
        self.row_ptr = [np.ascontiguousarray(r, dtype=np.int32) for r in row_ptr]
        self.col = [np.ascontiguousarray(c, dtype=np.int32) for c in col]
        self.w = [np.array(v, dtype=np.float64) for v in val]         # copies: training mutates them
        self.bias = [np.array(b, dtype=np.float64) for b in bias]
        self.clamp = float(np.float32(clamp))
        self.update_bias = bool(update_bias)
        for k in range(self.layers):
            if self.row_ptr[k].shape != (self.n + 1,) or self.col[k].shape != self.w[k].shape:
                raise ValueError("inconsistent CSR arrays")

    def quantize_state(self):
        """Rounds weights and biases to the nearest fp32 numbers (kept as float64).

        The GPU library stores its parameters in fp32 between steps.  A parity harness that wants both
        sides to START a step from identical numbers calls this and loads the result into the library;
        within the step all oracle arithmetic stays float64.  Not called by train_step itself."""
        self.w = [w.astype(np.float32).astype(np.float64) for w in self.w]
        self.bias = [b.astype(np.float32).astype(np.float64) for b in self.bias]

    # ---- single steps -------------------------------------------------------------------------
    def forward_layer(self, k: int, x_prev: np.ndarray, want_scale: bool = False):
        """Layer k (0-based: uses W^{k+1}) on x_prev [B, n] -> (z, x, scale); scale = |b| + sum|w x| or None."""
        x_prev = _f64(x_prev)
        nb = x_prev.shape[0]
        z = np.empty((nb, self.n))
        x = np.empty((nb, self.n))
        scale = np.empty((nb, self.n)) if want_scale else None
        _L().oracle_forward_layer(self.n, nb, _p(self.row_ptr[k]), _p(self.col[k]), _p(self.w[k]), _p(self.bias[k]),
                                  _p(x_prev), self.clamp, 1 if self.activation == "sigmoid" else 0, _p(z), _p(x), _p(scale))
        return z, x, scale

    def derivative_mask(self, z: np.ndarray) -> np.ndarray:
        """f'(z): clamped ReLU: a 0/1 array, 1 strictly inside (0, c); sigmoid: f(z) (1 - f(z))."""
        if self.activation == "sigmoid":
            f = 1.0 / (1.0 + np.exp(-z))
            return f * (1.0 - f)
        return ((z > 0.0) & (z < self.clamp)).astype(np.float64)

    def transposed_product(self, k: int, delta: np.ndarray) -> np.ndarray:
        delta = _f64(delta)
        s = np.empty_like(delta)
        _L().oracle_transposed_product(self.n, delta.shape[0], _p(self.row_ptr[k]), _p(self.col[k]), _p(self.w[k]),
                                       _p(delta), _p(s))
        return s

    def masked_gradient(self, k: int, delta: np.ndarray, x_prev: np.ndarray) -> np.ndarray:
        delta, x_prev = _f64(delta), _f64(x_prev)
        g = np.empty_like(self.w[k])
        _L().oracle_masked_gradient(self.n, delta.shape[0], _p(self.row_ptr[k]), _p(self.col[k]), _p(delta),
                                    _p(x_prev), _p(g))
        return g

    # ---- whole passes -------------------------------------------------------------------------
    def infer(self, x0, keep_all: bool = False):
        """Forward through all layers.  Returns x^L [B, n] (or the list x^0..x^L when keep_all)."""
        x = _f64(x0)
        xs = [x]
        for k in range(self.layers):
            _, x, _ = self.forward_layer(k, x)
            if keep_all:
                xs.append(x)
        return xs if keep_all else x

    def train_step(self, x0, y, eta: float, mask_hook=None, keep=("x", "delta", "grad")):
        """One minibatch SGD step; mutates the weights.

        mask_hook(k, z, scale, mask) -> mask, if given, may replace the derivative mask of layer
        output k (1-based) - the parity harness uses it for entries that sit on a kink within
        rounding error.  Returns dict(loss, x=[x^0..x^L], delta=[None, d^1..d^L], grad=[G^1..G^L],
        bias_grad=[...]) with the lists present as requested in `keep`.
        """
        x = _f64(x0)
        y = _f64(y, x.shape)
        nb = x.shape[0]
        eta = float(np.float32(eta))
        xs, masks = [x], [None]
        for k in range(self.layers):
            z, x, scale = self.forward_layer(k, x, want_scale=mask_hook is not None)
            m = self.derivative_mask(z)
            if mask_hook is not None and self.activation == "sigmoid":
                raise ValueError("mask_hook is for the kinks of the clamped ReLU; the sigmoid has none")
            if mask_hook is not None:
                m = mask_hook(k + 1, z, scale, m)
            xs.append(x)
            masks.append(m)
        diff = xs[-1] - y
        loss = float((diff * diff).sum() / (2.0 * nb))
        delta = diff * masks[-1]
        out = {"loss": loss}
        deltas = [None] * (self.layers + 1)
        grads = [None] * self.layers
        bgrads = [None] * self.layers
        for k in range(self.layers - 1, -1, -1):                 # paper's k = L..1 is k+1 here
            if "delta" in keep:
                deltas[k + 1] = delta
            s = self.transposed_product(k, delta) if k > 0 else None      # uses W before its update
            g = self.masked_gradient(k, delta, xs[k])
            self.w[k] -= eta * g
            if "grad" in keep:
                grads[k] = g
            bg = delta.mean(axis=0)
            if "grad" in keep:
                bgrads[k] = bg
            if self.update_bias:
                self.bias[k] -= eta * bg
            if k > 0:
                delta = s * masks[k]
        if "x" in keep:
            out["x"] = xs
        if "delta" in keep:
            out["delta"] = deltas
        if "grad" in keep:
            out["grad"] = grads
            out["bias_grad"] = bgrads
        out["masks"] = masks
        return out

    def derivative_from_activation(self, x: np.ndarray) -> np.ndarray:
        """f' written in terms of x = f(z): clamped ReLU: 1 strictly inside (0, c); sigmoid: x (1 - x)."""
        if self.activation == "sigmoid":
            return x * (1.0 - x)
        return ((x > 0.0) & (x < self.clamp)).astype(np.float64)

    def train_step_averaged(self, x0, y, eta: float):
        """Minibatch step in the averaged form (Discussion of Section 5): forward on the whole batch, delta^L averaged
        over the batch, one vector backpropagated as in Algorithm 1 with the batch means of the activations.
        Mutates the weights.  Returns dict(loss, x=[x^0..x^L] per input, xbar=[...], delta=[None, d^1..d^L] (each [1, n]),
        grad=[G^1..G^L] with G^k = delta^k (x) xbar^{k-1} on the stored entries)."""
        x = _f64(x0)
        y = _f64(y, x.shape)
        nb = x.shape[0]
        eta = float(np.float32(eta))
        xs = [x]
        z = None
        for k in range(self.layers):
            z, x, _ = self.forward_layer(k, x)
            xs.append(x)
        xbar = [v.mean(axis=0, keepdims=True) for v in xs]
        diff = xs[-1] - y
        loss = float((diff * diff).sum() / (2.0 * nb))
        delta = (diff * self.derivative_mask(z)).mean(axis=0, keepdims=True)     # average of the per-input output gradients
        deltas = [None] * (self.layers + 1)
        grads = [None] * self.layers
        for k in range(self.layers - 1, -1, -1):
            deltas[k + 1] = delta
            s = self.transposed_product(k, delta) if k > 0 else None      # uses W before its update
            g = self.masked_gradient(k, delta, xbar[k])
            self.w[k] -= eta * g
            grads[k] = g
            if self.update_bias:
                self.bias[k] -= eta * delta[0]
            if k > 0:
                delta = s * self.derivative_from_activation(xbar[k])
        return {"loss": loss, "x": xs, "xbar": xbar, "delta": deltas, "grad": grads}
