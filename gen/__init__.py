"""Seeded synthetic sparse-DNN workloads (patterns, weights, inputs, targets).

Data only: this package holds none of the method's arithmetic.  The CPU oracle
and the CUDA library are both fed from here so that they see identical arrays.
The numbers come from the counter-based generator in ``sdnn_gen.c`` (compiled
on first use with gcc); the shapes follow the grid of the paper's Section 6
(N neurons per layer x L layers, 60000 binary inputs), with synthetic uniform
or banded-permuted patterns of 32 nonzeros per row standing in for the
RadiX-Net topologies and thresholded MNIST inputs used there.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass, replace

import numpy as np

MASTER_SEED = 210411805

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "sdnn_gen.c")
_LIB = os.path.join(_HERE, "libsdnn_gen.so")

# stream ids (first component of every key)
S_PATTERN, S_PERM, S_VALUES, S_INPUT, S_TARGET, S_SHUFFLE = 1, 2, 3, 4, 5, 6


def build(force: bool = False) -> str:
    """Compile the generator library next to its source (no-op when up to date)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(
            ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-ffp-contract=off", "-o", _LIB, _SRC, "-lm"]
        )
    return _LIB


_lib = None


def _L():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        u64, i64, i32, dbl = ctypes.c_uint64, ctypes.c_int64, ctypes.c_int32, ctypes.c_double
        vp = ctypes.c_void_p
        lib.sdnn_gen_draw.restype = u64
        lib.sdnn_gen_draw.argtypes = [u64, u64, u64, u64, u64]
        lib.sdnn_gen_pattern_uniform.argtypes = [u64, u64, i64, i32, i32, vp]
        lib.sdnn_gen_permutation.argtypes = [u64, u64, i64, i32, vp]
        lib.sdnn_gen_pattern_windowed.argtypes = [u64, u64, i64, i32, i32, i32, vp, vp]
        lib.sdnn_gen_normal.argtypes = [u64, u64, i64, i64, dbl, vp]
        lib.sdnn_gen_bernoulli.argtypes = [u64, u64, i64, i64, dbl, vp]
        lib.sdnn_gen_uniform.argtypes = [u64, u64, i64, i64, vp]
        for f in (lib.sdnn_gen_pattern_uniform, lib.sdnn_gen_permutation, lib.sdnn_gen_pattern_windowed,
                  lib.sdnn_gen_normal, lib.sdnn_gen_bernoulli, lib.sdnn_gen_uniform):
            f.restype = None
        _lib = lib
    return _lib


def _ptr(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


@dataclass(frozen=True)
class NetSpec:
    """One synthetic network family (pattern + value rule + bias)."""
    name: str
    n: int                      # neurons per layer
    layers: int
    k: int = 32                 # nonzeros per row
    pattern: str = "uniform"    # "uniform" | "windowed"
    window: int = 1024
    values: str = "const"       # "const" (value `const`) | "normal" (std `sigma`) | "uniform_pm1" (uniform in [-1, 1))
    const: float = 1.0 / 16.0
    sigma: float = 32.0 ** -0.5
    bias: float = -0.30
    input_prob: float = 0.1
    config_id: int = 0          # separates the key spaces of the configs
    seed: int = MASTER_SEED
    shuffle: bool = False       # hidden structure: the neurons of every inner layer renumbered at random (see shuffled())

    # ---- companions that keep activations alive / drive them to the clamp ----
    def live(self) -> "NetSpec":
        """Same pattern; weights N(0, 2/k) (He scaling), bias 0: ~50 % of the neurons stay active."""
        return replace(self, name=self.name + "-live", values="normal", sigma=(2.0 / self.k) ** 0.5, bias=0.0)

    def saturating(self) -> "NetSpec":
        """Same pattern; all weights 1/16, bias -0.30, inputs Bernoulli(0.5): every neuron reaches the clamp."""
        return replace(self, name=self.name + "-sat", values="const", const=1.0 / 16.0, bias=-0.30, input_prob=0.5)

    def paper_setup(self) -> "NetSpec":
        """Same pattern with the training setup of the paper's Section 6: weights uniform in [-1, 1], bias 0 (to be
        used with the sigmoid activation and eta = 0.01; no neuron ever dies)."""
        return replace(self, name=self.name + "-paper", values="uniform_pm1", bias=0.0)

    def shuffled(self) -> "NetSpec":
        """The same network with the neurons of every inner layer renumbered by a seeded random permutation (rows of
        that layer's matrix permuted, columns of the next layer's matrix renamed to match; input and output neurons
        keep their numbers).  The function computed is unchanged; whatever block structure the pattern has is
        hidden behind the renumbering, as in a network that arrives in no particular neuron order."""
        return replace(self, name=self.name + "-shuffled", shuffle=True)

    def sliced(self, layers: int) -> "NetSpec":
        return replace(self, layers=layers)

    def scaled(self, n: int, layers: int) -> "NetSpec":
        """Same recipe at another size (reduced-size parity cases)."""
        return replace(self, n=n, layers=layers, window=min(self.window, n))

    @property
    def nnz_per_layer(self) -> int:
        return self.n * self.k

    @property
    def total_nnz(self) -> int:
        return self.n * self.k * self.layers


# The five benchmark configurations (inference nets: constant 1/16; training nets: N(0, 1/32)).
CFG1_INF = NetSpec("cfg1-inf", 1024, 120, values="const", bias=-0.30, config_id=1)
CFG1_TRAIN = NetSpec("cfg1-train", 1024, 120, values="normal", bias=-0.30, config_id=1)
CFG2 = NetSpec("cfg2-inf", 4096, 120, values="const", bias=-0.35, config_id=2)
CFG3 = NetSpec("cfg3-train", 16384, 480, values="normal", bias=-0.40, config_id=3)
CFG4 = NetSpec("cfg4-inf", 65536, 120, pattern="windowed", values="const", bias=-0.45, config_id=4)
CFG5 = NetSpec("cfg5-train", 65536, 1920, values="normal", bias=-0.45, config_id=5)

CONFIGS = {c.name: c for c in (CFG1_INF, CFG1_TRAIN, CFG2, CFG3, CFG4, CFG5)}


def row_ptr(spec: NetSpec) -> np.ndarray:
    return (np.arange(spec.n + 1, dtype=np.int64) * spec.k).astype(np.int32)


def _renumbering(spec: NetSpec, layer: int) -> np.ndarray:
    """q[new] = old number of the output neurons of layer `layer` (0-based); identity for the last layer and for layer -1
    (the inputs)."""
    if not spec.shuffle or layer < 0 or layer >= spec.layers - 1:
        return np.arange(spec.n, dtype=np.int32)
    q = np.empty(spec.n, dtype=np.int32)
    _L().sdnn_gen_permutation(spec.seed, (spec.config_id << 8) | S_SHUFFLE, layer, spec.n, _ptr(q))
    return q


def _renumbered(spec: NetSpec, layer: int, col: np.ndarray, val: np.ndarray | None):
    """Applies the renumbering of shuffled() to one layer given in the original numbering: pure index bookkeeping."""
    q_out, q_in = _renumbering(spec, layer), _renumbering(spec, layer - 1)
    inv_in = np.empty(spec.n, dtype=np.int32)
    inv_in[q_in] = np.arange(spec.n, dtype=np.int32)
    c = inv_in[col.reshape(spec.n, spec.k)[q_out]]
    order = np.argsort(c, axis=1, kind="stable")
    c = np.take_along_axis(c, order, axis=1).astype(np.int32).reshape(-1)
    if val is None:
        return c, None
    v = np.take_along_axis(val.reshape(spec.n, spec.k)[q_out], order, axis=1).reshape(-1)
    return c, np.ascontiguousarray(v)


def layer_pattern(spec: NetSpec, layer: int) -> np.ndarray:
    """Column indices of layer `layer` (0-based), int32 [n*k], ascending within each row."""
    if spec.shuffle:
        return _renumbered(spec, layer, layer_pattern(replace(spec, shuffle=False), layer), None)[0]
    col = np.empty(spec.n * spec.k, dtype=np.int32)
    if spec.pattern == "uniform":
        _L().sdnn_gen_pattern_uniform(spec.seed, (spec.config_id << 8) | S_PATTERN, layer, spec.n, spec.k, _ptr(col))
    elif spec.pattern == "windowed":
        perm = layer_permutation(spec, layer)
        _L().sdnn_gen_pattern_windowed(spec.seed, (spec.config_id << 8) | S_PATTERN, layer, spec.n, spec.k,
                                       spec.window, _ptr(perm), _ptr(col))
    else:
        raise ValueError(spec.pattern)
    return col


def layer_permutation(spec: NetSpec, layer: int) -> np.ndarray:
    perm = np.empty(spec.n, dtype=np.int32)
    _L().sdnn_gen_permutation(spec.seed, (spec.config_id << 8) | S_PERM, layer, spec.n, _ptr(perm))
    return perm


def layer_values(spec: NetSpec, layer: int) -> np.ndarray:
    """Weights of layer `layer` in CSR order, float32 [n*k]."""
    if spec.shuffle:
        base = replace(spec, shuffle=False)
        return _renumbered(spec, layer, layer_pattern(base, layer), layer_values(base, layer))[1]
    cnt = spec.n * spec.k
    if spec.values == "const":
        return np.full(cnt, np.float32(spec.const), dtype=np.float32)
    out = np.empty(cnt, dtype=np.float32)
    if spec.values == "uniform_pm1":
        _L().sdnn_gen_uniform(spec.seed, (spec.config_id << 8) | S_VALUES, layer, cnt, _ptr(out))
        return (2.0 * out - 1.0).astype(np.float32)
    _L().sdnn_gen_normal(spec.seed, (spec.config_id << 8) | S_VALUES, layer, cnt, float(spec.sigma), _ptr(out))
    return out


def layer_bias(spec: NetSpec, layer: int) -> np.ndarray:
    return np.full(spec.n, np.float32(spec.bias), dtype=np.float32)


def layer(spec: NetSpec, layer_idx: int):
    """(row_ptr, col, val, bias) of one layer."""
    return row_ptr(spec), layer_pattern(spec, layer_idx), layer_values(spec, layer_idx), layer_bias(spec, layer_idx)


def network(spec: NetSpec):
    """Whole net as four lists of per-layer arrays (row_ptr is shared between layers)."""
    rp = row_ptr(spec)
    cols, vals, biases = [], [], []
    for l in range(spec.layers):
        cols.append(layer_pattern(spec, l))
        vals.append(layer_values(spec, l))
        biases.append(layer_bias(spec, l))
    return [rp] * spec.layers, cols, vals, biases


def inputs(spec: NetSpec, count: int, step: int = 0, start: int = 0) -> np.ndarray:
    """Binary input vectors [count, n] (Bernoulli(input_prob)); `step` selects the minibatch stream,
    `start` the first input of a longer stream (inputs start..start+count-1 of that stream)."""
    lib = _L()
    out = np.empty((count, spec.n), dtype=np.float32)
    for r in range(count):  # one key per input vector, so any sub-range can be regenerated
        lib.sdnn_gen_bernoulli(spec.seed, (spec.config_id << 8) | S_INPUT, (step << 32) | (start + r), spec.n,
                               float(spec.input_prob), ctypes.c_void_p(out.ctypes.data + r * spec.n * 4))
    return out


def targets(spec: NetSpec, count: int, step: int = 0) -> np.ndarray:
    """Targets uniform in [0,1), [count, n]."""
    out = np.empty((count, spec.n), dtype=np.float32)
    _L().sdnn_gen_uniform(spec.seed, (spec.config_id << 8) | S_TARGET, step, count * spec.n, _ptr(out))
    return out


def circulant_pattern(n: int, k: int, stride: int) -> np.ndarray:
    """Row i holds columns (i + t*stride) mod n, t < k (k per row and per column); ascending per row."""
    i = np.arange(n, dtype=np.int64)[:, None]
    t = np.arange(k, dtype=np.int64)[None, :]
    col = np.sort((i + t * stride) % n, axis=1)
    if (np.diff(col, axis=1) == 0).any():
        raise ValueError("stride/k give duplicate columns")
    return col.astype(np.int32).reshape(-1)


def draw(stream: int, a: int, b: int, t: int, seed: int = MASTER_SEED) -> int:
    return int(_L().sdnn_gen_draw(seed, stream, a, b, t))
