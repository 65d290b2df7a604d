"""The harness rule for derivative decisions at the kinks of the clamped ReLU (parity_util.KinkProtocol), on the CPU.

The stand-in for the GPU is the float64 oracle itself run from a slightly perturbed layer input, so that its
decisions are exactly right for ITS inputs but differ from the unperturbed run's on entries that sit further
from a kink than one layer's rounding allowance: the protocol must settle those on the stand-in's own layer
input (second hearing) and flag nothing.  A planted wrong decision, far from any kink, must be flagged.
"""
import numpy as np

import gen
from oracle import OracleNet
from parity_util import KinkProtocol


def run(perturb, plant=None):
    spec = gen.CFG1_TRAIN.scaled(1024, 8).live()
    rp, col, val, bias = gen.network(spec)
    x0, y = gen.inputs(spec, 8), gen.targets(spec, 8)
    ora = OracleNet(rp, col, val, bias)
    # the stand-in's activations: the same net, its first layer's output nudged by a relative 2e-3
    other = OracleNet(rp, col, val, bias)
    xs = [x0.astype(np.float64)]
    for k in range(spec.layers):
        _, x, _ = other.forward_layer(k, xs[-1])
        if k == 0:
            x = x * (1.0 + perturb * np.cos(np.arange(x.size).reshape(x.shape)))
        xs.append(x)
    if plant is not None:
        k, b, i = plant
        xs[k] = xs[k].copy()
        xs[k][b, i] = 0.0 if xs[k][b, i] > 0.0 else 1.0          # the opposite decision, whatever the margin
    proto = KinkProtocol(lambda k: xs[k].astype(np.float32) if k else x0,
                         relayer=lambda k, xp: ora.forward_layer(k - 1, xp, want_scale=True)[::2])
    ora.train_step(x0, y, 1e-3, mask_hook=proto)
    return proto


def test_flips_caused_by_upstream_deviation_are_settled_on_the_layers_own_input():
    proto = run(perturb=2e-3)
    assert proto.flipped > 0 and proto.second_hearing > 0, "the perturbation should move some decisions outside tau"
    assert proto.hard_mismatch == 0


def test_a_planted_wrong_decision_is_flagged():
    clean = run(perturb=0.0)
    assert clean.hard_mismatch == 0 and clean.second_hearing == 0
    # pick an entry of layer 3 that is far from both kinks in the clean run: index found from the oracle's own forward pass
    spec = gen.CFG1_TRAIN.scaled(1024, 8).live()
    ora = OracleNet(*gen.network(spec))
    x = gen.inputs(spec, 8).astype(np.float64)
    for k in range(3):
        z, x, _ = ora.forward_layer(k, x)
    b, i = np.unravel_index(np.argmax(np.minimum(np.abs(z), np.abs(z - 32.0))), z.shape)
    assert run(perturb=0.0, plant=(3, int(b), int(i))).hard_mismatch >= 1
