"""Pins for the accumulation order of the oracle's network policies (CPU only).

The policies are the one place where the method specifies fused multiply-adds: every
unit is a left-to-right chain acc = fma(w_i, x_i, acc) that starts from its bias
(in-kernel policy inference is the paper's Sec. VI outlook; the chain order is this
build's definition, stated in include/cartpole.h). A float64 matrix product cannot tell
that order from another one, so these tests do:

* hidden activations are read out bit-exactly through one-hot output weights
  (fma(1, h, 0) == h and fma(0, h, acc) == acc), then every later chain is re-evaluated
  in exact rationals with one rounding per term and must match bit for bit;
* chains whose inputs cannot be read out exactly (they feed a tanh) get operands built so
  that any other order — reversed, pairwise, bias added last, multiply and add rounded
  separately — lands far away from the left-to-right fused result (absorption of small
  terms by 2^20, and a product whose rounding error is the whole result).
"""
from fractions import Fraction

import numpy as np
import pytest

from paper_2301_13062_b200 import inputs
from tests.exact_arith import fma_chain_exact, round_f32

BIG = np.float32(2.0 ** 20)     # ulp 2^-3: absorbs anything up to 2^-4
TOL_TANH = 3e-7                 # glibc tanhf against float64 tanh (a few ulp below 1)


class Shallow:
    """4 -> H (tanh) -> 2: W1[H][4], b1[H], W2[2][H], b2[2]."""

    def __init__(self, oracle, H, wide):
        self.H, self.size = H, 7 * H + 2
        self.call = (lambda w, z: oracle.mlp_logits_wide(w, H, z)) if wide else oracle.mlp_logits
        self.w1 = lambda j: slice(4 * j, 4 * j + 4)
        self.b1 = lambda j: 4 * H + j
        self.w2 = lambda k: slice(5 * H + k * H, 5 * H + (k + 1) * H)
        self.b2 = lambda k: 7 * H + k

    def hidden(self, w, z):
        """Hidden activations, bit-exact, read through one-hot output weights."""
        h = np.empty(self.H, np.float32)
        for j in range(self.H):
            probe = np.array(w, np.float32)
            probe[5 * self.H:] = 0.0
            probe[5 * self.H + j] = 1.0
            h[j] = self.call(probe, z)[0]
        return h


NETS = {"mlp16": (16, False), "wide16": (16, True), "wide32": (32, True), "wide64": (64, True)}


@pytest.fixture(params=sorted(NETS))
def net(request, oracle):
    H, wide = NETS[request.param]
    return Shallow(oracle, H, wide)


def _weights(net, seed):
    kind = {16: inputs.POLICY_MLP, 32: inputs.POLICY_MLP32, 64: inputs.POLICY_MLP64}[net.H]
    return inputs.policy_weights(kind, seed)


def test_hidden_units_and_logit_chains_in_exact_rationals(net):
    w = _weights(net, 5)
    zs = inputs.random_states(12, seed=8, spread="live")
    for i in range(zs.shape[1]):
        z = zs[:, i]
        h = net.hidden(w, z)
        for j in range(net.H):
            acc = fma_chain_exact(w[net.w1(j)], z, w[net.b1(j)])  # exact first-layer chain
            assert abs(float(h[j]) - np.tanh(float(acc))) <= TOL_TANH
        got = net.call(w, z)
        for k in range(2):
            want = fma_chain_exact(w[net.w2(k)], h, w[net.b2(k)])
            assert got[k].view(np.uint32) == want.view(np.uint32)


def _first_layer_probes():
    """(b, w[4], z[4], value of the left-to-right fused chain, what a wrong reading would give)."""
    s = np.float32(2.0 ** -6)
    one = np.ones(4, np.float32)
    e = np.float32(1.0 + 2.0 ** -12)
    return [
        # reversed order absorbs both small terms: 0
        (0.0, [BIG, -BIG, s, s], one, 2.0 ** -5, 0.0),
        # pairwise (a+b)+(c+d) absorbs both: 0
        (0.0, [s, BIG, -BIG, s], one, 2.0 ** -6, 0.0),
        # bias added last: 0
        (BIG, [-BIG, s, s, s], one, 3 * 2.0 ** -6, 0.0),
        # multiply rounded before the add: (1+2^-12)^2 = 1 + 2^-11 + 2^-24 rounds to 1 + 2^-11 -> 0
        (-(1.0 + 2.0 ** -11), [e, 0, 0, 0], np.array([e, 1, 1, 1], np.float32), 2.0 ** -24, 0.0),
    ]


def test_first_layer_is_a_left_to_right_fused_chain_from_the_bias(net):
    amp = np.float32(2.0 ** 20)
    for j in (0, net.H // 2, net.H - 1):
        for b, wrow, z, value, wrong in _first_layer_probes():
            w = np.zeros(net.size, np.float32)
            w[net.w1(j)] = wrow
            w[net.b1(j)] = b
            w[5 * net.H + j] = amp            # logit 0 = amp * h_j, exact scaling
            assert float(fma_chain_exact(wrow, z, b)) == value  # the probe's own arithmetic
            got = float(net.call(w, z)[0]) / float(amp)
            want = np.tanh(value)
            assert abs(got - want) <= 2e-6 * want, (j, value, got)
            assert abs(want - np.tanh(wrong)) > 1e3 * 2e-6 * want  # the probe separates the readings


def _chain_probes(H):
    """(bias, weights[H], left-to-right sum with every multiplier equal to 1.0f)."""
    s = np.float32(2.0 ** -12)
    a = np.full(H, s, np.float32)
    a[0], a[1] = BIG, -BIG                    # reversed: the small terms are absorbed by -2^20
    b = np.full(H, s, np.float32)
    b[1], b[2] = BIG, -BIG                    # pairwise / tree orders lose b[0] or b[3]
    c = np.full(H, s, np.float32)
    c[0] = -BIG                               # with bias 2^20: added last it absorbs everything
    return [(0.0, a, (H - 2) * 2.0 ** -12), (0.0, b, (H - 3) * 2.0 ** -12), (float(BIG), c, (H - 1) * 2.0 ** -12)]


def test_logit_chain_order_with_unit_activations(net):
    z = np.zeros(4, np.float32)
    base = np.zeros(net.size, np.float32)
    base[4 * net.H:5 * net.H] = 30.0           # every hidden unit is tanhf(30) = 1.0f
    assert np.all(net.hidden(base, z) == np.float32(1.0))
    for k in range(2):
        for bias, row, value in _chain_probes(net.H):
            w = base.copy()
            w[net.w2(k)] = row
            w[net.b2(k)] = bias
            assert float(net.call(w, z)[k]) == value
    # signs: tanhf(-30) = -1.0f flips a term exactly
    w = base.copy()
    w[net.b1(3)] = -30.0
    w[net.w2(1)] = 0.0
    w[5 * net.H + net.H + 3] = 0.375
    w[net.b2(1)] = 0.125
    assert float(net.call(w, z)[1]) == 0.125 - 0.375


# ---------------------------------------------------------------- two hidden layers
# W1[16][4] (0), b1[16] (64), W2[16][16] (80), b2[16] (336), W3[2][16] (352), b3[2] (384)
def _deep_hidden2(oracle, w, z):
    """Second-layer activations of the deep network, bit-exact, through one-hot W3."""
    h2 = np.empty(16, np.float32)
    for k in range(16):
        probe = np.array(w, np.float32)
        probe[352:] = 0.0
        probe[352 + k] = 1.0
        h2[k] = oracle.mlp_deep_logits(probe, z)[0]
    return h2


def test_deep_network_chains_in_exact_rationals(oracle):
    w = inputs.policy_weights(inputs.POLICY_MLP_DEEP, 7)
    shallow = Shallow(oracle, 16, False)
    first = np.zeros(114, np.float32)
    first[:80] = w[:80]                        # same first layer in the one-hidden-layer routine
    zs = inputs.random_states(10, seed=9, spread="live")
    for i in range(zs.shape[1]):
        z = zs[:, i]
        h1 = shallow.hidden(first, z)          # bit-exact first-layer activations
        h2 = _deep_hidden2(oracle, w, z)
        for k in range(16):
            acc = fma_chain_exact(w[80 + 16 * k:96 + 16 * k], h1, w[336 + k])
            assert abs(float(h2[k]) - np.tanh(float(acc))) <= TOL_TANH
        got = oracle.mlp_deep_logits(w, z)
        for m in range(2):
            want = fma_chain_exact(w[352 + 16 * m:368 + 16 * m], h2, w[384 + m])
            assert got[m].view(np.uint32) == want.view(np.uint32)


def test_deep_first_layer_order(oracle):
    amp = np.float32(2.0 ** 20)
    for j in (0, 7, 15):
        for b, wrow, z, value, wrong in _first_layer_probes():
            w = np.zeros(386, np.float32)
            w[4 * j:4 * j + 4] = wrow
            w[64 + j] = b
            w[80 + 16 * j + j] = 1.0           # second-layer unit j sees h1_j alone
            w[352 + j] = amp
            got = float(oracle.mlp_deep_logits(w, z)[0]) / float(amp)
            want = np.tanh(np.tanh(value))
            assert abs(got - want) <= 3e-6 * want, (j, value, got)
            assert abs(want - np.tanh(np.tanh(wrong))) > 1e3 * 3e-6 * want


def test_deep_second_and_third_layer_order(oracle):
    z = np.zeros(4, np.float32)
    # second layer: h1 = 1.0f everywhere, chain probes on row k, read through one-hot W3
    for k in (0, 9, 15):
        for bias, row, value in _chain_probes(16):
            w = np.zeros(386, np.float32)
            w[64:80] = 30.0
            w[80 + 16 * k:96 + 16 * k] = row
            w[336 + k] = bias
            w[352 + 16 + k] = 1.0              # logit 1 = h2_k
            got = float(oracle.mlp_deep_logits(w, z)[1])
            assert abs(got - np.tanh(value)) <= TOL_TANH and np.tanh(value) > 1e-3
    # third layer: h2 = 1.0f everywhere (b2 = 30, W2 = 0), exact sums
    for m in range(2):
        for bias, row, value in _chain_probes(16):
            w = np.zeros(386, np.float32)
            w[336:352] = 30.0
            w[352 + 16 * m:368 + 16 * m] = row
            w[384 + m] = bias
            assert float(oracle.mlp_deep_logits(w, z)[m]) == value


def test_deep_second_layer_is_fused(oracle):
    # b2 = -RN(w * h1): a fused chain returns the product's rounding error (exactly representable),
    # separate rounding returns 0. h1 comes bit-exact from the one-hidden-layer routine.
    shallow = Shallow(oracle, 16, False)
    base = inputs.policy_weights(inputs.POLICY_MLP_DEEP, 7)
    z = inputs.random_states(1, seed=4, spread="live")[:, 0]
    first = np.zeros(114, np.float32)
    first[:80] = base[:80]
    h1 = shallow.hidden(first, z)
    amp = np.float32(2.0 ** 26)
    seen = 0
    for j, wv in ((0, 0.7371), (5, -1.2113), (11, 0.3337)):
        wv = np.float32(wv)
        prod = Fraction(float(wv)) * Fraction(float(h1[j]))
        rounded = round_f32(prod)
        resid = float(prod - Fraction(float(rounded)))
        if resid == 0.0:
            continue
        seen += 1
        w = np.zeros(386, np.float32)
        w[:80] = base[:80]
        w[80 + 16 * 2 + j] = wv                # unit 2 of the second layer
        w[336 + 2] = -rounded
        w[352 + 2] = amp
        got = float(oracle.mlp_deep_logits(w, z)[0])
        assert abs(got - resid * float(amp)) <= 1e-5 * abs(resid) * float(amp) and got != 0.0
    assert seen >= 2
