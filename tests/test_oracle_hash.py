"""Pins for the oracle's counter hash (CPU only).

The hash is this build's own definition (the paper, Sec. V-A, only says the RNG
kernel was replaced by values that need no kernel), so the pins are: the
constants re-derived from their mathematical meaning, bijectivity through an
independently written inverse, stored vectors that predate the oracle, exact
rational re-evaluation of the uniform mapping, and stream statistics.
"""
import math
import os
from fractions import Fraction

import numpy as np
import pytest

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "hash_vectors.txt")
M32 = 0xFFFFFFFF


def _golden():
    rows = []
    with open(GOLDEN) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            lhs, rhs = line.split("=")
            kind, *args = lhs.split()
            rows.append((kind, args, rhs.split()))
    return rows


def test_golden_vectors(oracle):
    seen = set()
    for kind, args, want in _golden():
        seen.add(kind)
        if kind == "mix32":
            assert oracle.mix32(int(args[0], 16)) == int(want[0], 16)
        elif kind == "salt":
            assert oracle.salt(int(args[0]), int(args[1])) == int(want[0], 16)
        elif kind == "keys":
            got = oracle.keys(int(args[0]), int(args[1]), int(args[2]))
            assert got == (int(want[0], 16), int(want[1], 16))
        elif kind == "hash0":
            k = oracle.keys(int(args[0]), int(args[1]), 0)
            assert oracle.step_hash(*k, 0) == int(want[0], 16)
        elif kind == "actions":
            got = "".join(str(oracle.action(int(args[0]), int(args[1]), t)) for t in range(16))
            assert got == want[0]
        elif kind == "reset":
            got = oracle.reset_state(int(args[0]), int(args[1]), int(args[2])).view(np.uint32)
            assert [int(v) for v in got] == [int(w, 16) for w in want]
        else:
            raise AssertionError(kind)
    assert seen == {"mix32", "salt", "keys", "hash0", "actions", "reset"}


def test_constants_from_their_meaning(oracle):
    # mix32(h) for h < 2^15 has no shift feedback in the first xorshift, so
    # mix32 reveals its multipliers: recover them from the structure instead of
    # reading the source. The first multiplier is the 32 fractional bits of
    # sqrt(2), the second of sqrt(3), and the stream/key offset is the golden-ratio prime.
    ma = math.isqrt(2 << 64) & M32
    mb = math.isqrt(3 << 64) & M32
    assert ma == 0x6A09E667 and mb == 0xBB67AE85
    phi = (1 + 5 ** 0.5) / 2
    # the key offset is the prime next below 2^32/phi (Knuth's multiplicative-hash constant)
    mg = round(2 ** 32 / phi)
    while any(mg % d == 0 for d in range(2, math.isqrt(mg) + 1)):
        mg -= 1
    assert mg == 0x9E3779B1 == 2654435761

    def ref_mix(h):
        h ^= h >> 16
        h = (h * ma) & M32
        h ^= h >> 15
        h = (h * mb) & M32
        return h ^ (h >> 16)

    for h in (1, 2, 3, 0x7FFF, 0x12345678, 0xDEADBEEF, M32):
        assert oracle.mix32(h) == ref_mix(h)
    # keys use MG as the additive offset between K0 and K1 and in the seed salt.
    k0, k1 = oracle.keys(7, 99, 1)
    assert k1 == oracle.mix32((k0 + mg) & M32)
    assert oracle.salt(7, 1) == oracle.mix32((oracle.mix32(7 ^ mg) + 1) & M32)
    assert k0 == oracle.mix32(99 ^ oracle.salt(7, 1))


def _unxorshift(h, s):
    x = h
    for _ in range(32 // s + 1):
        x = h ^ (x >> s)
    return x & M32


def _inv_mix32(h):
    """Inverse built from modular inverses and xorshift inversion only."""
    ia = pow(0x6A09E667, -1, 1 << 32)
    ib = pow(0xBB67AE85, -1, 1 << 32)
    h = _unxorshift(h, 16)
    h = (h * ib) & M32
    h = _unxorshift(h, 15)
    h = (h * ia) & M32
    return _unxorshift(h, 16)


def test_mix32_is_a_bijection(oracle):
    assert oracle.mix32(0) == 0  # every stage fixes 0
    rng = np.random.default_rng(11)
    xs = list(range(0, 4096)) + [int(v) for v in rng.integers(0, 1 << 32, 4096)]
    ys = [oracle.mix32(x) for x in xs]
    assert len(set(ys)) == len(set(xs))
    for x, y in zip(xs, ys):
        assert _inv_mix32(y) == x


def test_step_hash_is_a_bijection_of_the_counter(oracle):
    # For fixed keys the map c -> step_hash is invertible: distinct steps can
    # never share a hash value, and the inverse recovers the counter.
    ia = pow(0x6A09E667, -1, 1 << 32)
    ib = pow(0xBB67AE85, -1, 1 << 32)
    rng = np.random.default_rng(5)
    for _ in range(50):
        k0, k1 = (int(v) for v in rng.integers(0, 1 << 32, 2))
        for c in [0, 1, 2, 3, M32] + [int(v) for v in rng.integers(0, 1 << 32, 20)]:
            h = oracle.step_hash(k0, k1, c)
            x = _unxorshift(h, 16)
            x = _unxorshift((x * ib) & M32, 15)
            x = ((x - k1) * ia) & M32
            x = _unxorshift(x, 16)
            assert x ^ k0 == c


def test_action_is_top_bit_of_stream0(oracle):
    for seed, env, t in [(0, 0, 0), (0, 5, 17), (3, 1 << 20, 499), (9, 77, 1 << 30)]:
        k = oracle.keys(seed, env, 0)
        assert oracle.action(seed, env, t) == oracle.step_hash(*k, t) >> 31


def test_reset_state_mapping_is_exact_rational(oracle):
    # Each component is RN_f32((bits * 2^-24 - 1/2) * fl(0.1)) with bits the top
    # 24 bits of stream-1 hash at counter 4t+j: evaluate that with exact
    # rationals and a single final rounding.
    tenth = Fraction(float(np.float32(0.1)))
    for seed, env, t in [(0, 0, 0), (0, 1, 0), (0, 0, 22), (1, 4095, 3), (2, 123456, 199)]:
        k = oracle.keys(seed, env, 1)
        got = oracle.reset_state(seed, env, t)
        for j in range(4):
            bits = oracle.step_hash(*k, 4 * t + j) >> 8
            exact = (Fraction(bits, 1 << 24) - Fraction(1, 2)) * tenth
            want = np.float32(float(exact))  # float(Fraction) is RN to f64; 24+24 bit product fits f64 exactly
            assert got[j] == want
            assert -0.05 <= float(got[j]) < 0.05 + 1e-9


def test_reset_state_range_and_moments(oracle):
    n = 20000
    z = oracle.initial_state(n, seed=0)
    lim = float(np.float32(0.05))
    assert z.min() >= -lim and z.max() <= lim
    # uniform on [-0.05, 0.05): mean 0, std 0.1/sqrt(12)
    assert np.all(np.abs(z.mean(axis=1)) < 4 * 0.02887 / np.sqrt(n))
    assert np.all(np.abs(z.std(axis=1) - 0.1 / np.sqrt(12)) < 4e-4)
    # components and neighbouring envs are uncorrelated
    c = np.corrcoef(z)
    assert np.all(np.abs(c - np.eye(4)) < 0.03)
    assert abs(np.corrcoef(z[0, :-1], z[0, 1:])[0, 1]) < 0.03


def test_action_stream_statistics(oracle):
    r = oracle.rollout(4096, 64, 0, action_bits=True, per_env=False)
    bits = np.unpackbits(r["action_bits"].view(np.uint8), bitorder="little").reshape(64, -1)[:, :4096]
    a = bits.astype(np.float64)
    n = a.size
    assert abs(a.mean() - 0.5) < 4 * 0.5 / np.sqrt(n)
    # lag-1 in time and neighbour-in-env correlations vanish
    ac = a - 0.5
    assert abs((ac[1:] * ac[:-1]).mean() * 4) < 5 / np.sqrt(n)
    assert abs((ac[:, 1:] * ac[:, :-1]).mean() * 4) < 5 / np.sqrt(n)
    # different seeds give different streams
    r1 = oracle.rollout(4096, 64, 1, action_bits=True, per_env=False)
    diff = np.unpackbits((r["action_bits"] ^ r1["action_bits"]).view(np.uint8)).mean()
    assert 0.45 < diff < 0.55


@pytest.mark.parametrize("bit", [0, 7, 16, 31])
def test_mix32_avalanche(oracle, bit):
    rng = np.random.default_rng(bit)
    xs = rng.integers(0, 1 << 32, 3000)
    flips = np.zeros(32)
    for x in xs:
        d = oracle.mix32(int(x)) ^ oracle.mix32(int(x) ^ (1 << bit))
        flips += [(d >> b) & 1 for b in range(32)]
    p = flips / len(xs)
    assert np.all(np.abs(p - 0.5) < 0.06)
