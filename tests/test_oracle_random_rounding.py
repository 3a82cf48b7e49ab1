"""Pins of the oracle's random rounding (rounding = 1): the Philox-4x32-10 generator against its published
known-answer vectors and against a second implementation with Python integers; the uniform draw; the
rounding rule against exact rational arithmetic; unbiasedness; reproducibility."""
import os
from fractions import Fraction

import numpy as np

from oracle import fho
from paper_2510_11400_b200 import synth

GOLD = os.path.join(os.path.dirname(__file__), "golden", "hand_cases.txt")


def philox_python(ctr, key):
    """Philox-4x32-10 from its published definition, with unbounded Python integers."""
    c, k = list(ctr), list(key)
    for _ in range(10):
        p0, p1 = 0xD2511F53 * c[0], 0xCD9E8D57 * c[2]
        c = [(p1 >> 32) ^ c[1] ^ k[0], p1 & 0xFFFFFFFF, (p0 >> 32) ^ c[3] ^ k[1], p0 & 0xFFFFFFFF]
        k = [(k[0] + 0x9E3779B9) & 0xFFFFFFFF, (k[1] + 0xBB67AE85) & 0xFFFFFFFF]
    return c


def test_philox_known_answer_vectors():
    seen = 0
    for line in open(GOLD):
        if not line.startswith("philox_"):
            continue
        _, ctr, key, out = [f.strip() for f in line.split("|")]
        ctr, key, out = ([int(w, 16) for w in f.split()] for f in (ctr, key, out))
        assert fho.philox4x32_10(ctr, key) == out
        assert philox_python(ctr, key) == out
        seen += 1
    assert seen == 3


def test_philox_agrees_with_the_integer_implementation_on_random_inputs():
    rng = np.random.default_rng(5)
    for _ in range(200):
        ctr = [int(v) for v in rng.integers(0, 2**32, 4)]
        key = [int(v) for v in rng.integers(0, 2**32, 2)]
        assert fho.philox4x32_10(ctr, key) == philox_python(ctr, key)


def test_rounding_rule_against_exact_arithmetic():
    """q = min(floor(t) + [floor(frac(t) * 2^24) + (word >> 8) >= 2^24], L) with t the fp32 product:
    recomputed with NumPy's fp32 product and exact rationals."""
    rng = np.random.default_rng(11)
    for bits in (2, 4, 8):
        L = (1 << bits) - 1
        lo, hi = np.float32(-1.25), np.float32(2.5)
        inv, _ = fho.quant_params(float(lo), float(hi), bits)
        for _ in range(500):
            x = np.float32(rng.uniform(float(lo), float(hi)))
            word = int(rng.integers(0, 2**32))
            t = Fraction(float(np.float32(x - lo) * np.float32(inv)))
            n = int(np.floor(float(t)))
            fi = int(np.floor(float((t - n) * 2**24)))
            want = min(n + (1 if fi + (word >> 8) >= 2**24 else 0), L)
            assert fho.quant_code_random(float(x), float(lo), inv, bits, word) == want
    # the probability of going up is floor(frac * 2^24) / 2^24: count over all 2^24 draws in closed form
    inv, _ = fho.quant_params(0.0, 3.0, 2)
    x = 1.3
    t = Fraction(float(np.float32(x) * np.float32(inv)))
    fi = int(np.floor(float((t - 1) * 2**24)))
    assert fho.quant_code_random(x, 0.0, inv, 2, ((2**24 - fi) << 8)) == 2       # smallest draw that goes up
    assert fho.quant_code_random(x, 0.0, inv, 2, ((2**24 - fi - 1) << 8) | 0xFF) == 1


def test_exact_positions_are_never_moved():
    """When (x - lo) * inv is an integer no draw changes the code."""
    for bits in (2, 4, 8):
        L = (1 << bits) - 1
        inv, scale = fho.quant_params(0.0, float(L), bits)
        assert inv == 1.0
        for q in range(L + 1):
            for w in (0, 0x7FFFFFFF, 0xFFFFFFFF):
                assert fho.quant_code_random(float(q), 0.0, inv, bits, w) == q


def test_restored_values_are_unbiased():
    """Mean over many seeds of the restored value equals the input to within sampling error."""
    shape = (1, 2, 8, 8)
    x = synth.normal(2 * 64, 9)
    d = fho.desc(shape, fho.F32, tensor_id=3)
    acc = np.zeros(x.size, dtype=np.float64)
    n = 400
    for seed in range(n):
        st, buf, _ = fho.compress(x, d, fho.params(bits=2, salient_mode=fho.OFF, rounding=1, seed=seed))
        assert st == fho.OK
        acc += fho.decompress(buf, d)[1]
    mean = acc / n
    scale = (x.reshape(2, 64).max(1) - x.reshape(2, 64).min(1)) / 3.0
    tol = np.repeat(scale, 64) * 0.5 / np.sqrt(n) * 5        # 5 sigma of a step-sized Bernoulli
    assert (np.abs(mean - x) <= tol + 1e-6).all()
    # round-to-nearest at 2 bits is visibly biased on the same data
    st, buf, _ = fho.compress(x, d, fho.params(bits=2, salient_mode=fho.OFF))
    assert (np.abs(fho.decompress(buf, d)[1] - x) > tol + 1e-6).any()


def test_reproducible_and_keyed_by_seed_tensor_and_position():
    shape = (2, 3, 8, 8)
    x = synth.normal(6 * 64, 4)
    base = fho.compress(x, fho.desc(shape, fho.F32, tensor_id=1), fho.params(bits=4, salient_mode=fho.OFF, rounding=1, seed=77))[1]
    again = fho.compress(x, fho.desc(shape, fho.F32, tensor_id=1), fho.params(bits=4, salient_mode=fho.OFF, rounding=1, seed=77))[1]
    assert np.array_equal(base, again)
    assert fho.parse_header(base)["rounding"] == 1
    other_seed = fho.compress(x, fho.desc(shape, fho.F32, tensor_id=1), fho.params(bits=4, salient_mode=fho.OFF, rounding=1, seed=78))[1]
    other_id = fho.compress(x, fho.desc(shape, fho.F32, tensor_id=2), fho.params(bits=4, salient_mode=fho.OFF, rounding=1, seed=77))[1]
    slots = 64 + 16 * 6
    assert not np.array_equal(base[slots:], other_seed[slots:]) and not np.array_equal(base[slots:], other_id[slots:])
    # the same plane content at another plane index draws other numbers
    y = np.concatenate([x[:64], x[:64]])
    two = fho.compress(y, fho.desc((1, 2, 8, 8), fho.F32), fho.params(bits=4, salient_mode=fho.OFF, rounding=1, seed=1))[1]
    s2 = 64 + 16 * 2
    assert not np.array_equal(two[s2:s2 + 32], two[s2 + 32:s2 + 64])
