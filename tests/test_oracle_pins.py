"""Pins for the CPU oracle: hand cases, closed forms, invariants, library routines and brute force.

Nothing here touches the CUDA path.  Each test states which passage of the paper (arXiv
2510.11400, Section 4.4.1, Eq. 7-9) or which piece of mathematics fixes the expected value.
"""
import os

import numpy as np
import pytest
import scipy.sparse as sp

from oracle import fho
from paper_2510_11400_b200 import synth
from tests import helpers as hp

GOLD = os.path.join(os.path.dirname(__file__), "golden", "hand_cases.txt")


def enc(x, shape, dtype=fho.F32, **kw):
    d = fho.desc(shape, dtype)
    p = fho.params(**kw)
    st, buf, total = fho.compress(x, d, p)
    assert st == fho.OK
    assert total == buf.size
    return d, p, buf


def dec(buf, d):
    st, out = fho.decompress(buf, d)
    assert st == fho.OK
    return out


def golden():
    out = {}
    for line in open(GOLD):
        if line.startswith("#") or "|" not in line:
            continue
        parts = [s.strip() for s in line.split("|")]
        out[parts[0]] = parts[1:]
    return out


# ------------------------------------------------------------------------------------------------
# Quantiser (normal planes)
# ------------------------------------------------------------------------------------------------

@pytest.mark.parametrize("name,vals", [("quant_identity", [0, 1, 2, 3]), ("quant_ties", [0, 0.5, 1.5, 3]),
                                       ("quant_skewed", [0, 0, 0, 9])])
def test_quant_hand_cases(name, vals):
    exp = golden()[name][1].split()
    codes = [int(v) for v in exp[1:5]]
    word = int(exp[6], 16)
    x = np.array(vals, dtype=np.float32)
    d, p, buf = enc(x, (1, 1, 2, 2), bits=2, salient_mode=fho.OFF)
    t = hp.table(buf, 1)
    assert list(hp.normal_codes(buf, int(t["off"][0]), 4, 2)) == codes
    assert int(buf[int(t["off"][0]):int(t["off"][0]) + 4].view(np.uint32)[0]) == word
    if "scale" in exp:
        assert t["scale"][0] == np.float32(float(exp[exp.index("scale") + 1]))
    assert t["lo"][0] == 0.0


@pytest.mark.parametrize("bits", [2, 4, 8])
def test_packing_is_little_endian_bitstream(bits):
    """Brute force: the payload equals the big integer sum(q_i << (i*b)) written little-endian."""
    rng = np.random.default_rng(7)
    hw = 5 * 7
    x = rng.standard_normal(hw).astype(np.float32)
    d, p, buf = enc(x, (1, 1, 5, 7), bits=bits, salient_mode=fho.OFF)
    t = hp.table(buf, 1)
    off = int(t["off"][0])
    inv, scale = fho.quant_params(float(x.min()), float(x.max()), bits)
    q = [fho.quant_code(float(v), float(x.min()), inv, bits) for v in x]
    big = 0
    for i, qi in enumerate(q):
        big |= qi << (i * bits)
    nbytes = 4 * ((hw * bits + 31) // 32)
    assert bytes(buf[off:off + nbytes]) == big.to_bytes(nbytes, "little")
    # padding to 16 bytes is zero, and the container ends there
    assert buf.size == off + hp.a16(nbytes)
    assert not buf[off + nbytes:].any()


@pytest.mark.parametrize("bits", [2, 4, 8])
def test_quant_codes_against_exact_rational_rounding(bits):
    """q must be the round-half-even of the exact product (x-lo)*inv; checked with Fractions."""
    from fractions import Fraction
    rng = np.random.default_rng(11)
    x = (rng.standard_normal(257) * 3).astype(np.float32)
    lo, hi = float(x.min()), float(x.max())
    inv, _ = fho.quant_params(lo, hi, bits)
    L = (1 << bits) - 1
    for v in x:
        dlt = np.float32(v) - np.float32(lo)
        t = Fraction(float(dlt)) * Fraction(float(inv))
        fl = t.numerator // t.denominator
        rem = t - fl
        r = fl + (1 if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and fl % 2 == 1) else 0)
        assert fho.quant_code(float(v), lo, inv, bits) == min(max(r, 0), L)


@pytest.mark.parametrize("bits,hi_hex,x_hex,want", [
    (2, "0x1.15aca4p+2", "0x1.ceca68p+1", 3), (2, "0x1.e75a0cp+2", "0x1.44e6b4p+0", 1),
    (4, "0x1.d664b6p+1", "0x1.1a3c6ep+0", 5), (4, "0x1.224f0cp+2", "0x1.bd23dep+1", 11),
    (8, "0x1.c2fd0cp+1", "0x1.e820f2p-2", 35), (8, "0x1.49d0c8p+1", "0x1.dfd96ap+0", 185)])
def test_quant_product_is_not_rounded_before_the_integer_rounding(bits, hi_hex, x_hex, want):
    """Inputs where rounding (x-lo)*inv to fp32 first would land on a tie and give another code.
    The expected code is recomputed here with exact rational arithmetic."""
    from fractions import Fraction
    hi, xv = float.fromhex(hi_hex), float.fromhex(x_hex)
    L = (1 << bits) - 1
    inv = np.float32(L) / np.float32(hi)
    t = Fraction(xv) * Fraction(float(inv))
    fl = t.numerator // t.denominator
    rem = t - fl
    exact = fl + (1 if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and fl % 2 == 1) else 0)
    assert exact == want
    x = np.array([0.0, xv, hi, 0.0], dtype=np.float32)
    d, p, buf = enc(x, (1, 1, 2, 2), bits=bits, salient_mode=fho.OFF)
    q = hp.normal_codes(buf, int(hp.table(buf, 1)["off"][0]), 4, bits)
    assert list(q) == [0, want, L, 0]


@pytest.mark.parametrize("bits", [2, 4, 8])
@pytest.mark.parametrize("kind", ["relu", "normal"])
def test_quant_error_bound_and_endpoints(bits, kind):
    """Uniform quantisation: |x - xhat| <= scale/2 (+ rounding of the fp32 ops) <= range/(2^b-1);
    the minimum maps to code 0 and the maximum to code 2^b-1."""
    shape = (2, 3, 9, 13)
    hw = 9 * 13
    x = synth.relu_normal(2 * 3 * hw, 5) if kind == "relu" else synth.normal(2 * 3 * hw, 5)
    d, p, buf = enc(x, shape, bits=bits, salient_mode=fho.OFF)
    xh = dec(buf, d)
    t = hp.table(buf, 6)
    L = (1 << bits) - 1
    for pl in range(6):
        xs, xr = x[pl * hw:(pl + 1) * hw], xh[pl * hw:(pl + 1) * hw]
        lo, hi = xs.min(), xs.max()
        rng_ = np.float64(hi) - np.float64(lo)
        assert t["lo"][pl] == lo
        assert abs(np.float64(t["scale"][pl]) - rng_ / L) <= 1e-6 * rng_
        q = hp.normal_codes(buf, int(t["off"][pl]), hw, bits)
        assert q[np.argmin(xs)] == 0 and q[np.argmax(xs)] == L
        err = np.abs(xs.astype(np.float64) - xr.astype(np.float64))
        ulp = np.spacing(np.float32(max(abs(lo), abs(hi))))
        assert err.max() <= np.float64(t["scale"][pl]) / 2 + 2 * ulp
        assert err.max() <= rng_ / L
        if kind == "relu":  # lo == 0: every zero is reproduced exactly
            assert lo == 0 and np.all(xr[xs == 0] == 0)


def test_quant_constant_plane_exact_and_8bit_lossless_on_bytes():
    x = np.full(50, 3.25, dtype=np.float32)
    d, p, buf = enc(x, (1, 2, 5, 5), bits=4, salient_mode=fho.OFF)
    t = hp.table(buf, 2)
    assert np.all(t["scale"] == 0) and np.all(t["lo"] == np.float32(3.25))
    assert np.array_equal(dec(buf, d), x)
    # integers 0..255 at 8 bits: scale = 1, codes = values
    y = np.random.default_rng(3).permutation(256).astype(np.float32)
    d, p, buf = enc(y, (1, 1, 16, 16), bits=8, salient_mode=fho.OFF)
    assert np.array_equal(hp.normal_codes(buf, int(hp.table(buf, 1)["off"][0]), 256, 8), y.astype(np.int64))
    assert np.array_equal(dec(buf, d), y)


@pytest.mark.parametrize("bits", [2, 4, 8])
def test_reencoding_decoded_plane_is_idempotent(bits):
    x = synth.normal(4 * 64, 9)
    d, p, buf = enc(x, (1, 4, 8, 8), bits=bits, salient_mode=fho.OFF)
    xh = dec(buf, d)
    d2, p2, buf2 = enc(xh, (1, 4, 8, 8), bits=bits, salient_mode=fho.OFF)
    for pl in range(4):
        o1, o2 = int(hp.table(buf, 4)["off"][pl]), int(hp.table(buf2, 4)["off"][pl])
        assert np.array_equal(hp.normal_codes(buf, o1, 64, bits), hp.normal_codes(buf2, o2, 64, bits))
    assert np.array_equal(dec(buf2, d2), xh)


def test_quant_decode_is_single_fma():
    """xhat = fma(q, scale, lo): compare with exact rational arithmetic rounded once to fp32."""
    from fractions import Fraction
    rng = np.random.default_rng(1)
    for _ in range(200):
        q = int(rng.integers(0, 256))
        scale = float(np.float32(rng.standard_normal() * 0.01))
        lo = float(np.float32(rng.standard_normal()))
        exact = Fraction(q) * Fraction(scale) + Fraction(lo)
        got = fho.dequant(q, lo, scale)
        # nearest fp32 to the exact value
        cand = np.float32(float(exact))
        assert got == cand


def test_bf16_input_is_widened_exactly_and_output_rounded_half_even():
    x32 = synth.normal(3 * 35, 21)
    xb = synth.to_bf16_bits(x32)
    xw = synth.bf16_bits_to_f32(xb)
    d16, p, b16 = enc(xb, (1, 3, 5, 7), dtype=fho.BF16, bits=8, salient_mode=fho.OFF)
    d32, _, b32 = enc(xw, (1, 3, 5, 7), dtype=fho.F32, bits=8, salient_mode=fho.OFF)
    # same codes and table as the exactly widened fp32 tensor
    assert np.array_equal(b16[64:], b32[64:])
    out16 = dec(b16, d16)
    out32 = dec(b32, d32)
    assert np.array_equal(out16, synth.to_bf16_bits(out32))


# ------------------------------------------------------------------------------------------------
# Sizes and container
# ------------------------------------------------------------------------------------------------

def test_size_closed_forms():
    exp = int(golden()["size_config1"][1])
    d = fho.desc((32, 16, 32, 32))
    assert fho.compressed_bytes(d, fho.params(bits=2), 0) == exp == 139328
    assert fho.compressed_bytes(d, fho.params(bits=2), 1) == 64 + 512 * (16 + 4096)
    # odd plane: HW = 49, b = 2 -> 98 bits -> 4 words = 16 bytes
    d = fho.desc((2, 3, 7, 7), fho.BF16)
    assert fho.compressed_bytes(d, fho.params(bits=2), 0) == 64 + 6 * (16 + 16)
    assert fho.compressed_bytes(d, fho.params(bits=8), 0) == 64 + 6 * (16 + 64)   # 52 -> 64
    assert fho.compressed_bytes(d, fho.params(bits=2), 1) == 64 + 6 * (16 + 112)  # 98 -> 112


def test_config1_size_and_header():
    spec = synth.config1()[0]
    x = synth.make(spec)
    d, p, buf = enc(x, spec.shape, bits=2)
    h = fho.parse_header(buf)
    P = 512
    t = hp.table(buf, P)
    # total = 64 + 16P + sum of padded payloads, offsets are the running sum
    sizes = np.where(t["cls"] == fho.NORMAL, 256, 0)
    assert h["total_bytes"] == buf.size
    assert h["magic"] == int.from_bytes(b"FHC1", "little") and h["version"] == 1
    assert (h["n"], h["c"], h["h"], h["w"]) == spec.shape
    if h["n_salient"] == 0 and h["n_raw"] == 0:
        assert buf.size == 139328
        assert np.array_equal(t["off"], 64 + 16 * P + np.arange(P) * 256)
    assert h["n_salient"] == int((t["cls"] == fho.SALIENT).sum())
    assert h["n_raw"] == int((t["cls"] == fho.RAW).sum())
    assert sizes.sum() > 0


def test_slots_and_overflow_offsets_mixed_classes():
    """Every plane owns a slot at a closed-form offset; payloads longer than the slot continue in the
    overflow region in plane order, each continuation padded to 16 bytes; total = fixed part + sum."""
    spec = synth.TensorSpec("s", (2, 32, 24, 40), synth.F32, "spiky_relu", 77)
    x = synth.make(spec)
    d, p, buf = enc(x, spec.shape, bits=4)
    P, H, W = 64, 24, 40
    npay = hp.a16(4 * ((H * W * 4 + 31) // 32))
    assert npay == hp.npay_of(buf, H * W)
    t = hp.table(buf, P)
    assert (t["cls"] == fho.SALIENT).sum() >= 4 and (t["cls"] == fho.NORMAL).sum() >= 32
    slots = 64 + 16 * P
    ovf = slots + P * npay
    for pl in range(P):
        if t["cls"][pl] == fho.NORMAL:
            assert t["off"][pl] == slots + pl * npay
            continue
        if t["cls"][pl] == fho.RAW:
            sz = 4 * H * W
        else:
            s = hp.salient_plane(buf, P, pl, H, W, 4)
            sz = s["size"]
            assert s["pad"] == 0
            assert sz == 16 + 4 * ((15 + 31) // 32) + 4 * (H + 1) + hp.a4(2 * s["nnz_s"]) + 4 * s["nnz_s"] \
                + 64 * s["n_dense"] + 4 * s["n_out_d"]
        if sz <= npay:
            assert t["off"][pl] == 0
            assert not buf[slots + pl * npay + sz: slots + (pl + 1) * npay].any()
        else:
            assert t["off"][pl] == ovf
            assert not buf[ovf + sz - npay: ovf + hp.a16(sz) - npay].any()
            ovf += hp.a16(sz) - npay
    assert ovf == buf.size == fho.parse_header(buf)["total_bytes"]


def test_short_salient_payload_stays_inside_its_slot():
    """A salient plane whose payload is no longer than a slot has no continuation (offset 0)."""
    x = np.zeros(32 * 32, dtype=np.float32)
    x[5] = 3.0
    d, p, buf = enc(x, (1, 1, 32, 32), bits=8, salient_mode=fho.ALL)   # slot = 1024 bytes
    t = hp.table(buf, 1)
    s = hp.salient_plane(buf, 1, 0, 32, 32, 4)
    assert t["cls"][0] == fho.SALIENT and t["off"][0] == 0 and s["size"] <= 1024
    assert buf.size == 64 + 16 + 1024
    assert np.array_equal(dec(buf, d), x)


# ------------------------------------------------------------------------------------------------
# Three-sigma rule and plane classification
# ------------------------------------------------------------------------------------------------

def test_sigma_hand_case_spike():
    exp = golden()["sigma_spike"][1].split()
    x = np.zeros(16, dtype=np.float32)
    x[5] = 16
    lo, dlo, dhi, n = fho.plane_sigma(x)
    Is, Iq, e, applies = fho.plane_sums(x)
    assert (lo, e, applies) == (0.0, 4, 1)
    assert (Is * 2.0 ** (e - 18), Iq * 2.0 ** (2 * e - 16)) == (16.0, 256.0)     # sum d, sum d^2
    assert n == int(exp[1])
    assert abs(lo + dhi - float(exp[5])) < 1e-5 and abs(lo + dlo - float(exp[7])) < 1e-5
    d, p, buf = enc(x, (1, 1, 4, 4), bits=2, eps=0.0625)
    t = hp.table(buf, 1)
    assert t["n_out"][0] == 1
    assert t["cls"][0] in (fho.SALIENT, fho.RAW)  # outlier-rich; RAW only because a 4x4 plane cannot gain


def _numpy_three_sigma(xs):
    """The rule in float64: thresholds, outlier count, and the distance of the closest element to a threshold."""
    x64 = xs.astype(np.float64)
    mu, sd = x64.mean(), x64.std()
    thi, tlo = mu + 3 * sd, mu - 3 * sd
    margin = np.minimum(np.abs(x64 - thi), np.abs(x64 - tlo)).min()
    return mu, sd, tlo, thi, int(((x64 > thi) | (x64 < tlo)).sum()), margin


@pytest.mark.parametrize("kind,seed", [("normal", 1), ("relu", 2), ("laplace", 3)])
def test_sigma_count_matches_numpy_float64(kind, seed):
    """mu, sigma are the plain mean and population standard deviation: NumPy float64 agrees on the
    thresholds to 1e-5 of the range and on the outlier count whenever no element sits that close to a
    threshold.  (The integer sums resolve 2^-18 of the range per group of four.)"""
    hw = 56 * 56
    x = {"normal": synth.normal, "relu": synth.relu_normal, "laplace": synth.laplace}[kind](8 * hw, seed)
    for pl in range(8):
        xs = x[pl * hw:(pl + 1) * hw]
        lo, dlo, dhi, n = fho.plane_sigma(xs)
        mu, sd, tlo, thi, want, margin = _numpy_three_sigma(xs)
        rng_ = float(xs.max()) - float(xs.min())
        assert abs(float(lo) + dhi - thi) <= 1e-5 * rng_ and abs(float(lo) + dlo - tlo) <= 1e-5 * rng_
        if margin > 2e-5 * rng_:
            assert n == want
        assert n <= hw / 9  # Chebyshev: P(|x-mu| > 3 sigma) <= 1/9


@pytest.mark.parametrize("offset,sigma", [(1000.0, 0.01), (-37.0, 1.0), (3.0e4, 0.5), (-1.0e6, 2.0), (255.0, 1e-3)])
@pytest.mark.parametrize("kind", ["normal", "relu", "spiky"])
def test_sigma_rule_on_planes_with_an_offset(offset, sigma, kind):
    """|mu| up to 10^5..10^6 sigma (a biased pre-activation, a plane far from zero): the rule has the same plain
    answer as for centred data, because the moments are taken of the distances from the plane's minimum.
    One-pass raw moments E[x^2] - mu^2 would be rounding noise here."""
    rng = np.random.default_rng(int(abs(offset)) + len(kind))
    hw = 28 * 28
    for _ in range(6):
        z = rng.standard_normal(hw)
        if kind == "relu":
            z = np.maximum(z, 0.0)
        elif kind == "spiky":                       # 6 % far outliers: the plane must come out outlier-rich
            z = np.where(rng.random(hw) < 0.06, 12.0 + np.abs(z), np.maximum(z, 0.0) * 0.2)
        xs = (offset + sigma * z).astype(np.float32)
        lo, dlo, dhi, n = fho.plane_sigma(xs)
        mu, sd, tlo, thi, want, margin = _numpy_three_sigma(xs)
        rng_ = float(xs.max()) - float(xs.min())
        assert abs(float(lo) + dhi - thi) <= 1e-5 * rng_ and abs(float(lo) + dlo - tlo) <= 1e-5 * rng_
        if margin > 2e-5 * rng_:
            assert n == want
        if kind == "spiky":
            assert n * 32 > hw
        else:
            assert n * 32 <= hw
    # the container carries the same count and class
    d, p, buf = enc(xs, (1, 1, 28, 28), bits=4)
    t = hp.table(buf, 1)
    assert t["n_out"][0] == n and (t["cls"][0] != fho.NORMAL) == (n * 32 > hw)


def test_sigma_rule_on_bf16_planes_with_an_offset():
    """bf16 activations around 100 with a spread of a few units (8 mantissa bits: steps of 0.5): widened exactly,
    then the same rule."""
    rng = np.random.default_rng(5)
    hw = 32 * 32
    xs = synth.bf16_bits_to_f32(synth.to_bf16_bits((100.0 + 3.0 * rng.standard_normal(hw)).astype(np.float32)))
    lo, dlo, dhi, n = fho.plane_sigma(xs)
    mu, sd, tlo, thi, want, margin = _numpy_three_sigma(xs)
    assert abs(float(lo) + dhi - thi) <= 1e-4 and abs(float(lo) + dlo - tlo) <= 1e-4
    assert margin > 1e-3 and n == want
    d, p, buf = enc(synth.to_bf16_bits(xs), (1, 1, 32, 32), dtype=fho.BF16, bits=2)
    assert hp.table(buf, 1)["n_out"][0] == n


@pytest.mark.parametrize("scale,offset", [(1.0, 0.0), (1e-3, 0.0), (3e4, 7e5), (2.0 ** -38, 0.0), (2.0 ** 55, 0.0), (0.25, -1e3)])
def test_fixed_point_sums_are_exact_integers_of_the_stated_roundings(scale, offset):
    """I_s and I_q are sums of round-half-even(s_g * 2^(18-e)) and (q_g * 2^(16-2e)) over the distances from
    the minimum: recomputed here with exact rational arithmetic from fp32 group values, for planes of very
    different magnitude and offset, and shown to be independent of the order of the groups."""
    from fractions import Fraction
    rng = np.random.default_rng(17)
    x = (offset + rng.standard_normal(203) * scale).astype(np.float32)   # 203: ragged last group
    Is, Iq, e, applies = fho.plane_sums(x)
    lo = x.min()
    span = float(np.float32(x.max() - lo))
    assert applies == 1 and e == int(np.floor(np.log2(span)))

    def rne(t):
        fl = t.numerator // t.denominator
        rem = t - fl
        return fl + (1 if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and fl % 2 == 1) else 0)
    dd = (x - lo).astype(np.float32)                                     # fp32 subtraction, element by element
    assert (dd >= 0).all()
    dp = np.concatenate([dd, np.zeros(1, np.float32)]).reshape(-1, 4)
    es = eq = 0
    for v in dp:
        sg = np.float32(np.float32(v[0] + v[2]) + np.float32(v[1] + v[3]))
        f = [Fraction(float(t)) for t in v]
        q02 = np.float32(float(f[2] * f[2] + Fraction(float(np.float32(v[0] * v[0])))))   # fma: one rounding
        q13 = np.float32(float(f[3] * f[3] + Fraction(float(np.float32(v[1] * v[1])))))
        qg = np.float32(q02 + q13)
        es += rne(Fraction(float(sg)) * Fraction(2) ** (18 - e))
        eq += rne(Fraction(float(qg)) * Fraction(2) ** (16 - 2 * e))
    assert (Is, Iq) == (es, eq)
    # a permutation of whole groups leaves the integers unchanged
    xp = np.concatenate([x, np.full(1, lo, np.float32)]).reshape(-1, 4)
    perm = rng.permutation(xp.shape[0])
    Is2, Iq2, _, _ = fho.plane_sums(xp[perm].reshape(-1))
    assert (Is2, Iq2) == (Is, Iq)
    # and the sums are close to the real ones
    d64 = x.astype(np.float64) - float(lo)
    assert abs(Is * 2.0 ** (e - 18) - d64.sum()) <= 51 * span * 2.0 ** -18
    assert abs(Iq * 2.0 ** (2 * e - 16) - (d64 ** 2).sum()) <= 51 * span * span * 2.0 ** -15


def test_sigma_tail_group_padding_constant_plane_and_domain():
    # HW not a multiple of 4: the padded group members add nothing, and the divisor is HW
    x = np.array([1, 2, 3, 4, 5, 6, 7], dtype=np.float32)
    lo, dlo, dhi, n = fho.plane_sigma(x)
    Is, Iq, e, applies = fho.plane_sums(x)
    assert (Is * 2.0 ** (e - 18), Iq * 2.0 ** (2 * e - 16)) == (21.0, 91.0)          # distances 0..6
    mu, sd = 4.0, 2.0
    assert lo == 1.0 and lo + dhi == np.float32(mu + 3 * sd) and lo + dlo == np.float32(mu - 3 * sd) and n == 0
    # constant plane: no spread, no outliers
    lo, dlo, dhi, n = fho.plane_sigma(np.full(10, -2.5, dtype=np.float32))
    assert (lo, n) == (-2.5, 0) and fho.plane_sums(np.full(10, -2.5, dtype=np.float32))[3] == 0
    # the rule is applied for ranges in [2^-40, 2^61) and for no other
    spike = np.zeros(64, dtype=np.float32)
    spike[:3] = 1.0                                  # 3 of 64 elements far out: outlier-rich wherever the rule applies
    for k, want in ((-41, 0), (-40, 1), (0, 1), (60, 1), (61, 0)):
        xs = spike * np.float32(2.0 ** k)
        assert fho.plane_sums(xs)[3] == want
        assert fho.plane_sigma(xs)[3] == (3 if want else 0)
        d, p, buf = enc(xs, (1, 1, 8, 8), bits=2)
        assert (hp.table(buf, 1)["cls"][0] != fho.NORMAL) == bool(want)


def test_classification_threshold_is_strict_fraction():
    """outlier-rich iff n_out/HW > rho (strict): HW = 64, two symmetric spikes -> n_out = 2 = HW/32."""
    x = np.zeros(64, dtype=np.float32)
    x[3], x[40] = 100, -100
    d, p, buf = enc(x, (1, 1, 8, 8), bits=2)
    t = hp.table(buf, 1)
    assert t["n_out"][0] == 2 and t["cls"][0] == fho.NORMAL     # 2*32 > 64 is false
    d, p, buf = enc(x, (1, 1, 8, 8), bits=2, rho=(1, 33))
    assert hp.table(buf, 1)["cls"][0] != fho.NORMAL               # 2*33 > 64
    # mode switches override the rule and record no count
    d, p, buf = enc(x, (1, 1, 8, 8), bits=2, salient_mode=fho.OFF, rho=(1, 33))
    t = hp.table(buf, 1)
    assert t["cls"][0] == fho.NORMAL and t["n_out"][0] == 0


def test_laplace_channel_outliers_classify_by_channel():
    spec = synth.TensorSpec("l", (2, 16, 28, 28), synth.BF16, "laplace_ch", 301)
    x = synth.make(spec)
    d, p, buf = enc(x, spec.shape, dtype=fho.BF16, bits=4)
    t = hp.table(buf, 32)
    ch = np.arange(32) % 16
    assert np.all(t["cls"][ch % 8 == 0] != fho.NORMAL)
    assert np.all(t["cls"][ch % 8 != 0] == fho.NORMAL)


# ------------------------------------------------------------------------------------------------
# Block-wise path: mask, pooling, CSR, Lorenzo
# ------------------------------------------------------------------------------------------------

def spiky_plane(H, W, seed):
    spec = synth.TensorSpec("p", (1, 1, H, W), synth.F32, "spiky_relu", seed)
    return synth.make(spec)


@pytest.mark.parametrize("H,W", [(24, 40), (21, 30), (8, 8), (9, 70)])
def test_block_classes_equal_average_pooled_mask(H, W):
    """Average pooling of the non-zero mask with an 8x8 window and zero padding, compared with
    tau = 1/4 (Section 4.4.1), computed with torch.nn.functional.avg_pool2d."""
    import torch
    x = spiky_plane(H, W, 5).reshape(H, W)
    d, p, buf = enc(x.reshape(-1), (1, 1, H, W), bits=2, salient_mode=fho.ALL)
    t = hp.table(buf, 1)
    if t["cls"][0] == fho.RAW:
        pytest.skip("plane stored verbatim")
    s = hp.salient_plane(buf, 1, 0, H, W, 4)
    Hp, Wp = 8 * ((H + 7) // 8), 8 * ((W + 7) // 8)
    m = torch.zeros(1, 1, Hp, Wp)
    m[0, 0, :H, :W] = torch.from_numpy((x != 0).astype(np.float32))
    pooled = torch.nn.functional.avg_pool2d(m, 8).reshape(-1).numpy()
    assert np.array_equal(s["dense"], (pooled >= 0.25).astype(np.int64))
    # reshape-sum gives the same counts
    cnt = m[0, 0].numpy().reshape(Hp // 8, 8, Wp // 8, 8).sum((1, 3)).reshape(-1)
    assert np.array_equal(s["dense"], (cnt * 4 >= 64).astype(np.int64))
    assert s["n_dense"] == int(s["dense"].sum())


def test_block_threshold_at_15_16_nonzeros():
    for nnz, want in [(15, 0), (16, 1)]:
        x = np.zeros((8, 16), dtype=np.float32)
        x.reshape(-1)[:0] = 0
        idx = np.random.default_rng(nnz).permutation(64)[:nnz]
        blk = np.zeros(64, dtype=np.float32)
        blk[idx] = 1.0
        x[:, 8:] = blk.reshape(8, 8)
        d, p, buf = enc(x.reshape(-1), (1, 1, 8, 16), bits=2, salient_mode=fho.ALL)
        t = hp.table(buf, 1)
        assert t["cls"][0] == fho.SALIENT
        s = hp.salient_plane(buf, 1, 0, 8, 16, 4)
        assert list(s["dense"]) == [0, want]


@pytest.mark.parametrize("H,W,dtype", [(24, 40, synth.F32), (21, 30, synth.F32), (33, 17, synth.BF16)])
def test_csr_equals_scipy(H, W, dtype):
    """Sparse blocks are stored as the textbook CSR of the plane with dense-block elements zeroed."""
    x = spiky_plane(H, W, 8)
    raw = x if dtype == synth.F32 else synth.to_bf16_bits(x)
    xv = x if dtype == synth.F32 else synth.bf16_bits_to_f32(raw)
    e = 4 if dtype == synth.F32 else 2
    d, p, buf = enc(raw, (1, 1, H, W), dtype=dtype, bits=2, salient_mode=fho.ALL)
    t = hp.table(buf, 1)
    assert t["cls"][0] == fho.SALIENT
    s = hp.salient_plane(buf, 1, 0, H, W, e)
    nbx = (W + 7) // 8
    yy, xx = np.mgrid[0:H, 0:W]
    in_sparse = s["dense"][(yy // 8) * nbx + xx // 8] == 0
    ref = sp.csr_matrix(np.where(in_sparse, xv.reshape(H, W), 0).astype(np.float32))
    ref.sort_indices()
    assert np.array_equal(s["row_ptr"], ref.indptr)
    assert np.array_equal(s["col"], ref.indices)
    vals = s["val"].view(np.float32) if e == 4 else synth.bf16_bits_to_f32(s["val"])
    assert np.array_equal(vals, ref.data)
    assert s["nnz_s"] == ref.nnz


def test_lorenzo_hand_case():
    exp = golden()["lorenzo_affine"][1]
    codes = [int(v) for v in exp.split("codes")[1].replace("/", " ").split()]
    # put the 2x3 field in the corner of a dense 8x8 block; fill the rest so the block is dense
    x = np.zeros((8, 8), dtype=np.float32)
    i, j = np.mgrid[0:8, 0:8]
    x[:] = i + j + 1
    d, p, buf = enc(x.reshape(-1), (1, 1, 8, 8), bits=2, salient_mode=fho.ALL, eps=0.5)
    t = hp.table(buf, 1)
    s = hp.salient_plane(buf, 1, 0, 8, 8, 4)
    assert s["n_dense"] == 1 and s["n_out_d"] == 0 and s["nnz_s"] == 0
    c = s["codes"][0]
    assert list(c[0, :3]) + list(c[1, :3]) == codes
    # affine integer field: zero residual everywhere off the first row and column
    assert np.all(c[1:, 1:] == 128) and np.all(c[0, 1:] == 129) and np.all(c[1:, 0] == 129)


@pytest.mark.parametrize("a,b,c", [(1, 2, -5), (-3, 1, 7), (2, -2, 0)])
def test_lorenzo_affine_fields_have_zero_interior_residual(a, b, c):
    """The first-order Lorenzo coefficients (+1, +1, -1) sum to one, so any field
    2*eps*(a*i + b*j + c) with integer a, b, c is predicted exactly in the interior."""
    eps = 0.25
    i, j = np.mgrid[0:16, 0:24]
    x = (2 * eps * (a * i + b * j + c)).astype(np.float32)
    x[x == 0] = 2 * eps * 64  # keep blocks dense without breaking integrality much
    d, p, buf = enc(x.reshape(-1), (1, 1, 16, 24), bits=2, salient_mode=fho.ALL, eps=eps)
    t = hp.table(buf, 1)
    s = hp.salient_plane(buf, 1, 0, 16, 24, 4)
    k = np.rint(x / (2 * eps)).astype(np.int64)
    for bi, blk in enumerate(np.flatnonzero(s["dense"])):
        by, bx = divmod(int(blk), 3)
        kb = k[by * 8:by * 8 + 8, bx * 8:bx * 8 + 8]
        delta = s["codes"][bi] - 128
        good = s["codes"][bi] != 0
        # inverse Lorenzo is a 2-D running sum when no element is stored verbatim
        if good.all():
            assert np.array_equal(np.cumsum(np.cumsum(delta, 0), 1), kb)
    xh = dec(buf, d)
    assert np.array_equal(xh, x.reshape(-1))


@pytest.mark.parametrize("H,W,eps", [(24, 40, 0.0625), (21, 30, 0.5), (40, 24, 0.1)])
def test_dense_blocks_error_bound_outliers_verbatim_zeros_kept(H, W, eps):
    """Eq. 9: residuals inside the bound are quantised -> |x - xhat| <= eps; unpredictable values are
    kept intact; sparse-block values are lossless; zeros stay zeros (Section 4.4.1)."""
    x = spiky_plane(H, W, 13)
    x[5] = 100.0          # residual far outside 8 bits -> verbatim
    x[W + 7] = -1.0e9     # beyond the 2^24 integer range -> verbatim
    d, p, buf = enc(x, (1, 1, H, W), bits=2, salient_mode=fho.ALL, eps=eps)
    t = hp.table(buf, 1)
    assert t["cls"][0] == fho.SALIENT
    s = hp.salient_plane(buf, 1, 0, H, W, 4)
    assert s["n_out_d"] >= 2
    xh = dec(buf, d)
    nbx = (W + 7) // 8
    yy, xx = np.mgrid[0:H, 0:W]
    blk = ((yy // 8) * nbx + xx // 8).reshape(-1)
    in_dense = s["dense"][blk] == 1
    assert np.array_equal(xh[~in_dense], x[~in_dense])          # CSR part is lossless
    err = np.abs(xh.astype(np.float64) - x.astype(np.float64))
    slack = 0.0 if np.log2(eps) == np.floor(np.log2(eps)) else eps * 2.0 ** -21
    assert err[in_dense].max() <= eps + slack
    assert xh[5] == x[5] and xh[W + 7] == x[W + 7]
    # x == 0 -> xhat == 0 on a salient plane
    assert np.all(xh[x == 0] == 0)
    # outlier list holds exactly the elements whose code is 0, in block-then-raster order
    vals = []
    for bi, b in enumerate(np.flatnonzero(s["dense"])):
        by, bx = divmod(int(b), nbx)
        for i in range(8):
            for j in range(8):
                y, xc = by * 8 + i, bx * 8 + j
                if y < H and xc < W:
                    if s["codes"][bi][i, j] == 0:
                        vals.append(x[y * W + xc])
                else:
                    assert s["codes"][bi][i, j] == 128
    assert np.array_equal(np.array(vals, dtype=np.float32), s["outl"].view(np.float32))


def test_residual_code_range_is_symmetric_127():
    """Residual codes are delta + 128 for -127 <= delta <= 127; code 0 marks a verbatim value, so a
    residual of -128 cannot be coded and must be stored verbatim too."""
    x = np.full((8, 8), 1.0, dtype=np.float32)   # eps = 0.5: k = x; uniform field -> residual 0
    x[1, 1] = 128   # residuals +127 at (1,1),(2,2) and -127 at (1,2),(2,1): all codable
    x[4, 4] = 129   # residuals +128 at (4,4),(5,5) and -128 at (4,5),(5,4): none codable
    d, p, buf = enc(x.reshape(-1), (1, 1, 8, 8), bits=2, salient_mode=fho.ALL, eps=0.5)
    s = hp.salient_plane(buf, 1, 0, 8, 8, 4)
    c = s["codes"][0]
    assert (c[1, 1], c[1, 2], c[2, 1], c[2, 2]) == (255, 1, 1, 255)
    assert (c[4, 4], c[4, 5], c[5, 4], c[5, 5]) == (0, 0, 0, 0)
    assert list(s["outl"].view(np.float32)) == [129.0, 1.0, 1.0, 1.0]
    assert np.array_equal(dec(buf, d), x.reshape(-1))


def test_predictor_sees_reconstructed_values():
    """"predictions utilize decompressed rather than original values": rebuilding k from the codes by
    a raster walk that only uses already-reconstructed neighbours gives exactly rint(x / 2 eps)."""
    H, W, eps = 16, 16, 0.0625
    x = (np.random.default_rng(4).standard_normal(H * W) * 2 + 3).astype(np.float32)
    d, p, buf = enc(x, (1, 1, H, W), bits=2, salient_mode=fho.ALL, eps=eps)
    t = hp.table(buf, 1)
    s = hp.salient_plane(buf, 1, 0, H, W, 4)
    assert s["n_dense"] == 4 and s["n_out_d"] == 0
    k_true = np.rint(x.reshape(H, W) / np.float32(2 * eps)).astype(np.int64)
    for bi in range(4):
        by, bx = divmod(bi, 2)
        k = np.zeros((9, 9), dtype=np.int64)
        for i in range(8):
            for j in range(8):
                pred = k[i, j + 1] + k[i + 1, j] - k[i, j]
                k[i + 1, j + 1] = pred + s["codes"][bi][i, j] - 128
        assert np.array_equal(k[1:, 1:], k_true[by * 8:by * 8 + 8, bx * 8:bx * 8 + 8])
    xh = dec(buf, d)
    assert np.array_equal(xh, (k_true * np.float32(2 * eps)).astype(np.float32).reshape(-1))


def test_raw_rule_when_nothing_is_gained():
    """A plane of unpredictable values costs more than it saves: stored verbatim."""
    rng = np.random.default_rng(2)
    x = (rng.standard_normal(64 * 64) * 1e6).astype(np.float32)
    d, p, buf = enc(x, (1, 1, 64, 64), bits=2, salient_mode=fho.ALL, eps=0.0625)
    t = hp.table(buf, 1)
    assert t["cls"][0] == fho.RAW and fho.parse_header(buf)["n_raw"] == 1
    assert buf.size == 64 + 16 + 4 * 64 * 64 and hp.table(buf, 1)["off"][0] == 64 + 16 + 1024
    assert np.array_equal(dec(buf, d), x)


# ------------------------------------------------------------------------------------------------
# Whole-tensor invariants and errors
# ------------------------------------------------------------------------------------------------

@pytest.mark.parametrize("dtype", [synth.F32, synth.BF16])
@pytest.mark.parametrize("bits", [2, 8])
def test_round_trip_mixed_tensor(dtype, bits):
    spec = synth.TensorSpec("m", (3, 16, 14, 14), dtype, "spiky_relu", 31)
    raw = synth.make(spec)
    x = raw if dtype == synth.F32 else synth.bf16_bits_to_f32(raw)
    d, p, buf = enc(raw, spec.shape, dtype=dtype, bits=bits)
    out = dec(buf, d)
    xh = out if dtype == synth.F32 else synth.bf16_bits_to_f32(out)
    t = hp.table(buf, 48)
    hw = 196
    L = (1 << bits) - 1
    for pl in range(48):
        xs, xr = x[pl * hw:(pl + 1) * hw].astype(np.float64), xh[pl * hw:(pl + 1) * hw].astype(np.float64)
        if t["cls"][pl] == fho.RAW:
            assert np.array_equal(xs, xr)
        elif t["cls"][pl] == fho.NORMAL:
            tol = (xs.max() - xs.min()) / L
            if dtype == synth.BF16:
                tol += np.abs(xs).max() * 2.0 ** -8
            assert np.abs(xs - xr).max() <= tol
        else:
            tol = 0.0625 + (np.abs(xs).max() * 2.0 ** -8 if dtype == synth.BF16 else 0)
            assert np.abs(xs - xr).max() <= tol
            assert np.all(xr[xs == 0] == 0)


def test_errors_capacity_nonfinite_corrupt_args():
    x = synth.relu_normal(2 * 64, 1)
    d = fho.desc((1, 2, 8, 8))
    p = fho.params(bits=2)
    need = fho.compressed_bytes(d, p, 0)
    st, buf, total = fho.compress(x, d, p, capacity=need - 1)
    assert st == fho.ERR_CAPACITY and total == need
    st, buf, total = fho.compress(x, d, p, capacity=need)
    assert st == fho.OK
    for bad in (np.nan, np.inf, -np.inf):
        y = x.copy()
        y[70] = bad
        st, _, _ = fho.compress(y, d, p)
        assert st == fho.ERR_NONFINITE
    y = x.copy()
    y[0], y[1] = 3e38, -3e38   # finite values whose range overflows
    assert fho.compress(y, d, p)[0] == fho.ERR_NONFINITE
    # corrupt header / wrong expectation / truncated buffer
    good = buf.copy()
    b = good.copy(); b[0] ^= 1
    assert fho.decompress(b, d)[0] == fho.ERR_CORRUPT
    assert fho.decompress(good, fho.desc((1, 2, 8, 4)))[0] == fho.ERR_CORRUPT
    assert fho.decompress(good[:-1], d)[0] == fho.ERR_CORRUPT
    assert fho.compress(x, d, fho.params(bits=3))[0] == fho.ERR_UNSUPPORTED
    assert fho.compress(x, d, fho.params(eps=0.0))[0] == fho.ERR_ARG
    # -0.0 counts as zero
    z = np.zeros(64, dtype=np.float32)
    z[::3] = -0.0
    z[1] = 5
    dd, pp, bb = enc(z, (1, 1, 8, 8), bits=2, salient_mode=fho.ALL)
    s = hp.salient_plane(bb, 1, 0, 8, 8, 4)
    assert s["nnz_s"] == 1 and s["n_dense"] == 0
    out = dec(bb, dd)
    assert out[1] == 5 and np.all(out.view(np.uint32)[np.arange(64) != 1] == 0)


def test_threads_do_not_change_bytes():
    spec = synth.TensorSpec("m", (2, 32, 14, 14), synth.F32, "spiky_relu", 3)
    x = synth.make(spec)
    fho.set_threads(1)
    _, _, b1 = enc(x, spec.shape, bits=4)
    fho.set_threads(4)
    _, _, b4 = enc(x, spec.shape, bits=4)
    fho.set_threads(1)
    assert np.array_equal(b1, b4)
