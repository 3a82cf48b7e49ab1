"""Pins of the oracle's tensor-wide three-sigma mode (salient_mode = TENSOR): mu and sigma over the whole
activation tensor fix what an outlier is; a plane is outlier-rich by its own share of such outliers."""
import numpy as np

from oracle import fho
from paper_2510_11400_b200 import synth
from tests import helpers as hp


def test_single_plane_tensor_reduces_to_the_per_plane_mode():
    spec = synth.TensorSpec("t", (1, 1, 28, 28), synth.F32, "spiky_relu", 41)
    raw = synth.make(spec)
    d = fho.desc(spec.shape, spec.dtype)
    a = fho.compress(raw, d, fho.params(bits=4, salient_mode=fho.AUTO))[1]
    t = fho.compress(raw, d, fho.params(bits=4, salient_mode=fho.TENSOR))[1]
    assert a.size == t.size and a[27] == fho.AUTO and t[27] == fho.TENSOR
    a2, t2 = a.copy(), t.copy()
    a2[27] = t2[27] = 0
    assert np.array_equal(a2, t2)


def test_counts_follow_the_tensor_wide_thresholds_and_classes_the_planes_own_share():
    n, c, h, w = 5, 12, 14, 14
    rng = np.random.default_rng(42)
    x = rng.standard_normal((n, c, h * w)).astype(np.float32)
    x[:, 3] *= 4.0                      # one loud channel: most outliers of the tensor sit there
    x[2, 7, :3] = 9.0                   # a few spikes in an otherwise quiet plane
    d = fho.desc((n, c, h, w), fho.F32)
    st, buf, _ = fho.compress(x.reshape(-1), d, fho.params(bits=2, salient_mode=fho.TENSOR))
    assert st == fho.OK
    t = hp.table(buf, n * c)
    x64 = x.astype(np.float64)
    mu, sd = x64.mean(), x64.std()
    thi, tlo = mu + 3 * sd, mu - 3 * sd
    margin = 2e-5 * (float(x.max()) - float(x.min()))
    flat = x.reshape(n * c, h * w)
    want = ((flat > thi) | (flat < tlo)).sum(axis=1)
    near = ((np.abs(flat - thi) < margin) | (np.abs(flat - tlo) < margin)).sum(axis=1)
    assert (np.abs(t["n_out"].astype(np.int64) - want) <= near).all()
    assert want.sum() > 0
    assert ((t["cls"] != fho.NORMAL) == (t["n_out"].astype(np.int64) * 32 > h * w)).all()
    # the oracle's own statistic over all planes gives the same total
    assert int(t["n_out"].sum()) == fho.channel_sigma(flat)[3]
    cls = t["cls"].reshape(n, c)
    assert (cls[:, 3] != fho.NORMAL).all()                 # sigma of the tensor is ~1.5: a third of 4 N(0,1) lies outside
    assert cls[2, 7] == fho.NORMAL                         # 3 of 196 elements: below 1/32
    assert (np.delete(cls, 3, axis=1) == fho.NORMAL).all()


def test_the_three_scopes_differ_where_they_should():
    """A loud channel is normal by its own statistics (per plane, per channel) and outlier-rich by the tensor's."""
    n, c, hw = 4, 8, 196
    rng = np.random.default_rng(43)
    x = rng.standard_normal((n, c, hw)).astype(np.float32)
    x[:, 5] *= 6.0
    d = fho.desc((n, c, 14, 14), fho.F32)
    cls = {m: hp.table(fho.compress(x.reshape(-1), d, fho.params(salient_mode=m))[1], n * c)["cls"].reshape(n, c)
           for m in (fho.AUTO, fho.CHANNEL, fho.TENSOR)}
    assert (cls[fho.AUTO][:, 5] == fho.NORMAL).all() and (cls[fho.CHANNEL][:, 5] == fho.NORMAL).all()
    assert (cls[fho.TENSOR][:, 5] != fho.NORMAL).all()


def test_round_trip_and_bf16():
    spec = synth.TensorSpec("t", (3, 16, 14, 14), synth.BF16, "spiky_relu", 44)
    raw = synth.make(spec)
    d = fho.desc(spec.shape, spec.dtype)
    st, buf, total = fho.compress(raw, d, fho.params(bits=8, salient_mode=fho.TENSOR))
    assert st == fho.OK and total == buf.size
    st, out = fho.decompress(buf, d)
    assert st == fho.OK
    t = hp.table(buf, 48)
    x = synth.bf16_bits_to_f32(raw).reshape(48, 196)
    y = synth.bf16_bits_to_f32(out).reshape(48, 196)
    normal = np.nonzero(t["cls"] == fho.NORMAL)[0]
    assert 0 < normal.size < 48
    for p in normal:   # half a quantisation step plus the rounding of the restored value to bf16
        assert np.abs(x[p] - y[p]).max() <= 0.5 * t["scale"][p] * 1.01 + 2.0 ** -8 * np.abs(x[p]).max()


def test_non_finite_input_is_reported():
    x = np.ones(2 * 3 * 16, dtype=np.float32)
    x[17] = np.inf
    st, _, _ = fho.compress(x, fho.desc((2, 3, 4, 4), fho.F32), fho.params(salient_mode=fho.TENSOR))
    assert st == fho.ERR_NONFINITE
