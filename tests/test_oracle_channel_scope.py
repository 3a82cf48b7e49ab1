"""Pins of the oracle's channel-wide three-sigma mode (salient_mode = CHANNEL): mu and sigma over the N
planes of a channel, one class per channel."""
import numpy as np

from oracle import fho
from paper_2510_11400_b200 import synth
from tests import helpers as hp


def test_channel_thresholds_and_count_against_numpy_float64():
    rng = np.random.default_rng(3)
    for n, hw in ((4, 49), (8, 196), (3, 1024), (16, 16)):
        x = rng.standard_normal((n, hw)).astype(np.float32)
        x[rng.random((n, hw)) < 0.02] *= 6.0
        lo, dlo, dhi, cnt = fho.channel_sigma(x)
        tlo, thi = float(lo) + dlo, float(lo) + dhi
        mu, sd = x.astype(np.float64).mean(), x.astype(np.float64).std()
        span = float(x.max()) - float(x.min())
        assert abs(thi - (mu + 3 * sd)) < 1e-5 * span and abs(tlo - (mu - 3 * sd)) < 1e-5 * span
        margin = 2e-5 * span
        near = ((np.abs(x - thi) < margin) | (np.abs(x - tlo) < margin)).sum()
        want = int(((x > mu + 3 * sd) | (x < mu - 3 * sd)).sum())
        assert abs(cnt - want) <= near
        assert cnt <= x.size / 9          # Chebyshev
    # one plane: the channel is the plane
    x = rng.standard_normal((1, 256)).astype(np.float32)
    assert fho.channel_sigma(x) == fho.plane_sigma(x[0])
    # a channel far from zero: the same plain answer (moments of the distances from the channel's minimum)
    x = (500.0 + 0.05 * rng.standard_normal((8, 196))).astype(np.float32)
    x[rng.random((8, 196)) < 0.02] += 1.0
    lo, dlo, dhi, cnt = fho.channel_sigma(x)
    mu, sd = x.astype(np.float64).mean(), x.astype(np.float64).std()
    span = float(x.max()) - float(x.min())
    assert abs(float(lo) + dhi - (mu + 3 * sd)) < 1e-5 * span and abs(float(lo) + dlo - (mu - 3 * sd)) < 1e-5 * span
    near = ((np.abs(x - (mu + 3 * sd)) < 2e-5 * span) | (np.abs(x - (mu - 3 * sd)) < 2e-5 * span)).sum()
    assert abs(cnt - int(((x > mu + 3 * sd) | (x < mu - 3 * sd)).sum())) <= near and cnt > 0


def test_batch_of_one_reduces_to_the_per_plane_mode():
    spec = synth.TensorSpec("t", (1, 24, 14, 14), synth.F32, "spiky_relu", 31)
    raw = synth.make(spec)
    d = fho.desc(spec.shape, spec.dtype)
    a = fho.compress(raw, d, fho.params(bits=4, salient_mode=fho.AUTO))[1]
    c = fho.compress(raw, d, fho.params(bits=4, salient_mode=fho.CHANNEL))[1]
    assert a.size == c.size and a[27] == fho.AUTO and c[27] == fho.CHANNEL
    a2, c2 = a.copy(), c.copy()
    a2[27] = c2[27] = 0
    assert np.array_equal(a2, c2)


def test_one_class_per_channel_and_counts_add_up():
    shape = (6, 20, 14, 14)
    spec = synth.TensorSpec("t", shape, synth.F32, "spiky_relu", 32)     # channels 0 and 16 are spiky in every sample
    raw = synth.make(spec)
    d = fho.desc(shape, spec.dtype)
    st, buf, _ = fho.compress(raw, d, fho.params(bits=2, salient_mode=fho.CHANNEL))
    assert st == fho.OK
    t = hp.table(buf, 6 * 20)
    cls = t["cls"].reshape(6, 20)
    x = raw.reshape(6, 20, 196)
    for c in range(20):
        assert len(set((cls[:, c] != fho.NORMAL).tolist())) == 1          # the whole channel or none of it
        cnt = fho.channel_sigma(x[:, c])[3]
        assert int(t["n_out"].reshape(6, 20)[:, c].sum()) == cnt
        assert (cls[0, c] != fho.NORMAL) == (cnt * 32 > 6 * 196)
    assert (cls[:, 0] != fho.NORMAL).all() and (cls[:, 16] != fho.NORMAL).all() and (cls[:, 1:16] == fho.NORMAL).all()
    # round trip: restored values of normal planes within the quantiser's bound, zeros kept on the others
    st, out = fho.decompress(buf, d)
    assert st == fho.OK
    out = out.reshape(6, 20, 196)
    assert ((x[:, 0] == 0) <= (out[:, 0] == 0)).all()


def test_a_single_spiky_sample_does_not_mark_the_channel():
    """Per plane the spiky plane is outlier-rich; over a batch of 32 its outliers are 1/32 of the channel's
    elements' share and the channel stays normal -- the two readings differ exactly here."""
    n, hw = 32, 196
    rng = np.random.default_rng(8)
    x = np.maximum(rng.standard_normal((n, 1, hw)), 0).astype(np.float32)
    x[5, 0, :16] = 40.0                                   # 16 of 196 elements of one plane
    d = fho.desc((n, 1, 14, 14), fho.F32)
    per_plane = hp.table(fho.compress(x.reshape(-1), d, fho.params(salient_mode=fho.AUTO))[1], n)["cls"]
    per_channel = hp.table(fho.compress(x.reshape(-1), d, fho.params(salient_mode=fho.CHANNEL))[1], n)["cls"]
    assert per_plane[5] != fho.NORMAL
    assert (per_channel == fho.NORMAL).all()
