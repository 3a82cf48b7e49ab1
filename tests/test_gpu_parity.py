"""Parity of the CUDA path with the CPU oracle, through the C ABI, on seeded synthetic activations.

Bar: container bytes (header, plane table, payloads) and sizes bit-exact; restored values
bit-identical (the contract allows 1 ulp; -0.0 and +0.0 compare equal).
"""
import ctypes as C

import numpy as np
import pytest

from oracle import fho
from paper_2510_11400_b200 import api, build, synth
from tests import helpers as hp

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _lib():
    build.build()
    api.lib()
    yield
    api.shutdown()


def to_dev(raw):
    import torch
    t = torch.from_numpy(raw.view(np.int16) if raw.dtype == np.uint16 else raw)
    return t.cuda()


def gpu_compress(raw, shape, dtype, **kw):
    p = api.default_params(**kw)
    st, packed, total = api.compress_tensor(to_dev(raw), shape, dtype, p)
    return st, packed, total


def oracle_compress(raw, shape, dtype, **kw):
    d = fho.desc(shape, dtype)
    p = fho.params(**kw)
    st, buf, total = fho.compress(raw, d, p)
    return st, buf, total, d


def check_same_values(a, b, dtype):
    """Bit-identical except that -0.0 == +0.0."""
    if dtype == synth.F32:
        a32, b32 = a.view(np.uint32), b.view(np.uint32)
        diff = (a32 != b32) & ~(((a32 | b32) & 0x7FFFFFFF) == 0)
    else:
        diff = (a != b) & ~(((a | b) & 0x7FFF) == 0)
    assert not diff.any(), f"{int(diff.sum())} values differ, first at {int(np.flatnonzero(diff)[0])}"


def full_parity(spec, **kw):
    raw = synth.make(spec)
    st_o, buf_o, total_o, d = oracle_compress(raw, spec.shape, spec.dtype, **kw)
    assert st_o == fho.OK
    st_g, packed, total_g = gpu_compress(raw, spec.shape, spec.dtype, **kw)
    assert st_g == api.FH_OK
    assert total_g == total_o
    buf_g = packed[:total_g].cpu().numpy()
    if not np.array_equal(buf_g, buf_o):
        P = spec.shape[0] * spec.shape[1]
        tg, to = hp.table(buf_g, P), hp.table(buf_o, P)
        for key in ("cls", "n_out", "off"):
            bad = np.flatnonzero(tg[key] != to[key])
            assert bad.size == 0, f"table field {key} differs at planes {bad[:8]}: gpu {tg[key][bad[:8]]} oracle {to[key][bad[:8]]}"
        assert np.array_equal(buf_g[:64], buf_o[:64]), "header differs"
        first = int(np.flatnonzero(buf_g != buf_o)[0])
        pl = int(np.searchsorted(to["off"], first, side="right") - 1)
        raise AssertionError(f"payload bytes differ first at byte {first} (plane {pl}, class {to['cls'][pl]})")
    st_d, out_g = api.decompress_tensor(packed, total_g, spec.shape, spec.dtype)
    assert st_d == api.FH_OK
    st_r, out_o = fho.decompress(buf_o, d)
    assert st_r == fho.OK
    out_g = out_g.cpu().numpy()
    if spec.dtype == synth.BF16:
        out_g = out_g.view(np.uint16)
    check_same_values(out_g, out_o, spec.dtype)
    return buf_o


def test_config1_round_trip_at_2_bits():
    buf = full_parity(synth.config1()[0], bits=2)
    h = fho.parse_header(buf)
    if h["n_salient"] == 0 and h["n_raw"] == 0:
        assert buf.size == 139328


SHAPES = [
    (3, 5, 7, 7),      # 49-element planes: unaligned plane starts, tensor size not a multiple of 16 bytes
    (2, 9, 14, 14),    # sub-warp teams
    (1, 7, 1, 1),      # single-element planes
    (2, 3, 3, 1),
    (1, 5, 5, 7),
    (2, 6, 33, 17),    # ragged 8x8 blocks in both directions
    (1, 12, 32, 32),   # one warp per plane, vector loads
    (2, 8, 28, 28),
    (1, 6, 56, 56),    # whole-CTA teams of 128 threads
    (1, 3, 112, 112),  # whole-CTA teams of 512 threads
    (1, 2, 64, 100),
    (1, 2, 128, 120),  # 60 KB planes
    (300, 1, 4, 4),    # many tiny planes, several tiles with a ragged last tile
]


@pytest.mark.parametrize("shape", SHAPES)
@pytest.mark.parametrize("dtype", [synth.F32, synth.BF16])
@pytest.mark.parametrize("bits", [2, 4, 8])
def test_parity_auto_mode_mixed_planes(shape, dtype, bits):
    kind = "spiky_relu" if (shape[1] >= 3) else "relu"
    spec = synth.TensorSpec("t", shape, dtype, kind, 40 + bits)
    full_parity(spec, bits=bits)


# Planes of 257 to 4096 groups run on the CTA-team kernel that keeps a thread's groups in registers: one shape per
# (threads, groups per thread) it is built for, each with a plane that fills the threads exactly and one that does
# not, and one shape beyond it (the kernel that sweeps the plane in shared memory).
CTA_SHAPES = [
    (1, 4, 56, 64), (1, 4, 57, 60),      # 896 groups = 128 x 7; 855
    (1, 4, 64, 64), (1, 4, 40, 100),     # 1024 = 128 x 8; 1000
    (1, 4, 64, 112), (1, 4, 60, 100),    # 1792 = 256 x 7; 1500
    (1, 4, 128, 64), (1, 4, 80, 100),    # 2048 = 256 x 8; 2000
    (1, 4, 112, 112), (1, 4, 100, 120),  # 3136 = 448 x 7; 3000
    (1, 4, 128, 128), (1, 4, 100, 160),  # 4096 = 512 x 8; 4000
    (1, 3, 160, 164),                    # 6560 groups: beyond the register variant
]


@pytest.mark.parametrize("shape", CTA_SHAPES)
@pytest.mark.parametrize("dtype", [synth.F32, synth.BF16])
def test_parity_cta_team_kernels(shape, dtype):
    full_parity(synth.TensorSpec("t", shape, dtype, "spiky_relu", 61), bits=2)
    full_parity(synth.TensorSpec("t", shape, dtype, "normal", 62), bits=8, salient_mode=api.FH_SALIENT_OFF)


@pytest.mark.parametrize("dtype", [synth.F32, synth.BF16])
def test_moment_sums_of_a_cta_team_beyond_32_bits(dtype):
    """Planes whose elements all lie near the maximum, with a single small one: every group's scaled sums are
    near their largest, and over 3136 groups the integer moment sums pass 2^32 (a warp team's never can)."""
    shape = (1, 6, 112, 112)
    rng = np.random.default_rng(5)
    x = (1000.0 + rng.random(shape, dtype=np.float32)).astype(np.float32)
    x[0, :, 3, 5] = 0.0                                  # the minimum: distances of about the range everywhere else
    x[0, 1::2, 60:70, 40:90] = 2000.0                    # every other plane: 500 far elements (outlier-rich or not, the oracle says)
    raw = synth.to_bf16_bits(x).reshape(shape) if dtype == synth.BF16 else x
    st_o, buf_o, total_o, d = oracle_compress(raw, shape, dtype, bits=4)
    assert st_o == fho.OK
    st_g, packed, total_g = gpu_compress(raw, shape, dtype, bits=4)
    assert st_g == api.FH_OK and total_g == total_o
    assert np.array_equal(packed[:total_g].cpu().numpy(), buf_o)


@pytest.mark.parametrize("shape", SHAPES)
@pytest.mark.parametrize("dtype", [synth.F32, synth.BF16])
@pytest.mark.parametrize("mode", [api.FH_SALIENT_OFF, api.FH_SALIENT_ALL])
def test_parity_forced_modes(shape, dtype, mode):
    spec = synth.TensorSpec("t", shape, dtype, "normal" if mode == api.FH_SALIENT_OFF else "spiky_relu", 90)
    full_parity(spec, bits=4, salient_mode=mode)


@pytest.mark.parametrize("shape", SHAPES)
@pytest.mark.parametrize("dtype", [synth.F32, synth.BF16])
def test_parity_huffman_stage(shape, dtype):
    """entropy = 1: the dense-block residual codes of outlier-rich planes go through the Huffman stage (one
    code per plane); container (version 2) identical to the oracle's byte for byte, restored values identical,
    in the three-sigma mode on mixed planes and with every plane forced down the block-wise path."""
    kind = "spiky_relu" if (shape[1] >= 3) else "relu"
    buf = full_parity(synth.TensorSpec("t", shape, dtype, kind, 71), bits=4, entropy=1, eps=0.25)
    assert fho.parse_header(buf)["version"] == 2
    buf = full_parity(synth.TensorSpec("t", shape, dtype, "relu", 72), bits=2, entropy=1, eps=0.25, salient_mode=api.FH_SALIENT_ALL)
    plain = fho.compress(synth.make(synth.TensorSpec("t", shape, dtype, "relu", 72)), fho.desc(shape, dtype),
                         fho.params(bits=2, eps=0.25, salient_mode=fho.ALL))[1]
    assert buf.size <= plain.size


def test_huffman_stage_gain_on_the_supplementary_workload():
    """Every 16th channel sparse-spiky (the recipe that drives planes down the block-wise path), ResNet-shaped
    56x56 planes: the stage shrinks the container, and the GPU's bytes are the oracle's."""
    spec = synth.supplement([synth.TensorSpec("s", (8, 64, 56, 56), synth.F32, "relu", 130)])[0]
    plain = full_parity(spec, bits=2, eps=0.0625)
    coded = full_parity(spec, bits=2, eps=0.0625, entropy=1)
    assert coded.size < plain.size
    print(f"supplement 8x64x56x56: {plain.size} B plain, {coded.size} B with the Huffman stage")


@pytest.mark.parametrize("kind", ["relu", "normal", "laplace_ch", "laplace_iid", "spiky_normal"])
@pytest.mark.parametrize("dtype", [synth.F32, synth.BF16])
def test_parity_value_distributions(kind, dtype):
    spec = synth.TensorSpec("t", (4, 16, 28, 28), dtype, kind, 7)
    full_parity(spec, bits=2)


@pytest.mark.parametrize("eps,tau,rho", [(0.5, (1, 4), (1, 32)), (0.1, (1, 2), (1, 64)), (0.0625, (1, 64), (1, 16)),
                                         (0.01, (3, 4), (0, 1))])
def test_parity_other_parameters(eps, tau, rho):
    spec = synth.TensorSpec("t", (2, 32, 24, 40), synth.F32, "spiky_relu", 11)
    full_parity(spec, bits=4, eps=eps, tau=tau, rho=rho)


def test_parity_multi_tile_scan_with_mixed_sizes():
    """Many tiles whose sizes differ (salient, raw and normal planes mixed): the plane-ordered offsets
    come from the look-back scan across tiles."""
    spec = synth.TensorSpec("t", (64, 48, 14, 14), synth.F32, "spiky_relu", 5)
    buf = full_parity(spec, bits=2)
    t = hp.table(buf, 64 * 48)
    assert (t["cls"] == fho.SALIENT).sum() > 100
    spec = synth.TensorSpec("t", (16, 32, 56, 56), synth.BF16, "laplace_ch", 6)
    full_parity(spec, bits=8)


def test_special_values_constant_planes_negative_zero_tiny_range():
    x = synth.normal(8 * 64, 3).reshape(8, 64)
    x[0] = 2.5                      # constant plane: scale 0, exact
    x[1] = 0.0
    x[1, ::3] = -0.0                # signed zeros
    x[2] = 1e-42                    # denormals, constant
    x[3, :] = np.float32(1e-40) * np.arange(64)   # denormal range: inv overflows -> all codes 0
    x[4] *= 1e30                    # huge but finite
    x[5] = np.arange(64) % 4        # exact codes at 2 bits
    raw = np.ascontiguousarray(x.reshape(-1), dtype=np.float32)
    for mode in (api.FH_SALIENT_OFF, api.FH_SALIENT_AUTO, api.FH_SALIENT_ALL):
        st_o, buf_o, total_o, d = oracle_compress(raw, (1, 8, 8, 8), synth.F32, bits=2, salient_mode=mode)
        st_g, packed, total_g = gpu_compress(raw, (1, 8, 8, 8), synth.F32, bits=2, salient_mode=mode)
        assert (st_o, st_g) == (0, 0) and total_o == total_g
        assert np.array_equal(packed[:total_g].cpu().numpy(), buf_o)
        st_d, out_g = api.decompress_tensor(packed, total_g, (1, 8, 8, 8), synth.F32)
        _, out_o = fho.decompress(buf_o, d)
        check_same_values(out_g.cpu().numpy(), out_o, synth.F32)


def test_device_side_errors_nonfinite_capacity_corrupt():
    import torch
    shape = (2, 16, 16, 16)
    raw = synth.relu_normal(2 * 16 * 256, 1)
    # non-finite input
    for bad in (np.nan, np.inf, -np.inf):
        y = raw.copy()
        y[5000] = bad
        st, _, _ = gpu_compress(y, shape, synth.F32, bits=2)
        assert st == api.FH_ERR_NONFINITE
    y = raw.copy()
    y[0], y[1] = 3e38, -3e38
    assert gpu_compress(y, shape, synth.F32, bits=2)[0] == api.FH_ERR_NONFINITE
    # capacity one byte short: error, needed size reported, nothing written past the capacity
    p = api.default_params(bits=2, salient_mode=api.FH_SALIENT_OFF)
    d = api.desc(shape)
    need = api.compressed_bytes(d, p, 0)
    x = to_dev(raw)
    dst = torch.full((need + 64,), 0xAB, dtype=torch.uint8, device="cuda")
    out2 = torch.zeros(2, dtype=torch.int64, device="cuda")
    assert api.fh_compress(d, p, x, dst, out2, capacity=need - 1) == api.FH_OK
    torch.cuda.synchronize()
    assert out2.tolist() == [need, api.FH_ERR_CAPACITY]
    assert bool((dst[need - 1:] == 0xAB).all())
    assert api.fh_compress(d, p, x, dst, out2, capacity=need) == api.FH_OK
    torch.cuda.synchronize()
    assert out2.tolist() == [need, api.FH_OK]
    assert bool((dst[need:] == 0xAB).all())
    # corrupt container: magic, shape expectation, truncation, table offset
    good = dst[:need].clone()
    st, _ = api.decompress_tensor(good, need, shape, synth.F32)
    assert st == api.FH_OK
    b = good.clone(); b[0] ^= 1
    assert api.decompress_tensor(b, need, shape, synth.F32)[0] == api.FH_ERR_CORRUPT
    assert api.decompress_tensor(good, need, (2, 16, 16, 8), synth.F32)[0] == api.FH_ERR_CORRUPT
    assert api.decompress_tensor(good, need - 1, shape, synth.F32)[0] == api.FH_ERR_CORRUPT
    b = good.clone(); b[64 + 16 * 3 + 3] = 0xFF   # plane 3 points far outside the container
    assert api.decompress_tensor(b, need, shape, synth.F32)[0] == api.FH_ERR_CORRUPT


def test_corrupt_salient_payload_is_rejected_without_out_of_bounds_reads():
    spec = synth.TensorSpec("t", (1, 16, 24, 40), synth.F32, "spiky_relu", 77)
    raw = synth.make(spec)
    st, packed, total = gpu_compress(raw, spec.shape, spec.dtype, bits=4)
    assert st == api.FH_OK
    buf = packed[:total].cpu().numpy()
    t = hp.table(buf, 16)
    pl = int(np.flatnonzero(t["cls"] == fho.SALIENT)[0])
    off = 64 + 16 * 16 + pl * hp.npay_of(buf, 24 * 40)     # the payload starts in the plane's slot
    for field, val in ((0, 0x7FFFFFFF), (4, 0x7FFFFFFF), (8, 0x7FFFFFFF)):
        b = packed.clone()
        b[off + field:off + field + 4] = to_dev(np.frombuffer(np.uint32(val).tobytes(), dtype=np.uint8).copy())
        assert api.decompress_tensor(b, total, spec.shape, spec.dtype)[0] == api.FH_ERR_CORRUPT
    # a continuation offset that points outside the overflow region
    b = packed.clone()
    b[64 + 16 * pl:64 + 16 * pl + 4] = to_dev(np.frombuffer(np.uint32(5).tobytes(), dtype=np.uint8).copy())
    assert api.decompress_tensor(b, total, spec.shape, spec.dtype)[0] == api.FH_ERR_CORRUPT


def test_repeated_calls_reuse_the_scratch_and_stay_exact():
    spec = synth.TensorSpec("t", (8, 32, 14, 14), synth.F32, "spiky_relu", 21)
    raw = synth.make(spec)
    _, buf_o, total_o, _ = oracle_compress(raw, spec.shape, spec.dtype, bits=2)
    for _ in range(5):
        st, packed, total = gpu_compress(raw, spec.shape, spec.dtype, bits=2)
        assert st == 0 and total == total_o
        assert np.array_equal(packed[:total].cpu().numpy(), buf_o)


def test_schedule_forward_compress_reverse_decompress():
    import torch
    specs = [synth.TensorSpec(f"s{i}", s, synth.F32, "spiky_relu" if i == 2 else "relu", 500 + i, compress=(i % 2 == 0))
             for i, s in enumerate([(4, 16, 32, 32), (4, 16, 32, 32), (4, 32, 16, 16), (4, 32, 16, 16),
                                    (4, 64, 8, 8), (4, 64, 8, 8), (4, 128, 4, 4)])]
    p = api.default_params(bits=2)
    items, raws, restored = [], [], []
    for s in specs:
        raw = synth.make(s)
        raws.append(raw)
        dense = to_dev(raw)
        rest = torch.zeros_like(dense)
        restored.append(rest)
        items.append(api.SchedItem(api.desc(s.shape, s.dtype, tensor_id=s.seed),
                                   api.FH_COMPRESS if s.compress else api.FH_KEEP, dense, rest))
    arena = torch.zeros(8 << 20, dtype=torch.uint8, device="cuda")
    rep = api.fh_run_schedule(items, p, arena)
    assert rep.status == api.FH_OK
    off = 0
    tot_packed = 0
    for s, raw, rest in zip(specs, raws, restored):
        if not s.compress:
            assert not bool(rest.any())
            continue
        d = fho.desc(s.shape, s.dtype, tensor_id=s.seed)
        st, buf_o, total_o = fho.compress(raw, d, fho.params(bits=2))
        assert np.array_equal(arena[off:off + total_o].cpu().numpy(), buf_o)
        _, out_o = fho.decompress(buf_o, d)
        check_same_values(rest.cpu().numpy(), out_o, s.dtype)
        tot_packed += total_o
        off += (total_o + 255) & ~255
    assert rep.total_packed_bytes == tot_packed
    assert rep.peak_packed_bytes == off
    assert rep.total_dense_bytes == sum(s.dense_bytes for s in specs if s.compress)
    assert rep.ms_forward > 0 and rep.ms_backward > 0
    # an arena that is too small: error, and the tensors that did not fit are not restored from stale bytes
    small = arena[:off - 4096]
    for r in restored:
        r.zero_()
    rep = api.fh_run_schedule(items, p, small)
    assert rep.status == api.FH_ERR_CAPACITY
    assert not bool(restored[-1].any())          # the last tensor did not fit: left untouched
    assert bool(restored[0].any())               # the first one did and was restored


def test_host_buffer_entry_points():
    import torch
    spec = synth.TensorSpec("t", (4, 16, 28, 28), synth.BF16, "laplace_ch", 9)
    raw = synth.make(spec)
    d = api.desc(spec.shape, spec.dtype)
    p = api.default_params(bits=4)
    work = torch.empty(api.host_work_bytes(d, p), dtype=torch.uint8, device="cuda")
    h_src = torch.from_numpy(raw.view(np.int16)).pin_memory()
    h_dst = torch.empty(api.compressed_bytes(d, p, 1), dtype=torch.uint8).pin_memory()
    st, total = api.fh_compress_host(d, p, h_src, h_dst, work)
    assert st == api.FH_OK
    _, buf_o, total_o, od = oracle_compress(raw, spec.shape, spec.dtype, bits=4)
    assert total == total_o and np.array_equal(h_dst[:total].numpy(), buf_o)
    h_out = torch.empty_like(h_src)
    assert api.fh_decompress_host(h_dst, total, d, h_out, work) == api.FH_OK
    _, out_o = fho.decompress(buf_o, od)
    check_same_values(h_out.numpy().view(np.uint16), out_o, spec.dtype)


def test_launch_counter_counts_our_kernels():
    before = api.kernel_launches()
    raw = synth.relu_normal(2 * 4 * 64, 1)
    # a compress call is one kernel, a decompress call is one kernel, whatever the mode
    st, packed, total = gpu_compress(raw, (2, 4, 8, 8), synth.F32, bits=2)
    api.decompress_tensor(packed, total, (2, 4, 8, 8), synth.F32)
    assert api.kernel_launches() == before + 2
    st, packed, total = gpu_compress(raw, (2, 4, 8, 8), synth.F32, bits=2, salient_mode=api.FH_SALIENT_OFF)
    api.decompress_tensor(packed, total, (2, 4, 8, 8), synth.F32)
    assert api.kernel_launches() == before + 4
    # the channel-wide mode adds its three statistics passes
    st, packed, total = gpu_compress(raw, (2, 4, 8, 8), synth.F32, bits=2, salient_mode=api.FH_SALIENT_CHANNEL)
    assert api.kernel_launches() == before + 8


def test_back_to_back_calls_without_host_synchronisation():
    """Several tensors with outlier-rich planes, compressed and restored back to back on one stream for
    three rounds with no host synchronisation in between: kernels of consecutive calls overlap at their
    edges, share the per-stream counters and alternate between the two sets of the placement scan's group
    sums; every wait must still end (every status word 0); the last round is compared with the oracle."""
    import torch
    specs = [synth.TensorSpec("a", (8, 96, 112, 112), synth.BF16, "laplace_ch", 21),
             synth.TensorSpec("b", (16, 144, 56, 56), synth.BF16, "laplace_ch", 22),
             synth.TensorSpec("c", (32, 64, 14, 14), synth.F32, "spiky_relu", 23)]
    ts = []
    for i, sp in enumerate(specs):
        raw = synth.make(sp)
        d = api.desc(sp.shape, sp.dtype)
        cap = api.compressed_bytes(d, api.default_params(bits=8), 1)
        x = to_dev(raw)
        ts.append(dict(sp=sp, raw=raw, d=d, x=x, cap=cap, dst=torch.empty(cap, dtype=torch.uint8, device="cuda"),
                       out=torch.empty_like(x)))
    words = []
    for rnd in range(3):
        for bits in (2, 4, 8):
            p = api.default_params(bits=bits)
            o2 = [torch.zeros(2, dtype=torch.int64, device="cuda") for _ in ts]
            st = [torch.zeros(1, dtype=torch.int64, device="cuda") for _ in ts]
            words.append((o2, st))
            for t, o in zip(ts, o2):
                assert api.fh_compress(t["d"], p, t["x"], t["dst"], o, capacity=t["cap"]) == api.FH_OK
            for t, q in zip(reversed(ts), reversed(st)):
                assert api.fh_decompress(t["dst"], t["cap"], t["d"], t["out"], q) == api.FH_OK
    torch.cuda.synchronize()
    for o2, st in words:
        assert [int(o[1]) for o in o2] == [0] * len(ts)
        assert [int(q[0]) for q in st] == [0] * len(ts)
    for t in ts:   # the last round ran at 8 bits
        st_o, buf_o, total_o, d = oracle_compress(t["raw"], t["sp"].shape, t["sp"].dtype, bits=8)
        assert st_o == fho.OK
        assert np.array_equal(t["dst"][:total_o].cpu().numpy(), buf_o)
        _, out_o = fho.decompress(buf_o, d)
        got = t["out"].cpu().numpy()
        check_same_values(got.view(np.uint16) if t["sp"].dtype == synth.BF16 else got, out_o, t["sp"].dtype)


def _full_size(spec, bits_list):
    """One tensor at its benchmark size: the container of every code width and the restored values against the
    oracle (the input is made once, the oracle runs on all host cores)."""
    raw = synth.make(spec)
    x = to_dev(raw)
    d_o = fho.desc(spec.shape, spec.dtype)
    out = {}
    for bits in bits_list:
        st_o, buf_o, total_o = fho.compress(raw, d_o, fho.params(bits=bits))
        assert st_o == fho.OK
        st_g, packed, total_g = api.compress_tensor(x, spec.shape, spec.dtype, api.default_params(bits=bits))
        assert st_g == api.FH_OK and total_g == total_o
        assert np.array_equal(packed[:total_g].cpu().numpy(), buf_o), f"container differs at {bits} bits"
        st_d, out_g = api.decompress_tensor(packed, total_g, spec.shape, spec.dtype)
        assert st_d == api.FH_OK
        st_r, out_o = fho.decompress(buf_o, d_o)
        assert st_r == fho.OK
        got = out_g.cpu().numpy()
        check_same_values(got.view(np.uint16) if spec.dtype == synth.BF16 else got, out_o, spec.dtype)
        out[bits] = buf_o
        del packed, out_g
    return out


def test_calls_with_and_without_the_placement_scan_interleaved_on_one_stream():
    """Calls that place overflow parts alternate between two sets of group sums, and a call clears the set of
    the last call that used the scan; calls with the three-sigma rule off use neither.  Mixed on one stream,
    with tensors of different tile counts, every container must still equal the oracle's."""
    import torch
    seq = [("a", (4, 40, 14, 14), "spiky_relu", api.FH_SALIENT_AUTO), ("b", (2, 64, 7, 7), "normal", api.FH_SALIENT_OFF),
           ("c", (16, 96, 7, 7), "spiky_relu", api.FH_SALIENT_AUTO), ("d", (1, 8, 56, 56), "spiky_relu", api.FH_SALIENT_ALL),
           ("e", (2, 9, 14, 14), "relu", api.FH_SALIENT_OFF), ("f", (1, 300, 4, 4), "spiky_relu", api.FH_SALIENT_AUTO),
           ("g", (4, 40, 14, 14), "spiky_relu", api.FH_SALIENT_AUTO)]
    items = []
    for i, (name, shape, kind, mode) in enumerate(seq):
        sp = synth.TensorSpec(name, shape, synth.F32, kind, 70 + i)
        raw = synth.make(sp)
        d = api.desc(shape, synth.F32)
        p = api.default_params(bits=4, salient_mode=mode)
        cap = api.compressed_bytes(d, p, 1)
        items.append(dict(sp=sp, raw=raw, d=d, p=p, cap=cap, x=to_dev(raw), mode=mode,
                          dst=torch.empty(cap, dtype=torch.uint8, device="cuda"),
                          o=torch.zeros(2, dtype=torch.int64, device="cuda")))
    for rnd in range(3):
        for t in items:
            assert api.fh_compress(t["d"], t["p"], t["x"], t["dst"], t["o"], capacity=t["cap"]) == api.FH_OK
    torch.cuda.synchronize()
    for t in items:
        assert int(t["o"][1]) == 0
        st_o, buf_o, total_o, _ = oracle_compress(t["raw"], t["sp"].shape, synth.F32, bits=4, salient_mode=t["mode"])
        assert st_o == fho.OK and int(t["o"][0]) == total_o
        assert np.array_equal(t["dst"][:total_o].cpu().numpy(), buf_o), t["sp"].name



@pytest.mark.parametrize("index", range(17))
def test_config2_every_tensor_at_full_size_and_every_code_width(index):
    """The 17 ResNet-18-shaped tensors of the benchmark's default workload (batch 64), at 2, 4 and 8 bits,
    through the entry points and launch configuration the benchmark times."""
    fho.set_threads(fho.max_threads())
    _full_size(synth.config2(64)[index], (2, 4, 8))


@pytest.mark.parametrize("stress", [False, True])
@pytest.mark.parametrize("index", range(5))
def test_config3_every_tensor_at_full_size(index, stress):
    """The MobileNetV2-shaped bf16 tensors (batch 128): channel-clustered outliers (every eighth channel must
    come out outlier-rich, the rest normal) and the i.i.d. stress variant (every plane stays normal)."""
    fho.set_threads(fho.max_threads())
    spec = synth.config3(128, stress=stress)[index]
    buf = _full_size(spec, (2,))[2]
    P = spec.shape[0] * spec.shape[1]
    t = hp.table(buf, P)
    ch = np.arange(P) % spec.shape[1]
    if not stress:
        # (on small planes the share of planted outliers fluctuates; above about 11 % they inflate sigma so
        # much that they no longer lie beyond three sigma, and the plane counts as normal)
        marked = (t["cls"][ch % 8 == 0] != fho.NORMAL).mean()
        assert marked == 1.0 if spec.shape[2] >= 56 else marked > 0.5
    # a plane without the planted outliers is outlier-rich only through sampling noise on small planes
    assert (t["cls"][ch % 8 != 0] == fho.NORMAL).mean() > (0.99 if spec.shape[2] >= 14 else 0.85)


@pytest.mark.parametrize("dtype", [synth.F32, synth.BF16])
@pytest.mark.parametrize("mib", [64, 256, 1024])
def test_config4_size_sweep_whole_tensors(mib, dtype):
    """The roofline sweep's tensors (32x32 planes, ReLU(N(0,1))), whole, at the smallest code width."""
    fho.set_threads(fho.max_threads())
    buf = _full_size(synth.config4(mib, dtype)[0], (2,))[2]
    h = fho.parse_header(buf)
    assert h["n_salient"] + h["n_raw"] < 1e-3 * h["n"] * h["c"]     # outlier-rich only by rare sampling noise


def test_config5_schedule_at_batch_128():
    """The 20 CIFAR-ResNet-shaped tensors at batch 128, every other one marked compress, through
    fh_run_schedule: arena bytes, footprint figures and restored values against the oracle."""
    import torch
    fho.set_threads(fho.max_threads())
    specs = synth.config5(128)
    p = api.default_params(bits=2)
    items, raws, restored, need = [], [], [], 0
    for i, s in enumerate(specs):
        raw = synth.make(s)
        raws.append(raw)
        dense = to_dev(raw)
        rest = torch.zeros_like(dense) if s.compress else None
        restored.append(rest)
        d = api.desc(s.shape, s.dtype, tensor_id=i)
        items.append(api.SchedItem(d, api.FH_COMPRESS if s.compress else api.FH_KEEP, dense, rest if rest is not None else dense))
        if s.compress:
            need += (api.compressed_bytes(d, p, 1) + 255) & ~255
    arena = torch.zeros(need, dtype=torch.uint8, device="cuda")
    rep = api.fh_run_schedule(items, p, arena)
    assert rep.status == api.FH_OK
    off = tot = 0
    for i, (s, raw, rest) in enumerate(zip(specs, raws, restored)):
        if not s.compress:
            continue
        d = fho.desc(s.shape, s.dtype, tensor_id=i)
        st, buf_o, total_o = fho.compress(raw, d, fho.params(bits=2))
        assert st == fho.OK
        assert np.array_equal(arena[off:off + total_o].cpu().numpy(), buf_o), f"container of tensor {i} differs"
        check_same_values(rest.cpu().numpy(), fho.decompress(buf_o, d)[1], s.dtype)
        tot += total_o
        off += (total_o + 255) & ~255
    assert rep.total_packed_bytes == tot and rep.peak_packed_bytes == off
    assert rep.total_dense_bytes == sum(s.dense_bytes for s in specs if s.compress)


def test_a_device_side_wait_that_runs_out_is_reported_and_leaves_the_library_usable():
    """Error path of the bounded device-side waits.  The placement of an outlier-rich plane waits, with a limit,
    until every earlier tile has published its size.  The fault is made on the host: one tile is told never to
    publish and the limit is shortened, so the wait of a later tile gives up and returns -- nothing traps or
    spins for ever.  The call must report FH_ERR_TIMEOUT, leave no valid header, and the next call on the same
    stream must be exact again."""
    import torch
    spec = synth.TensorSpec("t", (8, 32, 14, 14), synth.F32, "spiky_relu", 21)    # 256 planes in 8 tiles of 32
    raw = synth.make(spec)
    x = to_dev(raw)
    d = api.desc(spec.shape, spec.dtype)
    p = api.default_params(bits=2)
    cap = api.compressed_bytes(d, p, 1)
    st_o, buf_o, total_o = fho.compress(raw, fho.desc(spec.shape, spec.dtype), fho.params(bits=2))
    assert st_o == fho.OK and fho.parse_header(buf_o)["n_salient"] > 8
    dst = torch.zeros(cap, dtype=torch.uint8, device="cuda")
    out2 = torch.zeros(2, dtype=torch.int64, device="cuda")
    try:
        assert api.debug_set(api.FH_DEBUG_WAIT_POLLS, 2000) == api.FH_OK       # a fraction of a millisecond
        assert api.debug_set(api.FH_DEBUG_SILENT_TILE, 0) == api.FH_OK         # the first tile never publishes
        assert api.fh_compress(d, p, x, dst, out2, capacity=cap) == api.FH_OK
        torch.cuda.synchronize()
        assert int(out2[1]) == api.FH_ERR_TIMEOUT
        assert int(dst[:4].cpu().numpy().view(np.uint32)[0]) != 0x31434846       # no magic: not a valid container
        st = torch.zeros(1, dtype=torch.int64, device="cuda")
        rest = torch.empty_like(x)
        assert api.fh_decompress(dst, cap, d, rest, st) == api.FH_OK
        torch.cuda.synchronize()
        assert int(st[0]) == api.FH_ERR_CORRUPT
    finally:
        assert api.debug_set(api.FH_DEBUG_SILENT_TILE, 2 ** 64 - 1) == api.FH_OK
        assert api.debug_set(api.FH_DEBUG_WAIT_POLLS, 1 << 22) == api.FH_OK
    for _ in range(2):     # the scratch is clean: the same stream compresses exactly again
        dst.zero_()
        assert api.fh_compress(d, p, x, dst, out2, capacity=cap) == api.FH_OK
        torch.cuda.synchronize()
        assert out2.tolist() == [total_o, api.FH_OK]
        assert np.array_equal(dst[:total_o].cpu().numpy(), buf_o)
    assert api.debug_set(99, 0) == api.FH_ERR_ARG


def test_tensor_beyond_4_gib_on_sampled_planes():
    """A tensor a little over 4 GiB (byte offsets past 2^32, 2^30 elements): the oracle cannot take it whole
    in reasonable time, but planes are coded independently, so sampled planes -- the first, the last 64
    (which lie beyond 2^32 bytes) and a seeded random hundred -- are compared with the oracle run on just
    those planes: table entry, slot bytes and restored values.  Input: seeded normal draws on the device,
    ReLU'd; the oracle sees the very bytes copied back."""
    import torch
    P = (1 << 20) + 64
    shape = (P // 64, 64, 32, 32)
    gen = torch.Generator(device="cuda")
    gen.manual_seed(20251011)
    x = torch.empty(P * 1024, dtype=torch.float32, device="cuda")
    x.normal_(generator=gen)
    x.relu_()
    d = api.desc(shape, api.FH_F32)
    p = api.default_params(bits=2)
    st, packed, total = api.compress_tensor(x, shape, api.FH_F32, p)
    assert st == api.FH_OK
    hdr = packed[:64].cpu().numpy()
    assert int(hdr[56:64].view(np.uint64)[0]) == total
    npay, slots = 256, 64 + 16 * P
    assert total >= slots + P * npay
    rng = np.random.default_rng(7)
    idx = np.unique(np.concatenate([np.arange(4), np.arange(P - 64, P), rng.integers(0, P, 100)]))
    sample = x.view(P, 1024)[torch.from_numpy(idx).cuda()].cpu().numpy().reshape(-1)
    st_o, buf_o, total_o, d_o = oracle_compress(sample, (1, len(idx), 32, 32), synth.F32, bits=2)
    assert st_o == fho.OK
    to = hp.table(buf_o, len(idx))
    tab = packed[64:64 + 16 * P].view(torch.int32).view(P, 4)[torch.from_numpy(idx).cuda()].cpu().numpy().view(np.uint32)
    assert np.array_equal(tab[:, 1] & 3, to["cls"]) and np.array_equal(tab[:, 1] >> 2, to["n_out"])
    st_d, out = api.decompress_tensor(packed, total, shape, api.FH_F32)
    assert st_d == api.FH_OK
    _, out_o = fho.decompress(buf_o, d_o)
    got = out.view(P, 1024)[torch.from_numpy(idx).cuda()].cpu().numpy().reshape(-1)
    check_same_values(got, out_o, synth.F32)
    slots_o = 64 + 16 * len(idx)
    for k, pl in enumerate(idx):
        if to["cls"][k] != fho.NORMAL:
            continue
        assert tab[k, 0] * 16 == slots + int(pl) * npay
        assert np.array_equal(tab[k, 2:4], np.stack([to["lo"][k:k + 1].view(np.uint32), to["scale"][k:k + 1].view(np.uint32)], 1)[0])
        a0 = slots + int(pl) * npay
        assert np.array_equal(packed[a0:a0 + npay].cpu().numpy(), buf_o[slots_o + k * npay: slots_o + (k + 1) * npay])
    # every zero of a post-ReLU plane comes back as zero (normal planes have lo = 0; the block-wise path keeps zeros)
    probe = torch.from_numpy(idx[:32]).cuda()
    assert bool(((x.view(P, 1024)[probe] == 0) <= (out.view(P, 1024)[probe] == 0)).all())


@pytest.mark.parametrize("shape", [(3, 5, 7, 7), (2, 9, 14, 14), (1, 12, 32, 32), (2, 8, 28, 28), (1, 6, 56, 56), (1, 3, 112, 112),
                                   (2, 6, 33, 17), (300, 1, 4, 4)])
@pytest.mark.parametrize("dtype", [synth.F32, synth.BF16])
@pytest.mark.parametrize("bits", [2, 4, 8])
def test_parity_random_rounding(shape, dtype, bits):
    """rounding = 1: the draws come from the same counter-based generator on both sides, so the container
    is still identical byte for byte (normal planes carry randomly rounded codes, outlier-rich planes are
    coded as before)."""
    kind = "spiky_relu" if shape[1] >= 3 else "relu"
    spec = synth.TensorSpec("t", shape, dtype, kind, 60 + bits)
    raw = synth.make(spec)
    kw = dict(bits=bits, rounding=1, seed=0x1234567887654321 + bits)
    st_o, buf_o, total_o = fho.compress(raw, fho.desc(shape, dtype, tensor_id=0xABCDEF0123), fho.params(**kw))
    assert st_o == fho.OK and fho.parse_header(buf_o)["rounding"] == 1
    p = api.default_params(**kw)
    st_g, packed, total_g = api.compress_tensor(to_dev(raw), shape, dtype, p, tensor_id=0xABCDEF0123)
    assert st_g == api.FH_OK and total_g == total_o
    assert np.array_equal(packed[:total_g].cpu().numpy(), buf_o)
    st_d, out_g = api.decompress_tensor(packed, total_g, shape, dtype)
    assert st_d == api.FH_OK
    _, out_o = fho.decompress(buf_o, fho.desc(shape, dtype))
    got = out_g.cpu().numpy()
    check_same_values(got.view(np.uint16) if dtype == synth.BF16 else got, out_o, dtype)
    # another seed gives other codes
    st_2, packed2, _ = api.compress_tensor(to_dev(raw), shape, dtype, api.default_params(bits=bits, rounding=1, seed=5), tensor_id=0xABCDEF0123)
    assert st_2 == api.FH_OK and not np.array_equal(packed2[:total_g].cpu().numpy(), buf_o)


def test_generated_plan_drives_the_schedule():
    """Algorithm 1 end to end: the costs of compression are measured from this library on this device
    (fh_plan_measure: PC, RC and the freed space of Eq. 5), a plan is generated for one training step under a
    memory budget (recomputation costs made up), and its per-tensor actions are what fh_run_schedule executes."""
    import torch
    shapes = [(8, 32, 32, 32), (8, 32, 32, 32), (8, 64, 16, 16), (8, 64, 16, 16), (8, 128, 8, 8), (8, 128, 8, 8)]
    specs = [synth.TensorSpec(f"p{i}", sh, synth.F32, "relu", 700 + i) for i, sh in enumerate(shapes)]
    n = len(specs)
    p = api.default_params(bits=2)
    raws = [synth.make(sp) for sp in specs]
    dense = [to_dev(r) for r in raws]
    descs = [api.desc(sp.shape, sp.dtype, tensor_id=sp.seed) for sp in specs]
    work = torch.empty(max(api.host_work_bytes(d, p) for d in descs), dtype=torch.uint8, device="cuda")
    rc, tensors = api.plan_measure(descs, p, dense, work, repeats=5, t_recompute=[(10e-6 if i == 1 else 400e-6) for i in range(n)])
    assert rc == api.FH_OK
    for t, sp, d in zip(tensors, specs, descs):
        st_o, _, total_o = fho.compress(synth.make(sp), fho.desc(sp.shape, sp.dtype, tensor_id=sp.seed), fho.params(bits=2))
        assert st_o == fho.OK and t["bytes"] == sp.dense_bytes and t["packed_bytes"] == total_o
        assert 1e-6 < t["t_compress"] < 1e-3 and 1e-6 < t["t_decompress"] < 1e-3
    ops = [dict(time=100e-6, inputs=[k - 1] if k else [], outputs=[k]) for k in range(n)]
    ops += [dict(time=200e-6, inputs=[k], outputs=[]) for k in reversed(range(n))]
    budget = int(0.6 * sum(t["bytes"] for t in tensors))
    rc, actions, events, rep = api.plan_generate(ops, tensors, budget)
    assert rc == api.FH_OK and rep.peak_bytes < budget
    assert api.FH_COMPRESS in actions and api.FH_EVICT in actions       # the hybrid: both techniques get used
    items, rest = [], []
    for sp, act, dn, dsc in zip(specs, actions, dense, descs):
        out = torch.zeros_like(dn)
        rest.append(out)
        items.append(api.SchedItem(dsc, act, dn, out))
    arena = torch.zeros(4 << 20, dtype=torch.uint8, device="cuda")
    srep = api.fh_run_schedule(items, p, arena)
    assert srep.status == api.FH_OK
    assert srep.total_dense_bytes == sum(t["bytes"] for t, a in zip(tensors, actions) if a == api.FH_COMPRESS)
    for sp, raw, out, act in zip(specs, raws, rest, actions):
        if act != api.FH_COMPRESS:
            assert not bool(out.any())
            continue
        d = fho.desc(sp.shape, sp.dtype, tensor_id=sp.seed)
        _, buf_o, _ = fho.compress(raw, d, fho.params(bits=2))
        check_same_values(out.cpu().numpy(), fho.decompress(buf_o, d)[1], sp.dtype)


@pytest.mark.parametrize("shape", [(6, 20, 14, 14), (3, 5, 7, 7), (4, 12, 32, 32), (5, 8, 28, 28), (3, 6, 56, 56), (2, 3, 112, 112),
                                   (4, 6, 33, 17), (40, 7, 4, 4)])
@pytest.mark.parametrize("dtype", [synth.F32, synth.BF16])
def test_parity_channel_wide_three_sigma(shape, dtype):
    """salient_mode = CHANNEL: statistics and class per channel over the batch; container identical to the
    oracle's, and every channel is normal or outlier-rich as a whole."""
    for kind, bits in (("spiky_relu", 2), ("laplace_ch", 8)):
        spec = synth.TensorSpec("t", shape, dtype, kind, 83)
        buf = full_parity(spec, bits=bits, salient_mode=api.FH_SALIENT_CHANNEL)
        cls = hp.table(buf, shape[0] * shape[1])["cls"].reshape(shape[0], shape[1])
        assert ((cls != fho.NORMAL).all(0) | (cls == fho.NORMAL).all(0)).all()
    assert fho.parse_header(buf)["salient_mode"] == fho.CHANNEL


@pytest.mark.parametrize("shape", [(6, 20, 14, 14), (3, 5, 7, 7), (4, 12, 32, 32), (5, 8, 28, 28), (3, 6, 56, 56), (2, 3, 112, 112),
                                   (4, 6, 33, 17), (40, 7, 4, 4)])
@pytest.mark.parametrize("dtype", [synth.F32, synth.BF16])
def test_parity_tensor_wide_three_sigma(shape, dtype):
    """salient_mode = TENSOR: thresholds from the whole tensor's mu and sigma, class by each plane's own count;
    container identical to the oracle's, both classes present on the spiky data."""
    for kind, bits in (("spiky_relu", 2), ("laplace_ch", 8)):
        spec = synth.TensorSpec("t", shape, dtype, kind, 84)
        buf = full_parity(spec, bits=bits, salient_mode=api.FH_SALIENT_TENSOR)
        t = hp.table(buf, shape[0] * shape[1])
        assert ((t["cls"] != fho.NORMAL) == (t["n_out"].astype(np.int64) * 32 > shape[2] * shape[3])).all()
    assert fho.parse_header(buf)["salient_mode"] == fho.TENSOR
