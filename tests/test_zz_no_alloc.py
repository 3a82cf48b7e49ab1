"""fh_compress_static: the compress entry point that allocates nothing.

It serves callers that cannot call cudaMalloc when they need the codec -- an engine that compresses
because its device-memory budget is already spent, a process whose memory is wholly held by a
framework pool, a loop that cannot take the synchronisation an allocation may imply.  Its
book-keeping scratch is a fixed array inside the library, shared by all calls on a device and cleared
by each call.  The test drives it through the C ABI and requires the same container, byte for byte, as
fh_compress and as the CPU oracle, twice in a row (the second call sees the first call's leftovers in
the array), and checks that a tensor beyond the fixed limit is refused.

Collected last on purpose, and self-contained: it must pass alone in a fresh process and after the
other GPU tests.
"""
import numpy as np
import pytest

from oracle import fho
from paper_2510_11400_b200 import api, build, synth

pytestmark = pytest.mark.gpu


def _compress_both(spec, bits):
    import torch
    raw = synth.make(spec)
    x = torch.from_numpy(raw.view(np.int16) if raw.dtype == np.uint16 else raw).cuda()
    d = api.desc(spec.shape, spec.dtype, tensor_id=7)
    p = api.default_params(bits=bits)
    cap = api.compressed_bytes(d, p, 1)
    outs = []
    for fn in (api.fh_compress, api.fh_compress_static):
        dst = torch.full((cap,), 0x5A, dtype=torch.uint8, device="cuda")
        out2 = torch.full((2,), -1, dtype=torch.int64, device="cuda")
        assert fn(d, p, x, dst, out2, capacity=cap) == api.FH_OK
        torch.cuda.synchronize()
        total, st = out2.tolist()
        assert st == api.FH_OK
        outs.append(dst[:total].cpu().numpy())
    st_o, buf_o, total_o = fho.compress(raw, fho.desc(spec.shape, spec.dtype, tensor_id=7), fho.params(bits=bits))
    assert st_o == fho.OK and np.array_equal(outs[1], buf_o), "fh_compress_static differs from the oracle"
    return outs


def test_static_scratch_entry_point_matches_fh_compress_on_two_calls_in_a_row():
    build.build()
    api.lib()
    # first call: many planes of mixed classes, so the placement words of the fixed scratch are really used
    a = synth.TensorSpec("za", (64, 48, 14, 14), synth.F32, "spiky_relu", 5)
    ref, got = _compress_both(a, 2)
    assert ref.size == got.size and np.array_equal(ref, got)
    # second call, right after: fewer, larger planes over the same array
    b = synth.TensorSpec("zb", (8, 24, 56, 56), synth.BF16, "laplace_ch", 6)
    ref, got = _compress_both(b, 8)
    assert ref.size == got.size and np.array_equal(ref, got)
    # and the first tensor again: identical bytes to the first time
    ref2, got2 = _compress_both(a, 2)
    assert np.array_equal(got2, ref2)


def test_static_scratch_entry_point_refuses_tensors_beyond_its_limit():
    import torch
    build.build()
    planes = api.FH_STATIC_MAX_PLANES + 64           # one batch row more than the fixed scratch holds
    d = api.desc((planes // 64, 64, 4, 4), api.FH_F32)
    p = api.default_params(bits=2)
    x = torch.zeros(planes * 16, dtype=torch.float32, device="cuda")
    dst = torch.empty(api.compressed_bytes(d, p, 1), dtype=torch.uint8, device="cuda")
    assert api.fh_compress_static(d, p, x, dst, None) == api.FH_ERR_UNSUPPORTED
    assert api.fh_compress(d, p, x, dst, None) == api.FH_OK   # the allocating entry point takes it
    torch.cuda.synchronize()
    api.shutdown()
