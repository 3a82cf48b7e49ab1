"""Pins of the oracle's Huffman stage on the dense-block residual codes (Section 4.4.1: "a Huffman tree is
constructed from the quantization array for encoding"; "Decompression involves Huffman decoding").

Nothing here touches the CUDA path.  The pins: a hand-built case, Kraft equality, prefix-freeness, optimality
against an independent textbook construction, the stated tie-break, the stream's size against the sum of the
code lengths, losslessness of the stage, and rejection of damaged sections."""
import heapq
import os

import numpy as np
import pytest

from oracle import fho
from paper_2510_11400_b200 import synth
from tests import helpers as hp

GOLD = os.path.join(os.path.dirname(__file__), "golden", "hand_cases.txt")


def golden(name):
    for line in open(GOLD):
        if line.startswith(name):
            return [s.strip() for s in line.split("|")][1:]
    raise KeyError(name)


def hist_of(pairs):
    h = [0] * 256
    for sym, cnt in pairs:
        h[sym] = cnt
    return h


def test_hand_case_four_symbols():
    inp, exp = golden("huffman_four")
    pairs = [tuple(int(v) for v in tok.split(":")) for tok in inp.split()]
    toks = exp.split()
    want_len = [int(v) for v in toks[1:5]]
    want_code = toks[6:10]
    lens = fho.huffman_lengths(hist_of(pairs))
    codes = fho.canonical_codes(lens)
    assert [lens[s] for s, _ in pairs] == want_len
    assert [format(codes[s], "0%db" % lens[s]) for s, _ in pairs] == want_code
    assert sum(c * lens[s] for s, c in pairs) == int(toks[-1])
    assert sum(lens) == sum(want_len)            # symbols that do not occur get no code


def textbook_cost(hist):
    """Total code length of an optimal prefix code by the textbook heap construction (any tie-break gives the
    same total)."""
    heap = [w for w in hist if w]
    if len(heap) == 1:
        return heap[0]
    heapq.heapify(heap)
    cost = 0
    while len(heap) > 1:
        a, b = heapq.heappop(heap), heapq.heappop(heap)
        cost += a + b
        heapq.heappush(heap, a + b)
    return cost


@pytest.mark.parametrize("seed", range(20))
def test_lengths_are_optimal_complete_and_prefix_free(seed):
    rng = np.random.default_rng(seed)
    n = int(rng.integers(2, 200))
    syms = rng.choice(256, n, replace=False)
    kind = seed % 4
    w = {0: rng.integers(1, 5, n), 1: rng.integers(1, 10000, n), 2: (2.0 ** rng.integers(0, 14, n)).astype(np.int64),
         3: np.maximum(1, (3000 * np.exp(-0.5 * ((np.arange(n) - n / 2) / 3.0) ** 2)).astype(np.int64))}[kind]   # like residuals around 128
    hist = hist_of(zip(syms.tolist(), [int(v) for v in w]))
    lens = fho.huffman_lengths(hist)
    assert all((lens[s] > 0) == (hist[s] > 0) for s in range(256))
    from fractions import Fraction
    assert sum(Fraction(1, 2 ** l) for l in lens if l) == 1                     # Kraft equality: the tree is complete
    assert sum(hist[s] * lens[s] for s in range(256)) == textbook_cost(hist)    # as short as any prefix code can be
    codes = fho.canonical_codes(lens)
    words = sorted(format(codes[s], "0%db" % lens[s]) for s in range(256) if lens[s])
    assert len(set(words)) == len(words)
    assert not any(b.startswith(a) for a, b in zip(words, words[1:]))           # sorted: a prefix would be adjacent
    # canonical: by (length, symbol) the code values increase, and only the lengths were needed to make them
    order = sorted((lens[s], s) for s in range(256) if lens[s])
    vals = [codes[s] << (32 - l) for l, s in order]
    assert vals == sorted(vals)


def test_tie_break_and_degenerate_histograms():
    # equal weights: nodes are ordered by (weight, id), a leaf's id is its symbol, a merged node's 256 + its order
    lens = fho.huffman_lengths(hist_of([(5, 1), (9, 1), (200, 1)]))
    assert (lens[5], lens[9], lens[200]) == (2, 2, 1)          # 5 and 9 are merged first; 200 then meets the merged node
    # a leaf that ties with a merged node goes first (its id is smaller): weights 1, 1, 2, 2 give the balanced
    # tree, not the chain 3, 3, 2, 1 of the same cost
    lens = fho.huffman_lengths(hist_of([(1, 1), (2, 1), (3, 2), (4, 2)]))
    assert [lens[s] for s in (1, 2, 3, 4)] == [2, 2, 2, 2]
    lens = fho.huffman_lengths(hist_of([(1, 7), (2, 7), (3, 7), (4, 7)]))
    assert [lens[s] for s in (1, 2, 3, 4)] == [2, 2, 2, 2]
    lens = fho.huffman_lengths(hist_of([(77, 12)]))
    assert lens[77] == 1 and sum(lens) == 1                     # a single symbol still takes one bit
    assert sum(fho.huffman_lengths([0] * 256)) == 0
    # Fibonacci weights give the deepest tree: depth stays far below the limit of 24 for any plane size
    fib = [1, 1]
    while len(fib) < 20:
        fib.append(fib[-1] + fib[-2])
    lens = fho.huffman_lengths(hist_of(list(enumerate(fib, start=1))))
    assert max(lens) == 19 and sum(fib) < 2 ** 17


def coded_planes(buf, P, H, W, esize):
    """(plane, section size, parsed header) of every plane whose dense section went through the Huffman stage."""
    t = hp.table(buf, P)
    out = []
    for pl in np.flatnonzero(t["cls"] == fho.SALIENT):
        pay = hp.logical_payload(buf, P, int(pl), H * W)
        hdr = np.ascontiguousarray(pay[:16]).view(np.uint32)
        if hdr[3]:
            out.append((int(pl), int(hdr[3]), pay))
    return out


@pytest.mark.parametrize("dtype", [fho.F32, fho.BF16])
@pytest.mark.parametrize("shape,eps,kind,mode", [((2, 16, 28, 28), 0.0625, "spiky_relu", fho.AUTO),
                                                 ((1, 16, 56, 56), 0.25, "spiky_relu", fho.AUTO),
                                                 ((2, 4, 14, 14), 0.25, "relu", fho.ALL),      # every block dense
                                                 ((1, 16, 33, 17), 0.25, "relu", fho.ALL)])
def test_stage_is_lossless_never_larger_and_its_stream_has_the_stated_size(shape, eps, kind, mode, dtype):
    spec = synth.TensorSpec("t", shape, dtype, kind, 50)
    raw = synth.make(spec)
    d = fho.desc(shape, dtype)
    st0, plain, _ = fho.compress(raw, d, fho.params(bits=4, eps=eps, entropy=0, salient_mode=mode))
    st1, coded, _ = fho.compress(raw, d, fho.params(bits=4, eps=eps, entropy=1, salient_mode=mode))
    assert st0 == st1 == fho.OK
    assert fho.parse_header(plain)["version"] == 1 and fho.parse_header(coded)["version"] == 2
    assert coded.size <= plain.size
    # the stage is lossless: both containers restore the same values
    _, a = fho.decompress(plain, d)
    _, b = fho.decompress(coded, d)
    assert np.array_equal(a, b)
    n, c, H, W = shape
    esize = 4 if dtype == fho.F32 else 2
    planes = coded_planes(coded, n * c, H, W, esize)
    assert planes, "no plane took the stage: the case does not test it"
    for pl, sec_bytes, pay in planes:
        ref = hp.salient_plane(plain, n * c, pl, H, W, esize)             # the same plane with plain code bytes
        nnz_s, n_dense = ref["nnz_s"], ref["n_dense"]
        nblk = ((H + 7) // 8) * ((W + 7) // 8)
        off = 16 + 4 * ((nblk + 31) // 32) + 4 * (H + 1) + hp.a4(2 * nnz_s) + hp.a4(esize * nnz_s)
        sec = pay[off:off + sec_bytes]
        assert sec_bytes < 64 * n_dense and sec_bytes % 4 == 0
        # lengths as stored, against those of the plane's own histogram
        symbols = ref["codes"].reshape(n_dense, 64)
        hist = np.bincount(symbols.reshape(-1), minlength=256)
        lens = fho.huffman_lengths(hist.tolist())
        smin, smax = int(sec[1]), int(sec[2])
        present = [s for s in range(1, 256) if lens[s]]
        assert (smin, smax) == ((present[0], present[-1]) if present else (1, 1))
        assert int(sec[0]) == lens[0] and [int(v) for v in sec[4:4 + smax - smin + 1]] == lens[smin:smax + 1]
        # every chunk takes ceil(sum of its symbols' code lengths / 8) bytes, and the section nothing else
        chunk = sec[4 + hp.a4(smax - smin + 1):][:n_dense].astype(np.int64)
        want = [(int(sum(lens[s] for s in symbols[b])) + 7) // 8 for b in range(n_dense)]
        assert chunk.tolist() == want
        assert sec_bytes == hp.a4(4 + hp.a4(smax - smin + 1) + hp.a4(n_dense) + sum(want))
        # first chunk, bit by bit
        codes = fho.canonical_codes(lens)
        bits = "".join(format(codes[s], "0%db" % lens[s]) for s in symbols[0])
        start = 4 + hp.a4(smax - smin + 1) + hp.a4(n_dense)
        got = "".join(format(int(v), "08b") for v in sec[start:start + want[0]])
        assert got[:len(bits)] == bits and set(got[len(bits):]) <= {"0"}


def test_planes_that_gain_nothing_keep_their_plain_codes():
    """A plane whose residuals are spread evenly over many values: the table and the chunk lengths cost more
    than the code saves, the section is not used, and the payload is that of entropy = 0."""
    rng = np.random.default_rng(9)
    x = (rng.integers(-100, 100, (1, 1, 8, 8)) * 0.125).astype(np.float32)      # one dense block of unrelated values
    d = fho.desc((1, 1, 8, 8), fho.F32)
    a = fho.compress(x.reshape(-1), d, fho.params(bits=2, salient_mode=fho.ALL, eps=0.0625, entropy=0))[1]
    b = fho.compress(x.reshape(-1), d, fho.params(bits=2, salient_mode=fho.ALL, eps=0.0625, entropy=1))[1]
    assert a.size == b.size and b[4] == 2 and a[4] == 1
    a2, b2 = a.copy(), b.copy()
    a2[4] = b2[4] = 0
    assert np.array_equal(a2, b2)


def test_damaged_sections_are_rejected():
    spec = synth.TensorSpec("t", (1, 16, 28, 28), fho.F32, "relu", 51)
    raw = synth.make(spec)
    d = fho.desc(spec.shape, fho.F32)
    st, buf, _ = fho.compress(raw, d, fho.params(bits=4, entropy=1, eps=0.25, salient_mode=fho.ALL))
    assert st == fho.OK
    pl, sec_bytes, pay = coded_planes(buf, 16, 28, 28, 4)[0]
    assert fho.decompress(buf, d)[0] == fho.OK
    slots = 64 + 16 * 16
    npay = hp.npay_of(buf, 28 * 28)
    hdr_at = slots + pl * npay
    # a version-1 header must not carry coded sections
    b = buf.copy(); b[4] = 1
    assert fho.decompress(b, d)[0] == fho.ERR_CORRUPT
    # a section size that is not smaller than the plain codes, or not a multiple of four
    for bad in (0x7FFFFFF0, sec_bytes + 1):
        b = buf.copy()
        b[hdr_at + 12:hdr_at + 16] = np.frombuffer(np.uint32(bad).tobytes(), dtype=np.uint8)
        assert fho.decompress(b, d)[0] == fho.ERR_CORRUPT
    # code lengths that do not form a complete code
    nnz_s = int(np.ascontiguousarray(pay[:4]).view(np.uint32)[0])
    off = 16 + 4 * 1 + 4 * 29 + hp.a4(2 * nnz_s) + hp.a4(4 * nnz_s)          # 16 blocks -> one bitmap word
    # the section starts `off` bytes into the payload; find it in the container (slot, then overflow part)
    t_off = int(hp.table(buf, 16)["off"][pl])
    at = hdr_at + off if off < npay else t_off + (off - npay)
    b = buf.copy()
    b[at] = (int(b[at]) + 1) % 25                                            # the length of symbol 0
    assert fho.decompress(b, d)[0] == fho.ERR_CORRUPT
