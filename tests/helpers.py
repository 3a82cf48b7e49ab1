"""Container readers used by the tests (layout knowledge only, no codec arithmetic)."""
import numpy as np


def a4(x):
    return (x + 3) & ~3


def a16(x):
    return (x + 15) & ~15


def table(buf, P):
    t = np.ascontiguousarray(buf[64:64 + 16 * P]).view(np.uint32).reshape(P, 4)
    return dict(off=t[:, 0].astype(np.int64) * 16, cls=(t[:, 1] & 3).astype(np.int64),
                n_out=(t[:, 1] >> 2).astype(np.int64), lo=t[:, 2].copy().view(np.float32),
                scale=t[:, 3].copy().view(np.float32))


def normal_codes(buf, off, hw, bits):
    nwords = (hw * bits + 31) // 32
    w = np.ascontiguousarray(buf[off:off + 4 * nwords]).view(np.uint32)
    i = np.arange(hw, dtype=np.int64) * bits
    return ((w[i // 32] >> (i % 32).astype(np.uint32)) & np.uint32((1 << bits) - 1)).astype(np.int64)


def npay_of(buf, hw):
    """Slot size of a container: A16(4 * ceil(HW * bits / 32)), bits from the header."""
    bits = int(buf[7])
    return a16(4 * ((hw * bits + 31) // 32))


def logical_payload(buf, P, pl, hw):
    """Payload bytes of a salient or raw plane: its slot followed by its continuation in the
    overflow region (returned up to the end of the container; callers parse what they need)."""
    npay = npay_of(buf, hw)
    slots = 64 + 16 * P
    slot = buf[slots + pl * npay: slots + (pl + 1) * npay]
    off = int(table(buf, P)["off"][pl])
    if off == 0:
        return np.concatenate([slot, np.zeros(16, dtype=np.uint8)])
    return np.concatenate([slot, buf[off:], np.zeros(16, dtype=np.uint8)])


def salient_plane(buf, P, pl, H, W, esize):
    return salient(logical_payload(buf, P, pl, H * W), 0, H, W, esize)


def salient(buf, off, H, W, esize):
    """Split a salient payload (contiguous bytes) into its sections."""
    nblk = ((H + 7) // 8) * ((W + 7) // 8)
    nbm = (nblk + 31) // 32
    hdr = np.ascontiguousarray(buf[off:off + 16]).view(np.uint32)
    nnz_s, n_dense, n_out_d = int(hdr[0]), int(hdr[1]), int(hdr[2])
    p = off + 16
    bm = np.ascontiguousarray(buf[p:p + 4 * nbm]).view(np.uint32)
    p += 4 * nbm
    dense = np.array([(bm[b // 32] >> (b % 32)) & 1 for b in range(nblk)], dtype=np.int64)
    row_ptr = np.ascontiguousarray(buf[p:p + 4 * (H + 1)]).view(np.uint32).astype(np.int64)
    p += 4 * (H + 1)
    col = np.ascontiguousarray(buf[p:p + 2 * nnz_s]).view(np.uint16).astype(np.int64)
    p += a4(2 * nnz_s)
    val = np.ascontiguousarray(buf[p:p + esize * nnz_s]).view(np.uint32 if esize == 4 else np.uint16)
    p += a4(esize * nnz_s)
    codes = np.ascontiguousarray(buf[p:p + 64 * n_dense]).reshape(n_dense, 8, 8).astype(np.int64)
    p += 64 * n_dense
    outl = np.ascontiguousarray(buf[p:p + esize * n_out_d]).view(np.uint32 if esize == 4 else np.uint16)
    p += a4(esize * n_out_d)
    return dict(nnz_s=nnz_s, n_dense=n_dense, n_out_d=n_out_d, dense=dense, row_ptr=row_ptr, col=col,
                val=val, codes=codes, outl=outl, size=p - off, pad=int(hdr[3]))
