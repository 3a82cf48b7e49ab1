// Compress kernels: one pass over the dense tensor.
//
// Container recap: every plane owns a slot of npay bytes at a closed-form offset; a normal plane's
// codes fill its slot; the payload of a salient or raw plane runs through its slot and continues in
// the overflow region, in plane order.  Normal planes therefore never wait for anything: statistics,
// class, codes and the stores happen in one sweep.  Only tiles that hold salient or raw planes need
// their place in the overflow region, which a decoupled look-back over per-tile scan words supplies.
//
// Two kernels share this file:
//   compress_fast<DT, SIGMA, G, CTA>  planes whose size is a multiple of 16 bytes and that fit the
//       register budget: tiles stream into shared memory through a multi-stage bulk-copy (TMA)
//       pipeline, every thread keeps its G groups in registers for all passes;
//   compress_generic<DT, BITS>        everything else (ragged planes, very large planes): staged with
//       plain loads, passes re-read shared memory.
#pragma once

#include "fh_device.cuh"

namespace fh {

struct SalientInfo {
  uint32_t nnz_s, n_dense, n_out_d, size;
};

struct CompressArgs {
  const uint8_t* src;
  uint8_t* dst_base;
  unsigned long long capacity;          // bytes available at dst_base (minus the offset below)
  const unsigned long long* d_off_in;   // optional: byte offset of the container in dst_base
  unsigned long long* d_off_out;        // optional: offset for the next container
  unsigned long long* out2;             // optional: {total bytes, status}
  Scratch* sc;
  ScanState scan;                       // scan words (tiles, segments), epoch, wait bound
  uint32_t nseg;                        // segments of this call (for the final clean-up)
};

// Where the bytes of a salient / raw payload go: offsets below npay land in the plane's slot, the
// rest in its overflow part.  Offsets and npay are multiples of the access size.
struct SplitOut {
  uint8_t* slot;
  uint8_t* ovf;
  uint32_t npay;
  __device__ __forceinline__ uint8_t* at(uint32_t o) const { return o < npay ? slot + o : ovf + (o - npay); }
  __device__ __forceinline__ void st32(uint32_t o, uint32_t v) const { *reinterpret_cast<uint32_t*>(at(o)) = v; }
  __device__ __forceinline__ void st16(uint32_t o, uint32_t v) const { *reinterpret_cast<uint16_t*>(at(o)) = (uint16_t)v; }
};

// Pre-quantised integer of the element at (y, x); positions outside the plane count as value 0.
template <int DT>
__device__ __forceinline__ int32_t plane_k(const uint8_t* plane, int H, int W, int y, int x, float inv2e, bool* big) {
  const float v = (y < H && x < W) ? load_elem<DT>(plane, (uint32_t)y * (uint32_t)W + (uint32_t)x) : 0.0f;
  return dense_k(v, inv2e, big);
}

// Residual codes of one dense 8x8 block (Eq. 7-9), by all 32 lanes of a warp: first-order Lorenzo
// prediction on the pre-quantised integers k, neighbours outside the block count as 0.  Every element
// is independent because prediction runs on k, which follows from the input alone.  Lane l takes the
// elements l and l + 32 of the block's raster order.  Returns the number of verbatim elements.
// WRITE: also emits the 64 code bytes (logical offset o_codes) and the verbatim values (from logical
// offset o_outl, raster order).
template <int DT, bool WRITE>
__device__ __forceinline__ uint32_t block_codes_warp(const uint8_t* plane, int H, int W, int by, int bx, float inv2e,
                                                     const SplitOut& out, uint32_t o_codes, uint32_t o_outl) {
  const uint32_t lane = threadIdx.x & 31u;
  const int j = (int)(lane & 7u);
  uint32_t n_out = 0;
#pragma unroll
  for (int half = 0; half < 2; ++half) {
    const int i = half * 4 + (int)(lane >> 3);
    const int y = by * 8 + i, x = bx * 8 + j;
    const bool inpl = (y < H) && (x < W);
    bool big, nb;
    const int32_t k = plane_k<DT>(plane, H, W, y, x, inv2e, &big);
    const int32_t up = i > 0 ? plane_k<DT>(plane, H, W, y - 1, x, inv2e, &nb) : 0;
    const int32_t left = j > 0 ? plane_k<DT>(plane, H, W, y, x - 1, inv2e, &nb) : 0;
    const int32_t ul = (i > 0 && j > 0) ? plane_k<DT>(plane, H, W, y - 1, x - 1, inv2e, &nb) : 0;
    const int32_t delta = k - (up + left - ul);
    const bool verbatim = inpl && (big || delta > 127 || delta < -127);
    const uint32_t code = !inpl ? 128u : (verbatim ? 0u : (uint32_t)(delta + 128));
    const uint32_t m = __ballot_sync(0xFFFFFFFFu, verbatim);
    if (WRITE) {
      if (verbatim) {
        const uint32_t rank = n_out + __popc(m & ((1u << lane) - 1u));
        const uint32_t idx = (uint32_t)y * (uint32_t)W + (uint32_t)x;
        if (DT == kF32) out.st32(o_outl + 4u * rank, reinterpret_cast<const uint32_t*>(plane)[idx]);
        else out.st16(o_outl + 2u * rank, reinterpret_cast<const uint16_t*>(plane)[idx]);
      }
      uint32_t w = code | (__shfl_down_sync(0xFFFFFFFFu, code, 1) << 8);
      w |= __shfl_down_sync(0xFFFFFFFFu, w, 2) << 16;
      if ((lane & 3u) == 0u) out.st32(o_codes + (uint32_t)half * 32u + lane, w);
    }
    n_out += __popc(m);
  }
  return n_out;
}

// Block-wise path, measuring part (Section 4.4.1): non-zero mask pooled per 8x8 block against tau,
// CSR row counts over the sparse blocks, verbatim counts of the dense blocks.  The team is a whole
// warp or a whole CTA.  Leaves in shared scratch: rowp[0..H] = CSR row pointers, blk_a[b] = 1 for
// dense blocks, blk_b[b] = rank of block b among the dense blocks, blk_c[b] = index of the block's
// first verbatim value.
template <int DT>
__device__ __noinline__ SalientInfo salient_measure(const Team& t, const Plan& pl, const uint8_t* plane, uint32_t* sal) {
  uint32_t* rowp = sal;
  uint32_t* blk_a = sal + pl.H + 1;
  uint32_t* blk_b = blk_a + pl.nblk;
  uint32_t* blk_c = blk_b + pl.nblk;
  const int H = pl.H, W = pl.W;
  const uint32_t nblk = pl.nblk, nbx = pl.nbx;
  const uint32_t nw = t.block ? t.nwarps : 1u, wid = t.block ? threadIdx.x >> 5 : 0u, lane32 = threadIdx.x & 31u;
  for (uint32_t b = t.lane; b < nblk; b += t.size) blk_a[b] = 0;
  for (uint32_t y = t.lane; y <= (uint32_t)H; y += t.size) rowp[y] = 0;
  team_sync(t);
  // pooled mask: non-zero count per block, accumulated from (block, row) items
  for (uint32_t r = t.lane; r < nblk * 8u; r += t.size) {
    const uint32_t b = r >> 3, i = r & 7u;
    const int y = (int)(b / nbx) * 8 + (int)i, x0 = (int)(b % nbx) * 8;
    if (y < H) {
      uint32_t cnt = 0;
      const int x1 = min(W, x0 + 8);
      for (int x = x0; x < x1; ++x) cnt += load_elem<DT>(plane, (uint32_t)y * W + x) != 0.0f;
      if (cnt) atomicAdd(&blk_a[b], cnt);
    }
  }
  team_sync(t);
  for (uint32_t b = t.lane; b < nblk; b += t.size) {
    const uint32_t dense = (uint64_t)blk_a[b] * pl.tau_den >= (uint64_t)pl.tau_num * 64u;
    blk_a[b] = dense;
    blk_b[b] = dense;
  }
  team_sync(t);
  SalientInfo info;
  info.n_dense = team_excl_scan(t, blk_b, nblk);
  // CSR row counts: non-zeros of the sparse blocks, again from (block, row) items
  for (uint32_t r = t.lane; r < nblk * 8u; r += t.size) {
    const uint32_t b = r >> 3, i = r & 7u;
    const int y = (int)(b / nbx) * 8 + (int)i, x0 = (int)(b % nbx) * 8;
    if (y < H && !blk_a[b]) {
      uint32_t cnt = 0;
      const int x1 = min(W, x0 + 8);
      for (int x = x0; x < x1; ++x) cnt += load_elem<DT>(plane, (uint32_t)y * W + x) != 0.0f;
      if (cnt) atomicAdd(&rowp[y], cnt);
    }
  }
  team_sync(t);
  info.nnz_s = team_excl_scan(t, rowp, (uint32_t)H + 1u);
  // verbatim counts of the dense blocks, one warp per block
  const float inv2e = __fdiv_rn(1.0f, __fmul_rn(2.0f, pl.eps));
  const SplitOut none = {nullptr, nullptr, 0};
  for (uint32_t b = wid; b < nblk; b += nw) {
    uint32_t n = 0;
    if (blk_a[b]) n = block_codes_warp<DT, false>(plane, H, W, (int)(b / nbx), (int)(b % nbx), inv2e, none, 0, 0);
    if (lane32 == 0) blk_c[b] = n;
  }
  team_sync(t);
  info.n_out_d = team_excl_scan(t, blk_c, nblk);
  const uint32_t e = (uint32_t)pl.esize;
  info.size = 16u + 4u * pl.nbm + 4u * ((uint32_t)H + 1u) + a4(2u * info.nnz_s) + a4(e * info.nnz_s) +
              64u * info.n_dense + a4(e * info.n_out_d);
  return info;
}

// Block-wise path, writing part; `sal` holds what salient_measure left.
template <int DT>
__device__ __noinline__ void salient_write(const Team& t, const Plan& pl, const uint8_t* plane, const SalientInfo& info,
                                           const uint32_t* sal, const SplitOut& out) {
  const uint32_t* rowp = sal;
  const uint32_t* blk_a = sal + pl.H + 1;
  const uint32_t* blk_b = blk_a + pl.nblk;
  const uint32_t* blk_c = blk_b + pl.nblk;
  const int H = pl.H, W = pl.W;
  const uint32_t nblk = pl.nblk, nbx = pl.nbx, e = (uint32_t)pl.esize;
  const uint32_t nw = t.block ? t.nwarps : 1u, wid = t.block ? threadIdx.x >> 5 : 0u, lane32 = threadIdx.x & 31u;
  const uint32_t o_bm = 16u, o_rp = o_bm + 4u * pl.nbm, o_col = o_rp + 4u * ((uint32_t)H + 1u);
  const uint32_t o_val = o_col + a4(2u * info.nnz_s), o_codes = o_val + a4(e * info.nnz_s);
  const uint32_t o_outl = o_codes + 64u * info.n_dense;
  if (t.lane == 0) {
    out.st32(0, info.nnz_s);
    out.st32(4, info.n_dense);
    out.st32(8, info.n_out_d);
    out.st32(12, 0);
    // pads the section writers leave: col (2 bytes), val / verbatim values (bf16: 2 bytes)
    if (info.nnz_s & 1u) out.st16(o_col + 2u * info.nnz_s, 0);
    if (DT == kBF16 && (info.nnz_s & 1u)) out.st16(o_val + 2u * info.nnz_s, 0);
    if (DT == kBF16 && (info.n_out_d & 1u)) out.st16(o_outl + 2u * info.n_out_d, 0);
  }
  // zero padding up to the end of the slot / of the 16-byte padded overflow part
  const uint32_t end = max(pl.npay, a16(info.size));
  for (uint32_t o = info.size + 4u * t.lane; o < end; o += 4u * t.size) out.st32(o, 0);
  for (uint32_t w = t.lane; w < pl.nbm; w += t.size) {
    uint32_t word = 0;
    const uint32_t hi = min(nblk, w * 32u + 32u);
    for (uint32_t b = w * 32u; b < hi; ++b) word |= blk_a[b] << (b & 31u);
    out.st32(o_bm + 4u * w, word);
  }
  for (uint32_t y = t.lane; y <= (uint32_t)H; y += t.size) out.st32(o_rp + 4u * y, rowp[y]);
  // CSR entries: one warp per row, columns in chunks of 32, positions by ballot
  for (int y = (int)wid; y < H; y += (int)nw) {
    uint32_t o = rowp[y];
    const uint32_t* brow = blk_a + (uint32_t)(y >> 3) * nbx;
    for (int x0 = 0; x0 < W; x0 += 32) {
      const int x = x0 + (int)lane32;
      const uint32_t idx = (uint32_t)y * W + (uint32_t)x;
      const bool take = x < W && load_elem<DT>(plane, idx) != 0.0f && !brow[x >> 3];
      const uint32_t m = __ballot_sync(0xFFFFFFFFu, take);
      if (take) {
        const uint32_t pos = o + __popc(m & ((1u << lane32) - 1u));
        out.st16(o_col + 2u * pos, (uint32_t)x);
        if (DT == kF32) out.st32(o_val + 4u * pos, reinterpret_cast<const uint32_t*>(plane)[idx]);
        else out.st16(o_val + 2u * pos, reinterpret_cast<const uint16_t*>(plane)[idx]);
      }
      o += __popc(m);
    }
  }
  const float inv2e = __fdiv_rn(1.0f, __fmul_rn(2.0f, pl.eps));
  for (uint32_t b = wid; b < nblk; b += nw)
    if (blk_a[b])
      block_codes_warp<DT, true>(plane, H, W, (int)(b / nbx), (int)(b % nbx), inv2e, out, o_codes + 64u * blk_b[b],
                                 o_outl + e * blk_c[b]);
}

// Raw plane: verbatim copy through the slot into the overflow part, zero padded.
__device__ __noinline__ void raw_write(const Team& t, const Plan& pl, const uint8_t* plane, const SplitOut& out) {
  const uint32_t n = (uint32_t)pl.plane_bytes, end = max(pl.npay, a16(n));
  for (uint32_t o = 2u * t.lane; o < end; o += 2u * t.size)
    out.st16(o, o < n ? (uint32_t)*reinterpret_cast<const uint16_t*>(plane + o) : 0u);
}

// Per-plane record kept in shared memory while a tile is processed.
struct Rec {
  float lo, scale;
  uint32_t meta;  // class | n_out << 2
  uint32_t size;  // payload bytes of a salient / raw plane (before padding)
};

// What every thread of a CTA knows about the destination.
struct Dest {
  uint8_t* dst;
  unsigned long long capacity, off_in;
  bool fits;  // header, table and slots fit the capacity
};
__device__ __forceinline__ Dest make_dest(const Plan& pl, const CompressArgs& a) {
  Dest d;
  d.off_in = a.d_off_in ? *a.d_off_in : 0ull;
  d.dst = a.dst_base + d.off_in;
  d.capacity = a.capacity > d.off_in ? a.capacity - d.off_in : 0ull;
  d.fits = d.capacity >= pl.ovf_off;
  return d;
}

// Tile-level placement, executed by warp 0 after the classes and sizes of the tile's planes are in
// rec[].  Computes each plane's overflow offset (roff[], 16-byte units relative to the tile),
// publishes the tile's overflow size and, when the tile has overflow parts, resolves the tile's
// base.  Returns through shared variables: *s_base16 (absolute, 16-byte units), *s_skip.
__device__ __noinline__ void tile_place(const Plan& pl, const CompressArgs& a, const Dest& d, uint32_t tile,
                                           uint32_t np, const Rec* rec, uint32_t* roff,
                                           unsigned long long* s_base16, uint32_t* s_skip) {
  const uint32_t lane = threadIdx.x & 31u;
  uint32_t carry = 0, nsal = 0, nraw = 0;
  for (uint32_t base = 0; base < np; base += 32) {
    const uint32_t i = base + lane;
    uint32_t v = 0, c = 0;
    if (i < np) {
      c = rec[i].meta & 3u;
      if (c != kClsNormal && a16(rec[i].size) > pl.npay) v = (a16(rec[i].size) - pl.npay) >> 4;
    }
    uint32_t incl = v;
    for (uint32_t o = 1; o < 32; o <<= 1) {
      const uint32_t up = __shfl_up_sync(0xFFFFFFFFu, incl, o);
      if (lane >= o) incl += up;
    }
    if (i < np) roff[i] = carry + incl - v;
    carry += __shfl_sync(0xFFFFFFFFu, incl, 31);
    nsal += __popc(__ballot_sync(0xFFFFFFFFu, c == kClsSalient));
    nraw += __popc(__ballot_sync(0xFFFFFFFFu, c == kClsRaw));
  }
  unsigned long long excl = 0;
  uint32_t skip = d.fits ? 0u : 1u;
  if (pl.mode != kModeOff) {
    if (lane == 0) scan_publish(a.scan, tile, carry);
    if (carry > 0 && tile > 0) {
      if (!scan_resolve(a.scan, tile, &a.sc->status, &excl)) {
        if (lane == 0) atomicMax(&a.sc->status, (unsigned long long)kErrTimeout);
        skip = 1;
      }
    }
    if (lane == 0) {
      if (carry) atomicAdd(&a.sc->ovf16, (unsigned long long)carry);
      if (nsal) atomicAdd(&a.sc->nsal, (unsigned long long)nsal);
      if (nraw) atomicAdd(&a.sc->nraw, (unsigned long long)nraw);
    }
  }
  if (lane == 0) {
    const unsigned long long base16 = (pl.ovf_off >> 4) + excl;
    if ((base16 + carry) * 16ull > d.capacity) skip = 1;  // never write past the capacity
    *s_base16 = base16;
    *s_skip = skip;
  }
}

// Last step of every CTA: count the exit; the last CTA to leave writes the header and the result
// words and returns the scratch counters to zero for the next call.
__device__ __forceinline__ void cta_exit(const Plan& pl, const CompressArgs& a, const Dest& d) {
  __threadfence();
  __syncthreads();
  if (threadIdx.x != 0) return;
  const unsigned long long prev = atomicAdd(&a.sc->exited, 1ull);
  if (prev != (unsigned long long)gridDim.x - 1ull) return;
  __threadfence();
  const unsigned long long ovf16 = ld_relaxed(&a.sc->ovf16);
  const unsigned long long nsal = ld_relaxed(&a.sc->nsal), nraw = ld_relaxed(&a.sc->nraw);
  uint32_t code = (uint32_t)ld_relaxed(&a.sc->status);
  const unsigned long long total = pl.ovf_off + ovf16 * 16ull;
  if (total > d.capacity && code < kErrCapacity) code = kErrCapacity;
  if (d.capacity >= 64) {
    uint32_t h[16];
    h[0] = code == kErrNone ? kMagic : 0u;  // a failed container must not pass for a valid one
    h[1] = 1u | ((uint32_t)pl.dtype << 16) | ((uint32_t)pl.bits << 24);
    h[2] = pl.N;
    h[3] = pl.C;
    h[4] = (uint32_t)pl.H;
    h[5] = (uint32_t)pl.W;
    h[6] = 8u | (8u << 8) | (0u << 16) | ((uint32_t)pl.mode << 24);
    h[7] = pl.rho_num | (pl.rho_den << 16);
    h[8] = pl.tau_num | (pl.tau_den << 16);
    h[9] = __float_as_uint(pl.eps);
    h[10] = (uint32_t)nsal;
    h[11] = (uint32_t)nraw;
    h[12] = (uint32_t)pl.tensor_id;
    h[13] = (uint32_t)(pl.tensor_id >> 32);
    h[14] = (uint32_t)total;
    h[15] = (uint32_t)(total >> 32);
    uint32_t* hd = reinterpret_cast<uint32_t*>(d.dst);
    for (int k = 0; k < 16; ++k) hd[k] = h[k];
  }
  if (a.out2) {
    a.out2[0] = total;
    a.out2[1] = status_word(code);
  }
  if (a.d_off_out) *a.d_off_out = code == kErrNone ? d.off_in + ((total + 255ull) & ~255ull) : (~0ull >> 1);
  if (pl.mode != kModeOff)
    for (uint32_t k = 0; k < a.nseg; ++k) st_relaxed(a.scan.seg_cs + k, 0ull);  // counters back to zero
  st_relaxed(&a.sc->ticket, 0ull);
  st_relaxed(&a.sc->status, 0ull);
  st_relaxed(&a.sc->ovf16, 0ull);
  st_relaxed(&a.sc->nsal, 0ull);
  st_relaxed(&a.sc->nraw, 0ull);
  st_relaxed(&a.sc->exited, 0ull);
}

__device__ __forceinline__ void store_table_entry(const Dest& d, uint64_t plane, uint32_t off16, const Rec& r) {
  uint4 e;
  e.x = off16;
  e.y = r.meta;
  e.z = __float_as_uint(r.lo);
  e.w = __float_as_uint(r.scale);
  reinterpret_cast<uint4*>(d.dst + 64)[plane] = e;
}

// Writes a salient or raw plane whose record and overflow offset (absolute, 16-byte units) are known.
template <int DT>
__device__ __forceinline__ void write_nonnormal(const Team& t, const Plan& pl, const Dest& d, const uint8_t* plane,
                                                uint64_t gp, const Rec& r, unsigned long long off16, uint32_t* sal) {
  SplitOut out;
  out.slot = d.dst + pl.slots_off + gp * pl.npay;
  out.ovf = d.dst + off16 * 16ull;
  out.npay = pl.npay;
  const bool has_ovf = a16(r.size) > pl.npay;
  if ((r.meta & 3u) == kClsRaw) {
    raw_write(t, pl, plane, out);
  } else {
    const SalientInfo info = salient_measure<DT>(t, pl, plane, sal);
    salient_write<DT>(t, pl, plane, info, sal, out);
  }
  if (t.lane == 0) store_table_entry(d, gp, has_ovf ? (uint32_t)off16 : 0u, r);
}

// =================================================================================================
// Generic kernel
// =================================================================================================
template <int DT, int BITS>
__global__ void __launch_bounds__(kThreads) compress_generic(const Plan pl, const CompressArgs a) {
  extern __shared__ __align__(128) uint8_t smem[];
  __shared__ double s_red[kMaxWarps * 5];
  __shared__ uint32_t s_tile, s_skip;
  __shared__ unsigned long long s_base16;

  const uint32_t tid = threadIdx.x;
  uint8_t* tile_buf = smem + pl.sm_tile;
  uint8_t* out_buf = smem + pl.sm_out;
  Rec* rec = reinterpret_cast<Rec*>(smem + pl.sm_rec);
  uint32_t* roff = reinterpret_cast<uint32_t*>(smem + pl.sm_rec + 16u * pl.ppt);
  const Dest d = make_dest(pl, a);
  const Team team = make_team(pl.team, s_red);
  const uint32_t nteams = team.block ? 1u : kThreads / team.size;
  const uint32_t my_team = team.block ? 0u : tid / team.size;
  uint32_t* sal = reinterpret_cast<uint32_t*>(smem + pl.sm_sal + (uint64_t)my_team * pl.sm_sal_stride);
  constexpr uint32_t L = (1u << BITS) - 1u;
  const bool need_sigma = pl.mode == kModeAuto;
  uint32_t rp = 0;  // reduction counter (see red_half)
  if (!d.fits && tid == 0 && blockIdx.x == 0) atomicMax(&a.sc->status, (unsigned long long)kErrCapacity);

  for (;;) {
    if (tid == 0) s_tile = (uint32_t)atomicAdd(&a.sc->ticket, 1ull);
    __syncthreads();
    const uint32_t tile = s_tile;
    if (tile >= pl.ntiles) break;
    const uint64_t p0 = (uint64_t)tile * pl.ppt;
    const uint32_t np = (uint32_t)min((uint64_t)pl.ppt, pl.P - p0);

    // ---- stage the tile: whole 16-byte chunks, then the ragged end of the tensor byte by byte
    const uint64_t start = p0 * pl.plane_bytes, end = start + (uint64_t)np * pl.plane_bytes;
    const uint64_t a0 = start & ~15ull;
    const uint32_t head = (uint32_t)(start - a0);
    const uint64_t a1 = min((end + 15ull) & ~15ull, pl.dense_bytes & ~15ull);
    {
      const uint4* s16 = reinterpret_cast<const uint4*>(a.src + a0);
      uint4* t16 = reinterpret_cast<uint4*>(tile_buf);
      const uint32_t n16 = (uint32_t)((a1 - a0) >> 4);
      for (uint32_t i = tid; i < n16; i += kThreads) t16[i] = __ldg(s16 + i);
      for (uint64_t i = a1 + tid; i < end; i += kThreads) tile_buf[i - a0] = a.src[i];
    }
    __syncthreads();

    // ---- phase A: per-plane statistics, class, codes / sizes
    for (uint32_t lp = my_team; lp < np; lp += nteams) {
      const uint8_t* plane = tile_buf + head + (uint64_t)lp * pl.plane_bytes;
      const bool vec = (smem_u32(plane) & (DT == kF32 ? 15u : 7u)) == 0u;
      const uint32_t HW = pl.HW, nfull = HW >> 2, groups = pl.groups;
      float lo = __int_as_float(0x7F800000), hi = __int_as_float(0xFF800000);
      for (uint32_t g = team.lane; g < nfull; g += team.size) {
        float v[4];
        load_group<DT>(plane, g, HW, vec, v);
        lo = min3_nan(lo, min_nan(v[0], v[1]), min_nan(v[2], v[3]));
        hi = max3_nan(hi, max_nan(v[0], v[1]), max_nan(v[2], v[3]));
      }
      if ((HW & 3u) && team.lane == 0) {  // ragged last group
        for (uint32_t i = nfull * 4u; i < HW; ++i) {
          const float x = load_elem<DT>(plane, i);
          lo = min_nan(lo, x);
          hi = max_nan(hi, x);
        }
      }
      team_minmax(team, lo, hi, rp);
      if (!(fabsf(__fsub_rn(hi, lo)) <= 3.402823466e38f) && team.lane == 0)
        atomicMax(&a.sc->status, (unsigned long long)kErrNonfinite);

      uint32_t cls = kClsNormal, n_out = 0;
      if (need_sigma) {
        const SigmaScale sc = sigma_scale(lo, hi);
        uint32_t as = 0, aq = 0, ng = 0;
        for (uint32_t g = team.lane; g < groups; g += team.size) {
          float v[4];
          load_group<DT>(plane, g, HW, vec, v);
          sigma_addends(v, sc, as, aq);
          ++ng;
        }
        long long Is, Iq;
        if (team.block)
          team_sum2_wide(team, (long long)(int32_t)(as - ng * kMagicBits), (long long)(int32_t)(aq - ng * kMagicBits),
                         Is, Iq, rp);
        else
          team_sum2(team, (int32_t)(as - ng * kMagicBits), (int32_t)(aq - ng * kMagicBits), Is, Iq, rp);
        float tlo, thi;
        sigma_thresholds(Is, Iq, sc, pl.inv_hw, tlo, thi);
        uint32_t cnt = 0;
        for (uint32_t g = team.lane; g < groups; g += team.size) {
          float v[4];
          load_group<DT>(plane, g, HW, vec, v);
#pragma unroll
          for (int k = 0; k < 4; ++k) cnt += (v[k] > thi) || (v[k] < tlo);
        }
        n_out = team_sum_u32(team, cnt, rp);
        if ((0.0f > thi) || (0.0f < tlo)) n_out -= 4u * groups - HW;  // padded zeros are not elements
        if ((uint64_t)n_out * pl.rho_den > (uint64_t)pl.rho_num * HW) cls = kClsSalient;
      } else if (pl.mode == kModeAll) {
        cls = kClsSalient;
      }

      Rec r;
      r.lo = 0.0f;
      r.scale = 0.0f;
      r.size = 0;
      if (cls == kClsSalient) {
        const SalientInfo info = salient_measure<DT>(team, pl, plane, sal);
        r.size = info.size;
        if (a16(info.size) >= a16((uint32_t)pl.plane_bytes)) {
          cls = kClsRaw;
          r.size = (uint32_t)pl.plane_bytes;
        }
      } else {
        float inv, scale;
        quant_params(lo, hi, L, inv, scale);
        r.lo = lo;
        r.scale = scale;
        uint8_t* o = out_buf + (uint64_t)lp * pl.npay;
        const uint32_t ogroups = pl.npay * 2u / BITS;
        for (uint32_t g = team.lane; g < ogroups; g += team.size) {
          uint32_t word = 0;
          if (g < groups) {
            float v[4];
            load_group<DT>(plane, g, HW, vec, v);
#pragma unroll
            for (int k = 0; k < 4; ++k) {
              uint32_t q = quant_code(v[k], lo, inv, L);
              if (g * 4u + k >= HW) q = 0;
              word |= q << (k * BITS);
            }
          }
          if (BITS == 2) o[g] = (uint8_t)word;
          else if (BITS == 4) reinterpret_cast<uint16_t*>(o)[g] = (uint16_t)word;
          else reinterpret_cast<uint32_t*>(o)[g] = word;
        }
      }
      r.meta = cls | (n_out << 2);
      if (team.lane == 0) rec[lp] = r;
    }
    __syncthreads();

    // ---- phase B: placement of the overflow parts
    if (tid < 32) tile_place(pl, a, d, tile, np, rec, roff, &s_base16, &s_skip);
    __syncthreads();

    // ---- phase C: table entries and payloads
    if (!s_skip) {
      const unsigned long long base16 = s_base16;
      const uint32_t chunks = pl.npay >> 4;
      uint4* slots = reinterpret_cast<uint4*>(d.dst + pl.slots_off + p0 * pl.npay);
      for (uint32_t i = tid; i < np * chunks; i += kThreads) {
        const uint32_t lp = i / chunks;
        if ((rec[lp].meta & 3u) == kClsNormal) slots[i] = reinterpret_cast<const uint4*>(out_buf)[i];
      }
      for (uint32_t i = tid; i < np; i += kThreads)
        if ((rec[i].meta & 3u) == kClsNormal)
          store_table_entry(d, p0 + i, (uint32_t)((pl.slots_off + (p0 + i) * pl.npay) >> 4), rec[i]);
      for (uint32_t lp = my_team; lp < np; lp += nteams) {
        if ((rec[lp].meta & 3u) == kClsNormal) continue;
        const uint8_t* plane = tile_buf + head + (uint64_t)lp * pl.plane_bytes;
        write_nonnormal<DT>(team, pl, d, plane, p0 + lp, rec[lp], base16 + roff[lp], sal);
      }
    }
    __syncthreads();
  }
  cta_exit(pl, a, d);
}

// =================================================================================================
// Fast kernel
// =================================================================================================
// One plane per team and tile.  Warp-team variant (CTA = false): kThreads / team planes per tile,
// each handled by `team` lanes of a warp.  CTA-team variant: one plane per tile, handled by all
// threads.  Thread t of a team owns groups t, t + team, ... (G of them) and keeps them in registers
// for every pass.  FULL: groups == G * team, so no group needs a bounds check.
//
// One sweep over a plane: min/max -> (fixed-point moments -> thresholds -> count -> class) ->
// codes, stored straight to the plane's slot together with its table entry.  Salient planes are
// measured by their team right away; their writes wait for the tile's placement.
// Codes of the thread's groups, packed and stored to the plane's slot (used inside plane_sweep, on
// its register-resident groups x[k][e]).  Four codes of a group are the sum of
// (magic + q_e) << (e * BITS) minus the magic's contribution.
#define FH_STORE_CODES(BITS)                                                                                  \
  {                                                                                                           \
    constexpr uint32_t bias = kMagicBits * (1u + (1u << (BITS)) + (1u << (2 * (BITS))) + (1u << (3 * (BITS)))); \
    _Pragma("unroll") for (int k = 0; k < G; ++k) {                                                           \
      const uint32_t g = lane + (uint32_t)(k * TT);                                                           \
      if (FULL || g < groups) {                                                                               \
        uint32_t word = __float_as_uint(__fmaf_rn(__fsub_rn(x[k][0], lo), inv, kMagicF));                     \
        word += __float_as_uint(__fmaf_rn(__fsub_rn(x[k][1], lo), inv, kMagicF)) << (BITS);                   \
        word += __float_as_uint(__fmaf_rn(__fsub_rn(x[k][2], lo), inv, kMagicF)) << (2 * (BITS));             \
        word += __float_as_uint(__fmaf_rn(__fsub_rn(x[k][3], lo), inv, kMagicF)) << (3 * (BITS));             \
        word -= bias;                                                                                         \
        if (!VEC) { /* ragged last group: elements past the plane carry no code */                            \
          const uint32_t valid = min(4u, pl.HW - g * 4u);                                                     \
          if (valid < 4u) word &= (1u << (valid * (BITS))) - 1u;                                              \
        }                                                                                                     \
        if ((BITS) == 2) slot[g] = (uint8_t)word;                                                             \
        else if ((BITS) == 4) reinterpret_cast<uint16_t*>(slot)[g] = (uint16_t)word;                          \
        else reinterpret_cast<uint32_t*>(slot)[g] = word;                                                     \
      }                                                                                                       \
    }                                                                                                         \
  }

// TT: team size (1..32, or kThreads for the CTA team), a compile-time constant so that the strides
// between a thread's groups are immediates.  FULL: groups == G * TT.  VEC: planes are whole 16-byte
// chunks (vector loads, no ragged last group).
template <int DT, bool SIGMA, int G, int TT, bool FULL, bool VEC>
__device__ __forceinline__ void plane_sweep(const Team& team, const Plan& pl, const Dest& d, const CompressArgs& a,
                                            const uint8_t* plane, uint64_t gp, uint32_t& rp, Rec& r) {
  const uint32_t groups = pl.groups, lane = team.lane;
  float x[G][4];
  float lo = __int_as_float(0x7F800000), hi = __int_as_float(0xFF800000), lo1 = lo, hi1 = hi;
  uint32_t ng = 0, npad = 0;  // groups of this thread; zero-padded elements among them
#pragma unroll
  for (int k = 0; k < G; ++k) {
    const uint32_t g = lane + (uint32_t)(k * TT);
    if (FULL || g < groups) {
      if (VEC) {
        if (DT == kF32) {
          const float4 t4 = (reinterpret_cast<const float4*>(plane) + lane)[k * TT];
          x[k][0] = t4.x; x[k][1] = t4.y; x[k][2] = t4.z; x[k][3] = t4.w;
        } else {
          const uint2 t2 = (reinterpret_cast<const uint2*>(plane) + lane)[k * TT];
          x[k][0] = __uint_as_float(t2.x << 16); x[k][1] = __uint_as_float(t2.x & 0xFFFF0000u);
          x[k][2] = __uint_as_float(t2.y << 16); x[k][3] = __uint_as_float(t2.y & 0xFFFF0000u);
        }
        // per-group partial results keep the dependency chains short
        const float gl = min_nan(min3_nan(x[k][0], x[k][1], x[k][2]), x[k][3]);
        const float gh = max_nan(max3_nan(x[k][0], x[k][1], x[k][2]), x[k][3]);
        if (k & 1) {
          lo1 = min_nan(lo1, gl);
          hi1 = max_nan(hi1, gh);
        } else {
          lo = min_nan(lo, gl);
          hi = max_nan(hi, gh);
        }
      } else {  // plane not on a 16-byte boundary, possibly with a ragged last group
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const uint32_t i = g * 4u + e;
          const bool in = i < pl.HW;
          x[k][e] = in ? load_elem<DT>(plane, i) : 0.0f;
          if (in) {
            lo = min_nan(lo, x[k][e]);
            hi = max_nan(hi, x[k][e]);
          } else {
            ++npad;
          }
        }
      }
      ++ng;
    }
  }
  lo = min_nan(lo, lo1);
  hi = max_nan(hi, hi1);
  team_minmax(team, lo, hi, rp);
  if (!(fabsf(__fsub_rn(hi, lo)) <= 3.402823466e38f) && lane == 0)
    atomicMax(&a.sc->status, (unsigned long long)kErrNonfinite);

  uint32_t cls = kClsNormal, n_out = 0;
  if (SIGMA) {
    const SigmaScale sc = sigma_scale(lo, hi);
    uint32_t as = 0, aq = 0;
#pragma unroll
    for (int k = 0; k < G; ++k)
      if (FULL || lane + (uint32_t)(k * TT) < groups) sigma_addends4(x[k][0], x[k][1], x[k][2], x[k][3], sc, as, aq);
    if (FULL) ng = G;
    long long Is, Iq;
    team_sum2(team, (int32_t)(as - ng * kMagicBits), (int32_t)(aq - ng * kMagicBits), Is, Iq, rp);
    float tlo, thi;
    if (TT > 32) sigma_thresholds(Is, Iq, sc, pl.inv_hw, tlo, thi);
    else sigma_thresholds((int32_t)Is, (int32_t)Iq, sc, pl.inv_hw, tlo, thi);
    uint32_t cnt = 0;
    if (hi > thi || lo < tlo) {  // otherwise no element can lie outside: the count is zero
      uint32_t c[4] = {0, 0, 0, 0};  // four counters: short dependency chains
      if (lo >= tlo) {               // nothing below: one compare per element
#pragma unroll
        for (int k = 0; k < G; ++k)
          if (FULL || lane + (uint32_t)(k * TT) < groups) {
#pragma unroll
            for (int e = 0; e < 4; ++e) c[e] += x[k][e] > thi;
          }
        cnt = (c[0] + c[1]) + (c[2] + c[3]);
        if (!VEC && 0.0f > thi) cnt -= npad;  // padded zeros are not elements
      } else {
#pragma unroll
        for (int k = 0; k < G; ++k)
          if (FULL || lane + (uint32_t)(k * TT) < groups) {
#pragma unroll
            for (int e = 0; e < 4; ++e) c[e] += (x[k][e] > thi) || (x[k][e] < tlo);
          }
        cnt = (c[0] + c[1]) + (c[2] + c[3]);
        if (!VEC && ((0.0f > thi) || (0.0f < tlo))) cnt -= npad;
      }
      cnt = team_sum_u32(team, cnt, rp);
    }
    n_out = cnt;
    if ((uint64_t)n_out * pl.rho_den > (uint64_t)pl.rho_num * pl.HW) cls = kClsSalient;
  } else if (pl.mode == kModeAll) {
    cls = kClsSalient;
  }

  r.lo = 0.0f;
  r.scale = 0.0f;
  r.size = 0;
  r.meta = cls | (n_out << 2);
  if (cls != kClsNormal) return;
  const uint32_t bits = (uint32_t)pl.bits;
  float inv, scale;
  quant_params(lo, hi, (1u << bits) - 1u, inv, scale);
  r.lo = lo;
  r.scale = scale;
  if (!d.fits) return;
  uint8_t* slot = d.dst + pl.slots_off + gp * pl.npay;
  if (bits == 2u) FH_STORE_CODES(2)
  else if (bits == 4u) FH_STORE_CODES(4)
  else FH_STORE_CODES(8)
  // zero padding of the slot behind the codes
  const uint32_t code_bytes = groups * bits / 2u;
  if (code_bytes < pl.npay) {
    for (uint32_t o = code_bytes + lane; o < a4(code_bytes); o += TT) slot[o] = 0;
    for (uint32_t o = a4(code_bytes) + 4u * lane; o < pl.npay; o += 4u * TT)
      *reinterpret_cast<uint32_t*>(slot + o) = 0u;
  }
  if (lane == 0) store_table_entry(d, gp, (uint32_t)((pl.slots_off + gp * pl.npay) >> 4), r);
}

// Picks the specialisation of the sweep.  FULLVEC kernels are launched only for planes of exactly
// G * TT whole groups, so they carry nothing but the lean variant; the others choose at run time.
template <int DT, bool SIGMA, int G, int TT, bool FULLVEC>
__device__ __forceinline__ void plane_sweep_any(const Team& team, const Plan& pl, const Dest& d,
                                                const CompressArgs& a, const uint8_t* plane, uint64_t gp,
                                                bool vec, uint32_t& rp, Rec& r) {
  if (FULLVEC) plane_sweep<DT, SIGMA, G, TT, true, true>(team, pl, d, a, plane, gp, rp, r);
  else if (vec) plane_sweep<DT, SIGMA, G, TT, false, true>(team, pl, d, a, plane, gp, rp, r);
  else plane_sweep<DT, SIGMA, G, TT, false, false>(team, pl, d, a, plane, gp, rp, r);
}

// -------------------------------------------------------------------------------------------------
// Warp-team kernel: planes of at most 256 groups.  Eight consumer warps and one producer warp per
// CTA.  The producer hands out tiles and streams them into a ring of shared-memory stages with bulk
// copies.  The consumer warps never wait for each other on the common path: each sweeps its own
// planes of a tile (statistics, class, codes, stores) and arrives on the stage's barriers.  When a
// stage comes back, the producer publishes the tile's (zero) scan word.  Only warps that hold
// salient or raw planes take the slow path: they wait until the whole tile is classified, one of
// them places the tile's overflow parts, and they write their planes.
// -------------------------------------------------------------------------------------------------
constexpr int kWarpKernelThreads = kThreads + 32;

// Placement of a tile with salient / raw planes, executed by one warp.  ovf16[i] holds the overflow
// size of plane i of the tile in 16-byte units (0 for normal planes); the
// sizes are left alone; poff[i] receives the plane's offset relative to the tile's base.
__device__ __noinline__ void tile_place_sparse(const Plan& pl, const CompressArgs& a, const Dest& d, uint32_t tile,
                                               uint32_t np, const uint32_t* ovf16, uint32_t* poff,
                                               unsigned long long* s_base16, uint32_t* s_skip) {
  const uint32_t lane = threadIdx.x & 31u;
  uint32_t carry = 0;
  for (uint32_t base = 0; base < np; base += 32) {
    const uint32_t i = base + lane;
    const uint32_t v = i < np ? ovf16[i] : 0u;
    uint32_t incl = v;
    for (uint32_t o = 1; o < 32; o <<= 1) {
      const uint32_t up = __shfl_up_sync(0xFFFFFFFFu, incl, o);
      if (lane >= o) incl += up;
    }
    if (i < np) poff[i] = carry + incl - v;
    carry += __shfl_sync(0xFFFFFFFFu, incl, 31);
  }
  unsigned long long excl = 0;
  uint32_t skip = d.fits ? 0u : 1u;
  if (lane == 0) scan_publish(a.scan, tile, carry);
  if (carry > 0 && tile > 0) {
    if (!scan_resolve(a.scan, tile, &a.sc->status, &excl)) {
      if (lane == 0) atomicMax(&a.sc->status, (unsigned long long)kErrTimeout);
      skip = 1;
    }
  }
  if (lane == 0) {
    if (carry) atomicAdd(&a.sc->ovf16, (unsigned long long)carry);
    const unsigned long long base16 = (pl.ovf_off >> 4) + excl;
    if ((base16 + carry) * 16ull > d.capacity) skip = 1;  // never write past the capacity
    *s_base16 = base16;
    *s_skip = skip;
  }
}

template <int DT, bool SIGMA, int TT, bool FULLVEC>
__global__ void __launch_bounds__(kWarpKernelThreads, 3) compress_warp(const Plan pl, const CompressArgs a) {
  extern __shared__ __align__(128) uint8_t smem[];
  __shared__ double s_red[kMaxWarps * 5];
  __shared__ __align__(8) uint64_t s_full[kMaxStages], s_empty[kMaxStages], s_classified[kMaxStages];
  __shared__ uint32_t s_tiles[kMaxStages], s_nn[kMaxStages], s_nnmask[kMaxStages], s_skip[kMaxStages];
  __shared__ volatile uint32_t s_placed[kMaxStages];  // tile + 1 once the tile's overflow parts are placed
  __shared__ unsigned long long s_base16[kMaxStages];
  __shared__ volatile uint32_t s_abort;
  __shared__ Plan s_pl;          // copies for the outlined slow path (salient planes, placement):
  __shared__ CompressArgs s_a;   // its functions take them by address

  const uint32_t tid = threadIdx.x, lane = tid & 31u, warp = tid >> 5;
  const Dest d = make_dest(pl, a);
  const uint32_t nstage = pl.nstage;
  uint32_t* ovf16_all = reinterpret_cast<uint32_t*>(smem + pl.sm_rec);  // nstage x ppt words, zero when idle
  if (!d.fits && tid == 0 && blockIdx.x == 0) atomicMax(&a.sc->status, (unsigned long long)kErrCapacity);
  if (tid == 0) {
    s_pl = pl;
    s_a = a;
    for (uint32_t s = 0; s < nstage; ++s) {
      mbar_init(&s_full[s], 1);
      mbar_init(&s_empty[s], kWarps);
      mbar_init(&s_classified[s], kWarps);
      s_nn[s] = 0;
      s_nnmask[s] = 0;
      s_placed[s] = 0;
    }
    fence_mbar_init();
    s_abort = 0;
  }
  for (uint32_t i = tid; i < nstage * pl.ppt; i += kWarpKernelThreads) ovf16_all[i] = 0;
  __syncthreads();

  if (warp == (uint32_t)kWarps) {
    // ======================= producer (all 32 lanes walk the loop, lane 0 issues) =======================
    uint32_t s = 0, empty_phase = 0;
    bool aborted = false;
    // Drains stage q: waits until every consumer warp is done with its tile, then gives a tile without
    // salient planes its scan word (tiles with salient planes were published by their consumers).
    auto drain = [&](uint32_t q) -> bool {
      bool ok = mbar_wait_abortable(&s_empty[q], (empty_phase >> q) & 1u, 1u << 20, &s_abort);
      ok = __all_sync(0xFFFFFFFFu, ok);
      if (!ok) return false;
      empty_phase ^= 1u << q;
      if (pl.mode != kModeOff) {
        if (lane == 0) {
          if (*reinterpret_cast<volatile uint32_t*>(&s_nn[q]) == 0) scan_publish(a.scan, s_tiles[q], 0u);
          s_nn[q] = 0;
          s_nnmask[q] = 0;
        }
        __syncwarp();
      }
      return true;
    };
    for (uint32_t n = 0;; ++n) {
      if (n >= nstage && !drain(s)) {
        aborted = true;
        break;
      }
      uint32_t t = 0;
      if (lane == 0) t = (uint32_t)atomicAdd(&a.sc->ticket, 1ull);
      t = __shfl_sync(0xFFFFFFFFu, t, 0);
      if (t >= pl.ntiles) {
        // no more tiles: wake the consumers at this stage, then drain the tiles still in the ring
        const uint32_t first = n >= nstage ? n - nstage + 1u : 0u;
        uint32_t q = first % nstage;
        __syncwarp();
        if (lane == 0) {
          s_tiles[s] = t;
          mbar_arrive(&s_full[s]);
        }
        for (uint32_t m = first; m < n; ++m) {
          if (!drain(q)) {
            aborted = true;
            break;
          }
          q = q + 1 == nstage ? 0 : q + 1;
        }
        break;
      }
      if (lane == 0) {
        s_tiles[s] = t;
        const uint32_t p0 = t * pl.ppt;
        const uint32_t np = (uint32_t)min((uint64_t)pl.ppt, pl.P - p0);
        const uint32_t bytes = np * (uint32_t)pl.plane_bytes;
        uint8_t* stage = smem + pl.sm_tile + (uint64_t)s * pl.stage_bytes;
        if ((bytes & 15u) == 0u) {
          fence_proxy_async();
          mbar_expect_tx(&s_full[s], bytes);
          bulk_g2s(stage, a.src + (uint64_t)p0 * pl.plane_bytes, bytes, &s_full[s]);
        } else {  // ragged last tile of a tensor of ragged planes: plain loads by this thread
          const uint16_t* g = reinterpret_cast<const uint16_t*>(a.src + (uint64_t)p0 * pl.plane_bytes);
          for (uint32_t i = 0; i < bytes / 2u; ++i) reinterpret_cast<uint16_t*>(stage)[i] = g[i];
          mbar_arrive(&s_full[s]);
        }
      }
      __syncwarp();
      s = s + 1 == nstage ? 0 : s + 1;
    }
    if (aborted) {  // wait (bounded) for copies still in flight before the CTA may exit
      s_abort = 1;
      if (lane == 0) {
        atomicMax(&a.sc->status, (unsigned long long)kErrTimeout);
        for (uint32_t k = 0; k < nstage; ++k) {
          mbar_wait(&s_full[k], 0u, 1u << 10);
          mbar_wait(&s_full[k], 1u, 1u << 10);
        }
      }
    }
  } else {
    // ======================= consumers =======================
    constexpr int G = 8;  // groups per thread: a plane has at most 8 * TT groups
    const Team team = make_team(TT, s_red);
    const uint32_t my_team = tid / TT;
    const bool vec = (pl.plane_bytes & 15u) == 0u;
    uint32_t rp = 0, s = 0, phase = 0;
    for (;;) {
      const uint32_t par = (phase >> s) & 1u;
      bool ok = mbar_wait_abortable(&s_full[s], par, 1u << 20, &s_abort);
      ok = __all_sync(0xFFFFFFFFu, ok);
      if (!ok) {
        s_abort = 1;
        break;
      }
      phase ^= 1u << s;
      const uint32_t tile = s_tiles[s];
      if (tile >= pl.ntiles) break;
      const uint32_t p0 = tile * pl.ppt;
      const uint32_t np = (uint32_t)min((uint64_t)pl.ppt, pl.P - p0);
      const uint32_t lp = my_team;
      const bool active = lp < np;
      const uint8_t* plane = smem + pl.sm_tile + (uint64_t)s * pl.stage_bytes + (uint64_t)lp * pl.plane_bytes;
      Rec r;
      r.meta = kClsNormal;
      if (active) plane_sweep_any<DT, SIGMA, G, TT, FULLVEC>(team, pl, d, a, plane, (uint64_t)p0 + lp, vec, rp, r);
      const bool mine_nn = active && (r.meta & 3u) != kClsNormal;
      if (!__any_sync(0xFFFFFFFFu, mine_nn)) {
        // ---- common path: this warp is done with the tile
        if (lane == 0) {
          mbar_arrive(&s_classified[s]);
          mbar_arrive(&s_empty[s]);
        }
      } else {
        // ---- slow path: salient / raw planes in this warp.  Each of them is handled by all 32 lanes.
        const Team wteam = make_warp_team(s_red);
        uint32_t* ovf16 = ovf16_all + s * pl.ppt;
        uint32_t* poff = ovf16_all + nstage * pl.ppt + s * pl.ppt;  // offsets inside the tile, from the placement
        uint32_t* sinfo = ovf16_all + 2u * nstage * pl.ppt + (s * pl.ppt) * 4u;  // per plane: size, nnz_s, n_dense, n_out_d
        const uint32_t leaders = __ballot_sync(0xFFFFFFFFu, mine_nn && team.lane == 0);
        const uint8_t* stage = smem + pl.sm_tile + (uint64_t)s * pl.stage_bytes;
        uint32_t raw_mask = 0;  // bit L: the plane led by lane L turned out raw
        for (uint32_t m = leaders; m; m &= m - 1u) {
          const uint32_t L = (uint32_t)__ffs(m) - 1u, tlp = (warp * 32u + L) / TT;
          const uint8_t* tplane = stage + (uint64_t)tlp * pl.plane_bytes;
          uint32_t* tsal = reinterpret_cast<uint32_t*>(smem + pl.sm_sal + (uint64_t)tlp * pl.sm_sal_stride);
          const SalientInfo info = salient_measure<DT>(wteam, s_pl, tplane, tsal);
          uint32_t size = info.size;
          const bool raw = a16(info.size) >= a16((uint32_t)pl.plane_bytes);
          if (raw) {
            size = (uint32_t)pl.plane_bytes;
            raw_mask |= 1u << L;
          }
          if (lane == 0) {
            ovf16[tlp] = a16(size) > pl.npay ? (a16(size) - pl.npay) >> 4 : 0u;
            sinfo[tlp * 4u + 0] = size;
            sinfo[tlp * 4u + 1] = info.nnz_s;
            sinfo[tlp * 4u + 2] = info.n_dense;
            sinfo[tlp * 4u + 3] = info.n_out_d;
            atomicAdd(raw ? &a.sc->nraw : &a.sc->nsal, 1ull);
          }
        }
        __syncwarp();
        if (lane == 0) {
          atomicAdd(&s_nn[s], 1u);
          atomicOr(&s_nnmask[s], 1u << warp);
          __threadfence_block();
          mbar_arrive(&s_classified[s]);
        }
        bool done = mbar_wait_abortable(&s_classified[s], par, 1u << 20, &s_abort);  // the whole tile is classified
        done = __all_sync(0xFFFFFFFFu, done);
        if (done) {
          __threadfence_block();
          const uint32_t mask = *reinterpret_cast<volatile uint32_t*>(&s_nnmask[s]);
          if ((uint32_t)__ffs(mask) - 1u == warp) {  // the first such warp places the tile
            tile_place_sparse(s_pl, s_a, d, tile, np, ovf16, poff, &s_base16[s], &s_skip[s]);
            __threadfence_block();
            __syncwarp();
            if (lane == 0) s_placed[s] = tile + 1u;
          }
          done = false;
          for (uint32_t i = 0; i < (1u << 22); ++i) {
            if (s_placed[s] == tile + 1u) {
              done = true;
              break;
            }
            if (s_abort) break;
            __nanosleep(64);
          }
          done = __all_sync(0xFFFFFFFFu, done);
        }
        if (!done) {
          s_abort = 1;
          if (lane == 0) atomicMax(&a.sc->status, (unsigned long long)kErrTimeout);
        } else {
          __threadfence_block();
          const bool skip = s_skip[s] != 0;
          for (uint32_t m = leaders; m; m &= m - 1u) {
            const uint32_t L = (uint32_t)__ffs(m) - 1u, tlp = (warp * 32u + L) / TT;
            const uint32_t meta_n = __shfl_sync(0xFFFFFFFFu, r.meta, L);  // the plane's three-sigma count
            if (!skip) {
              const uint8_t* tplane = stage + (uint64_t)tlp * pl.plane_bytes;
              const uint32_t* tsal = reinterpret_cast<const uint32_t*>(smem + pl.sm_sal + (uint64_t)tlp * pl.sm_sal_stride);
              const unsigned long long off16 = s_base16[s] + poff[tlp];
              SalientInfo info;
              info.size = sinfo[tlp * 4u + 0];
              info.nnz_s = sinfo[tlp * 4u + 1];
              info.n_dense = sinfo[tlp * 4u + 2];
              info.n_out_d = sinfo[tlp * 4u + 3];
              const bool raw = (raw_mask >> L) & 1u;
              SplitOut out;
              out.slot = d.dst + pl.slots_off + ((uint64_t)p0 + tlp) * pl.npay;
              out.ovf = d.dst + off16 * 16ull;
              out.npay = pl.npay;
              if (raw) raw_write(wteam, s_pl, tplane, out);
              else salient_write<DT>(wteam, s_pl, tplane, info, tsal, out);
              if (lane == 0) {
                Rec tr;
                tr.lo = 0.0f;
                tr.scale = 0.0f;
                tr.size = info.size;
                tr.meta = (meta_n & ~3u) | (raw ? kClsRaw : kClsSalient);
                store_table_entry(d, (uint64_t)p0 + tlp, a16(info.size) > pl.npay ? (uint32_t)off16 : 0u, tr);
              }
            }
            __syncwarp();
            if (lane == 0) ovf16[tlp] = 0;  // leave the array clean for the stage's next tile
          }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&s_empty[s]);
      }
      if (s_abort) break;
      s = s + 1 == nstage ? 0 : s + 1;
    }
  }
  cta_exit(pl, a, d);
}

// -------------------------------------------------------------------------------------------------
// CTA-team kernel: planes of more than 256 groups (whole 16-byte chunks).  One plane per tile, all
// NT threads of the CTA work on it.  The plane stays in its shared-memory stage and is swept two or
// three times (min/max; fixed-point moments; count + codes), so that few registers are needed and
// several CTAs fit an SM.  Thread 0 keeps the next ticket in flight while the CTA works.
// -------------------------------------------------------------------------------------------------
template <int DT>
__device__ __forceinline__ void lds_group(const uint8_t* plane, uint32_t g, float (&v)[4]) {
  if (DT == kF32) {
    const float4 t4 = reinterpret_cast<const float4*>(plane)[g];
    v[0] = t4.x; v[1] = t4.y; v[2] = t4.z; v[3] = t4.w;
  } else {
    const uint2 t2 = reinterpret_cast<const uint2*>(plane)[g];
    v[0] = __uint_as_float(t2.x << 16); v[1] = __uint_as_float(t2.x & 0xFFFF0000u);
    v[2] = __uint_as_float(t2.y << 16); v[3] = __uint_as_float(t2.y & 0xFFFF0000u);
  }
}

#define FH_CTA_STORE_CODES(BITS)                                                                              \
  {                                                                                                           \
    constexpr uint32_t bias = kMagicBits * (1u + (1u << (BITS)) + (1u << (2 * (BITS))) + (1u << (3 * (BITS)))); \
    _Pragma("unroll 2") for (uint32_t g = tid; g < groups; g += NT) {                                         \
      float v[4];                                                                                             \
      lds_group<DT>(plane, g, v);                                                                             \
      uint32_t word = __float_as_uint(__fmaf_rn(__fsub_rn(v[0], lo), inv, kMagicF));                          \
      word += __float_as_uint(__fmaf_rn(__fsub_rn(v[1], lo), inv, kMagicF)) << (BITS);                        \
      word += __float_as_uint(__fmaf_rn(__fsub_rn(v[2], lo), inv, kMagicF)) << (2 * (BITS));                  \
      word += __float_as_uint(__fmaf_rn(__fsub_rn(v[3], lo), inv, kMagicF)) << (3 * (BITS));                  \
      word -= bias;                                                                                           \
      if ((BITS) == 2) slot[g] = (uint8_t)word;                                                               \
      else if ((BITS) == 4) reinterpret_cast<uint16_t*>(slot)[g] = (uint16_t)word;                            \
      else reinterpret_cast<uint32_t*>(slot)[g] = word;                                                       \
      if (COUNT) {                                                                                            \
        if (one_sided) {                                                                                      \
          c0 += (v[0] > thi) + (v[2] > thi);                                                                  \
          c1 += (v[1] > thi) + (v[3] > thi);                                                                  \
        } else {                                                                                              \
          c0 += ((v[0] > thi) || (v[0] < tlo)) + ((v[2] > thi) || (v[2] < tlo));                              \
          c1 += ((v[1] > thi) || (v[1] < tlo)) + ((v[3] > thi) || (v[3] < tlo));                              \
        }                                                                                                     \
      }                                                                                                       \
    }                                                                                                         \
  }

template <int DT, bool SIGMA, int NT>
__global__ void __launch_bounds__(NT) compress_cta(const Plan pl, const CompressArgs a) {
  constexpr int NW = NT / 32;
  constexpr bool COUNT = SIGMA;
  extern __shared__ __align__(128) uint8_t smem[];
  __shared__ double s_red[kMaxWarps * 5];
  __shared__ __align__(8) uint64_t s_full[kMaxStages];
  __shared__ uint32_t s_tiles[kMaxStages];
  __shared__ uint32_t s_skip, s_abort;
  __shared__ unsigned long long s_base16;
  __shared__ Plan s_pl;          // copies for the outlined slow path
  __shared__ CompressArgs s_a;

  const uint32_t tid = threadIdx.x, lane = tid & 31u, warp = tid >> 5;
  if (tid == 0) {
    s_pl = pl;
    s_a = a;
  }
  Rec* rec = reinterpret_cast<Rec*>(smem + pl.sm_rec);
  uint32_t* roff = reinterpret_cast<uint32_t*>(smem + pl.sm_rec + 16u);
  uint32_t* sal = reinterpret_cast<uint32_t*>(smem + pl.sm_sal);
  const Dest d = make_dest(pl, a);
  const Team team = make_team(NT, s_red);
  const uint32_t nstage = pl.nstage, groups = pl.groups, bits = (uint32_t)pl.bits;
  uint32_t rp = 0;
  if (!d.fits && tid == 0 && blockIdx.x == 0) atomicMax(&a.sc->status, (unsigned long long)kErrCapacity);

  if (tid == 0) {
    for (uint32_t s = 0; s < nstage; ++s) mbar_init(&s_full[s], 1);
    fence_mbar_init();
    s_abort = 0;
  }
  __syncthreads();
  uint32_t next_ticket = 0;  // thread 0: the ticket for the next load, requested one tile ahead
  auto issue = [&](uint32_t s) {
    const uint32_t t = next_ticket;
    s_tiles[s] = t;
    if (t < pl.ntiles) {
      fence_proxy_async();
      mbar_expect_tx(&s_full[s], (uint32_t)pl.plane_bytes);
      bulk_g2s(smem + pl.sm_tile + (uint64_t)s * pl.stage_bytes, a.src + (uint64_t)t * pl.plane_bytes,
               (uint32_t)pl.plane_bytes, &s_full[s]);
      next_ticket = (uint32_t)atomicAdd(&a.sc->ticket, 1ull);
    }
  };
  if (tid == 0) {
    next_ticket = (uint32_t)atomicAdd(&a.sc->ticket, 1ull);
    for (uint32_t s = 0; s < nstage; ++s) issue(s);
  }
  __syncthreads();

  uint32_t s = 0, phase = 0;
  for (;;) {
    const uint32_t tile = s_tiles[s];
    if (tile >= pl.ntiles) break;
    bool ready = mbar_wait(&s_full[s], (phase >> s) & 1u, 1u << 20);
    ready = __all_sync(0xFFFFFFFFu, ready);
    phase ^= 1u << s;
    if (!ready) s_abort = 1;
    const uint8_t* plane = smem + pl.sm_tile + (uint64_t)s * pl.stage_bytes;
    const uint64_t gp = tile;

    // ---- sweep 1: minimum and maximum
    float lo = __int_as_float(0x7F800000), hi = __int_as_float(0xFF800000), lo1 = lo, hi1 = hi;
    if (ready) {
#pragma unroll 2
      for (uint32_t g = tid; g < groups; g += 2 * NT) {
        float v[4];
        lds_group<DT>(plane, g, v);
        lo = min_nan(lo, min_nan(min3_nan(v[0], v[1], v[2]), v[3]));
        hi = max_nan(hi, max_nan(max3_nan(v[0], v[1], v[2]), v[3]));
        if (g + NT < groups) {
          lds_group<DT>(plane, g + NT, v);
          lo1 = min_nan(lo1, min_nan(min3_nan(v[0], v[1], v[2]), v[3]));
          hi1 = max_nan(hi1, max_nan(max3_nan(v[0], v[1], v[2]), v[3]));
        }
      }
    }
    lo = min_nan(lo, lo1);
    hi = max_nan(hi, hi1);
    team_minmax(team, lo, hi, rp);  // one barrier: also tells every thread about an abort
    if (s_abort) break;
    if (!(fabsf(__fsub_rn(hi, lo)) <= 3.402823466e38f) && tid == 0)
      atomicMax(&a.sc->status, (unsigned long long)kErrNonfinite);

    // ---- sweep 2: fixed-point moments, thresholds
    float tlo = 0.0f, thi = 0.0f;
    bool one_sided = true, need_count = false;
    if (SIGMA) {
      const SigmaScale sc = sigma_scale(lo, hi);
      uint32_t as = 0, aq = 0, ng = 0;
#pragma unroll 2
      for (uint32_t g = tid; g < groups; g += NT) {
        float v[4];
        lds_group<DT>(plane, g, v);
        sigma_addends4(v[0], v[1], v[2], v[3], sc, as, aq);
        ++ng;
      }
      long long Is, Iq;
      team_sum2(team, (int32_t)(as - ng * kMagicBits), (int32_t)(aq - ng * kMagicBits), Is, Iq, rp);
      sigma_thresholds(Is, Iq, sc, pl.inv_hw, tlo, thi);
      need_count = hi > thi || lo < tlo;  // otherwise no element can lie outside
      one_sided = lo >= tlo;
    }

    // ---- sweep 3: codes into the plane's slot (and the outlier count).  A plane that turns out
    // salient has its slot rewritten by the slow path below.
    float inv, scale;
    quant_params(lo, hi, (1u << bits) - 1u, inv, scale);
    uint8_t* slot = d.dst + pl.slots_off + gp * pl.npay;
    uint32_t c0 = 0, c1 = 0;
    if (d.fits && pl.mode != kModeAll) {
      if (!need_count) {
        thi = __int_as_float(0x7F800000);  // nothing is counted
        one_sided = true;
      }
      if (bits == 2u) FH_CTA_STORE_CODES(2)
      else if (bits == 4u) FH_CTA_STORE_CODES(4)
      else FH_CTA_STORE_CODES(8)
      const uint32_t code_bytes = groups * bits / 2u;
      for (uint32_t o = a4(code_bytes) + 4u * tid; o < pl.npay; o += 4u * NT) *reinterpret_cast<uint32_t*>(slot + o) = 0u;
      if (tid == 0)
        for (uint32_t o = code_bytes; o < a4(code_bytes); ++o) slot[o] = 0;
    } else if (SIGMA && need_count) {  // nothing may be stored: count only
      for (uint32_t g = tid; g < groups; g += NT) {
        float v[4];
        lds_group<DT>(plane, g, v);
#pragma unroll
        for (int e = 0; e < 4; ++e) c0 += (v[e] > thi) || (v[e] < tlo);
      }
    }
    uint32_t cls = kClsNormal, n_out = 0;
    if (SIGMA) {
      n_out = team_sum_u32(team, c0 + c1, rp);
      if ((uint64_t)n_out * pl.rho_den > (uint64_t)pl.rho_num * pl.HW) cls = kClsSalient;
    } else {
      if (pl.mode == kModeAll) cls = kClsSalient;
      __syncthreads();  // every thread is done with the stage
    }

    Rec r;
    r.lo = 0.0f;
    r.scale = 0.0f;
    r.size = 0;
    r.meta = cls | (n_out << 2);
    if (cls == kClsNormal) {
      r.lo = lo;
      r.scale = scale;
      if (tid == 0) {
        if (d.fits) store_table_entry(d, gp, (uint32_t)((pl.slots_off + gp * pl.npay) >> 4), r);
        if (pl.mode != kModeOff) scan_publish(a.scan, tile, 0u);
      }
    } else {
      // ---- slow path: the block-wise encoding of a salient plane, by the whole CTA
      const SalientInfo info = salient_measure<DT>(team, s_pl, plane, sal);
      r.size = info.size;
      if (a16(info.size) >= a16((uint32_t)pl.plane_bytes)) {
        r.meta = (r.meta & ~3u) | kClsRaw;
        r.size = (uint32_t)pl.plane_bytes;
      }
      if (tid == 0) rec[0] = r;
      __syncthreads();
      if (warp == 0) tile_place(s_pl, s_a, d, tile, 1u, rec, roff, &s_base16, &s_skip);
      __syncthreads();
      if (!s_skip) {
        SplitOut out;
        out.slot = slot;
        out.ovf = d.dst + (s_base16 + roff[0]) * 16ull;
        out.npay = pl.npay;
        if ((r.meta & 3u) == kClsRaw) raw_write(team, s_pl, plane, out);
        else salient_write<DT>(team, s_pl, plane, info, sal, out);
        if (tid == 0) store_table_entry(d, gp, a16(r.size) > pl.npay ? (uint32_t)(s_base16 + roff[0]) : 0u, r);
      }
      __syncthreads();
    }
    // ---- the stage is free: next load (thread 0), next stage
    if (tid == 0) issue(s);
    s = s + 1 == nstage ? 0 : s + 1;
    // s_tiles[s] for the next iteration was written at least one barrier ago (nstage >= 2)
  }

  if (s_abort && tid == 0) {  // a load timed out: report, then wait (bounded) for copies still in flight
    atomicMax(&a.sc->status, (unsigned long long)kErrTimeout);
    for (uint32_t k = 0; k < nstage; ++k)
      if (s_tiles[k] < pl.ntiles) {
        mbar_wait(&s_full[k], 0u, 1u << 10);
        mbar_wait(&s_full[k], 1u, 1u << 10);
      }
  }
  cta_exit(pl, a, d);
}

}  // namespace fh
