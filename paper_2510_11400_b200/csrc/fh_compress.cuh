// Compress kernels.
//
// Container recap: every plane owns a slot of npay bytes at a closed-form offset; a normal plane's
// codes fill its slot; the payload of an outlier-rich (salient) or raw plane runs through its slot and
// continues in the overflow region, in plane order.
//
// A call is ONE kernel, one pass over the dense tensor.  Tiles (runs of consecutive planes) are handed
// out in order by a ticket.  Per plane: statistics, three-sigma class, and
//   normal plane:   codes and table entry, written at once (the slot's offset is closed-form);
//   other planes:   measured at once while they lie in shared memory (block classes, CSR and code sizes,
//                   salient versus raw); the tile publishes the overflow size of its planes, obtains the sum
//                   over all earlier tiles from the placement scan (fh_device.cuh) and writes the payloads.
// Three variants by plane size:
//   compress_warp<DT, SIGMA, TT, FULLVEC>  planes of at most 256 groups: bulk-copy (TMA) pipeline, a sub-warp
//       team per plane, groups kept in registers; a warp handles the outlier-rich planes of its slice;
//   compress_cta<DT, SIGMA, NT>            larger planes of whole 16-byte chunks: one plane per CTA and tile;
//   compress_generic<DT, BITS>             everything else (ragged large planes, random rounding).
// The kernel's last CTA writes the header and the result words and returns the scratch to its idle state.
#pragma once

#include "fh_device.cuh"

namespace fh {

struct SalientInfo {
  uint32_t nnz_s, n_dense, n_out_d, size;
  uint32_t coded;  // bytes of the Huffman-coded section that replaces the dense blocks' code bytes; 0: plain codes
};

struct CompressArgs {
  const uint8_t* src;
  uint8_t* dst_base;
  unsigned long long capacity;          // bytes available at dst_base (minus the offset below)
  const unsigned long long* d_off_in;   // optional: byte offset of the container in dst_base
  unsigned long long* d_off_out;        // optional: offset for the next container
  unsigned long long* out2;             // optional: {total bytes, status}
  Scratch* sc;
  Scan scan;                            // placement of overflow parts (unused with salient_mode OFF)
  uint32_t* defer_next;                 // one word per tile: links the tiles a CTA has put off (see BlockCtl)
  uint32_t parity;                      // which of the two ticket counters this call uses
  uint32_t early_ticket;                // 1: tiles may be requested before the previous kernel on the stream has completed
  // channel-wide three-sigma mode: per-channel outlier counts and per-plane counts from the statistics passes
  const unsigned long long* chan_nout;  // stride: 4 words (see ChanStat)
  const uint32_t* plane_nout;
};

// Class and outlier count of plane gp when mu and sigma are taken per channel over the batch (the class is
// the channel's) or over the whole tensor (the class follows from the plane's own count).
__device__ __forceinline__ uint32_t channel_class(const Plan& pl, const CompressArgs& a, uint64_t gp, uint32_t& n_out) {
  n_out = a.plane_nout[gp];
  if (pl.mode == kModeTensor)
    return (uint64_t)n_out * pl.rho_den > (uint64_t)pl.rho_num * pl.HW ? kClsSalient : kClsNormal;
  const unsigned long long total = a.chan_nout[(gp % pl.C) * 4ull];
  return total * pl.rho_den > (unsigned long long)pl.rho_num * pl.N * pl.HW ? kClsSalient : kClsNormal;
}

// A CTA whose threads change one of the call's counters (error code, overflow size, plane counts) notes it in
// this flag; cta_exit passes it on through the exit counter, so that the last CTA of a call in which nobody did
// -- every plane normal, no error: the usual case -- neither fences nor reads the counters back.
__device__ __forceinline__ volatile uint32_t* cta_dirty() {
  __shared__ uint32_t flag;
  return &flag;
}
__device__ __forceinline__ void report_error(const CompressArgs& a, uint32_t code) {
  *cta_dirty() = 1u;
  atomicMax(&a.sc->status, (unsigned long long)code);
}

// Where the bytes of a salient / raw payload go: offsets below npay land in the plane's slot, the
// rest in its overflow part.  Offsets and npay are multiples of the access size.
struct SplitOut {
  uint8_t* slot;
  uint8_t* ovf;
  uint32_t npay;
  __device__ __forceinline__ uint8_t* at(uint32_t o) const { return o < npay ? slot + o : ovf + (o - npay); }
  __device__ __forceinline__ void st32(uint32_t o, uint32_t v) const { *reinterpret_cast<uint32_t*>(at(o)) = v; }
  __device__ __forceinline__ void st16(uint32_t o, uint32_t v) const { *reinterpret_cast<uint16_t*>(at(o)) = (uint16_t)v; }
  __device__ __forceinline__ void st8(uint32_t o, uint32_t v) const { *at(o) = (uint8_t)v; }
};

// One 8x8 block in the registers of a warp: lane l holds the elements (l >> 3, l & 7) and
// ((l >> 3) + 4, l & 7) of the block, i.e. raster positions l and l + 32.  Positions outside the
// plane count as value 0.
struct BlockRegs {
  float x0, x1;    // values (rows 0-3, rows 4-7)
  bool in0, in1;   // the positions lie inside the plane
  uint32_t idx0;   // plane index of the first position; the second is idx0 + 4 W
};
template <int DT>
__device__ __forceinline__ BlockRegs block_load(const uint8_t* plane, int H, int W, int by, int bx, uint32_t lane) {
  BlockRegs r;
  const int y0 = by * 8 + (int)(lane >> 3), x = bx * 8 + (int)(lane & 7u);
  r.in0 = y0 < H && x < W;
  r.in1 = y0 + 4 < H && x < W;
  r.idx0 = (uint32_t)y0 * (uint32_t)W + (uint32_t)x;
  r.x0 = r.in0 ? load_elem<DT>(plane, r.idx0) : 0.0f;
  r.x1 = r.in1 ? load_elem<DT>(plane, r.idx0 + 4u * (uint32_t)W) : 0.0f;
  return r;
}

// Residual codes of a dense block (Eq. 7-9): first-order Lorenzo prediction on the pre-quantised
// integers k, neighbours outside the block count as 0.  Every element is independent because
// prediction runs on k, which follows from the input alone; the neighbours' k come from the other
// lanes by shuffle.  code0/code1: the lane's two code bytes; m0/m1: ballots of the verbatim elements.
__device__ __forceinline__ void block_codes(const BlockRegs& r, float inv2e, uint32_t lane, uint32_t& code0,
                                            uint32_t& code1, uint32_t& m0, uint32_t& m1) {
  const uint32_t full = 0xFFFFFFFFu, c = lane & 7u, r0 = lane >> 3;
  bool big0, big1;
  const int32_t k0 = dense_k(r.x0, inv2e, &big0), k1 = dense_k(r.x1, inv2e, &big1);
  int32_t left0 = __shfl_up_sync(full, k0, 1), up0 = __shfl_up_sync(full, k0, 8), ul0 = __shfl_up_sync(full, k0, 9);
  int32_t left1 = __shfl_up_sync(full, k1, 1), up1 = __shfl_up_sync(full, k1, 8), ul1 = __shfl_up_sync(full, k1, 9);
  const int32_t up1r = __shfl_sync(full, k0, 24 + (int)c), ul1r = __shfl_sync(full, k0, 23 + (int)c);  // row 3 feeds row 4
  if (r0 == 0) {
    up0 = 0;
    ul0 = 0;
    up1 = up1r;
    ul1 = ul1r;
  }
  if (c == 0) {
    left0 = 0;
    ul0 = 0;
    left1 = 0;
    ul1 = 0;
  }
  const int32_t d0 = k0 - (up0 + left0 - ul0), d1 = k1 - (up1 + left1 - ul1);
  const bool v0 = r.in0 && (big0 || d0 > 127 || d0 < -127), v1 = r.in1 && (big1 || d1 > 127 || d1 < -127);
  code0 = !r.in0 ? 128u : (v0 ? 0u : (uint32_t)(d0 + 128));
  code1 = !r.in1 ? 128u : (v1 ? 0u : (uint32_t)(d1 + 128));
  m0 = __ballot_sync(full, v0);
  m1 = __ballot_sync(full, v1);
}

// Block-wise path, measuring part (Section 4.4.1): one pass over the plane's 8x8 blocks, a warp per
// block.  The non-zero mask of a block is two ballots; its pooled density against tau says dense or
// sparse; a sparse block adds its row counts to the CSR row counters, a dense block is coded once to
// count its verbatim elements.  The team is a whole warp or a whole CTA.  Leaves in shared scratch:
// rowp[0..H] = CSR row pointers, blk_a[b] = 1 for dense blocks, blk_b[b] = rank of block b among the
// dense blocks, blk_c[b] = index of the block's first verbatim value.
template <int DT>
__device__ __noinline__ SalientInfo salient_measure(const Team& t, const Plan& pl, const uint8_t* plane, uint32_t* sal) {
  uint32_t* rowp = sal;
  uint32_t* blk_a = sal + pl.H + 1;
  uint32_t* blk_b = blk_a + pl.nblk;
  uint32_t* blk_c = blk_b + pl.nblk;
  const int H = pl.H, W = pl.W;
  const uint32_t nblk = pl.nblk, nbx = pl.nbx;
  const uint32_t nw = t.block ? t.nwarps : 1u, wid = t.block ? threadIdx.x >> 5 : 0u, lane32 = threadIdx.x & 31u;
  const float inv2e = __fdiv_rn(1.0f, __fmul_rn(2.0f, pl.eps));
  for (uint32_t y = t.lane; y <= (uint32_t)H; y += t.size) rowp[y] = 0;
  team_sync(t);
  for (uint32_t b = wid; b < nblk; b += nw) {
    const uint32_t by = b / nbx, bx = b - by * nbx;
    const BlockRegs r = block_load<DT>(plane, H, W, (int)by, (int)bx, lane32);
    const uint32_t z0 = __ballot_sync(0xFFFFFFFFu, r.x0 != 0.0f), z1 = __ballot_sync(0xFFFFFFFFu, r.x1 != 0.0f);
    const uint32_t nnz = __popc(z0) + __popc(z1);
    const bool dense = (uint64_t)nnz * pl.tau_den >= (uint64_t)pl.tau_num * 64u;
    uint32_t n_out = 0;
    if (dense) {
      uint32_t c0, c1, m0, m1;
      block_codes(r, inv2e, lane32, c0, c1, m0, m1);
      n_out = __popc(m0) + __popc(m1);
    } else if (lane32 < 8u) {  // lane r: non-zeros of row r of the block
      const uint32_t cnt = __popc(((lane32 < 4u ? z0 : z1) >> ((lane32 & 3u) * 8u)) & 0xFFu);
      if (cnt) atomicAdd(&rowp[by * 8u + lane32], cnt);
    }
    if (lane32 == 0) {
      blk_a[b] = dense;
      blk_b[b] = dense;
      blk_c[b] = n_out;
    }
  }
  team_sync(t);
  SalientInfo info;
  info.n_dense = team_excl_scan(t, blk_b, nblk);
  info.nnz_s = team_excl_scan(t, rowp, (uint32_t)H + 1u);
  info.n_out_d = team_excl_scan(t, blk_c, nblk);
  info.coded = 0;
  if (pl.entropy && info.n_dense) {
    // Huffman stage (Section 4.4.1): histogram of the plane's code bytes, the code, the size of every chunk
    uint32_t* blk_d = blk_c + nblk;   // bytes of a dense block's chunk
    uint32_t* blk_e = blk_d + nblk;   // ... and where it starts
    HufEncode* h = reinterpret_cast<HufEncode*>(blk_e + nblk);
    for (uint32_t i = t.lane; i < 256u; i += t.size) h->hist[i] = 0;
    team_sync(t);
    for (uint32_t b = wid; b < nblk; b += nw) {
      if (!blk_a[b]) continue;
      const uint32_t by = b / nbx, bx = b - by * nbx;
      const BlockRegs r = block_load<DT>(plane, H, W, (int)by, (int)bx, lane32);
      uint32_t c0, c1, m0, m1;
      block_codes(r, inv2e, lane32, c0, c1, m0, m1);
      atomicAdd(&h->hist[c0], 1u);
      atomicAdd(&h->hist[c1], 1u);
    }
    team_sync(t);
    if (t.lane == 0) huffman_build(h);
    team_sync(t);
    if (h->maxlen <= kHufMaxLen) {
      for (uint32_t b = wid; b < nblk; b += nw) {
        uint32_t bits = 0;
        if (blk_a[b]) {
          const uint32_t by = b / nbx, bx = b - by * nbx;
          const BlockRegs r = block_load<DT>(plane, H, W, (int)by, (int)bx, lane32);
          uint32_t c0, c1, m0, m1;
          block_codes(r, inv2e, lane32, c0, c1, m0, m1);
          bits = (uint32_t)h->len[c0] + (uint32_t)h->len[c1];
          asm volatile("redux.sync.add.u32 %0, %0, %1;" : "+r"(bits) : "r"(0xFFFFFFFFu));
        }
        if (lane32 == 0) blk_d[b] = blk_e[b] = (bits + 7u) >> 3;
      }
      team_sync(t);
      const uint32_t chunks = team_excl_scan(t, blk_e, nblk);
      const uint32_t section = a4(4u + a4(h->nlens) + a4(info.n_dense) + chunks);
      if (section < 64u * info.n_dense) info.coded = section;
    }
  }
  const uint32_t e = (uint32_t)pl.esize;
  info.size = 16u + 4u * pl.nbm + 4u * ((uint32_t)H + 1u) + a4(2u * info.nnz_s) + a4(e * info.nnz_s) +
              (info.coded ? info.coded : 64u * info.n_dense) + a4(e * info.n_out_d);
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
  const uint32_t o_outl = o_codes + (info.coded ? info.coded : 64u * info.n_dense);
  if (t.lane == 0) {
    out.st32(0, info.nnz_s);
    out.st32(4, info.n_dense);
    out.st32(8, info.n_out_d);
    out.st32(12, info.coded);
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
  if (info.nnz_s) {
    for (int y = (int)wid; y < H; y += (int)nw) {
      uint32_t o = rowp[y];
      if (o == rowp[y + 1]) continue;
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
  }
  // dense blocks: 64 code bytes each (or their Huffman-coded chunk), verbatim values in raster order
  const float inv2e = __fdiv_rn(1.0f, __fmul_rn(2.0f, pl.eps));
  const uint32_t lt = (1u << lane32) - 1u;
  const uint32_t* blk_d = blk_c + nblk;
  const uint32_t* blk_e = blk_d + nblk;
  HufEncode* h = reinterpret_cast<HufEncode*>(const_cast<uint32_t*>(blk_e + nblk));  // (only looked at when info.coded)
  uint32_t o_chunks = 0;
  if (info.coded) {  // the section's head: code lengths, then the bytes of every chunk; pads are zero
    const uint32_t nl = h->nlens, o_cb = o_codes + 4u + a4(nl);
    o_chunks = o_cb + a4(info.n_dense);
    if (t.lane == 0) {
      out.st8(o_codes, h->len[0]);
      out.st8(o_codes + 1u, h->smin);
      out.st8(o_codes + 2u, h->smax);
      out.st8(o_codes + 3u, 0);
      for (uint32_t o = o_codes + 4u + nl; o < o_cb; ++o) out.st8(o, 0);
      for (uint32_t o = o_cb + info.n_dense; o < o_chunks; ++o) out.st8(o, 0);
      uint32_t last_end = 0;  // end of the chunks: the last dense block's start + bytes
      for (uint32_t b = nblk; b-- > 0;)
        if (blk_a[b]) {
          last_end = blk_e[b] + blk_d[b];
          break;
        }
      for (uint32_t o = o_chunks + last_end; o < o_codes + info.coded; ++o) out.st8(o, 0);
    }
    for (uint32_t i = t.lane; i < nl; i += t.size) out.st8(o_codes + 4u + i, h->len[h->smin + i]);
    for (uint32_t b = t.lane; b < nblk; b += t.size)
      if (blk_a[b]) out.st8(o_cb + blk_b[b], blk_d[b]);
  }
  for (uint32_t b = wid; b < nblk; b += nw) {
    if (!blk_a[b]) continue;
    const uint32_t by = b / nbx, bx = b - by * nbx;
    const BlockRegs r = block_load<DT>(plane, H, W, (int)by, (int)bx, lane32);
    uint32_t c0, c1, m0, m1;
    block_codes(r, inv2e, lane32, c0, c1, m0, m1);
    const uint32_t oc = o_codes + 64u * blk_b[b], oo = o_outl + e * blk_c[b];
    if ((m0 >> lane32) & 1u) {
      const uint32_t rank = __popc(m0 & lt);
      if (DT == kF32) out.st32(oo + 4u * rank, reinterpret_cast<const uint32_t*>(plane)[r.idx0]);
      else out.st16(oo + 2u * rank, reinterpret_cast<const uint16_t*>(plane)[r.idx0]);
    }
    if ((m1 >> lane32) & 1u) {
      const uint32_t rank = __popc(m0) + __popc(m1 & lt), idx1 = r.idx0 + 4u * (uint32_t)W;
      if (DT == kF32) out.st32(oo + 4u * rank, reinterpret_cast<const uint32_t*>(plane)[idx1]);
      else out.st16(oo + 2u * rank, reinterpret_cast<const uint16_t*>(plane)[idx1]);
    }
    if (info.coded) {
      // the chunk's bits are assembled in shared memory (a code goes in most significant bit first, the words
      // hold the stream big-endian) and leave byte by byte
      uint32_t* stg = h->stage[wid];
      for (uint32_t i = lane32; i < kHufStageWords; i += 32u) stg[i] = 0;
      __syncwarp();
      const uint32_t l0 = h->len[c0], l1 = h->len[c1];
      uint32_t i0 = l0, i1 = l1;  // inclusive prefix sums of the lengths, raster positions l and l + 32
      for (uint32_t o = 1; o < 32u; o <<= 1) {
        const uint32_t u0 = __shfl_up_sync(0xFFFFFFFFu, i0, o), u1 = __shfl_up_sync(0xFFFFFFFFu, i1, o);
        if (lane32 >= o) {
          i0 += u0;
          i1 += u1;
        }
      }
      const uint32_t first_half = __shfl_sync(0xFFFFFFFFu, i0, 31);
#pragma unroll
      for (int half = 0; half < 2; ++half) {
        const uint32_t len = half ? l1 : l0, at = half ? first_half + i1 - l1 : i0 - l0, cv = h->code[half ? c1 : c0];
        const uint32_t wi = at >> 5;
        const int shift = 32 - (int)(at & 31u) - (int)len;
        if (shift >= 0) {
          atomicOr(&stg[wi], cv << shift);
        } else {
          atomicOr(&stg[wi], cv >> (-shift));
          atomicOr(&stg[wi + 1u], cv << (32 + shift));
        }
      }
      __syncwarp();
      for (uint32_t j = lane32; j < blk_d[b]; j += 32u) out.st8(o_chunks + blk_e[b] + j, (stg[j >> 2] >> (24u - 8u * (j & 3u))) & 0xFFu);
      __syncwarp();
      continue;
    }
    uint32_t w0 = c0 | (__shfl_down_sync(0xFFFFFFFFu, c0, 1) << 8);
    w0 |= __shfl_down_sync(0xFFFFFFFFu, w0, 2) << 16;
    uint32_t w1 = c1 | (__shfl_down_sync(0xFFFFFFFFu, c1, 1) << 8);
    w1 |= __shfl_down_sync(0xFFFFFFFFu, w1, 2) << 16;
    if ((lane32 & 3u) == 0u) {
      out.st32(oc + lane32, w0);
      out.st32(oc + 32u + lane32, w1);
    }
  }
}

// Raw plane: verbatim copy through the slot into the overflow part, zero padded.
__device__ __noinline__ void raw_write(const Team& t, const Plan& pl, const uint8_t* plane, const SplitOut& out) {
  const uint32_t n = (uint32_t)pl.plane_bytes, end = max(pl.npay, a16(n));
  for (uint32_t o = 2u * t.lane; o < end; o += 2u * t.size)
    out.st16(o, o < n ? (uint32_t)*reinterpret_cast<const uint16_t*>(plane + o) : 0u);
}

// -------------------------------------------------------------------------------------------------
// Small planes (at most kSmallBlocks blocks and fewer than 32 rows: 7x7, 8x8, 14x14, 16x16, ...) take the
// block-wise path in the registers of one warp: no measuring scratch, no second look at the plane.  The
// results are those of salient_measure / salient_write.
// -------------------------------------------------------------------------------------------------
constexpr uint32_t kSmallBlocks = 4;
__device__ __forceinline__ bool is_small_plane(const Plan& pl) { return pl.nblk <= kSmallBlocks && pl.H < 32; }

struct SmallBlocks {
  uint32_t z0[kSmallBlocks], z1[kSmallBlocks];  // non-zero masks of the block's two halves (ballots)
  uint32_t m0[kSmallBlocks], m1[kSmallBlocks];  // verbatim elements of a dense block (ballots)
  uint32_t c0[kSmallBlocks], c1[kSmallBlocks];  // this lane's two residual codes
  uint32_t w0[kSmallBlocks], w1[kSmallBlocks];  // this lane's two elements, verbatim bits
  uint32_t dense;                               // bit b: block b is dense
  uint32_t rowp;                                // lane y: CSR row pointer of row y; lane H: nnz_s
  SalientInfo info;
};
// Non-zero bits of row rr (0..7) of a block.
__device__ __forceinline__ uint32_t block_row_bits(uint32_t z0, uint32_t z1, uint32_t rr) {
  return ((rr < 4u ? z0 : z1) >> ((rr & 3u) * 8u)) & 0xFFu;
}

template <int DT>
__device__ __forceinline__ void small_blocks(const Plan& pl, const uint8_t* plane, SmallBlocks& sb) {
  const uint32_t lane = threadIdx.x & 31u, full = 0xFFFFFFFFu;
  const float inv2e = __fdiv_rn(1.0f, __fmul_rn(2.0f, pl.eps));
  sb.dense = 0;
  uint32_t n_dense = 0, n_out_d = 0;
#pragma unroll
  for (uint32_t b = 0; b < kSmallBlocks; ++b) {
    sb.z0[b] = sb.z1[b] = sb.m0[b] = sb.m1[b] = 0;
    sb.c0[b] = sb.c1[b] = 128u;
    sb.w0[b] = sb.w1[b] = 0;
    if (b < pl.nblk) {
      const uint32_t by = b / pl.nbx, bx = b - by * pl.nbx;
      const BlockRegs r = block_load<DT>(plane, pl.H, pl.W, (int)by, (int)bx, lane);
      sb.w0[b] = DT == kF32 ? __float_as_uint(r.x0) : __float_as_uint(r.x0) >> 16;
      sb.w1[b] = DT == kF32 ? __float_as_uint(r.x1) : __float_as_uint(r.x1) >> 16;
      sb.z0[b] = __ballot_sync(full, r.x0 != 0.0f);
      sb.z1[b] = __ballot_sync(full, r.x1 != 0.0f);
      const uint32_t nnz = __popc(sb.z0[b]) + __popc(sb.z1[b]);
      if ((uint64_t)nnz * pl.tau_den >= (uint64_t)pl.tau_num * 64u) {  // (the same for every lane)
        sb.dense |= 1u << b;
        ++n_dense;
        block_codes(r, inv2e, lane, sb.c0[b], sb.c1[b], sb.m0[b], sb.m1[b]);
        n_out_d += __popc(sb.m0[b]) + __popc(sb.m1[b]);
      }
    }
  }
  // CSR row pointers: lane y counts the non-zeros of row y that lie in sparse blocks
  uint32_t cnt = 0;
  {
    const uint32_t by = lane >> 3, rr = lane & 7u;
#pragma unroll
    for (uint32_t b = 0; b < kSmallBlocks; ++b)
      if (b < pl.nblk && !((sb.dense >> b) & 1u) && b / pl.nbx == by && lane < (uint32_t)pl.H)
        cnt += __popc(block_row_bits(sb.z0[b], sb.z1[b], rr));
  }
  uint32_t incl = cnt;
  for (uint32_t o = 1; o < 32u; o <<= 1) {
    const uint32_t up = __shfl_up_sync(full, incl, o);
    if (lane >= o) incl += up;
  }
  sb.rowp = incl - cnt;
  const uint32_t nnz_s = __shfl_sync(full, incl, 31), e = (uint32_t)pl.esize;
  sb.info.nnz_s = nnz_s;
  sb.info.n_dense = n_dense;
  sb.info.n_out_d = n_out_d;
  sb.info.coded = 0;
  sb.info.size = 16u + 4u * pl.nbm + 4u * ((uint32_t)pl.H + 1u) + a4(2u * nnz_s) + a4(e * nnz_s) + 64u * n_dense +
                 a4(e * n_out_d);
}

template <int DT>
__device__ __forceinline__ void small_write(const Plan& pl, const SmallBlocks& sb, const SplitOut& out) {
  const uint32_t lane = threadIdx.x & 31u, full = 0xFFFFFFFFu, e = (uint32_t)pl.esize, H = (uint32_t)pl.H;
  const SalientInfo& info = sb.info;
  const uint32_t o_bm = 16u, o_rp = o_bm + 4u * pl.nbm, o_col = o_rp + 4u * (H + 1u);
  const uint32_t o_val = o_col + a4(2u * info.nnz_s), o_codes = o_val + a4(e * info.nnz_s);
  const uint32_t o_outl = o_codes + 64u * info.n_dense;
  if (lane == 0) {
    out.st32(0, info.nnz_s);
    out.st32(4, info.n_dense);
    out.st32(8, info.n_out_d);
    out.st32(12, 0);
    out.st32(o_bm, sb.dense);  // (at most kSmallBlocks blocks: one bitmap word)
    // pads the section writers leave: col (2 bytes), val / verbatim values (bf16: 2 bytes)
    if (info.nnz_s & 1u) out.st16(o_col + 2u * info.nnz_s, 0);
    if (DT == kBF16 && (info.nnz_s & 1u)) out.st16(o_val + 2u * info.nnz_s, 0);
    if (DT == kBF16 && (info.n_out_d & 1u)) out.st16(o_outl + 2u * info.n_out_d, 0);
  }
  // zero padding up to the end of the slot / of the 16-byte padded overflow part
  const uint32_t end = max(pl.npay, a16(info.size));
  for (uint32_t o = info.size + 4u * lane; o < end; o += 128u) out.st32(o, 0);
  if (lane <= H) out.st32(o_rp + 4u * lane, sb.rowp);
  const uint32_t lt = (1u << lane) - 1u, c = lane & 7u, r0 = lane >> 3;
  uint32_t dense_rank = 0, outl_at = 0;
#pragma unroll
  for (uint32_t b = 0; b < kSmallBlocks; ++b) {
    if (b >= pl.nblk) continue;
    const uint32_t by = b / pl.nbx, bx = b - by * pl.nbx;
    if ((sb.dense >> b) & 1u) {
      const uint32_t oc = o_codes + 64u * dense_rank, oo = o_outl + e * outl_at;
      if ((sb.m0[b] >> lane) & 1u) {
        const uint32_t rank = __popc(sb.m0[b] & lt);
        if (DT == kF32) out.st32(oo + 4u * rank, sb.w0[b]);
        else out.st16(oo + 2u * rank, sb.w0[b]);
      }
      if ((sb.m1[b] >> lane) & 1u) {
        const uint32_t rank = __popc(sb.m0[b]) + __popc(sb.m1[b] & lt);
        if (DT == kF32) out.st32(oo + 4u * rank, sb.w1[b]);
        else out.st16(oo + 2u * rank, sb.w1[b]);
      }
      uint32_t v0 = sb.c0[b] | (__shfl_down_sync(full, sb.c0[b], 1) << 8);
      v0 |= __shfl_down_sync(full, v0, 2) << 16;
      uint32_t v1 = sb.c1[b] | (__shfl_down_sync(full, sb.c1[b], 1) << 8);
      v1 |= __shfl_down_sync(full, v1, 2) << 16;
      if ((lane & 3u) == 0u) {
        out.st32(oc + lane, v0);
        out.st32(oc + 32u + lane, v1);
      }
      ++dense_rank;
      outl_at += __popc(sb.m0[b]) + __popc(sb.m1[b]);
    } else {
      // CSR entries of the block's two halves: row pointer of the element's row, plus the non-zeros of that
      // row in sparse blocks to the left, plus those before it in the block's row
#pragma unroll
      for (uint32_t half = 0; half < 2u; ++half) {
        const uint32_t rr = r0 + 4u * half, y = by * 8u + rr;
        uint32_t pos = __shfl_sync(full, sb.rowp, (int)(y & 31u));
#pragma unroll
        for (uint32_t bl = 0; bl < kSmallBlocks; ++bl)
          if (bl < b && bl / pl.nbx == by && !((sb.dense >> bl) & 1u)) pos += __popc(block_row_bits(sb.z0[bl], sb.z1[bl], rr));
        const uint32_t bits = block_row_bits(sb.z0[b], sb.z1[b], rr);
        pos += __popc(bits & ((1u << c) - 1u));
        if ((bits >> c) & 1u) {
          out.st16(o_col + 2u * pos, bx * 8u + c);
          const uint32_t w = half ? sb.w1[b] : sb.w0[b];
          if (DT == kF32) out.st32(o_val + 4u * pos, w);
          else out.st16(o_val + 2u * pos, w);
        }
      }
    }
  }
}

// A warp measures an outlier-rich plane that lies in shared memory: small planes in registers, others through
// the measuring scratch `sal`.
template <int DT>
__device__ __forceinline__ SalientInfo warp_plane_measure(const Team& warp_team, const Plan& pl, const uint8_t* plane,
                                                          uint32_t* sal) {
  if (is_small_plane(pl)) {
    SmallBlocks sb;
    small_blocks<DT>(pl, plane, sb);
    return sb.info;
  }
  return salient_measure<DT>(warp_team, pl, plane, sal);
}

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

__device__ __forceinline__ uint32_t salient_size(const Plan& pl, uint32_t nnz_s, uint32_t n_dense, uint32_t n_out_d) {
  const uint32_t e = (uint32_t)pl.esize;
  return 16u + 4u * pl.nbm + 4u * ((uint32_t)pl.H + 1u) + a4(2u * nnz_s) + a4(e * nnz_s) + 64u * n_dense +
         a4(e * n_out_d);
}
// Overflow size, in 16-byte units, of a payload of `size` bytes.
__device__ __forceinline__ uint32_t ovf_units(const Plan& pl, uint32_t size) {
  return a16(size) > pl.npay ? (a16(size) - pl.npay) >> 4 : 0u;
}
// A measured plane is stored salient, or raw when that would not be smaller; returns its overflow units.
__device__ __forceinline__ uint32_t plane_units(const Plan& pl, const SalientInfo& info, bool& raw) {
  raw = a16(info.size) >= a16((uint32_t)pl.plane_bytes);
  return ovf_units(pl, raw ? (uint32_t)pl.plane_bytes : info.size);
}

// Per-call counters of a tile's outlier-rich planes (one thread): nsal and nraw share a word.
__device__ __forceinline__ void count_blockwise(const CompressArgs& a, uint32_t units, uint32_t nsal, uint32_t nraw) {
  if (units | nsal | nraw) *cta_dirty() = 1u;
  if (units) atomicAdd(&a.sc->ovf16, (unsigned long long)units);
  if (nsal | nraw) atomicAdd(&a.sc->nsal, (unsigned long long)nsal | ((unsigned long long)nraw << 32));
}

// Writes the payload of the measured plane gp (`plane` in shared memory, `info` and `sal` from
// salient_measure) with its overflow part `at` units into the overflow region, and its table entry.
template <int DT>
__device__ __forceinline__ void write_blockwise(const Team& t, const Plan& pl, const Dest& d, uint64_t gp,
                                                const uint8_t* plane, const SalientInfo& info, const uint32_t* sal,
                                                uint32_t n_out, uint32_t at) {
  bool raw;
  const uint32_t my_units = plane_units(pl, info, raw);
  const unsigned long long off16 = (pl.ovf_off >> 4) + at;
  if (!d.fits || (off16 + my_units) * 16ull > d.capacity) return;  // never write past the capacity
  SplitOut out;
  out.slot = d.dst + pl.slots_off + gp * pl.npay;
  out.ovf = d.dst + off16 * 16ull;
  out.npay = pl.npay;
  if (raw) raw_write(t, pl, plane, out);
  else salient_write<DT>(t, pl, plane, info, sal, out);
  if (t.lane == 0)
    reinterpret_cast<uint4*>(d.dst + 64)[gp] =
        make_uint4(my_units ? (uint32_t)off16 : 0u, (raw ? kClsRaw : kClsSalient) | (n_out << 2), 0u, 0u);
}

// A warp measures the outlier-rich plane gp (in shared memory) and writes it with its overflow part `at` units
// into the overflow region: small planes in registers, others through the measuring scratch `sal`.
template <int DT>
__device__ __forceinline__ void warp_plane_write(const Team& warp_team, const Plan& pl, const Dest& d, uint64_t gp,
                                                 const uint8_t* plane, uint32_t* sal, uint32_t n_out, uint32_t at) {
  if (!is_small_plane(pl)) {
    const SalientInfo info = salient_measure<DT>(warp_team, pl, plane, sal);
    write_blockwise<DT>(warp_team, pl, d, gp, plane, info, sal, n_out, at);
    return;
  }
  SmallBlocks sb;
  small_blocks<DT>(pl, plane, sb);
  bool raw;
  const uint32_t my_units = plane_units(pl, sb.info, raw);
  const unsigned long long off16 = (pl.ovf_off >> 4) + at;
  if (!d.fits || (off16 + my_units) * 16ull > d.capacity) return;  // never write past the capacity
  SplitOut out;
  out.slot = d.dst + pl.slots_off + gp * pl.npay;
  out.ovf = d.dst + off16 * 16ull;
  out.npay = pl.npay;
  if (raw) raw_write(warp_team, pl, plane, out);
  else small_write<DT>(pl, sb, out);
  if (warp_team.lane == 0)
    reinterpret_cast<uint4*>(d.dst + 64)[gp] =
        make_uint4(my_units ? (uint32_t)off16 : 0u, (raw ? kClsRaw : kClsSalient) | (n_out << 2), 0u, 0u);
}

// One thread, after everything else of the call is done: header, result words, and every counter the
// call touched back to zero.
// `touched`: some CTA of the call has changed a counter; otherwise all of them are known to be zero.
__device__ __forceinline__ void finalize(const Plan& pl, const CompressArgs& a, const Dest& d, bool touched) {
  unsigned long long ovf16 = 0, cnt = 0;
  uint32_t code = kErrNone;
  if (touched) {
    __threadfence();  // the counters as the other CTAs left them before they were counted out
    ovf16 = ld_relaxed(&a.sc->ovf16);
    cnt = ld_relaxed(&a.sc->nsal);
    code = (uint32_t)ld_relaxed(&a.sc->status);
  }
  const uint32_t nsal = (uint32_t)cnt, nraw = (uint32_t)(cnt >> 32);
  const unsigned long long total = pl.ovf_off + ovf16 * 16ull;
  if (total > d.capacity && code < kErrCapacity) code = kErrCapacity;
  if (d.capacity >= 64) {
    uint4* hd = reinterpret_cast<uint4*>(d.dst);
    // a failed container must not pass for a valid one: no magic
    // (version 2: payloads may carry Huffman-coded sections)
    hd[0] = make_uint4(code == kErrNone ? kMagic : 0u, (pl.entropy ? 2u : 1u) | ((uint32_t)pl.dtype << 16) | ((uint32_t)pl.bits << 24),
                       pl.N, pl.C);
    hd[1] = make_uint4((uint32_t)pl.H, (uint32_t)pl.W, 8u | (8u << 8) | ((uint32_t)pl.rounding << 16) | ((uint32_t)pl.mode << 24),
                       pl.rho_num | (pl.rho_den << 16));
    hd[2] = make_uint4(pl.tau_num | (pl.tau_den << 16), __float_as_uint(pl.eps), nsal, nraw);
    hd[3] = make_uint4((uint32_t)pl.tensor_id, (uint32_t)(pl.tensor_id >> 32), (uint32_t)total, (uint32_t)(total >> 32));
  }
  if (a.out2) {
    a.out2[0] = total;
    a.out2[1] = status_word(code);
  }
  if (a.d_off_out) *a.d_off_out = code == kErrNone ? d.off_in + ((total + 255ull) & ~255ull) : (~0ull >> 1);
  if (ovf16) st_relaxed(&a.sc->ovf16, 0ull);
  if (cnt) st_relaxed(&a.sc->nsal, 0ull);
  if (code) st_relaxed(&a.sc->status, 0ull);
}

// Last step of every CTA: the last CTA to leave returns the group sums of the previous call's placement scan and
// the hand-out counters to zero and finishes the container.
// The exit counter carries the CTAs that have left in its low half and, in its high half, how many of them had
// changed a counter of the call (cta_dirty); only such a CTA fences -- its updates must be performed before it is
// counted out -- so a call without outlier-rich planes and without errors ends with one atomic per CTA and no
// read-back.  The container itself needs no fence: its readers are later kernels.
__device__ __forceinline__ void cta_exit(const Plan& pl, const CompressArgs& a, const Dest& d, uint32_t* s_last) {
  __syncthreads();  // every thread's note in the flag is in
  const bool dirty = *cta_dirty() != 0u;  // (the same for every thread)
  if (dirty) {
    __threadfence();
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    const unsigned long long old = atomicAdd(&a.sc->exited, 1ull | (dirty ? 1ull << 32 : 0ull));
    const bool last = (uint32_t)old == gridDim.x - 1u;
    *s_last = last ? (((old >> 32) != 0ull || dirty) ? 3u : 1u) : 0u;
  }
  __syncthreads();
  const uint32_t last = *s_last;
  if (!last) return;
  if (pl.mode != kModeOff)
    for (uint32_t k = threadIdx.x; k < a.scan.clear_groups; k += blockDim.x) a.scan.grp_clear[k] = 0ull;
  if (threadIdx.x != 0) return;
  // (what follows is read by later kernels only, which start work after this one has completed: no fence)
  st_relaxed(&a.sc->ticket[a.parity], 0ull);
  st_relaxed(&a.sc->exited, 0ull);
  finalize(pl, a, d, (last & 2u) != 0u);
}

__device__ __forceinline__ void store_table_entry(const Dest& d, uint64_t plane, uint32_t off16, uint32_t meta, float lo,
                                                  float scale) {
  reinterpret_cast<uint4*>(d.dst + 64)[plane] = make_uint4(off16, meta, __float_as_uint(lo), __float_as_uint(scale));
}

// Table entry of a plane that takes the block-wise path, until its payload is written: class salient, the
// three-sigma count; phase 1 leaves the plane's overflow size (16-byte units) where the offset will go.
__device__ __forceinline__ void store_marker(const Dest& d, uint64_t plane, uint32_t meta, uint32_t units) {
  reinterpret_cast<uint4*>(d.dst + 64)[plane] = make_uint4(units, (meta & ~3u) | kClsSalient, 0u, 0u);
}
__device__ __forceinline__ uint2 load_marker(const Dest& d, uint64_t plane) {
  const volatile uint32_t* e = reinterpret_cast<const volatile uint32_t*>(d.dst + 64 + 16ull * plane);
  return make_uint2(e[0], e[1]);
}

// The block-wise path runs in two phases so that nothing in the streaming phase ever waits for another CTA.
// Phase 1, while a tile lies in shared memory: its outlier-rich planes are measured, the tile publishes the
// overflow size of its planes to the scan, and the CTA links the tile into its own list (newest first;
// `defer_next[tile]` holds the tile listed before it).  Phase 2, when the CTA has run out of tiles: it takes
// its listed tiles again (they come from the L2 cache when the tensor is small), obtains each tile's place
// from the scan -- every tile before it has been published, or is about to be, by a CTA in phase 1 -- and
// writes the payloads.  This block sits in shared memory: what the outlined functions of both phases need.
constexpr uint32_t kNoTile = 0xFFFFFFFFu;
struct BlockCtl {
  Plan pl;
  CompressArgs a;
  Dest d;
  uint32_t U[kMaxStages], C[kMaxStages], arr[kMaxStages];  // warp-team kernel, per stage: units, counts, warps done
  uint32_t wcnt[kMaxWarps];                                // phase 2: outlier-rich planes per warp's slice
  uint32_t base, ok;
  uint32_t head;                                           // the tile this CTA listed last
  uint32_t held[kMaxStages];                               // warp-team kernel: the tile each stage buffer holds
  // phase 2 of the warp-team kernel: the outlier-rich planes of the tile in hand, in plane order
  uint32_t list_at[256];                                   // overflow units, then (scanned) the place within the tile's part
  uint32_t list_meta[256];
  uint16_t list_lp[256];
};

// One thread: tile `tile` has `units` of overflow in `nsal` salient and `nraw` raw planes.
__device__ __forceinline__ void publish_tile(BlockCtl* c, uint32_t tile, uint32_t units, uint32_t nsal, uint32_t nraw) {
  scan_publish(c->a.scan, tile, units);
  count_blockwise(c->a, units, nsal, nraw);
  if ((nsal | nraw) && c->d.fits) c->a.defer_next[tile] = atomicExch(&c->head, tile);
}

// Copies planes [p0, p0 + np) into `buf` (whole 16-byte chunks from the aligned start, the ragged end of the
// tensor byte-wise; all threads of the CTA) and returns the offset of plane p0 in it.
__device__ __forceinline__ uint32_t stage_planes(const Plan& pl, const uint8_t* src, uint64_t p0, uint32_t np, uint8_t* buf) {
  const uint64_t start = p0 * pl.plane_bytes, end = start + (uint64_t)np * pl.plane_bytes;
  const uint64_t a0 = start & ~15ull;
  const uint64_t a1 = min((end + 15ull) & ~15ull, pl.dense_bytes & ~15ull);
  const uint4* s16 = reinterpret_cast<const uint4*>(src + a0);
  uint4* t16 = reinterpret_cast<uint4*>(buf);
  const uint32_t n16 = (uint32_t)((a1 - a0) >> 4);
  for (uint32_t i = threadIdx.x; i < n16; i += blockDim.x) t16[i] = __ldg(s16 + i);
  for (uint64_t i = a1 + threadIdx.x; i < end; i += blockDim.x) buf[i - a0] = src[i];
  return (uint32_t)(start - a0);
}

// Distances d = x - lo of group g of a plane; positions past HW read as 0.
template <int DT>
__device__ __forceinline__ void load_dist(const uint8_t* plane, uint32_t g, uint32_t HW, bool vec, float lo, float d[4]) {
  float v[4];
  load_group<DT>(plane, g, HW, vec, v);
#pragma unroll
  for (int k = 0; k < 4; ++k) d[k] = (g * 4u + k < HW) ? __fsub_rn(v[k], lo) : 0.0f;
}

// Per-plane record kept in shared memory while a tile of the generic kernel is processed.
struct Rec {
  float lo, scale;
  uint32_t meta;   // class | n_out << 2
  uint32_t units;  // overflow units of a salient / raw plane
};

// =================================================================================================
// Generic streaming kernel
// =================================================================================================
// Tiles of consecutive planes are staged in shared memory with plain loads (planes need not start
// on a 16-byte boundary); a team per plane computes statistics and class; the codes of normal planes
// are staged in shared memory and leave with 16-byte stores.  Outlier-rich planes of the tile are then
// measured one after the other by the whole CTA, and written the same way in phase 2 (this kernel serves the
// odd shapes and is not tuned).
template <int DT, int BITS>
__global__ void __launch_bounds__(kThreads) compress_generic(const Plan pl, const CompressArgs a) {
  extern __shared__ __align__(128) uint8_t smem[];
  __shared__ double s_red[kMaxWarps * 5];
  __shared__ uint32_t s_tile, s_last;
  __shared__ BlockCtl s_ctl;

  const uint32_t tid = threadIdx.x;
  if (tid == 0) *cta_dirty() = 0u;
  if (tid == 0 && a.early_ticket) s_tile = (uint32_t)atomicAdd(&a.sc->ticket[a.parity], 1ull);
  if (tid == 0 && pl.mode != kModeOff) {  // (before the wait for the previous kernel, whose tail hides it)
    s_ctl.pl = pl;
    s_ctl.a = a;
    s_ctl.head = kNoTile;
  }
  dep_wait();     // the previous kernel on the stream has completed
  dep_trigger();  // the next kernel on the stream may become resident as this one drains
  uint8_t* tile_buf = smem + pl.sm_tile;
  uint8_t* out_buf = smem + pl.sm_out;
  Rec* rec = reinterpret_cast<Rec*>(smem + pl.sm_rec);
  uint32_t* sal = reinterpret_cast<uint32_t*>(smem + pl.sm_sal);
  const Dest d = make_dest(pl, a);
  if (tid == 0 && pl.mode != kModeOff) s_ctl.d = d;
  const Team team = make_team(pl.team, s_red);
  const Team cta = make_team(kThreads, s_red);
  const uint32_t nteams = team.block ? 1u : kThreads / team.size;
  const uint32_t my_team = team.block ? 0u : tid / team.size;
  constexpr uint32_t L = (1u << BITS) - 1u;
  const bool need_sigma = pl.mode == kModeAuto;
  uint32_t rp = 0;  // reduction counter (see red_half)
  if (!d.fits && tid == 0 && blockIdx.x == 0) report_error(a, kErrCapacity);

  for (bool first = true;; first = false) {
    if (tid == 0 && !(first && a.early_ticket)) s_tile = (uint32_t)atomicAdd(&a.sc->ticket[a.parity], 1ull);
    __syncthreads();
    const uint32_t tile = s_tile;
    if (tile >= pl.ntiles) break;
    const uint64_t p0 = (uint64_t)tile * pl.ppt;
    const uint32_t np = (uint32_t)min((uint64_t)pl.ppt, pl.P - p0);

    // ---- stage the tile
    const uint32_t head = stage_planes(pl, a.src, p0, np, tile_buf);
    __syncthreads();

    // ---- phase A: per-plane statistics, class, codes
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
      const float range = __fsub_rn(hi, lo);
      if (!(fabsf(range) <= 3.402823466e38f) && team.lane == 0)
        report_error(a, kErrNonfinite);

      uint32_t cls = kClsNormal, n_out = 0;
      if (need_sigma) {
        const SigmaScale sc = sigma_scale(range);
        if (sc.applies) {  // (the same for every thread of the team)
          uint32_t as = 0, aq = 0, ng = 0;
          for (uint32_t g = team.lane; g < groups; g += team.size) {
            float dd[4];
            load_dist<DT>(plane, g, HW, vec, lo, dd);
            sigma_addends(dd, sc, as, aq);
            ++ng;
          }
          long long Is, Iq;
          if (team.block)
            team_sum2_wide(team, (long long)(int32_t)(as - ng * kMagicBits), (long long)(int32_t)(aq - ng * kMagicBits),
                           Is, Iq, rp);
          else
            team_sum2(team, (int32_t)(as - ng * kMagicBits), (int32_t)(aq - ng * kMagicBits), Is, Iq, rp);
          float dlo, dhi;
          sigma_thresholds(Is, Iq, sc, pl.inv_hw, dlo, dhi);
          uint32_t cnt = 0;
          for (uint32_t g = team.lane; g < groups; g += team.size) {
            float dd[4];
            load_dist<DT>(plane, g, HW, vec, lo, dd);
#pragma unroll
            for (int k = 0; k < 4; ++k) cnt += (g * 4u + k < HW) && ((dd[k] > dhi) || (dd[k] < dlo));
          }
          n_out = team_sum_u32(team, cnt, rp);
          if ((uint64_t)n_out * pl.rho_den > (uint64_t)pl.rho_num * HW) cls = kClsSalient;
        }
      } else if (pl.mode == kModeAll) {
        cls = kClsSalient;
      } else if (pl.mode >= kModeChannel) {
        cls = channel_class(pl, a, p0 + lp, n_out);
      }

      Rec r;
      r.lo = 0.0f;
      r.scale = 0.0f;
      r.units = 0;
      if (cls == kClsNormal) {
        float inv, scale;
        quant_params(range, L, inv, scale);
        r.lo = lo;
        r.scale = scale;
        uint8_t* o = out_buf + (uint64_t)lp * pl.npay;
        const uint32_t ogroups = pl.npay * 2u / BITS;
        for (uint32_t g = team.lane; g < ogroups; g += team.size) {
          uint32_t word = 0;
          if (g < groups) {
            float dd[4];
            load_dist<DT>(plane, g, HW, vec, lo, dd);
            uint32_t rnd[4] = {0, 0, 0, 0};
            if (pl.rounding)  // one generator call per group: counter = (group, plane, tensor id), key = seed
              philox4x32_10(g, (uint32_t)(p0 + lp), (uint32_t)pl.tensor_id, (uint32_t)(pl.tensor_id >> 32),
                            (uint32_t)pl.seed, (uint32_t)(pl.seed >> 32), rnd);
#pragma unroll
            for (int k = 0; k < 4; ++k) {
              uint32_t q = pl.rounding ? quant_code_random(dd[k], inv, L, rnd[k]) : quant_code(dd[k], inv, L);
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

    // ---- phase B: table entries and slots of the normal planes
    if (d.fits) {
      const uint32_t chunks = pl.npay >> 4;
      uint4* slots = reinterpret_cast<uint4*>(d.dst + pl.slots_off + p0 * pl.npay);
      for (uint32_t i = tid; i < np * chunks; i += kThreads) {
        const uint32_t lp = i / chunks;
        if ((rec[lp].meta & 3u) == kClsNormal) slots[i] = reinterpret_cast<const uint4*>(out_buf)[i];
      }
      for (uint32_t i = tid; i < np; i += kThreads)
        if ((rec[i].meta & 3u) == kClsNormal)
          store_table_entry(d, p0 + i, (uint32_t)((pl.slots_off + (p0 + i) * pl.npay) >> 4), rec[i].meta, rec[i].lo,
                            rec[i].scale);
    }

    // ---- phase C: the other planes are measured, one after the other by the whole CTA; the tile publishes
    // their overflow size and is put off until the CTA has run out of tiles
    if (pl.mode != kModeOff) {
      uint32_t U = 0, nsal = 0, nraw = 0;  // (every thread keeps the same figures)
      for (uint32_t lp = 0; lp < np; ++lp) {
        if ((rec[lp].meta & 3u) == kClsNormal) continue;
        const SalientInfo info = salient_measure<DT>(cta, s_ctl.pl, tile_buf + head + (uint64_t)lp * pl.plane_bytes, sal);
        bool raw;
        const uint32_t u = plane_units(pl, info, raw);
        if (tid == 0 && d.fits) store_marker(d, p0 + lp, rec[lp].meta, u);
        U += u;
        nsal += raw ? 0u : 1u;
        nraw += raw ? 1u : 0u;
        __syncthreads();  // the measuring scratch is reused
      }
      if (tid == 0) publish_tile(&s_ctl, tile, U, nsal, nraw);
    }
    __syncthreads();
  }

  // ---- phase 2: the tiles put off, newest first
  __syncthreads();
  for (uint32_t tile = pl.mode != kModeOff ? s_ctl.head : kNoTile; tile != kNoTile;) {
    const uint32_t next = a.defer_next[tile];
    const uint64_t p0 = (uint64_t)tile * pl.ppt;
    const uint32_t np = (uint32_t)min((uint64_t)pl.ppt, pl.P - p0);
    const uint32_t head = stage_planes(pl, a.src, p0, np, tile_buf);
    uint32_t U = 0;
    for (uint32_t i = tid; i < np; i += kThreads) {
      const uint2 m = load_marker(d, p0 + i);
      rec[i].meta = m.y;
      rec[i].units = (m.y & 3u) != kClsNormal ? m.x : 0u;
      U += rec[i].units;
    }
    U = __syncthreads_or(U);  // (only whether the tile has any overflow matters here)
    if (tid < 32u) {
      bool ok = true;
      uint32_t base = 0;
      if (U) ok = scan_prefix(a.scan, tile, base);
      if (tid == 0) {
        if (!ok) report_error(a, kErrTimeout);
        s_ctl.base = base;
        s_ctl.ok = ok;
      }
    }
    __syncthreads();
    if (s_ctl.ok) {
      uint32_t at = s_ctl.base;
      for (uint32_t lp = 0; lp < np; ++lp) {
        if ((rec[lp].meta & 3u) == kClsNormal) continue;
        const uint8_t* plane = tile_buf + head + (uint64_t)lp * pl.plane_bytes;
        const SalientInfo info = salient_measure<DT>(cta, s_ctl.pl, plane, sal);
        write_blockwise<DT>(cta, s_ctl.pl, d, p0 + lp, plane, info, sal, rec[lp].meta >> 2, at);
        at += rec[lp].units;
        __syncthreads();
      }
    }
    __syncthreads();
    tile = next;
  }
  cta_exit(pl, a, d, &s_last);
}

// =================================================================================================
// Fast kernels
// =================================================================================================
// One plane per team.  Warp-team variant: kThreads / team planes per tile, each handled by `team` lanes of a
// warp; thread t of a team owns groups t, t + team, ... (G of them) and keeps them in registers for every
// pass.  FULL: groups == G * team, so no group needs a bounds check.
//
// One sweep over a plane: min/max -> distances from the minimum -> (integer moments -> thresholds -> count
// -> class) -> codes, stored straight to the plane's slot together with its table entry.
//
// Codes of the thread's groups, packed and stored to the plane's slot (used inside plane_sweep, on its
// register-resident distances x[k][e]).  Four codes of a group are the sum of (magic + q_e) << (e * BITS)
// minus the magic's contribution.
#define FH_STORE_CODES(BITS)                                                                                  \
  {                                                                                                           \
    constexpr uint32_t bias = kMagicBits * (1u + (1u << (BITS)) + (1u << (2 * (BITS))) + (1u << (3 * (BITS)))); \
    const f32x2 inv2 = pack2(inv, inv), mag2 = pack2(kMagicF, kMagicF);                                         \
    _Pragma("unroll") for (int k = 0; k < G; ++k) {                                                           \
      const uint32_t g = lane + (uint32_t)(k * TT);                                                           \
      uint32_t w0, w1, w2, w3;                                                                                \
      unpack2u(fma2(pack2(x[k][0], x[k][1]), inv2, mag2), w0, w1); /* packed pairs */                         \
      unpack2u(fma2(pack2(x[k][2], x[k][3]), inv2, mag2), w2, w3);                                            \
      uint32_t word = w0 + (w1 << (BITS)) + (w2 << (2 * (BITS))) + (w3 << (3 * (BITS))) - bias;               \
      if (FULL || g < groups) {                                                                               \
        if ((BITS) == 2) slot[g] = (uint8_t)word;                                                             \
        else if ((BITS) == 4) reinterpret_cast<uint16_t*>(slot)[g] = (uint16_t)word;                          \
        else reinterpret_cast<uint32_t*>(slot)[g] = word;                                                     \
      }                                                                                                       \
    }                                                                                                         \
  }

// TT: team size (1..32), a compile-time constant so that the strides between a thread's groups are
// immediates.  FULL: groups == G * TT.  VEC: planes are whole 16-byte chunks (vector loads, no ragged last
// group).  Returns class | n_out << 2; a normal plane is complete when the function returns.
// SIGMA: 0 no three-sigma statistics, 1 the plane's own, 2 the same with random rounding of the codes.
template <int DT, int SIGMA, int G, int TT, bool FULL, bool VEC>
__device__ __forceinline__ uint32_t plane_sweep(const Team& team, const Plan& pl, const Dest& d, const CompressArgs& a,
                                                const uint8_t* plane, uint64_t gp, uint32_t& rp) {
  // A thread's G group slots that lie past the plane, and the elements past a ragged last group, are
  // kept out of minimum and maximum with neutral values and then held as distance 0: they add exactly
  // nothing to the moments, are subtracted from the outlier count when 0 lies outside the thresholds, and
  // carry code 0 (a ragged last group) or are not stored at all.  The arithmetic runs unpredicated over all
  // G slots.
  const uint32_t groups = pl.groups, lane = team.lane;
  const float pinf = __int_as_float(0x7F800000), ninf = __int_as_float(0xFF800000);
  float x[G][4];
  float lo = pinf, hi = ninf, lo1 = pinf, hi1 = ninf;
  uint32_t npad = 0;  // padded elements among this thread's slots
#pragma unroll
  for (int k = 0; k < G; ++k) {
    const uint32_t g = lane + (uint32_t)(k * TT);
    if (VEC) {
      const bool act = FULL || g < groups;
      if (DT == kF32) {
        float4 t4 = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
        if (act) t4 = (reinterpret_cast<const float4*>(plane) + lane)[k * TT];
        x[k][0] = t4.x; x[k][1] = t4.y; x[k][2] = t4.z; x[k][3] = t4.w;
      } else {
        uint2 t2 = make_uint2(0u, 0u);
        if (act) t2 = (reinterpret_cast<const uint2*>(plane) + lane)[k * TT];
        x[k][0] = __uint_as_float(t2.x << 16); x[k][1] = __uint_as_float(t2.x & 0xFFFF0000u);
        x[k][2] = __uint_as_float(t2.y << 16); x[k][3] = __uint_as_float(t2.y & 0xFFFF0000u);
      }
      // per-group partial results keep the dependency chains short
      float gl = min_nan(min3_nan(x[k][0], x[k][1], x[k][2]), x[k][3]);
      float gh = max_nan(max3_nan(x[k][0], x[k][1], x[k][2]), x[k][3]);
      if (!FULL) {
        gl = act ? gl : pinf;
        gh = act ? gh : ninf;
        npad += act ? 0u : 4u;
      }
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
        if (e & 1) {
          lo1 = min_nan(lo1, in ? x[k][e] : pinf);
          hi1 = max_nan(hi1, in ? x[k][e] : ninf);
        } else {
          lo = min_nan(lo, in ? x[k][e] : pinf);
          hi = max_nan(hi, in ? x[k][e] : ninf);
        }
        npad += in ? 0u : 1u;
      }
    }
  }
  lo = min_nan(lo, lo1);
  hi = max_nan(hi, hi1);
  team_minmax(team, lo, hi, rp);
  const float range = __fsub_rn(hi, lo);
  if (!(fabsf(range) <= 3.402823466e38f) && lane == 0) report_error(a, kErrNonfinite);

  // distances from the minimum, in place (x - lo is x + (-lo): the same rounding)
  {
    const float nlo = -lo;
    const f32x2 nlo2 = pack2(nlo, nlo);
#pragma unroll
    for (int k = 0; k < G; ++k) {
      unpack2(add2(pack2(x[k][0], x[k][1]), nlo2), x[k][0], x[k][1]);
      unpack2(add2(pack2(x[k][2], x[k][3]), nlo2), x[k][2], x[k][3]);
      if (!(FULL && VEC)) {
        const uint32_t g = lane + (uint32_t)(k * TT);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const bool in = VEC ? g < groups : g * 4u + e < pl.HW;
          x[k][e] = in ? x[k][e] : 0.0f;
        }
      }
    }
  }

  uint32_t cls = kClsNormal, n_out = 0;
  if (SIGMA) {
    const SigmaScale sc = sigma_scale(range);
    if (sc.applies) {  // (the same for every thread of the team)
      uint32_t as = 0, aq = 0;
#pragma unroll
      for (int k = 0; k < G; ++k) sigma_addends4(x[k][0], x[k][1], x[k][2], x[k][3], sc, as, aq);
      long long Is, Iq;
      team_sum2(team, (int32_t)(as - (uint32_t)G * kMagicBits), (int32_t)(aq - (uint32_t)G * kMagicBits), Is, Iq, rp);
      float dlo, dhi;
      if (TT > 32) sigma_thresholds(Is, Iq, sc, pl.inv_hw, dlo, dhi);  // (a CTA team's sums may pass 32 bits)
      else sigma_thresholds((int32_t)Is, (int32_t)Iq, sc, pl.inv_hw, dlo, dhi);
      uint32_t cnt = 0;
      if (range > dhi || 0.0f < dlo) {  // otherwise no element can lie outside: the count is zero
        uint32_t c[4] = {0, 0, 0, 0};  // four counters: short dependency chains
        if (!(0.0f < dlo)) {           // nothing below: one compare per element
#pragma unroll
          for (int k = 0; k < G; ++k) {
#pragma unroll
            for (int e = 0; e < 4; ++e) c[e] += x[k][e] > dhi;
          }
          cnt = (c[0] + c[1]) + (c[2] + c[3]);
        } else {
#pragma unroll
          for (int k = 0; k < G; ++k) {
#pragma unroll
            for (int e = 0; e < 4; ++e) c[e] += (x[k][e] > dhi) || (x[k][e] < dlo);
          }
          cnt = (c[0] + c[1]) + (c[2] + c[3]);
          if (!(FULL && VEC)) cnt -= npad;  // padded positions (distance 0, below the lower threshold) are not elements
        }
        cnt = team_sum_u32(team, cnt, rp);
      }
      n_out = cnt;
      if ((uint64_t)n_out * pl.rho_den > (uint64_t)pl.rho_num * pl.HW) cls = kClsSalient;
    }
  } else if (pl.mode == kModeAll) {
    cls = kClsSalient;
  } else if (pl.mode >= kModeChannel) {
    cls = channel_class(pl, a, gp, n_out);
  }

  const uint32_t meta = cls | (n_out << 2);
  if (cls != kClsNormal || !d.fits) return meta;  // (the caller sees to a plane that is not normal)
  const uint32_t bits = (uint32_t)pl.bits;
  float inv, scale;
  quant_params(range, (1u << bits) - 1u, inv, scale);
  uint8_t* slot = d.dst + pl.slots_off + gp * pl.npay;
  if (SIGMA == 2) {
    // random rounding: one generator call per group, counter = (group, plane, tensor id), key = seed; a padded
    // position (distance 0) gets code 0 whatever the draw
    const uint32_t L = (1u << bits) - 1u;
#pragma unroll
    for (int k = 0; k < G; ++k) {
      const uint32_t g = lane + (uint32_t)(k * TT);
      if (FULL || g < groups) {
        uint32_t rnd[4];
        philox4x32_10(g, (uint32_t)gp, (uint32_t)pl.tensor_id, (uint32_t)(pl.tensor_id >> 32), (uint32_t)pl.seed,
                      (uint32_t)(pl.seed >> 32), rnd);
        uint32_t word = 0;
#pragma unroll
        for (int e = 0; e < 4; ++e) word |= quant_code_random(x[k][e], inv, L, rnd[e]) << (e * bits);
        if (bits == 2u) slot[g] = (uint8_t)word;
        else if (bits == 4u) reinterpret_cast<uint16_t*>(slot)[g] = (uint16_t)word;
        else reinterpret_cast<uint32_t*>(slot)[g] = word;
      }
    }
  } else if (bits == 2u) FH_STORE_CODES(2)
  else if (bits == 4u) FH_STORE_CODES(4)
  else FH_STORE_CODES(8)
  // zero padding of the slot behind the codes
  const uint32_t code_bytes = groups * bits / 2u;
  if (code_bytes < pl.npay) {
    for (uint32_t o = code_bytes + lane; o < a4(code_bytes); o += TT) slot[o] = 0;
    for (uint32_t o = a4(code_bytes) + 4u * lane; o < pl.npay; o += 4u * TT)
      *reinterpret_cast<uint32_t*>(slot + o) = 0u;
  }
  if (lane == 0) store_table_entry(d, gp, (uint32_t)((pl.slots_off + gp * pl.npay) >> 4), meta, lo, scale);
  return meta;
}

// Picks the specialisation of the sweep.  FULLVEC kernels are launched only for planes of exactly
// G * TT whole groups, so they carry nothing but the lean variant; the others choose at run time.
template <int DT, int SIGMA, int G, int TT, bool FULLVEC>
__device__ __forceinline__ uint32_t plane_sweep_any(const Team& team, const Plan& pl, const Dest& d,
                                                    const CompressArgs& a, const uint8_t* plane, uint64_t gp,
                                                    bool vec, uint32_t& rp) {
  if (FULLVEC) return plane_sweep<DT, SIGMA, G, TT, true, true>(team, pl, d, a, plane, gp, rp);
  if (vec) return plane_sweep<DT, SIGMA, G, TT, false, true>(team, pl, d, a, plane, gp, rp);
  return plane_sweep<DT, SIGMA, G, TT, false, false>(team, pl, d, a, plane, gp, rp);
}

// -------------------------------------------------------------------------------------------------
// Warp-team streaming kernel: planes of at most 256 groups.  Eight consumer warps and one producer
// warp per CTA.  The producer requests tiles and streams them into a ring of shared-memory stages
// with bulk copies.  A consumer warp sweeps its own planes of a tile (statistics, class, codes, stores)
// and never waits for another warp.  Outlier-rich planes are rare: a warp that has some in its slice
// measures them and adds their overflow size to the tile's sum in shared memory; the last of the tile's
// eight warps to get there publishes the tile and puts it on the CTA's list for phase 2.
// -------------------------------------------------------------------------------------------------
constexpr int kWarpKernelThreads = kThreads + 32;

// Phase 1, a warp with outlier-rich planes in its slice (`leaders`: the first lanes of their teams; lp0: first
// plane of the warp's slice): they are measured, their sizes go into the sums of the tile in stage s and into
// their table markers.
template <int DT, int TT>
__device__ __noinline__ void warp_tile_measure(BlockCtl* c, const uint8_t* tbuf, uint64_t p0, uint32_t s, uint32_t lp0,
                                               uint32_t leaders, uint32_t meta, uint32_t* sal) {
  const Team team = make_warp_team(nullptr);
  const Plan& pl = c->pl;
  uint32_t total = 0, nraw = 0, n = 0;
  for (uint32_t m = leaders; m; m &= m - 1u, ++n) {
    const uint32_t src = (uint32_t)__ffs((int)m) - 1u, lp = lp0 + src / TT;
    if (n) __syncwarp();
    const SalientInfo info = warp_plane_measure<DT>(team, pl, tbuf + (uint64_t)lp * pl.plane_bytes, sal);
    bool raw;
    const uint32_t u = plane_units(pl, info, raw);
    total += u;
    nraw += raw ? 1u : 0u;
    const uint32_t mt = __shfl_sync(0xFFFFFFFFu, meta, (int)src);
    if (team.lane == 0 && c->d.fits) store_marker(c->d, p0 + lp, mt, u);
  }
  if (team.lane == 0) {
    if (total) atomicAdd(&c->U[s], total);
    atomicAdd(&c->C[s], (n - nraw) | (nraw << 16));
  }
}

// Phase 1, the last of a tile's eight warps (one thread): the tile's sums are complete.
__device__ __noinline__ void warp_tile_publish(BlockCtl* c, uint32_t s, uint32_t tile) {
  __threadfence_block();  // the other warps' sums after their arrivals
  const uint32_t U = c->U[s], C = c->C[s];
  c->U[s] = 0;
  c->C[s] = 0;
  publish_tile(c, tile, U, C & 0xFFFFu, C >> 16);
}

// Phase 2 of the warp-team kernel: every tile the CTA has put off, newest first.  The tile's outlier-rich
// planes are listed in plane order (their markers carry class, count and size), placed by one scan over
// the list, and dealt out to the warps in turn.
template <int DT, int TT>
__device__ __noinline__ void warp_phase2(BlockCtl* c, uint8_t* stages, uint8_t* sal_base) {
  const Plan& pl = c->pl;
  const uint32_t tid = threadIdx.x, lane = tid & 31u, warp = tid >> 5;
  const Team team = make_warp_team(nullptr);
  uint32_t* sal = reinterpret_cast<uint32_t*>(sal_base + min(warp, (uint32_t)kWarps - 1u) * pl.sal_stride);
  // Two walks over the list: first the tiles that still lie in a stage buffer (the last ones the CTA streamed:
  // all of them when the tensor is small), then the others, fetched again into the first buffer.
  for (uint32_t walk = 0; walk < 2u; ++walk) {
    for (uint32_t tile = c->head; tile != kNoTile;) {
      const uint32_t next = c->a.defer_next[tile];
      uint32_t at_stage = kMaxStages;
      for (uint32_t s = 0; s < pl.nstage; ++s)
        if (c->held[s] == tile) at_stage = s;
      if ((at_stage < (uint32_t)kMaxStages) != (walk == 0u)) {  // (the same for every thread)
        tile = next;
        continue;
      }
      const uint32_t p0 = tile * pl.ppt;
      const uint32_t np = (uint32_t)min((uint64_t)pl.ppt, pl.P - p0);
      uint8_t* tbuf = stages + (uint64_t)(walk == 0u ? at_stage : 0u) * pl.stage_bytes;
      if (walk) stage_planes(pl, c->a.src, p0, np, tbuf);  // (tiles of this kernel start on 16-byte boundaries)
      uint2 mk = make_uint2(0u, 0u);
      bool mine = false;
      const uint32_t lp = tid / TT;
      if (warp < (uint32_t)kWarps && lp < np && (tid % TT) == 0u) {
        mk = load_marker(c->d, (uint64_t)p0 + lp);
        mine = (mk.y & 3u) != kClsNormal;
      }
      const uint32_t leaders = __ballot_sync(0xFFFFFFFFu, mine);
      if (lane == 0 && warp < (uint32_t)kWarps) c->wcnt[warp] = __popc(leaders);
      __syncthreads();
      uint32_t before = 0, total = 0;
      for (uint32_t w = 0; w < (uint32_t)kWarps; ++w) {
        before += w < warp ? c->wcnt[w] : 0u;
        total += c->wcnt[w];
      }
      if (mine) {
        const uint32_t r = before + __popc(leaders & ((1u << lane) - 1u));
        c->list_at[r] = mk.x;
        c->list_meta[r] = mk.y;
        c->list_lp[r] = (uint16_t)lp;
      }
      __syncthreads();
      if (warp == 0) {  // places within the tile's part of the overflow region, and the tile's place
        uint32_t run = 0;
        for (uint32_t r0 = 0; r0 < total; r0 += 32u) {
          const uint32_t v = r0 + lane < total ? c->list_at[r0 + lane] : 0u;
          uint32_t incl = v;
          for (uint32_t o = 1; o < 32u; o <<= 1) {
            const uint32_t up = __shfl_up_sync(0xFFFFFFFFu, incl, o);
            if (lane >= o) incl += up;
          }
          if (r0 + lane < total) c->list_at[r0 + lane] = run + incl - v;
          run += __shfl_sync(0xFFFFFFFFu, incl, 31);
        }
        bool ok = true;
        uint32_t base = 0;
        if (run) ok = scan_prefix(c->a.scan, tile, base);
        if (lane == 0) {
          if (!ok) report_error(c->a, kErrTimeout);
          c->base = base;
          c->ok = ok;
        }
      }
      __syncthreads();
      if (c->ok && warp < (uint32_t)kWarps)
        for (uint32_t r = warp; r < total; r += (uint32_t)kWarps) {
          const uint32_t pl_lp = c->list_lp[r];
          warp_plane_write<DT>(team, pl, c->d, (uint64_t)p0 + pl_lp, tbuf + (uint64_t)pl_lp * pl.plane_bytes, sal,
                               c->list_meta[r] >> 2, c->base + c->list_at[r]);
          __syncwarp();
        }
      __syncthreads();
      tile = next;
    }
  }
}

template <int DT, int SIGMA, int TT, bool FULLVEC>
__global__ void __launch_bounds__(kWarpKernelThreads, 3) compress_warp(const Plan pl, const CompressArgs a) {
  extern __shared__ __align__(128) uint8_t smem[];
  __shared__ double s_red[kMaxWarps * 5];
  __shared__ __align__(8) uint64_t s_full[kMaxStages], s_empty[kMaxStages];
  __shared__ uint32_t s_tiles[kMaxStages];
  __shared__ volatile uint32_t s_abort;
  __shared__ uint32_t s_last;
  __shared__ BlockCtl s_ctl;

  const uint32_t tid = threadIdx.x, lane = tid & 31u, warp = tid >> 5;
  const uint32_t nstage = pl.nstage;
  const bool scan_on = pl.mode != kModeOff;
  uint32_t first_ticket = 0;
  // Everything that needs no global memory comes before the wait for the previous kernel, whose tail hides it.
  if (tid == 0) {
    for (uint32_t s = 0; s < nstage; ++s) {
      mbar_init(&s_full[s], 1);
      mbar_init(&s_empty[s], kWarps);
    }
    fence_mbar_init();
    s_abort = 0;
    *cta_dirty() = 0u;
    if (scan_on) {
      s_ctl.pl = pl;
      s_ctl.a = a;
      s_ctl.head = kNoTile;
      for (uint32_t s = 0; s < nstage; ++s) {
        s_ctl.U[s] = s_ctl.C[s] = s_ctl.arr[s] = 0;
        s_ctl.held[s] = kNoTile;
      }
    }
  }
  // (the ticket counter of this call was returned to zero by the call before the previous one, which had
  // completed before the previous kernel let this one start)
  if (tid == (uint32_t)kThreads && a.early_ticket)
    first_ticket = (uint32_t)atomicAdd(&a.sc->ticket[a.parity], (unsigned long long)nstage);
  __syncthreads();
  dep_wait();     // the previous kernel on the stream has completed; global memory may be touched from here on
  dep_trigger();  // the next kernel on the stream may become resident as this one drains
  const Dest d = make_dest(pl, a);
  if (warp < (uint32_t)kWarps) {  // (the producer goes straight to its first loads)
    if (tid == 0) {
      if (!d.fits && blockIdx.x == 0) report_error(a, kErrCapacity);
      if (scan_on) s_ctl.d = d;
    }
    asm volatile("bar.sync 1, %0;" ::"n"(kThreads) : "memory");  // the consumer warps: s_ctl.d is in place
  }

  if (warp == (uint32_t)kWarps) {
    // ======================= producer (all 32 lanes walk the loop, lane 0 issues) =======================
    uint32_t s = 0, empty_phase = 0;
    bool aborted = false;
    if (!a.early_ticket && lane == 0)
      first_ticket = (uint32_t)atomicAdd(&a.sc->ticket[a.parity], (unsigned long long)nstage);
    first_ticket = __shfl_sync(0xFFFFFFFFu, first_ticket, 0);
    // Waits until every consumer warp is done with the tile in stage q.
    auto drain = [&](uint32_t q) -> bool {
      bool ok = mbar_wait_abortable(&s_empty[q], (empty_phase >> q) & 1u, 1u << 20, &s_abort);
      ok = __all_sync(0xFFFFFFFFu, ok);
      if (ok) empty_phase ^= 1u << q;
      return ok;
    };
    for (uint32_t n = 0;; ++n) {
      if (n >= nstage && !drain(s)) {
        aborted = true;
        break;
      }
      // tiles come in ticket order: the first nstage of them in one request, then one at a time
      uint32_t t = first_ticket + n;
      if (n >= nstage) {
        if (lane == 0) t = (uint32_t)atomicAdd(&a.sc->ticket[a.parity], 1ull);
        t = __shfl_sync(0xFFFFFFFFu, t, 0);
      }
      if (t >= pl.ntiles) {
        // no more tiles: wake the consumers at this stage, then wait for the tiles still in the ring
        const uint32_t first = n >= nstage ? n - nstage + 1u : 0u;
        uint32_t q = first % nstage;
        __syncwarp();
        if (lane == 0) {
          s_tiles[s] = kNoTile;
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
        if (scan_on) s_ctl.held[s] = t;
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
        report_error(a, kErrTimeout);
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
      const uint8_t* stage = smem + pl.sm_tile + (uint64_t)s * pl.stage_bytes;
      uint32_t meta = kClsNormal;
      if (active)
        meta = plane_sweep_any<DT, SIGMA, G, TT, FULLVEC>(team, pl, d, a, stage + (uint64_t)lp * pl.plane_bytes,
                                                          (uint64_t)p0 + lp, vec, rp);
      if (scan_on) {  // phase 1 of the block-wise path
        const uint32_t leaders = __ballot_sync(0xFFFFFFFFu, active && (meta & 3u) != kClsNormal && team.lane == 0);
        if (leaders)
          warp_tile_measure<DT, TT>(&s_ctl, stage, (uint64_t)p0, s, (warp * 32u) / TT, leaders, meta,
                                    reinterpret_cast<uint32_t*>(smem + pl.sm_sal + warp * pl.sal_stride));
        if (lane == 0) {
          if (leaders) __threadfence_block();  // the warp's sums before its arrival
          if ((atomicAdd(&s_ctl.arr[s], 1u) & 7u) == 7u) warp_tile_publish(&s_ctl, s, tile);
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&s_empty[s]);
      if (s_abort) break;
      s = s + 1 == nstage ? 0 : s + 1;
    }
  }
  if (scan_on) {
    __syncthreads();
    if (s_ctl.head != kNoTile && !s_abort) warp_phase2<DT, TT>(&s_ctl, smem + pl.sm_tile, smem + pl.sm_sal);
  }
  cta_exit(pl, a, d, &s_last);
}

// -------------------------------------------------------------------------------------------------
// CTA-team kernel: planes of more than 256 groups (whole 16-byte chunks).  One plane per tile, all
// NT threads of the CTA work on it.  The plane stays in its shared-memory stage and is swept two or
// three times (min/max; integer moments; count + codes), so that few registers are needed and
// shared memory alone limits how many CTAs fit an SM (two stages each).  What every warp repeats per
// plane -- reductions, thresholds, quantiser parameters -- does not shrink with the warp's share of the
// plane, so NT is kept small for small planes.  Thread 0 keeps the next ticket in flight while the CTA works.
// An outlier-rich plane is measured by the whole CTA while it lies in its stage and written in phase 2.
// -------------------------------------------------------------------------------------------------
// Phase 1: the plane in `plane` is measured, tile (= plane) `tile` published and put on the CTA's list.
template <int DT, int NT>
__device__ __noinline__ void cta_tile_measure(BlockCtl* c, double* red, const uint8_t* plane, uint32_t* sal, uint32_t tile,
                                              uint32_t meta) {
  const Team team = make_team(NT, red);
  const SalientInfo info = salient_measure<DT>(team, c->pl, plane, sal);
  bool raw;
  const uint32_t units = plane_units(c->pl, info, raw);
  if (threadIdx.x == 0) {
    if (c->d.fits) store_marker(c->d, tile, meta, units);
    publish_tile(c, tile, units, raw ? 0u : 1u, raw ? 1u : 0u);
  }
}

// Phase 2 of the CTA-team kernel: every plane the CTA has put off, newest first.
template <int DT, int NT>
__device__ __noinline__ void cta_phase2(BlockCtl* c, double* red, uint8_t* stage, uint32_t* sal, uint64_t* bar, uint32_t parity) {
  const Plan& pl = c->pl;
  const Team team = make_team(NT, red);
  const uint32_t tid = threadIdx.x;
  for (uint32_t tile = c->head; tile != kNoTile;) {
    const uint32_t next = c->a.defer_next[tile];
    if (tid == 0) {
      fence_proxy_async();
      mbar_expect_tx(bar, (uint32_t)pl.plane_bytes);
      bulk_g2s(stage, c->a.src + (uint64_t)tile * pl.plane_bytes, (uint32_t)pl.plane_bytes, bar);
    }
    bool ready = mbar_wait(bar, parity, 1u << 20);
    ready = __syncthreads_and(ready);
    parity ^= 1u;
    if (!ready) {  // the load timed out: report, wait (bounded) for the copy, give up
      if (tid == 0) {
        report_error(c->a, kErrTimeout);
        mbar_wait(bar, parity ^ 1u, 1u << 10);
      }
      return;
    }
    const SalientInfo info = salient_measure<DT>(team, pl, stage, sal);
    bool raw;
    const uint32_t units = plane_units(pl, info, raw);
    if (tid < 32u) {
      bool ok = true;
      uint32_t base = 0;
      if (units) ok = scan_prefix(c->a.scan, tile, base);
      if (tid == 0) {
        if (!ok) report_error(c->a, kErrTimeout);
        c->base = base;
        c->ok = ok;
      }
    }
    __syncthreads();
    if (c->ok) write_blockwise<DT>(team, pl, c->d, (uint64_t)tile, stage, info, sal, load_marker(c->d, tile).y >> 2, c->base);
    __syncthreads();
    tile = next;
  }
}

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
// The group's distances from lo (x - lo is x + (-lo): the same rounding).
template <int DT>
__device__ __forceinline__ void lds_dist(const uint8_t* plane, uint32_t g, float nlo, float (&v)[4]) {
  lds_group<DT>(plane, g, v);
  const f32x2 nlo2 = pack2(nlo, nlo);
  unpack2(add2(pack2(v[0], v[1]), nlo2), v[0], v[1]);
  unpack2(add2(pack2(v[2], v[3]), nlo2), v[2], v[3]);
}

#define FH_CTA_STORE_CODES(BITS)                                                                              \
  {                                                                                                           \
    constexpr uint32_t bias = kMagicBits * (1u + (1u << (BITS)) + (1u << (2 * (BITS))) + (1u << (3 * (BITS)))); \
    const f32x2 inv2 = pack2(inv, inv), mag2 = pack2(kMagicF, kMagicF);                                         \
    _Pragma("unroll 2") for (uint32_t g = tid; g < groups; g += NT) {                                         \
      float v[4];                                                                                             \
      lds_dist<DT>(plane, g, nlo, v);                                                                         \
      uint32_t w0, w1, w2, w3;                                                                                \
      unpack2u(fma2(pack2(v[0], v[1]), inv2, mag2), w0, w1);                                                  \
      unpack2u(fma2(pack2(v[2], v[3]), inv2, mag2), w2, w3);                                                  \
      uint32_t word = w0 + (w1 << (BITS)) + (w2 << (2 * (BITS))) + (w3 << (3 * (BITS))) - bias;               \
      if ((BITS) == 2) slot[g] = (uint8_t)word;                                                               \
      else if ((BITS) == 4) reinterpret_cast<uint16_t*>(slot)[g] = (uint16_t)word;                            \
      else reinterpret_cast<uint32_t*>(slot)[g] = word;                                                       \
      if (COUNT) {                                                                                            \
        if (one_sided) {                                                                                      \
          c0 += (v[0] > dhi) + (v[2] > dhi);                                                                  \
          c1 += (v[1] > dhi) + (v[3] > dhi);                                                                  \
        } else {                                                                                              \
          c0 += ((v[0] > dhi) || (v[0] < dlo)) + ((v[2] > dhi) || (v[2] < dlo));                              \
          c1 += ((v[1] > dhi) || (v[1] < dlo)) + ((v[3] > dhi) || (v[3] < dlo));                              \
        }                                                                                                     \
      }                                                                                                       \
    }                                                                                                         \
  }

template <int DT, bool SIGMA, int NT>
__global__ void __launch_bounds__(NT) compress_cta(const Plan pl, const CompressArgs a) {
  constexpr bool COUNT = SIGMA;
  extern __shared__ __align__(128) uint8_t smem[];
  __shared__ double s_red[kMaxWarps * 5];
  __shared__ __align__(8) uint64_t s_full[kMaxStages];
  __shared__ uint32_t s_tiles[kMaxStages];
  __shared__ uint32_t s_abort, s_last;
  __shared__ float2 s_thr;
  __shared__ BlockCtl s_ctl;

  const uint32_t tid = threadIdx.x;
  const Team team = make_team(NT, s_red);
  const uint32_t nstage = pl.nstage, groups = pl.groups, bits = (uint32_t)pl.bits;
  const bool scan_on = pl.mode != kModeOff;
  uint32_t* sal = reinterpret_cast<uint32_t*>(smem + pl.sm_sal);
  uint32_t rp = 0;
  // Thread 0 requests the tiles and issues the loads: the first nstage tiles in one request, later ones one
  // at a time, the request running one tile ahead of its use.  Tiles come in ticket order.
  uint32_t next_ticket = 0, issued = 0;
  if (tid == 0) {
    for (uint32_t s = 0; s < nstage; ++s) mbar_init(&s_full[s], 1);
    fence_mbar_init();
    s_abort = 0;
    *cta_dirty() = 0u;
    // (the ticket counter of this call was returned to zero by the call before the previous one, which had
    // completed before the previous kernel let this one start)
    if (a.early_ticket) next_ticket = (uint32_t)atomicAdd(&a.sc->ticket[a.parity], (unsigned long long)nstage);
  }
  if (tid == 0 && scan_on) {  // (before the wait for the previous kernel, whose tail hides it)
    s_ctl.pl = pl;
    s_ctl.a = a;
    s_ctl.head = kNoTile;
  }
  dep_wait();     // the previous kernel on the stream has completed; global memory may be touched from here on
  dep_trigger();  // the next kernel on the stream may become resident as this one drains
  auto issue = [&](uint32_t s) {
    const uint32_t t = next_ticket;
    s_tiles[s] = t;
    if (t < pl.ntiles) {
      fence_proxy_async();
      mbar_expect_tx(&s_full[s], (uint32_t)pl.plane_bytes);
      bulk_g2s(smem + pl.sm_tile + (uint64_t)s * pl.stage_bytes, a.src + (uint64_t)t * pl.plane_bytes,
               (uint32_t)pl.plane_bytes, &s_full[s]);
      ++issued;
      next_ticket = issued < nstage ? t + 1u : (uint32_t)atomicAdd(&a.sc->ticket[a.parity], 1ull);
    }
  };
  if (tid == 0) {  // the first loads before anything else
    if (!a.early_ticket) next_ticket = (uint32_t)atomicAdd(&a.sc->ticket[a.parity], (unsigned long long)nstage);
    for (uint32_t s = 0; s < nstage; ++s) issue(s);
  }
  const Dest d = make_dest(pl, a);
  if (tid == 0) {
    if (!d.fits && blockIdx.x == 0) report_error(a, kErrCapacity);
    if (scan_on) s_ctl.d = d;
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
    const float range = __fsub_rn(hi, lo), nlo = -lo;
    if (!(fabsf(range) <= 3.402823466e38f) && tid == 0) report_error(a, kErrNonfinite);

    // ---- sweep 2: integer moments of the distances from lo, thresholds
    float dlo = 0.0f, dhi = 0.0f;
    bool one_sided = true, need_count = false;
    if (SIGMA) {
      const SigmaScale sc = sigma_scale(range);
      if (sc.applies) {  // (the same for every thread)
        uint32_t as = 0, aq = 0, ng = 0;
#pragma unroll 2
        for (uint32_t g = tid; g < groups; g += NT) {
          float v[4];
          lds_dist<DT>(plane, g, nlo, v);
          sigma_addends4(v[0], v[1], v[2], v[3], sc, as, aq);
          ++ng;
        }
        {  // the first warp adds up the warps' sums and works out what depends on them, for all
          int32_t pa = (int32_t)(as - ng * kMagicBits), pb = (int32_t)(aq - ng * kMagicBits);
          asm volatile("redux.sync.add.s32 %0, %0, %1;" : "+r"(pa) : "r"(0xFFFFFFFFu));
          asm volatile("redux.sync.add.s32 %0, %0, %1;" : "+r"(pb) : "r"(0xFFFFFFFFu));
          int2* r = reinterpret_cast<int2*>(red_half(team, rp));
          const uint32_t wl = tid & 31u;
          if (wl == 0) r[tid >> 5] = make_int2(pa, pb);
          __syncthreads();
          if (tid < 32u) {
            const int2 pr = wl < team.nwarps ? r[wl] : make_int2(0, 0);
            const long long Is = warp_sum_s32_wide(pr.x), Iq = warp_sum_s32_wide(pr.y);
            float tl, th;
            sigma_thresholds(Is, Iq, sc, pl.inv_hw, tl, th);
            if (tid == 0) s_thr = make_float2(tl, th);
          }
          __syncthreads();
          dlo = s_thr.x;
          dhi = s_thr.y;
        }
        need_count = range > dhi || 0.0f < dlo;  // otherwise no element can lie outside
        one_sided = !(0.0f < dlo);
      }
    }

    // ---- sweep 3: codes into the plane's slot (and the outlier count).  A plane that turns out
    // outlier-rich has its slot rewritten below.
    float inv, scale;
    quant_params(range, (1u << bits) - 1u, inv, scale);
    uint8_t* slot = d.dst + pl.slots_off + gp * pl.npay;
    uint32_t c0 = 0, c1 = 0;
    if (d.fits && pl.mode != kModeAll) {
      if (!need_count) {
        dhi = __int_as_float(0x7F800000);  // nothing is counted
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
        lds_dist<DT>(plane, g, nlo, v);
#pragma unroll
        for (int e = 0; e < 4; ++e) c0 += (v[e] > dhi) || (v[e] < dlo);
      }
    }
    uint32_t cls = kClsNormal, n_out = 0;
    if (SIGMA) {
      n_out = team_sum_u32(team, c0 + c1, rp);  // its barrier: every thread is done with the sweeps
      if ((uint64_t)n_out * pl.rho_den > (uint64_t)pl.rho_num * pl.HW) cls = kClsSalient;
    } else {
      if (pl.mode == kModeAll) cls = kClsSalient;
      if (pl.mode >= kModeChannel) cls = channel_class(pl, a, gp, n_out);
      __syncthreads();  // every thread is done with the sweeps
    }
    if (cls == kClsNormal) {
      if (tid == 0) {
        if (d.fits) store_table_entry(d, gp, (uint32_t)((pl.slots_off + gp * pl.npay) >> 4), cls | (n_out << 2), lo, scale);
        if (scan_on) scan_publish(a.scan, tile, 0u);
        issue(s);  // the stage is free: next load
      }
    } else {  // (the same for every thread) phase 1 of the block-wise path
      cta_tile_measure<DT, NT>(&s_ctl, s_red, plane, sal, tile, cls | (n_out << 2));
      __syncthreads();  // every thread is done with the stage
      if (tid == 0) issue(s);
    }
    s = s + 1 == nstage ? 0 : s + 1;
    // s_tiles[s] for the next iteration was written at least one barrier ago (nstage >= 2)
  }

  if (s_abort && tid == 0) {  // a load timed out: report, then wait (bounded) for copies still in flight
    report_error(a, kErrTimeout);
    for (uint32_t k = 0; k < nstage; ++k)
      if (s_tiles[k] < pl.ntiles) {
        mbar_wait(&s_full[k], 0u, 1u << 10);
        mbar_wait(&s_full[k], 1u, 1u << 10);
      }
  }
  if (scan_on) {
    __syncthreads();
    if (s_ctl.head != kNoTile && !s_abort)
      cta_phase2<DT, NT>(&s_ctl, s_red, smem + pl.sm_tile, sal, &s_full[0], phase & 1u);
  }
  cta_exit(pl, a, d, &s_last);
}

// -------------------------------------------------------------------------------------------------
// CTA-team kernel, register variant: planes of 257 to NT * G groups (whole 16-byte chunks).  As compress_cta, but
// every thread takes its G groups out of the stage once and keeps them in registers for the whole sweep
// (plane_sweep with the CTA as the team): one pass over shared memory instead of three, the distances
// computed once.  A normal plane's stage is free as soon as the sweep returns -- its last read of the stage
// lies before the first reduction's barrier -- and takes the next load at once.
// -------------------------------------------------------------------------------------------------
template <int DT, bool SIGMA, int NT, int G, bool FULL>
__global__ void __launch_bounds__(NT, NT > 256 ? 2 : (NT > 128 ? 3 : 6)) compress_cta_regs(const Plan pl, const CompressArgs a) {
  extern __shared__ __align__(128) uint8_t smem[];
  __shared__ double s_red[kMaxWarps * 5];
  __shared__ __align__(8) uint64_t s_full[kMaxStages];
  __shared__ uint32_t s_tiles[kMaxStages];
  __shared__ uint32_t s_abort, s_last;
  __shared__ BlockCtl s_ctl;

  const uint32_t tid = threadIdx.x;
  const Team team = make_team(NT, s_red);
  const uint32_t nstage = pl.nstage;
  const bool scan_on = pl.mode != kModeOff;
  uint32_t* sal = reinterpret_cast<uint32_t*>(smem + pl.sm_sal);
  uint32_t rp = 0;
  // Thread 0 requests the tiles and issues the loads: the first nstage tiles in one request, later ones one
  // at a time, the request running one tile ahead of its use.  Tiles come in ticket order.
  uint32_t next_ticket = 0, issued = 0;
  if (tid == 0) {
    for (uint32_t s = 0; s < nstage; ++s) mbar_init(&s_full[s], 1);
    fence_mbar_init();
    s_abort = 0;
    *cta_dirty() = 0u;
    if (a.early_ticket) next_ticket = (uint32_t)atomicAdd(&a.sc->ticket[a.parity], (unsigned long long)nstage);
    if (scan_on) {  // (before the wait for the previous kernel, whose tail hides it)
      s_ctl.pl = pl;
      s_ctl.a = a;
      s_ctl.head = kNoTile;
    }
  }
  dep_wait();     // the previous kernel on the stream has completed; global memory may be touched from here on
  dep_trigger();  // the next kernel on the stream may become resident as this one drains
  auto issue = [&](uint32_t s) {
    const uint32_t t = next_ticket;
    s_tiles[s] = t;
    if (t < pl.ntiles) {
      fence_proxy_async();
      mbar_expect_tx(&s_full[s], (uint32_t)pl.plane_bytes);
      bulk_g2s(smem + pl.sm_tile + (uint64_t)s * pl.stage_bytes, a.src + (uint64_t)t * pl.plane_bytes,
               (uint32_t)pl.plane_bytes, &s_full[s]);
      ++issued;
      next_ticket = issued < nstage ? t + 1u : (uint32_t)atomicAdd(&a.sc->ticket[a.parity], 1ull);
    }
  };
  if (tid == 0) {  // the first loads before anything else
    if (!a.early_ticket) next_ticket = (uint32_t)atomicAdd(&a.sc->ticket[a.parity], (unsigned long long)nstage);
    for (uint32_t s = 0; s < nstage; ++s) issue(s);
  }
  const Dest d = make_dest(pl, a);
  if (tid == 0) {
    if (!d.fits && blockIdx.x == 0) report_error(a, kErrCapacity);
    if (scan_on) s_ctl.d = d;
  }
  __syncthreads();

  uint32_t s = 0, phase = 0;
  for (;;) {
    const uint32_t tile = s_tiles[s];
    if (tile >= pl.ntiles) break;
    bool ready = mbar_wait(&s_full[s], (phase >> s) & 1u, 1u << 20);
    phase ^= 1u << s;
    if (!__syncthreads_and(ready)) {  // a load timed out (the same answer for every thread)
      if (tid == 0) s_abort = 1;
      break;
    }
    const uint8_t* plane = smem + pl.sm_tile + (uint64_t)s * pl.stage_bytes;
    const uint32_t meta = plane_sweep<DT, SIGMA, G, NT, FULL, true>(team, pl, d, a, plane, (uint64_t)tile, rp);
    if ((meta & 3u) == kClsNormal) {  // (the same for every thread) complete; every read of the stage lies behind a barrier
      if (tid == 0) {
        if (scan_on) scan_publish(a.scan, tile, 0u);
        issue(s);
      }
    } else {  // phase 1 of the block-wise path
      cta_tile_measure<DT, NT>(&s_ctl, s_red, plane, sal, tile, meta);
      __syncthreads();  // every thread is done with the stage
      if (tid == 0) issue(s);
    }
    s = s + 1 == nstage ? 0 : s + 1;
    // s_tiles[s] for the next iteration was written at least one barrier ago (nstage >= 2)
  }
  __syncthreads();
  if (s_abort && tid == 0) {  // a load timed out: report, then wait (bounded) for copies still in flight
    report_error(a, kErrTimeout);
    for (uint32_t k = 0; k < nstage; ++k)
      if (s_tiles[k] < pl.ntiles) {
        mbar_wait(&s_full[k], 0u, 1u << 10);
        mbar_wait(&s_full[k], 1u, 1u << 10);
      }
  }
  if (scan_on) {
    __syncthreads();
    if (s_ctl.head != kNoTile && !s_abort)
      cta_phase2<DT, NT>(&s_ctl, s_red, smem + pl.sm_tile, sal, &s_full[0], phase & 1u);
  }
  cta_exit(pl, a, d, &s_last);
}

}  // namespace fh
