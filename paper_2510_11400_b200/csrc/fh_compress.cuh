// Compress kernels.
//
// Container recap: every plane owns a slot of npay bytes at a closed-form offset; a normal plane's
// codes fill its slot; the payload of a salient or raw plane runs through its slot and continues in
// the overflow region, in plane order.
//
// A call runs one or two kernels on its stream:
//   1. a streaming kernel (one pass over the dense tensor): per-plane statistics, three-sigma class,
//      and for normal planes the codes and the table entry.  Normal planes depend on nothing but
//      themselves, so this kernel has no cross-CTA waits.  A plane that takes the block-wise path only
//      gets a marker in the table and an entry in a work list.  Three variants by plane size:
//        compress_warp<DT, SIGMA, TT, FULLVEC>  planes of at most 256 groups: bulk-copy (TMA) pipeline,
//            a sub-warp team per plane, groups kept in registers;
//        compress_cta<DT, SIGMA, NT>            larger planes of whole 16-byte chunks: one plane per CTA;
//        compress_generic<DT, BITS>             everything else (ragged large planes);
//   2. blockwise_kernel<DT> (not with salient_mode OFF): measures every plane of the work list (block
//      classes, CSR and code sizes), decides salient versus raw, and after a barrier over its grid
//      places the payloads in the overflow region in plane order (so the bytes do not depend on
//      scheduling) and writes them; its last CTA writes the header and the result words.  With an
//      empty work list it only writes the header.
// With salient_mode OFF the streaming kernel finishes the container itself.
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
  uint32_t* worklist;                   // planes that take the block-wise path, in no particular order
  uint32_t* chunk_ovf;                  // per chunk of 2^chunk_shift planes: overflow size of its planes (16-byte units)
  uint32_t chunk_shift, nchunks;
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
  // dense blocks: 64 code bytes each, verbatim values in raster order
  const float inv2e = __fdiv_rn(1.0f, __fmul_rn(2.0f, pl.eps));
  const uint32_t lt = (1u << lane32) - 1u;
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

// One thread, after everything else of the call is done: header, result words, and every counter the
// call touched back to zero.
__device__ __forceinline__ void finalize(const Plan& pl, const CompressArgs& a, const Dest& d) {
  const unsigned long long ovf16 = ld_relaxed(&a.sc->ovf16);
  const unsigned long long nsal = ld_relaxed(&a.sc->nsal), nraw = ld_relaxed(&a.sc->nraw);
  const unsigned long long listed = ld_relaxed(&a.sc->wl_count);
  uint32_t code = (uint32_t)ld_relaxed(&a.sc->status);
  const unsigned long long total = pl.ovf_off + ovf16 * 16ull;
  if (total > d.capacity && code < kErrCapacity) code = kErrCapacity;
  if (d.capacity >= 64) {
    uint4* hd = reinterpret_cast<uint4*>(d.dst);
    // a failed container must not pass for a valid one: no magic
    hd[0] = make_uint4(code == kErrNone ? kMagic : 0u, 1u | ((uint32_t)pl.dtype << 16) | ((uint32_t)pl.bits << 24), pl.N, pl.C);
    hd[1] = make_uint4((uint32_t)pl.H, (uint32_t)pl.W, 8u | (8u << 8) | ((uint32_t)pl.rounding << 16) | ((uint32_t)pl.mode << 24),
                       pl.rho_num | (pl.rho_den << 16));
    hd[2] = make_uint4(pl.tau_num | (pl.tau_den << 16), __float_as_uint(pl.eps), (uint32_t)nsal, (uint32_t)nraw);
    hd[3] = make_uint4((uint32_t)pl.tensor_id, (uint32_t)(pl.tensor_id >> 32), (uint32_t)total, (uint32_t)(total >> 32));
  }
  if (a.out2) {
    a.out2[0] = total;
    a.out2[1] = status_word(code);
  }
  if (a.d_off_out) *a.d_off_out = code == kErrNone ? d.off_in + ((total + 255ull) & ~255ull) : (~0ull >> 1);
  if (listed) {  // (the chunk sums are cleared by the block-wise kernel's last CTA)
    st_relaxed(&a.sc->ovf16, 0ull);
    st_relaxed(&a.sc->nsal, 0ull);
    st_relaxed(&a.sc->nraw, 0ull);
    st_relaxed(&a.sc->wl_count, 0ull);
    st_relaxed(&a.sc->arrived, 0ull);
  }
  if (code) st_relaxed(&a.sc->status, 0ull);
}

// Last step of every CTA of a kernel that hands out tiles or counts exits: the last CTA to leave
// returns those counters to zero and, if this is the call's last kernel (FINAL), finishes the call.
template <bool FINAL>
__device__ __forceinline__ void cta_exit(const Plan& pl, const CompressArgs& a, const Dest& d) {
  __threadfence();
  __syncthreads();
  if (threadIdx.x != 0) return;
  const unsigned long long prev = atomicAdd(&a.sc->exited, 1ull);
  if (prev != (unsigned long long)gridDim.x - 1ull) return;
  __threadfence();
  st_relaxed(&a.sc->ticket, 0ull);
  st_relaxed(&a.sc->exited, 0ull);
  if (FINAL) finalize(pl, a, d);
}

__device__ __forceinline__ void store_table_entry(const Dest& d, uint64_t plane, uint32_t off16, const Rec& r) {
  uint4 e;
  e.x = off16;
  e.y = r.meta;
  e.z = __float_as_uint(r.lo);
  e.w = __float_as_uint(r.scale);
  reinterpret_cast<uint4*>(d.dst + 64)[plane] = e;
}


// Table marker of a plane that takes the block-wise path: class salient, the three-sigma count, no
// offset yet.  The block-wise kernels complete the entry.
__device__ __forceinline__ void store_marker(const Dest& d, uint64_t plane, uint32_t meta) {
  reinterpret_cast<uint4*>(d.dst + 64)[plane] = make_uint4(0u, (meta & ~3u) | kClsSalient, 0u, 0u);
}

// Appends plane `gp` to the work list of the block-wise kernels (one thread).
__device__ __forceinline__ void list_plane(const CompressArgs& a, uint64_t gp) {
  const unsigned long long at = atomicAdd(&a.sc->wl_count, 1ull);
  a.worklist[at] = (uint32_t)gp;
}

// =================================================================================================
// Generic streaming kernel
// =================================================================================================
// Tiles of consecutive planes are staged in shared memory with plain loads (planes need not start
// on a 16-byte boundary); a team per plane computes statistics and class; the codes of normal planes
// are staged in shared memory and leave with 16-byte stores.
template <int DT, int BITS>
__global__ void __launch_bounds__(kThreads) compress_generic(const Plan pl, const CompressArgs a) {
  extern __shared__ __align__(128) uint8_t smem[];
  __shared__ double s_red[kMaxWarps * 5];
  __shared__ uint32_t s_tile;
  dep_trigger();  // the next kernel on the stream may become resident as this one drains
  dep_wait();     // the previous kernel on the stream has completed

  const uint32_t tid = threadIdx.x;
  uint8_t* tile_buf = smem + pl.sm_tile;
  uint8_t* out_buf = smem + pl.sm_out;
  Rec* rec = reinterpret_cast<Rec*>(smem + pl.sm_rec);
  const Dest d = make_dest(pl, a);
  const Team team = make_team(pl.team, s_red);
  const uint32_t nteams = team.block ? 1u : kThreads / team.size;
  const uint32_t my_team = team.block ? 0u : tid / team.size;
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
      } else if (pl.mode >= kModeChannel) {
        cls = channel_class(pl, a, p0 + lp, n_out);
      }

      Rec r;
      r.lo = 0.0f;
      r.scale = 0.0f;
      r.size = 0;
      if (cls == kClsNormal) {
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
            uint32_t rnd[4] = {0, 0, 0, 0};
            if (pl.rounding)  // one generator call per group: counter = (group, plane, tensor id), key = seed
              philox4x32_10(g, (uint32_t)(p0 + lp), (uint32_t)pl.tensor_id, (uint32_t)(pl.tensor_id >> 32),
                            (uint32_t)pl.seed, (uint32_t)(pl.seed >> 32), rnd);
#pragma unroll
            for (int k = 0; k < 4; ++k) {
              uint32_t q = pl.rounding ? quant_code_random(v[k], lo, inv, L, rnd[k]) : quant_code(v[k], lo, inv, L);
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

    // ---- phase B: table entries and slots of the normal planes; markers and work-list entries of the others
    if (d.fits) {
      const uint32_t chunks = pl.npay >> 4;
      uint4* slots = reinterpret_cast<uint4*>(d.dst + pl.slots_off + p0 * pl.npay);
      for (uint32_t i = tid; i < np * chunks; i += kThreads) {
        const uint32_t lp = i / chunks;
        if ((rec[lp].meta & 3u) == kClsNormal) slots[i] = reinterpret_cast<const uint4*>(out_buf)[i];
      }
    }
    for (uint32_t i = tid; i < np; i += kThreads) {
      if ((rec[i].meta & 3u) == kClsNormal) {
        if (d.fits) store_table_entry(d, p0 + i, (uint32_t)((pl.slots_off + (p0 + i) * pl.npay) >> 4), rec[i]);
      } else {
        if (d.fits) store_marker(d, p0 + i, rec[i].meta);
        list_plane(a, p0 + i);
      }
    }
    __syncthreads();
  }
  if (pl.mode == kModeOff) cta_exit<true>(pl, a, d);
  else cta_exit<false>(pl, a, d);
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
    const f32x2 nlo2 = pack2(-lo, -lo), inv2 = pack2(inv, inv), mag2 = pack2(kMagicF, kMagicF);                 \
    _Pragma("unroll") for (int k = 0; k < G; ++k) {                                                           \
      const uint32_t g = lane + (uint32_t)(k * TT);                                                           \
      uint32_t w0, w1, w2, w3;                                                                                \
      if (DT == kBF16) { /* packed pairs; x - lo is x + (-lo): the same rounding */                          \
        unpack2u(fma2(add2(pack2(x[k][0], x[k][1]), nlo2), inv2, mag2), w0, w1);                              \
        unpack2u(fma2(add2(pack2(x[k][2], x[k][3]), nlo2), inv2, mag2), w2, w3);                              \
      } else {                                                                                                \
        w0 = __float_as_uint(__fmaf_rn(__fsub_rn(x[k][0], lo), inv, kMagicF));                                \
        w1 = __float_as_uint(__fmaf_rn(__fsub_rn(x[k][1], lo), inv, kMagicF));                                \
        w2 = __float_as_uint(__fmaf_rn(__fsub_rn(x[k][2], lo), inv, kMagicF));                                \
        w3 = __float_as_uint(__fmaf_rn(__fsub_rn(x[k][3], lo), inv, kMagicF));                                \
      }                                                                                                       \
      uint32_t word = w0 + (w1 << (BITS)) + (w2 << (2 * (BITS))) + (w3 << (3 * (BITS))) - bias;               \
      if (FULL || g < groups) {                                                                               \
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
  // A thread's G group slots that lie past the plane, and the elements past a ragged last group, are
  // held as zeros: they add exactly nothing to the fixed-point moments, are kept out of minimum and
  // maximum with neutral values, are subtracted from the outlier count when zero lies outside the
  // thresholds, and their codes are not stored.  The arithmetic runs unpredicated over all G slots.
  const uint32_t groups = pl.groups, lane = team.lane;
  const float pinf = __int_as_float(0x7F800000), ninf = __int_as_float(0xFF800000);
  float x[G][4];
  float lo = pinf, hi = ninf, lo1 = pinf, hi1 = ninf;
  uint32_t npad = 0;  // zero-padded elements among this thread's slots
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
  if (!(fabsf(__fsub_rn(hi, lo)) <= 3.402823466e38f) && lane == 0)
    atomicMax(&a.sc->status, (unsigned long long)kErrNonfinite);

  uint32_t cls = kClsNormal, n_out = 0;
  if (SIGMA) {
    const SigmaScale sc = sigma_scale(lo, hi);
    uint32_t as = 0, aq = 0;
#pragma unroll
    for (int k = 0; k < G; ++k) sigma_addends4<DT == kBF16>(x[k][0], x[k][1], x[k][2], x[k][3], sc, as, aq);
    long long Is, Iq;
    team_sum2(team, (int32_t)(as - (uint32_t)G * kMagicBits), (int32_t)(aq - (uint32_t)G * kMagicBits), Is, Iq, rp);
    float tlo, thi;
    if (TT > 32) sigma_thresholds(Is, Iq, sc, pl.inv_hw, tlo, thi);
    else sigma_thresholds((int32_t)Is, (int32_t)Iq, sc, pl.inv_hw, tlo, thi);
    uint32_t cnt = 0;
    if (hi > thi || lo < tlo) {  // otherwise no element can lie outside: the count is zero
      uint32_t c[4] = {0, 0, 0, 0};  // four counters: short dependency chains
      if (lo >= tlo) {               // nothing below: one compare per element
#pragma unroll
        for (int k = 0; k < G; ++k) {
#pragma unroll
          for (int e = 0; e < 4; ++e) c[e] += x[k][e] > thi;
        }
        cnt = (c[0] + c[1]) + (c[2] + c[3]);
        if (!(FULL && VEC) && 0.0f > thi) cnt -= npad;  // padded zeros are not elements
      } else {
#pragma unroll
        for (int k = 0; k < G; ++k) {
#pragma unroll
          for (int e = 0; e < 4; ++e) c[e] += (x[k][e] > thi) || (x[k][e] < tlo);
        }
        cnt = (c[0] + c[1]) + (c[2] + c[3]);
        if (!(FULL && VEC) && ((0.0f > thi) || (0.0f < tlo))) cnt -= npad;
      }
      cnt = team_sum_u32(team, cnt, rp);
    }
    n_out = cnt;
    if ((uint64_t)n_out * pl.rho_den > (uint64_t)pl.rho_num * pl.HW) cls = kClsSalient;
  } else if (pl.mode == kModeAll) {
    cls = kClsSalient;
  } else if (pl.mode >= kModeChannel) {
    cls = channel_class(pl, a, gp, n_out);
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
// Warp-team streaming kernel: planes of at most 256 groups.  Eight consumer warps and one producer
// warp per CTA.  The producer hands out tiles and streams them into a ring of shared-memory stages
// with bulk copies.  The consumer warps never wait for each other: each sweeps its own planes of a
// tile (statistics, class, codes, stores), lists the planes that take the block-wise path, and
// arrives on the stage's barrier.
// -------------------------------------------------------------------------------------------------
constexpr int kWarpKernelThreads = kThreads + 32;

template <int DT, bool SIGMA, int TT, bool FULLVEC>
__global__ void __launch_bounds__(kWarpKernelThreads, 3) compress_warp(const Plan pl, const CompressArgs a) {
  extern __shared__ __align__(128) uint8_t smem[];
  __shared__ double s_red[kMaxWarps * 5];
  __shared__ __align__(8) uint64_t s_full[kMaxStages], s_empty[kMaxStages];
  __shared__ uint32_t s_tiles[kMaxStages];
  __shared__ volatile uint32_t s_abort;

  const uint32_t tid = threadIdx.x, lane = tid & 31u, warp = tid >> 5;
  const uint32_t nstage = pl.nstage;
  dep_trigger();  // the next kernel on the stream may become resident as this one drains
  if (tid == 0) {
    for (uint32_t s = 0; s < nstage; ++s) {
      mbar_init(&s_full[s], 1);
      mbar_init(&s_empty[s], kWarps);
    }
    fence_mbar_init();
    s_abort = 0;
  }
  __syncthreads();
  dep_wait();  // the previous kernel on the stream has completed; global memory may be touched from here on
  const Dest d = make_dest(pl, a);
  if (!d.fits && tid == 0 && blockIdx.x == 0) atomicMax(&a.sc->status, (unsigned long long)kErrCapacity);

  if (warp == (uint32_t)kWarps) {
    // ======================= producer (all 32 lanes walk the loop, lane 0 issues) =======================
    uint32_t s = 0, empty_phase = 0;
    bool aborted = false;
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
      // the first tile of every stage follows from the CTA's index; later tiles are handed out
      uint32_t t = blockIdx.x + n * gridDim.x;
      if (n >= nstage) {
        if (lane == 0) t = nstage * gridDim.x + (uint32_t)atomicAdd(&a.sc->ticket, 1ull);
        t = __shfl_sync(0xFFFFFFFFu, t, 0);
      }
      if (t >= pl.ntiles) {
        // no more tiles: wake the consumers at this stage, then wait for the tiles still in the ring
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
      // planes that take the block-wise path: marker in the table, entry in the work list
      const bool mine = active && (r.meta & 3u) != kClsNormal && team.lane == 0;
      const uint32_t leaders = __ballot_sync(0xFFFFFFFFu, mine);
      if (leaders) {
        uint32_t base = 0;
        if (lane == 0) base = (uint32_t)atomicAdd(&a.sc->wl_count, (unsigned long long)__popc(leaders));
        base = __shfl_sync(0xFFFFFFFFu, base, 0);
        if (mine) {
          a.worklist[base + __popc(leaders & ((1u << lane) - 1u))] = p0 + lp;
          if (d.fits) store_marker(d, (uint64_t)p0 + lp, r.meta);
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&s_empty[s]);
      if (s_abort) break;
      s = s + 1 == nstage ? 0 : s + 1;
    }
  }
  if (pl.mode == kModeOff) cta_exit<true>(pl, a, d);
  else cta_exit<false>(pl, a, d);
}

// -------------------------------------------------------------------------------------------------
// CTA-team kernel: planes of more than 256 groups (whole 16-byte chunks).  One plane per tile, all
// NT threads of the CTA work on it.  The plane stays in its shared-memory stage and is swept two or
// three times (min/max; fixed-point moments; count + codes), so that few registers are needed and
// shared memory alone limits how many CTAs fit an SM (two stages each).  What every warp repeats per
// plane -- reductions, thresholds, quantiser parameters -- does not shrink with the warp's share of the
// plane, so NT is kept small for small planes.  Thread 0 keeps the next ticket in flight while the CTA works.
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
    const f32x2 nlo2 = pack2(-lo, -lo), inv2 = pack2(inv, inv), mag2 = pack2(kMagicF, kMagicF);                 \
    _Pragma("unroll 2") for (uint32_t g = tid; g < groups; g += NT) {                                         \
      float v[4];                                                                                             \
      lds_group<DT>(plane, g, v);                                                                             \
      uint32_t w0, w1, w2, w3;                                                                                \
      if (DT == kBF16) {                                                                                      \
        unpack2u(fma2(add2(pack2(v[0], v[1]), nlo2), inv2, mag2), w0, w1);                                    \
        unpack2u(fma2(add2(pack2(v[2], v[3]), nlo2), inv2, mag2), w2, w3);                                    \
      } else {                                                                                                \
        w0 = __float_as_uint(__fmaf_rn(__fsub_rn(v[0], lo), inv, kMagicF));                                   \
        w1 = __float_as_uint(__fmaf_rn(__fsub_rn(v[1], lo), inv, kMagicF));                                   \
        w2 = __float_as_uint(__fmaf_rn(__fsub_rn(v[2], lo), inv, kMagicF));                                   \
        w3 = __float_as_uint(__fmaf_rn(__fsub_rn(v[3], lo), inv, kMagicF));                                   \
      }                                                                                                       \
      uint32_t word = w0 + (w1 << (BITS)) + (w2 << (2 * (BITS))) + (w3 << (3 * (BITS))) - bias;               \
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
  constexpr bool COUNT = SIGMA;
  extern __shared__ __align__(128) uint8_t smem[];
  __shared__ double s_red[kMaxWarps * 5];
  __shared__ __align__(8) uint64_t s_full[kMaxStages];
  __shared__ uint32_t s_tiles[kMaxStages];
  __shared__ uint32_t s_abort;

  const uint32_t tid = threadIdx.x;
  const Team team = make_team(NT, s_red);
  const uint32_t nstage = pl.nstage, groups = pl.groups, bits = (uint32_t)pl.bits;
  uint32_t rp = 0;
  dep_trigger();  // the next kernel on the stream may become resident as this one drains
  if (tid == 0) {
    for (uint32_t s = 0; s < nstage; ++s) mbar_init(&s_full[s], 1);
    fence_mbar_init();
    s_abort = 0;
  }
  dep_wait();  // the previous kernel on the stream has completed; global memory may be touched from here on
  const Dest d = make_dest(pl, a);
  if (!d.fits && tid == 0 && blockIdx.x == 0) atomicMax(&a.sc->status, (unsigned long long)kErrCapacity);
  // Thread 0 issues the loads.  The first tile of every stage follows from the CTA's index; later tiles
  // are handed out, the request running one tile ahead of its use.
  uint32_t next_ticket = blockIdx.x, issued = 0;
  auto issue = [&](uint32_t s) {
    const uint32_t t = next_ticket;
    s_tiles[s] = t;
    if (t < pl.ntiles) {
      fence_proxy_async();
      mbar_expect_tx(&s_full[s], (uint32_t)pl.plane_bytes);
      bulk_g2s(smem + pl.sm_tile + (uint64_t)s * pl.stage_bytes, a.src + (uint64_t)t * pl.plane_bytes,
               (uint32_t)pl.plane_bytes, &s_full[s]);
      ++issued;
      next_ticket = issued < nstage ? blockIdx.x + issued * gridDim.x
                                    : nstage * gridDim.x + (uint32_t)atomicAdd(&a.sc->ticket, 1ull);
    }
  };
  if (tid == 0)
    for (uint32_t s = 0; s < nstage; ++s) issue(s);
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
        sigma_addends4<DT == kBF16>(v[0], v[1], v[2], v[3], sc, as, aq);
        ++ng;
      }
      long long Is, Iq;
      team_sum2(team, (int32_t)(as - ng * kMagicBits), (int32_t)(aq - ng * kMagicBits), Is, Iq, rp);
      sigma_thresholds(Is, Iq, sc, pl.inv_hw, tlo, thi);
      need_count = hi > thi || lo < tlo;  // otherwise no element can lie outside
      one_sided = lo >= tlo;
    }

    // ---- sweep 3: codes into the plane's slot (and the outlier count).  A plane that turns out
    // salient has its slot rewritten by the block-wise kernels.
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
      n_out = team_sum_u32(team, c0 + c1, rp);  // its barrier: every thread is done with the stage
      if ((uint64_t)n_out * pl.rho_den > (uint64_t)pl.rho_num * pl.HW) cls = kClsSalient;
    } else {
      if (pl.mode == kModeAll) cls = kClsSalient;
      if (pl.mode >= kModeChannel) cls = channel_class(pl, a, gp, n_out);
      __syncthreads();  // every thread is done with the stage
    }
    if (tid == 0) {
      Rec r;
      r.size = 0;
      r.meta = cls | (n_out << 2);
      if (cls == kClsNormal) {
        r.lo = lo;
        r.scale = scale;
        if (d.fits) store_table_entry(d, gp, (uint32_t)((pl.slots_off + gp * pl.npay) >> 4), r);
      } else {
        if (d.fits) store_marker(d, gp, r.meta);
        list_plane(a, gp);
      }
      issue(s);  // the stage is free: next load
    }
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
  if (pl.mode == kModeOff) cta_exit<true>(pl, a, d);
  else cta_exit<false>(pl, a, d);
}

// =================================================================================================
// Block-wise kernel: the planes of the work list
// =================================================================================================
// Runs after the streaming kernel whenever planes can take the block-wise path.  With an empty work
// list one thread finishes the container.  Otherwise a unit -- one warp for planes up to 8 KB, the
// whole CTA above -- takes entries i = unit, unit + units, ... of the list.
//
// Measuring phase: the unit copies the plane into its shared-memory buffer, measures it (block
// classes, CSR and code sizes), decides salient versus raw, completes the plane's table entry (class;
// the offset stays 0), leaves the three counts of a salient payload in the first 16 bytes of the
// plane's slot, and adds the plane's overflow size to the sum of its chunk (a chunk is a run of
// 2^chunk_shift consecutive planes; there are at most kMaxChunks chunks).
//
// A barrier over the grid separates the phases: all CTAs are resident (a cooperative launch of a grid
// sized to what the device holds at once); the wait is bounded all the same, and a wait that runs out
// ends the call with the time-out status instead of hanging.
//
// Writing phase: every CTA turns the chunk sums into chunk offsets.  A plane's place in the overflow
// region is its chunk's offset plus the overflow sizes of the listed planes before it in the same
// chunk, recomputed from their table classes and slot headers (nothing changes those words any more:
// whoever stores to them stores the value that is already there).  The unit walks its entries in
// reverse so that the plane it measured last is still in its buffer; the others are copied and
// measured again.  The last CTA to leave finishes the container.
__device__ __forceinline__ uint32_t salient_size(const Plan& pl, uint32_t nnz_s, uint32_t n_dense, uint32_t n_out_d) {
  const uint32_t e = (uint32_t)pl.esize;
  return 16u + 4u * pl.nbm + 4u * ((uint32_t)pl.H + 1u) + a4(2u * nnz_s) + a4(e * nnz_s) + 64u * n_dense +
         a4(e * n_out_d);
}
// Overflow size, in 16-byte units, of a payload of `size` bytes.
__device__ __forceinline__ uint32_t ovf_units(const Plan& pl, uint32_t size) {
  return a16(size) > pl.npay ? (a16(size) - pl.npay) >> 4 : 0u;
}

// Copies plane p into the unit's buffer (whole 16-byte chunks from the aligned start, the ragged end
// of the tensor byte-wise) and returns where the plane starts in it.
__device__ __forceinline__ const uint8_t* fetch_plane(const Team& t, const Plan& pl, const uint8_t* src, uint32_t p,
                                                      uint8_t* ubuf) {
  const uint64_t start = (uint64_t)p * pl.plane_bytes, end = start + pl.plane_bytes;
  const uint64_t a0 = start & ~15ull;
  const uint64_t a1 = min((end + 15ull) & ~15ull, pl.dense_bytes & ~15ull);
  const uint4* s16 = reinterpret_cast<const uint4*>(src + a0);
  uint4* t16 = reinterpret_cast<uint4*>(ubuf);
  const uint32_t n16 = (uint32_t)((a1 - a0) >> 4);
  for (uint32_t k = t.lane; k < n16; k += t.size) t16[k] = __ldg(s16 + k);
  for (uint64_t k = a1 + t.lane; k < end; k += t.size) ubuf[k - a0] = src[k];
  team_sync(t);
  return ubuf + (uint32_t)(start - a0);
}

constexpr uint32_t kGridWaitPolls = 1u << 21;  // about a second

template <int DT>
__global__ void __launch_bounds__(512) blockwise_kernel(const Plan pl, const CompressArgs a) {
  extern __shared__ __align__(128) uint8_t smem[];
  __shared__ double s_red[kMaxWarps * 5];
  __shared__ Plan s_pl;  // copy for the outlined measuring / writing functions, which take it by address
  __shared__ uint32_t s_ok;

  const uint32_t tid = threadIdx.x, lane32 = tid & 31u, warp = tid >> 5;
  // (launched in plain stream order: the streaming kernel has completed, its list, table and counters are visible)
  const Dest d = make_dest(pl, a);
  const uint32_t count = (uint32_t)ld_relaxed(&a.sc->wl_count);
  if (count == 0) {  // nothing listed: the container lacks only its header
    if (blockIdx.x == 0 && tid == 0) finalize(pl, a, d);
    return;
  }
  if (tid == 0) s_pl = pl;
  const bool unit_cta = pl.sk_cta != 0u;
  const uint32_t upc = unit_cta ? 1u : blockDim.x >> 5;
  const uint32_t unit = unit_cta ? blockIdx.x : blockIdx.x * upc + warp;
  const uint32_t units = gridDim.x * upc;
  const Team t = unit_cta ? make_team(blockDim.x, s_red) : make_warp_team(s_red);
  uint8_t* ubuf = smem + (unit_cta ? 0u : warp * pl.sk_unit_stride);
  // measuring areas of the unit: the n-th entry it takes uses area min(n, keep - 1); an area starts with
  // the four sizes of SalientInfo, the measuring scratch follows
  uint32_t* areas = reinterpret_cast<uint32_t*>(ubuf + pl.sk_sal_off);
  const uint32_t keep = pl.sk_keep, area_words = pl.sk_area_words;
  uint32_t* pre = reinterpret_cast<uint32_t*>(smem + pl.sk_pre_off);
  const uint4* table = reinterpret_cast<const uint4*>(d.dst + 64);
  const uint32_t raw_units = ovf_units(pl, (uint32_t)pl.plane_bytes);
  __syncthreads();

  // ---- measuring phase
  uint32_t taken = 0;  // entries this unit has measured; the plane of the last one stays in the buffer
  const uint8_t* plane = ubuf;
  SalientInfo info;
  info.nnz_s = info.n_dense = info.n_out_d = info.size = 0;
  for (uint32_t i = unit; i < count; i += units, ++taken) {
    if (taken) team_sync(t);  // the buffer is reused
    const uint32_t p = a.worklist[i];
    plane = fetch_plane(t, pl, a.src, p, ubuf);
    uint32_t* area = areas + min(taken, keep - 1u) * area_words;
    info = salient_measure<DT>(t, s_pl, plane, area + 4);
    if (t.lane == 0) {
      area[0] = info.nnz_s;
      area[1] = info.n_dense;
      area[2] = info.n_out_d;
      area[3] = info.size;
    }
    const bool raw = a16(info.size) >= a16((uint32_t)pl.plane_bytes);
    const uint32_t my_units = ovf_units(pl, raw ? (uint32_t)pl.plane_bytes : info.size);
    if (t.lane == 0) {
      if (d.fits) {
        // the streaming kernel's marker says salient (class bits 01); a raw plane flips them to 10
        if (raw)
          atomicXor(reinterpret_cast<uint32_t*>(d.dst + 64 + 16ull * p) + 1, 3u);
        else
          *reinterpret_cast<uint4*>(d.dst + pl.slots_off + (uint64_t)p * pl.npay) =
              make_uint4(info.nnz_s, info.n_dense, info.n_out_d, 0u);
      }
      if (my_units) {
        atomicAdd(&a.chunk_ovf[p >> a.chunk_shift], my_units);
        atomicAdd(&a.sc->ovf16, (unsigned long long)my_units);
      }
      atomicAdd(raw ? &a.sc->nraw : &a.sc->nsal, 1ull);
    }
  }

  // ---- barrier over the grid (bounded)
  __threadfence();
  __syncthreads();
  if (tid == 0) {
    atomicAdd(&a.sc->arrived, 1ull);
    uint32_t ok = 0;
    for (uint32_t k = 0; k < kGridWaitPolls; ++k) {
      if (ld_acquire(&a.sc->arrived) >= (unsigned long long)gridDim.x) {
        ok = 1;
        break;
      }
      __nanosleep(200);
    }
    if (!ok) atomicMax(&a.sc->status, (unsigned long long)kErrTimeout);
    s_ok = ok;
  }
  __syncthreads();
  // Only now may the next kernel on the stream become resident: before the barrier its CTAs could take
  // the place of CTAs of this grid that have not started yet, and the barrier would never complete.
  dep_trigger();

  // ---- writing phase
  if (s_ok && d.fits && (unit_cta ? blockIdx.x : blockIdx.x * upc) < count) {  // CTAs without entries are done
    // chunk offsets: exclusive prefix sum of the chunk sums (warp 0: consecutive chunks per lane)
    {
      uint32_t v[4];
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const uint32_t k = tid + (uint32_t)q * blockDim.x;
        v[q] = k < a.nchunks ? __ldcg(a.chunk_ovf + k) : 0u;
      }
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const uint32_t k = tid + (uint32_t)q * blockDim.x;
        if (k < kMaxChunks) pre[k] = v[q];
      }
    }
    __syncthreads();
    if (warp == 0) {
      constexpr uint32_t per = kMaxChunks / 32;
      uint32_t local = 0;
      for (uint32_t k = 0; k < per; ++k) local += pre[lane32 * per + k];
      uint32_t incl = local;
      for (uint32_t o = 1; o < 32; o <<= 1) {
        const uint32_t up = __shfl_up_sync(0xFFFFFFFFu, incl, o);
        if (lane32 >= o) incl += up;
      }
      uint32_t run = incl - local;
      for (uint32_t k = 0; k < per; ++k) {
        const uint32_t v = pre[lane32 * per + k];
        pre[lane32 * per + k] = run;
        run += v;
      }
    }
    __syncthreads();
    if (taken) {
      // last entry first: its plane is still in the buffer.  Entries whose area was not reused keep their
      // measuring results; the others are measured again.
      team_sync(t);
      for (uint32_t n = taken; n-- > 0;) {
        const uint32_t i = unit + n * units;
        const uint32_t p = a.worklist[i];
        uint32_t* area = areas + min(n, keep - 1u) * area_words;
        if (n + 1u != taken) {
          plane = fetch_plane(t, pl, a.src, p, ubuf);
          if (n >= keep - 1u) {
            info = salient_measure<DT>(t, s_pl, plane, area + 4);
          } else {
            info.nnz_s = area[0];
            info.n_dense = area[1];
            info.n_out_d = area[2];
            info.size = area[3];
          }
        }
        const uint32_t* sal = area + 4;
        const bool raw = a16(info.size) >= a16((uint32_t)pl.plane_bytes);
        const uint32_t my_units = ovf_units(pl, raw ? (uint32_t)pl.plane_bytes : info.size);
        // overflow units of the listed planes before p in its chunk (every warp of the unit computes them)
        uint32_t before = 0;
        for (uint32_t q0 = (p >> a.chunk_shift) << a.chunk_shift; q0 < p; q0 += 32u) {
          const uint32_t q = q0 + lane32;
          uint32_t v = 0;
          if (q < p) {
            const uint32_t cls = __ldcg(reinterpret_cast<const uint32_t*>(table + q) + 1) & 3u;
            if (cls == kClsRaw) {
              v = raw_units;
            } else if (cls == kClsSalient) {
              const uint4 h = __ldcg(reinterpret_cast<const uint4*>(d.dst + pl.slots_off + (uint64_t)q * pl.npay));
              v = ovf_units(pl, salient_size(pl, h.x, h.y, h.z));
            }
          }
          asm volatile("redux.sync.add.u32 %0, %0, %1;" : "+r"(v) : "r"(0xFFFFFFFFu));
          before += v;
        }
        const unsigned long long off16 = (pl.ovf_off >> 4) + pre[p >> a.chunk_shift] + before;
        if ((off16 + my_units) * 16ull <= d.capacity) {  // never write past the capacity
          SplitOut out;
          out.slot = d.dst + pl.slots_off + (uint64_t)p * pl.npay;
          out.ovf = d.dst + off16 * 16ull;
          out.npay = pl.npay;
          if (raw) raw_write(t, s_pl, plane, out);
          else salient_write<DT>(t, s_pl, plane, info, sal, out);
          if (t.lane == 0) *reinterpret_cast<uint32_t*>(d.dst + 64 + 16ull * p) = my_units ? (uint32_t)off16 : 0u;
        }
        team_sync(t);  // the buffer is reused
      }
    }
  }
  // last CTA to leave: clear the chunk sums (all threads), then finish the container (one thread)
  __threadfence();
  __syncthreads();
  if (tid == 0) s_ok = atomicAdd(&a.sc->exited, 1ull) == (unsigned long long)gridDim.x - 1ull;
  __syncthreads();
  if (!s_ok) return;
  for (uint32_t k = tid; k < a.nchunks; k += blockDim.x) a.chunk_ovf[k] = 0u;
  if (tid == 0) {
    __threadfence();
    st_relaxed(&a.sc->exited, 0ull);
    finalize(pl, a, d);
  }
}

}  // namespace fh
