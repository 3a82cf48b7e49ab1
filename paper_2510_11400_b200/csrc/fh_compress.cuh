// Compress kernel: one pass over the dense tensor.
//
// A persistent grid of CTAs takes tiles (runs of consecutive planes) from a ticket counter.  For
// each tile the CTA stages the planes in shared memory, and then, entirely on chip,
//   A. per plane (one team of threads each): min/max and three-sigma statistics, the plane class,
//      and either the packed codes of a normal plane (into a shared staging buffer) or the size of
//      the block-wise encoding of an outlier-rich plane;
//   B. sums the tile's payload sizes, publishes them, and finds the tile's byte offset in the
//      container by a decoupled look-back over the preceding tiles (bounded wait);
//   C. writes table entries and payloads.
// The dense tensor is read from DRAM exactly once and nothing but the container is written.
#pragma once

#include "fh_device.cuh"

namespace fh {

struct Rec {       // per-plane result of phase A, in shared memory
  float lo, scale;
  uint32_t meta;   // class | n_out << 2
  uint32_t size16; // padded payload size / 16
};

struct SalientInfo {
  uint32_t nnz_s, n_dense, n_out_d, size;
};

// Residual codes of one dense 8x8 block (Eq. 7-9): first-order Lorenzo prediction on the
// pre-quantised integers k, neighbours outside the block count as 0.  Returns the number of
// verbatim elements.  WRITE: also emits the 64 code bytes and the verbatim values.
template <int DT, bool WRITE>
__device__ __forceinline__ uint32_t block_codes(const uint8_t* plane, int H, int W, int by, int bx,
                                                float inv2e, uint32_t* g_codes, uint8_t* g_outl) {
  int32_t prev[8];
#pragma unroll
  for (int j = 0; j < 8; ++j) prev[j] = 0;
  uint32_t n_out = 0;
#pragma unroll 1
  for (int i = 0; i < 8; ++i) {
    const int y = by * 8 + i;
    int32_t left = 0, ul = 0;
    uint32_t w0 = 0, w1 = 0;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const int x = bx * 8 + j;
      const bool inpl = (y < H) && (x < W);
      const uint32_t idx = (uint32_t)y * (uint32_t)W + (uint32_t)x;
      const float v = inpl ? load_elem<DT>(plane, idx) : 0.0f;
      bool big;
      const int32_t k = dense_k(v, inv2e, &big);
      const int32_t up = prev[j];
      const int32_t delta = k - (up + left - ul);
      uint32_t code;
      if (!inpl) {
        code = 128u;
      } else if (big || delta > 127 || delta < -127) {
        code = 0u;
        if (WRITE) {
          if (DT == kF32)
            reinterpret_cast<uint32_t*>(g_outl)[n_out] = reinterpret_cast<const uint32_t*>(plane)[idx];
          else
            reinterpret_cast<uint16_t*>(g_outl)[n_out] = reinterpret_cast<const uint16_t*>(plane)[idx];
        }
        ++n_out;
      } else {
        code = (uint32_t)(delta + 128);
      }
      if (j < 4) w0 |= code << (8 * j);
      else w1 |= code << (8 * (j - 4));
      ul = up;
      left = k;
      prev[j] = k;
    }
    if (WRITE) {
      g_codes[2 * i] = w0;
      g_codes[2 * i + 1] = w1;
    }
  }
  return n_out;
}

// Block-wise path, measuring part (Section 4.4.1): non-zero mask pooled per 8x8 block against tau,
// CSR row counts over the sparse blocks, verbatim counts of the dense blocks.  Leaves in shared
// scratch: rowp[0..H] = CSR row pointers, blk_a[b] = 1 for dense blocks, blk_b[b] = rank of block b
// among the dense blocks, blk_c[b] = index of the block's first verbatim value.
template <int DT>
__device__ SalientInfo salient_measure(const Team& t, const Plan& pl, const uint8_t* plane,
                                       uint32_t* rowp, uint32_t* blk_a, uint32_t* blk_b, uint32_t* blk_c) {
  const int H = pl.H, W = pl.W;
  const uint32_t nblk = pl.nblk, nbx = pl.nbx;
  for (uint32_t b = t.lane; b < nblk; b += t.size) blk_a[b] = 0;
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
  // CSR over non-zeros in sparse blocks
  for (int y = (int)t.lane; y <= H; y += (int)t.size) {
    uint32_t cnt = 0;
    if (y < H) {
      const uint32_t* brow = blk_a + (uint32_t)(y >> 3) * nbx;
      for (int x = 0; x < W; ++x)
        cnt += (load_elem<DT>(plane, (uint32_t)y * W + x) != 0.0f) && !brow[x >> 3];
    }
    rowp[y] = cnt;
  }
  team_sync(t);
  info.nnz_s = team_excl_scan(t, rowp, (uint32_t)H + 1u);
  // verbatim counts of dense blocks
  const float two_eps = __fmul_rn(2.0f, pl.eps);
  const float inv2e = __fdiv_rn(1.0f, two_eps);
  for (uint32_t b = t.lane; b < nblk; b += t.size)
    blk_c[b] = blk_a[b] ? block_codes<DT, false>(plane, H, W, (int)(b / nbx), (int)(b % nbx), inv2e,
                                                 nullptr, nullptr)
                        : 0u;
  team_sync(t);
  info.n_out_d = team_excl_scan(t, blk_c, nblk);
  const uint32_t e = (uint32_t)pl.esize;
  info.size = 16u + 4u * pl.nbm + 4u * ((uint32_t)H + 1u) + a4(2u * info.nnz_s) + a4(e * info.nnz_s) +
              64u * info.n_dense + a4(e * info.n_out_d);
  return info;
}

// Block-wise path, writing part; the scratch arrays are those salient_measure left.
template <int DT>
__device__ void salient_write(const Team& t, const Plan& pl, const uint8_t* plane, const SalientInfo& info,
                              const uint32_t* rowp, const uint32_t* blk_a, const uint32_t* blk_b,
                              const uint32_t* blk_c, uint8_t* g) {
  const int H = pl.H, W = pl.W;
  const uint32_t nblk = pl.nblk, nbx = pl.nbx, e = (uint32_t)pl.esize;
  uint32_t* g32 = reinterpret_cast<uint32_t*>(g);
  uint32_t* g_bm = g32 + 4;
  uint32_t* g_rp = g_bm + pl.nbm;
  uint8_t* g_col = reinterpret_cast<uint8_t*>(g_rp + H + 1);
  uint8_t* g_val = g_col + a4(2u * info.nnz_s);
  uint8_t* g_codes = g_val + a4(e * info.nnz_s);
  uint8_t* g_outl = g_codes + 64u * info.n_dense;
  if (t.lane == 0) {
    g32[0] = info.nnz_s; g32[1] = info.n_dense; g32[2] = info.n_out_d; g32[3] = 0;
    // zero the pads the section writers leave: col (2 bytes), val / verbatim (bf16: 2 bytes), tail
    if (info.nnz_s & 1u) reinterpret_cast<uint16_t*>(g_col)[info.nnz_s] = 0;
    if (DT == kBF16 && (info.nnz_s & 1u)) reinterpret_cast<uint16_t*>(g_val)[info.nnz_s] = 0;
    if (DT == kBF16 && (info.n_out_d & 1u)) reinterpret_cast<uint16_t*>(g_outl)[info.n_out_d] = 0;
    for (uint32_t o = info.size; o < a16(info.size); o += 4) g32[o >> 2] = 0;
  }
  for (uint32_t w = t.lane; w < pl.nbm; w += t.size) {
    uint32_t word = 0;
    const uint32_t hi = min(nblk, w * 32u + 32u);
    for (uint32_t b = w * 32u; b < hi; ++b) word |= blk_a[b] << (b & 31u);
    g_bm[w] = word;
  }
  for (uint32_t y = t.lane; y <= (uint32_t)H; y += t.size) g_rp[y] = rowp[y];
  for (int y = (int)t.lane; y < H; y += (int)t.size) {
    uint32_t o = rowp[y];
    const uint32_t* brow = blk_a + (uint32_t)(y >> 3) * nbx;
    for (int x = 0; x < W; ++x) {
      const uint32_t idx = (uint32_t)y * W + x;
      if (load_elem<DT>(plane, idx) != 0.0f && !brow[x >> 3]) {
        reinterpret_cast<uint16_t*>(g_col)[o] = (uint16_t)x;
        if (DT == kF32)
          reinterpret_cast<uint32_t*>(g_val)[o] = reinterpret_cast<const uint32_t*>(plane)[idx];
        else
          reinterpret_cast<uint16_t*>(g_val)[o] = reinterpret_cast<const uint16_t*>(plane)[idx];
        ++o;
      }
    }
  }
  const float two_eps = __fmul_rn(2.0f, pl.eps);
  const float inv2e = __fdiv_rn(1.0f, two_eps);
  for (uint32_t b = t.lane; b < nblk; b += t.size)
    if (blk_a[b])
      block_codes<DT, true>(plane, H, W, (int)(b / nbx), (int)(b % nbx), inv2e,
                            reinterpret_cast<uint32_t*>(g_codes + 64u * blk_b[b]), g_outl + e * blk_c[b]);
}

struct CompressArgs {
  const uint8_t* src;
  uint8_t* dst_base;
  unsigned long long capacity;                 // bytes available at dst_base (+ offset below)
  const unsigned long long* d_off_in;          // optional: byte offset of the container in dst_base
  unsigned long long* d_off_out;               // optional: offset for the next container
  unsigned long long* out2;                    // optional: {total bytes, status}
  Scratch* sc;
  TileState* ts;
  uint32_t epoch;
  unsigned long long ticket_base, done_base;
  uint32_t spin_limit;
};

template <int DT, int BITS>
__global__ void __launch_bounds__(kThreads) compress_kernel(const Plan pl, const CompressArgs a) {
  extern __shared__ __align__(16) uint8_t smem[];
  __shared__ double s_red[kThreads / 32 * 4 + 8];
  __shared__ uint32_t s_tile;
  __shared__ unsigned long long s_base16, s_cnt_excl;
  __shared__ uint32_t s_tile16, s_tile_nsal, s_tile_nraw, s_skip;

  const uint32_t tid = threadIdx.x;
  uint8_t* tile_buf = smem + pl.sm_tile;
  uint8_t* out_buf = smem + pl.sm_out;
  Rec* rec = reinterpret_cast<Rec*>(smem + pl.sm_rec);
  uint32_t* roff = reinterpret_cast<uint32_t*>(smem + pl.sm_rec + 16u * pl.ppt);
  const unsigned long long off_in = a.d_off_in ? *a.d_off_in : 0ull;
  uint8_t* dst = a.dst_base + off_in;
  const unsigned long long capacity = a.capacity > off_in ? a.capacity - off_in : 0ull;
  const unsigned long long epoch_hi = (unsigned long long)a.epoch << 32;
  const unsigned long long table_end = 64ull + 16ull * pl.P;
  const Team team = make_team(pl.team, s_red);
  const uint32_t nteams = team.block ? 1u : kThreads / team.size;
  const uint32_t my_team = team.block ? 0u : tid / team.size;
  constexpr uint32_t L = (1u << BITS) - 1u;

  for (;;) {
    if (tid == 0) s_tile = (uint32_t)(atomicAdd(&a.sc->ticket, 1ull) - a.ticket_base);
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
      const bool vec = ((uint32_t)__cvta_generic_to_shared(plane) & (DT == kF32 ? 15u : 7u)) == 0u;
      const uint32_t HW = pl.HW, nfull = HW >> 2, groups = pl.groups;
      Stats s;
      s.lo = __int_as_float(0x7F800000);
      s.hi = __int_as_float(0xFF800000);
      s.S = 0.0;
      s.Q = 0.0;
      const bool need_sigma = pl.mode == kModeAuto;
      for (uint32_t g = team.lane; g < nfull; g += team.size) {
        float v[4];
        load_group<DT>(plane, g, HW, vec, v);
        s.lo = min_nan(s.lo, min_nan(min_nan(v[0], v[1]), min_nan(v[2], v[3])));
        s.hi = max_nan(s.hi, max_nan(max_nan(v[0], v[1]), max_nan(v[2], v[3])));
        if (need_sigma) {
          const float sg = __fadd_rn(__fadd_rn(v[0], v[1]), __fadd_rn(v[2], v[3]));
          const float q01 = __fmaf_rn(v[1], v[1], __fmul_rn(v[0], v[0]));
          const float q23 = __fmaf_rn(v[3], v[3], __fmul_rn(v[2], v[2]));
          s.S += (double)sg;
          s.Q += (double)__fadd_rn(q01, q23);
        }
      }
      if ((HW & 3u) && team.lane == 0) {  // ragged last group: zero padded for the sums only
        float v[4];
        load_group<DT>(plane, nfull, HW, false, v);
        for (uint32_t k = 0; k < (HW & 3u); ++k) {
          s.lo = min_nan(s.lo, v[k]);
          s.hi = max_nan(s.hi, v[k]);
        }
        if (need_sigma) {
          const float sg = __fadd_rn(__fadd_rn(v[0], v[1]), __fadd_rn(v[2], v[3]));
          const float q01 = __fmaf_rn(v[1], v[1], __fmul_rn(v[0], v[0]));
          const float q23 = __fmaf_rn(v[3], v[3], __fmul_rn(v[2], v[2]));
          s.S += (double)sg;
          s.Q += (double)__fadd_rn(q01, q23);
        }
      }
      s = team_reduce_stats(team, s);
      const float range = __fsub_rn(s.hi, s.lo);
      if (!(fabsf(range) <= 3.402823466e38f) && team.lane == 0)
        atomicMax(&a.sc->status, epoch_hi | kErrNonfinite);

      uint32_t cls = kClsNormal, n_out = 0;
      if (need_sigma) {
        const double hw = (double)HW;
        const double mu = __ddiv_rn(s.S, hw);
        double var = __dsub_rn(__ddiv_rn(s.Q, hw), __dmul_rn(mu, mu));
        if (!(var > 0.0)) var = 0.0;
        const double three = __dmul_rn(3.0, __dsqrt_rn(var));
        const float thi = __double2float_rn(__dadd_rn(mu, three));
        const float tlo = __double2float_rn(__dsub_rn(mu, three));
        uint32_t cnt = 0;
        for (uint32_t g = team.lane; g < groups; g += team.size) {
          float v[4];
          load_group<DT>(plane, g, HW, vec, v);
#pragma unroll
          for (int k = 0; k < 4; ++k) cnt += (v[k] > thi) || (v[k] < tlo);
        }
        n_out = team_sum_u32(team, cnt);
        if ((0.0f > thi) || (0.0f < tlo)) n_out -= 4u * groups - HW;  // padded zeros are not elements
        if ((uint64_t)n_out * pl.rho_den > (uint64_t)pl.rho_num * HW) cls = kClsSalient;
      } else if (pl.mode == kModeAll) {
        cls = kClsSalient;
      }

      float lo_out = 0.0f, scale_out = 0.0f;
      uint32_t size = 0;
      if (cls == kClsSalient) {
        uint32_t* sal = reinterpret_cast<uint32_t*>(smem + pl.sm_sal + (uint64_t)my_team * pl.sm_sal_stride);
        const SalientInfo info =
            salient_measure<DT>(team, pl, plane, sal, sal + pl.H + 1, sal + pl.H + 1 + pl.nblk,
                                sal + pl.H + 1 + 2 * pl.nblk);
        size = info.size;
        if (a16(size) >= a16((uint32_t)pl.plane_bytes)) {
          cls = kClsRaw;
          size = (uint32_t)pl.plane_bytes;
        }
      } else {
        float inv = __fdiv_rn((float)L, range), scale = __fdiv_rn(range, (float)L);
        if (range == 0.0f || !(fabsf(inv) <= 3.402823466e38f)) {
          inv = 0.0f;
          scale = 0.0f;
        }
        lo_out = s.lo;
        scale_out = scale;
        size = pl.npay;
        uint8_t* o = out_buf + (uint64_t)lp * pl.npay;
        const uint32_t ogroups = pl.npay * 2u / BITS;
        for (uint32_t g = team.lane; g < ogroups; g += team.size) {
          uint32_t word = 0;
          if (g < groups) {
            float v[4];
            load_group<DT>(plane, g, HW, vec, v);
#pragma unroll
            for (int k = 0; k < 4; ++k) {
              const float d = __fsub_rn(v[k], s.lo);
              const float r = __fmaf_rn(d, inv, 12582912.0f);  // exact product, rne to an integer
              uint32_t q = (__float_as_uint(r) - 0x4B400000u) & L;
              if (g * 4u + k >= HW) q = 0;
              word |= q << (k * BITS);
            }
          }
          if (BITS == 2) o[g] = (uint8_t)word;
          else if (BITS == 4) reinterpret_cast<uint16_t*>(o)[g] = (uint16_t)word;
          else reinterpret_cast<uint32_t*>(o)[g] = word;
        }
      }
      if (team.lane == 0) {
        Rec r;
        r.lo = lo_out;
        r.scale = scale_out;
        r.meta = cls | (n_out << 2);
        r.size16 = a16(size) >> 4;
        rec[lp] = r;
      }
    }
    __syncthreads();

    // ---- phase B: offsets inside the tile, then the tile's offset in the container
    if (tid < 32) {
      uint32_t carry = 0, nsal = 0, nraw = 0;
      for (uint32_t base = 0; base < np; base += 32) {
        const uint32_t i = base + tid;
        const uint32_t v = i < np ? rec[i].size16 : 0u;
        const uint32_t c = i < np ? (rec[i].meta & 3u) : 0u;
        uint32_t incl = v;
        for (uint32_t o = 1; o < 32; o <<= 1) {
          const uint32_t up = __shfl_up_sync(0xFFFFFFFFu, incl, o);
          if (tid >= o) incl += up;
        }
        if (i < np) roff[i] = carry + incl - v;
        carry += __shfl_sync(0xFFFFFFFFu, incl, 31);
        nsal += __popc(__ballot_sync(0xFFFFFFFFu, c == kClsSalient));
        nraw += __popc(__ballot_sync(0xFFFFFFFFu, c == kClsRaw));
      }
      if (tid == 0) {
        unsigned long long excl = 0, cnt_excl = 0;
        uint32_t skip = 0;
        const unsigned long long my_b = ((unsigned long long)nsal << 32) | nraw;
        if (pl.mode == kModeOff) {
          excl = (unsigned long long)tile * pl.ppt * (pl.npay >> 4);
        } else {
          TileState* me = a.ts + tile;
          if (tile > 0) {
            st_relaxed(&me->agg_b, my_b);
            st_release(&me->agg_a, epoch_hi | carry);
            long long j = (long long)tile - 1;
            uint32_t spins = 0;
            while (j >= 0) {
              const TileState* pr = a.ts + j;
              const unsigned long long ia = ld_acquire(&pr->inc_a);
              if ((ia >> 32) == a.epoch) {
                excl += (uint32_t)ia;
                cnt_excl += ld_relaxed(&pr->inc_b);
                break;
              }
              const unsigned long long aa = ld_acquire(&pr->agg_a);
              if ((aa >> 32) == a.epoch) {
                excl += (uint32_t)aa;
                cnt_excl += ld_relaxed(&pr->agg_b);
                --j;
                continue;
              }
              if (++spins > a.spin_limit) {  // the predecessor never published: give up cleanly
                atomicMax(&a.sc->status, epoch_hi | kErrTimeout);
                skip = 1;
                break;
              }
              __nanosleep(64);
            }
          }
          st_relaxed(&me->inc_b, cnt_excl + my_b);
          st_release(&me->inc_a, epoch_hi | (uint32_t)(excl + carry));
        }
        s_base16 = (table_end >> 4) + excl;
        s_cnt_excl = cnt_excl;
        s_tile16 = carry;
        s_tile_nsal = nsal;
        s_tile_nraw = nraw;
        // never write past the capacity
        if (((table_end >> 4) + excl + carry) * 16ull > capacity) skip = 1;
        if (64ull + 16ull * (p0 + np) > capacity) skip = 1;
        s_skip = skip;
      }
    }
    __syncthreads();

    // ---- phase C: table entries and payloads
    if (!s_skip) {
      const unsigned long long base16 = s_base16;
      uint4* table = reinterpret_cast<uint4*>(dst + 64) + p0;
      for (uint32_t i = tid; i < np; i += kThreads) {
        const Rec r = rec[i];
        uint4 e;
        e.x = (uint32_t)(base16 + roff[i]);
        e.y = r.meta;
        e.z = __float_as_uint(r.lo);
        e.w = __float_as_uint(r.scale);
        table[i] = e;
      }
      // normal payloads: straight 16-byte copies out of the staging buffer
      const uint32_t chunks = pl.npay >> 4;
      for (uint32_t i = tid; i < np * chunks; i += kThreads) {
        const uint32_t lp = i / chunks, c = i - lp * chunks;
        if ((rec[lp].meta & 3u) == kClsNormal)
          reinterpret_cast<uint4*>(dst + (base16 + roff[lp]) * 16ull)[c] =
              reinterpret_cast<const uint4*>(out_buf + (uint64_t)lp * pl.npay)[c];
      }
      if (s_tile_nsal + s_tile_nraw) {
        for (uint32_t lp = my_team; lp < np; lp += nteams) {
          const uint32_t cls = rec[lp].meta & 3u;
          if (cls == kClsNormal) continue;
          const uint8_t* plane = tile_buf + head + (uint64_t)lp * pl.plane_bytes;
          uint8_t* g = dst + (base16 + roff[lp]) * 16ull;
          if (cls == kClsRaw) {
            const uint32_t n = (uint32_t)pl.plane_bytes >> 1;  // copy as 16-bit units
            for (uint32_t i = team.lane; i < (a16((uint32_t)pl.plane_bytes) >> 1); i += team.size)
              reinterpret_cast<uint16_t*>(g)[i] = i < n ? reinterpret_cast<const uint16_t*>(plane)[i] : (uint16_t)0;
          } else {
            uint32_t* sal = reinterpret_cast<uint32_t*>(smem + pl.sm_sal + (uint64_t)my_team * pl.sm_sal_stride);
            uint32_t* rowp = sal;
            uint32_t* blk_a = sal + pl.H + 1;
            uint32_t* blk_b = blk_a + pl.nblk;
            uint32_t* blk_c = blk_b + pl.nblk;
            const SalientInfo info = salient_measure<DT>(team, pl, plane, rowp, blk_a, blk_b, blk_c);
            salient_write<DT>(team, pl, plane, info, rowp, blk_a, blk_b, blk_c, g);
          }
        }
      }
    }
    // the tile holding the last planes knows the totals: header
    if (tile == pl.ntiles - 1 && tid == 0) {
      const unsigned long long total = (s_base16 + s_tile16) * 16ull;
      st_relaxed(&a.sc->total, total);
      if (total > capacity) atomicMax(&a.sc->status, epoch_hi | kErrCapacity);
      if (!s_skip && capacity >= 64) {
        const unsigned long long cnt = s_cnt_excl + (((unsigned long long)s_tile_nsal << 32) | s_tile_nraw);
        uint32_t h[16];
        h[0] = kMagic;
        h[1] = 1u | ((uint32_t)pl.dtype << 16) | ((uint32_t)pl.bits << 24);
        h[2] = pl.N;
        h[3] = pl.C;
        h[4] = (uint32_t)pl.H;
        h[5] = (uint32_t)pl.W;
        h[6] = 8u | (8u << 8) | (0u << 16) | ((uint32_t)pl.mode << 24);
        h[7] = pl.rho_num | (pl.rho_den << 16);
        h[8] = pl.tau_num | (pl.tau_den << 16);
        h[9] = __float_as_uint(pl.eps);
        h[10] = (uint32_t)(cnt >> 32);
        h[11] = (uint32_t)cnt;
        h[12] = (uint32_t)pl.tensor_id;
        h[13] = (uint32_t)(pl.tensor_id >> 32);
        h[14] = (uint32_t)total;
        h[15] = (uint32_t)(total >> 32);
        uint32_t* hd = reinterpret_cast<uint32_t*>(dst);
        for (int k = 0; k < 16; ++k) hd[k] = h[k];
      }
    }
    __threadfence();
    __syncthreads();
    if (tid == 0) {
      const unsigned long long prev = atomicAdd(&a.sc->done, 1ull) - a.done_base;
      if (prev == (unsigned long long)pl.ntiles - 1ull) {  // every tile has finished
        __threadfence();
        const unsigned long long total = ld_relaxed(&a.sc->total);
        const unsigned long long st = ld_relaxed(&a.sc->status);
        const uint32_t code = (st >> 32) == a.epoch ? (uint32_t)st : kErrNone;
        if (a.out2) {
          a.out2[0] = total;
          a.out2[1] = status_word(code);
        }
        // a failed container must not be mistaken for a valid one, and nothing may follow it
        if (code != kErrNone && capacity >= 4) *reinterpret_cast<uint32_t*>(dst) = 0u;
        if (a.d_off_out) *a.d_off_out = code == kErrNone ? off_in + ((total + 255ull) & ~255ull) : (~0ull >> 1);
      }
    }
  }
}

}  // namespace fh
