// Decompress kernel: container -> dense tensor, one pass.
//
// Planes are independent and their slots sit at closed-form offsets, so the kernel needs no
// hand-out and no barrier: team t of the grid restores planes t, t + teams, ...  A team is a
// power-of-two slice of a warp (a whole warp for planes of 256 groups and more).  Normal planes are
// the fused unpack-and-dequantise: code bytes are read straight from the slot (they are 1/16 to 1/4
// of the output), four values per thread and step go out as one 16-byte (fp32) or 8-byte (bf16)
// store.  Raw planes are copied; outlier-rich planes take zero fill + CSR scatter + inverse Lorenzo
// walk of the dense blocks.  Every read of the container is bounds-checked against src_bytes; a
// plane whose table entry or payload is inconsistent is left unwritten and the call reports
// FH_ERR_CORRUPT.
#pragma once

#include "fh_device.cuh"

namespace fh {

struct DecompressArgs {
  const uint8_t* src_base;
  unsigned long long src_bytes;
  const unsigned long long* d_off_in;  // optional: byte offset of the container in src_base
  uint8_t* dst;
  unsigned long long* d_status;        // optional
  Scratch* sc;
  unsigned long long team_stride;      // a prime, at most the number of teams of the grid (see the kernel)
};

// Reads of a salient / raw payload: offsets below npay come from the plane's slot, the rest from its
// overflow part.
struct SplitIn {
  const uint8_t* slot;
  const uint8_t* ovf;
  uint32_t npay;
  __device__ __forceinline__ const uint8_t* at(uint32_t o) const { return o < npay ? slot + o : ovf + (o - npay); }
  __device__ __forceinline__ uint32_t ld32(uint32_t o) const { return __ldg(reinterpret_cast<const uint32_t*>(at(o))); }
  __device__ __forceinline__ uint32_t ld16(uint32_t o) const { return __ldg(reinterpret_cast<const uint16_t*>(at(o))); }
  __device__ __forceinline__ uint32_t ld8(uint32_t o) const { return __ldg(at(o)); }
};

// One thread decodes a dense block's chunk of the Huffman-coded section (`nbytes` bytes at payload offset
// `o_chunk`) into the block's 64 code bytes, four to a word.  False when the chunk is inconsistent.
template <typename In>
__device__ __noinline__ bool huffman_decode_chunk(const In& in, uint32_t o_chunk, uint32_t nbytes, const HufDecode* hd,
                                                  uint32_t* codes) {
  const uint32_t nbits = nbytes * 8u;
  uint32_t pos = 0, cur = 0;
  for (uint32_t i = 0; i < 16u; ++i) codes[i] = 0;
  for (uint32_t i = 0; i < 64u; ++i) {
    uint32_t acc = 0, sym = 256;
    for (uint32_t l = 1; l <= kHufMaxLen; ++l) {
      if (pos >= nbits) return false;
      if ((pos & 7u) == 0u) cur = in.ld8(o_chunk + (pos >> 3));
      acc = (acc << 1) | ((cur >> (7u - (pos & 7u))) & 1u);
      ++pos;
      const uint32_t k = acc - hd->first[l];
      if (k < (uint32_t)hd->count[l]) {
        sym = hd->sorted[hd->base[l] + k];
        break;
      }
    }
    if (sym > 255u) return false;
    codes[i >> 2] |= sym << (8u * (i & 3u));
  }
  return true;
}

template <int DT>
__device__ __forceinline__ void store_elem(uint8_t* plane, uint32_t i, float v) {
  if (DT == kF32) reinterpret_cast<float*>(plane)[i] = v;
  else reinterpret_cast<uint16_t*>(plane)[i] = (uint16_t)f32_to_bf16_bits(v);
}

// x = fma(q, scale, lo); q < 2^23 is turned into a float through its bit pattern.
__device__ __forceinline__ float dequant(uint32_t q, float scale, float lo) {
  const float qf = __fsub_rn(__uint_as_float(0x4B000000u | q), 8388608.0f);
  return __fmaf_rn(qf, scale, lo);
}

// Outlier-rich plane.  `scr` is the team's shared scratch: 2 * nblk words, followed by a HufDecode.  `ovf_avail`
// is the number of readable bytes behind in.ovf; `version` the container's (2: the dense blocks' codes may be
// Huffman-coded, Section 4.4.1 "Decompression involves Huffman decoding").
template <int DT>
__device__ __noinline__ bool decode_salient(const Team& t, const Plan& pl, const SplitIn& in, uint64_t ovf_avail, float eps,
                               uint8_t* out, uint32_t* scr, uint32_t version) {
  const int H = pl.H, W = pl.W;
  const uint32_t nblk = pl.nblk, nbx = pl.nbx, nbm = pl.nbm, e = (uint32_t)pl.esize, HW = pl.HW;
  const uint32_t nnz_s = in.ld32(0), n_dense = in.ld32(4), n_out_d = in.ld32(8), coded = in.ld32(12);
  if (nnz_s > HW || n_dense > nblk || n_out_d > HW) return false;
  if (coded && (version != 2u || (coded & 3u) || coded >= 64u * n_dense)) return false;
  const uint64_t size = 16ull + 4ull * nbm + 4ull * ((uint64_t)H + 1) + a4(2u * nnz_s) + a4(e * nnz_s) +
                        (coded ? (uint64_t)coded : 64ull * n_dense) + a4(e * n_out_d);
  if (size > in.npay && size - in.npay > ovf_avail) return false;
  const uint32_t o_bm = 16u, o_rp = o_bm + 4u * nbm, o_col = o_rp + 4u * ((uint32_t)H + 1u);
  const uint32_t o_val = o_col + a4(2u * nnz_s), o_codes = o_val + a4(e * nnz_s);
  const uint32_t o_outl = o_codes + (coded ? coded : 64u * n_dense);
  bool ok = true;
  // Huffman-coded section: decoding tables from the stored lengths, start of every chunk from the chunks' sizes
  uint32_t* cho = scr + nblk;  // by rank among the dense blocks
  HufDecode* hd = reinterpret_cast<HufDecode*>(scr + 2u * nblk);
  uint32_t o_chunks = 0, o_cb = 0;
  if (coded) {
    const uint32_t smin = in.ld8(o_codes + 1u), smax = in.ld8(o_codes + 2u);
    if (smin < 1u || smax < smin) return false;
    const uint32_t nl = smax - smin + 1u;
    o_cb = o_codes + 4u + a4(nl);
    o_chunks = o_cb + a4(n_dense);
    if (o_chunks - o_codes > coded) return false;
    for (uint32_t sym = t.lane; sym < 256u; sym += t.size)
      hd->len[sym] = sym == 0u ? (uint8_t)in.ld8(o_codes) : ((sym >= smin && sym <= smax) ? (uint8_t)in.ld8(o_codes + 4u + sym - smin) : (uint8_t)0);
    for (uint32_t r = t.lane; r < nblk; r += t.size) cho[r] = r < n_dense ? in.ld8(o_cb + r) : 0u;
    team_sync(t);
    if (t.lane == 0) huffman_tables(hd);
    const uint32_t chunks = team_excl_scan(t, cho, nblk);
    if (!hd->ok || o_chunks - o_codes + chunks > coded) return false;  // (the same for every thread)
  }
  // zero fill (16-bit units cover both element sizes)
  for (uint32_t i = t.lane; i < (uint32_t)(pl.plane_bytes >> 1); i += t.size) reinterpret_cast<uint16_t*>(out)[i] = 0;
  // verbatim counts of the dense blocks -> first verbatim index of each block
  for (uint32_t b = t.lane; b < nblk; b += t.size) {
    uint32_t cnt = 0;
    if ((in.ld32(o_bm + 4u * (b >> 5)) >> (b & 31u)) & 1u) {
      uint32_t rank = 0;
      for (uint32_t w = 0; w < (b >> 5); ++w) rank += __popc(in.ld32(o_bm + 4u * w));
      rank += __popc(in.ld32(o_bm + 4u * (b >> 5)) & ((1u << (b & 31u)) - 1u));
      if (rank < n_dense) {
        uint32_t cw[16];
        if (coded && !huffman_decode_chunk(in, o_chunks + cho[rank], in.ld8(o_cb + rank), hd, cw)) ok = false;
        for (uint32_t k = 0; k < 16; ++k) {
          const uint32_t w = coded ? cw[k] : in.ld32(o_codes + 64u * rank + 4u * k);
          cnt += ((w & 0xFFu) == 0) + ((w & 0xFF00u) == 0) + ((w & 0xFF0000u) == 0) + ((w & 0xFF000000u) == 0);
        }
      } else {
        ok = false;
      }
    }
    scr[b] = cnt;
  }
  team_sync(t);
  const uint32_t tot_out = team_excl_scan(t, scr, nblk);
  if (tot_out > n_out_d) ok = false;
  // CSR scatter
  for (int y = (int)t.lane; y < H; y += (int)t.size) {
    const uint32_t r0 = in.ld32(o_rp + 4u * y), r1 = in.ld32(o_rp + 4u * (y + 1));
    if (r0 > r1 || r1 > nnz_s) { ok = false; continue; }
    for (uint32_t k = r0; k < r1; ++k) {
      const uint32_t col = in.ld16(o_col + 2u * k);
      if (col >= (uint32_t)W) { ok = false; continue; }
      const uint32_t idx = (uint32_t)y * W + col;
      if (DT == kF32) reinterpret_cast<uint32_t*>(out)[idx] = in.ld32(o_val + 4u * k);
      else reinterpret_cast<uint16_t*>(out)[idx] = (uint16_t)in.ld16(o_val + 2u * k);
    }
  }
  // dense blocks: raster walk, k = pred + residual (Eq. 7-9), x = k * 2 eps
  const float two_eps = __fmul_rn(2.0f, eps);
  const float inv2e = __fdiv_rn(1.0f, two_eps);
  if (ok && tot_out <= n_out_d) {
    for (uint32_t b = t.lane; b < nblk; b += t.size) {
      if (!((in.ld32(o_bm + 4u * (b >> 5)) >> (b & 31u)) & 1u)) continue;
      uint32_t rank = 0;
      for (uint32_t w = 0; w < (b >> 5); ++w) rank += __popc(in.ld32(o_bm + 4u * w));
      rank += __popc(in.ld32(o_bm + 4u * (b >> 5)) & ((1u << (b & 31u)) - 1u));
      const uint32_t oc = o_codes + 64u * rank;
      uint32_t cw[16];
      if (coded && !huffman_decode_chunk(in, o_chunks + cho[rank], in.ld8(o_cb + rank), hd, cw)) {
        ok = false;
        continue;
      }
      uint32_t oi = scr[b];
      const int by = (int)(b / nbx), bx = (int)(b % nbx);
      int32_t prev[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) prev[j] = 0;
#pragma unroll 1
      for (int i = 0; i < 8; ++i) {
        const int y = by * 8 + i;
        const uint32_t w0 = coded ? cw[2 * i] : in.ld32(oc + 8u * i), w1 = coded ? cw[2 * i + 1] : in.ld32(oc + 8u * i + 4u);
        int32_t left = 0, ul = 0;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const int x = bx * 8 + j;
          const uint32_t code = ((j < 4 ? w0 : w1) >> (8 * (j & 3))) & 0xFFu;
          const int32_t up = prev[j];
          const int32_t pred = up + left - ul;
          int32_t k = pred;
          if (y < H && x < W) {
            const uint32_t idx = (uint32_t)y * W + x;
            if (code == 0u) {
              float v;
              if (DT == kF32) {
                const uint32_t raw = in.ld32(o_outl + 4u * oi);
                reinterpret_cast<uint32_t*>(out)[idx] = raw;
                v = __uint_as_float(raw);
              } else {
                const uint32_t raw = in.ld16(o_outl + 2u * oi);
                reinterpret_cast<uint16_t*>(out)[idx] = (uint16_t)raw;
                v = bf16_bits_to_f32(raw);
              }
              bool big;
              k = dense_k(v, inv2e, &big);
              ++oi;
            } else {
              k = pred + (int32_t)code - 128;
              store_elem<DT>(out, idx, __fmul_rn((float)k, two_eps));
            }
          }
          ul = up;
          left = k;
          prev[j] = k;
        }
      }
    }
  }
  return ok;
}

// Header of a container against what the caller expects: 0 if it does not fit, the container's version (1, 2)
// otherwise; also returns code width, eps and total size.
__device__ __forceinline__ uint32_t check_header(const Plan& pl, const uint8_t* src, unsigned long long src_bytes, uint32_t& bits,
                                                 float& eps, unsigned long long& total) {
  if (src_bytes < 64ull + 16ull * pl.P) return 0u;
  const uint32_t* h = reinterpret_cast<const uint32_t*>(src);
  bits = __ldg(h + 1) >> 24;
  const uint32_t version = __ldg(h + 1) & 0xFFFFu;
  bool ok = __ldg(h) == kMagic && (version == 1u || version == 2u) && ((__ldg(h + 1) >> 16) & 0xFFu) == (uint32_t)pl.dtype &&
            (bits == 2u || bits == 4u || bits == 8u) && __ldg(h + 2) == pl.N && __ldg(h + 3) == pl.C &&
            __ldg(h + 4) == (uint32_t)pl.H && __ldg(h + 5) == (uint32_t)pl.W && (__ldg(h + 6) & 0xFFFFu) == (8u | (8u << 8));
  total = (unsigned long long)__ldg(h + 14) | ((unsigned long long)__ldg(h + 15) << 32);
  eps = __uint_as_float(__ldg(h + 9));
  const unsigned long long npay = a16(4u * ((pl.HW * (bits & 15u) + 31u) / 32u));
  ok = ok && total <= src_bytes && total >= 64ull + 16ull * pl.P + pl.P * npay && eps >= 1e-30f && eps <= 1e30f;
  return ok ? version : 0u;
}

// Last step of every CTA.  The exit counter carries the CTAs that have left in its low half and, in its high half,
// how many of them had found something wrong; only such a CTA reports and fences, and the last CTA reads the
// status back only when there was one: a clean call ends with one atomic per CTA.  (The restored tensor needs no
// fence: its readers are later kernels.)
__device__ __forceinline__ void decompress_exit(const DecompressArgs& a, bool bad) {
  const bool any_bad = __syncthreads_or(bad) != 0;  // (the same for every thread)
  if (any_bad) {
    if (bad) atomicMax(&a.sc->status, (unsigned long long)kErrCorrupt);
    __threadfence();
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    const unsigned long long old = atomicAdd(&a.sc->exited, 1ull | (any_bad ? 1ull << 32 : 0ull));
    if ((uint32_t)old == gridDim.x - 1u) {
      uint32_t code = kErrNone;
      if ((old >> 32) != 0ull || any_bad) {
        __threadfence();
        code = (uint32_t)ld_relaxed(&a.sc->status);
        st_relaxed(&a.sc->status, 0ull);
      }
      if (a.d_status) *a.d_status = status_word(code);
      st_relaxed(&a.sc->exited, 0ull);
    }
  }
}

// Four restored values of one group leave as one 16-byte (fp32) or 8-byte (bf16) store.
template <int DT>
__device__ __forceinline__ void store_group(uint8_t* out, uint32_t g, float v0, float v1, float v2, float v3) {
  if (DT == kF32) {
    reinterpret_cast<float4*>(out)[g] = make_float4(v0, v1, v2, v3);
  } else {
    uint2 w;
    w.x = f32x2_to_bf16x2(v0, v1);
    w.y = f32x2_to_bf16x2(v2, v3);
    reinterpret_cast<uint2*>(out)[g] = w;
  }
}

// Normal plane, whole-warp team, one chunk of up to 256 groups starting at group g0 (a multiple of
// 256).  The chunk's code bytes are fetched as 32-bit words, one or more coalesced loads per lane
// issued before anything else, and handed to the lanes that need them by shuffle: lane l restores
// groups g0 + l, g0 + 32 + l, ...  `w` holds the lane's words: word j*32 + l of the chunk's codes.
template <int DT, int BITS>
__device__ __forceinline__ void decode_chunk32(const uint32_t (&w)[8], uint32_t lane, uint32_t g0, uint32_t g1,
                                               float scale, float lo, uint8_t* out) {
  constexpr uint32_t L = (1u << BITS) - 1u;
#pragma unroll
  for (int k = 0; k < 8; ++k) {
    const uint32_t g = g0 + (uint32_t)k * 32u + lane;
    uint32_t word;
    if (BITS == 2) {         // one code byte per group: byte k*32 + l = word k*8 + (l >> 2), byte l & 3
      const uint32_t src = __shfl_sync(0xFFFFFFFFu, w[k >> 2], (uint32_t)(k & 3) * 8u + (lane >> 2));
      word = (src >> ((lane & 3u) * 8u)) & 0xFFu;
    } else if (BITS == 4) {  // two code bytes per group: halfword k*32 + l = word k*16 + (l >> 1)
      const uint32_t src = __shfl_sync(0xFFFFFFFFu, w[k >> 1], (uint32_t)(k & 1) * 16u + (lane >> 1));
      word = (src >> ((lane & 1u) * 16u)) & 0xFFFFu;
    } else {                 // one word per group
      word = w[k];
    }
    if (g < g1)
      store_group<DT>(out, g, dequant(word & L, scale, lo), dequant((word >> BITS) & L, scale, lo),
                      dequant((word >> (2 * BITS)) & L, scale, lo), dequant((word >> (3 * BITS)) & L, scale, lo));
  }
}

// The same for bf16 planes of whole 16-byte chunks: a lane restores two neighbouring groups at a time -- groups
// g0 + 64 k + 2 l and the one after it -- so that eight values leave as one 16-byte store (four stores of 512
// contiguous bytes per warp and chunk instead of eight of 256).
template <int BITS>
__device__ __forceinline__ void decode_chunk32_bf16_pairs(const uint32_t (&w)[8], uint32_t lane, uint32_t g0, uint32_t g1,
                                                          float scale, float lo, uint8_t* out) {
  constexpr uint32_t L = (1u << BITS) - 1u, full = 0xFFFFFFFFu;
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const uint32_t g = g0 + (uint32_t)k * 64u + 2u * lane;
    uint32_t wa, wb;  // code words of groups g and g + 1
    if (BITS == 2) {         // a byte per group: halfword 32 k + l of the chunk = word 16 k + (l >> 1)
      const uint32_t src = __shfl_sync(full, w[k >> 1], (uint32_t)(k & 1) * 16u + (lane >> 1));
      const uint32_t h = src >> ((lane & 1u) * 16u);
      wa = h & 0xFFu;
      wb = (h >> 8) & 0xFFu;
    } else if (BITS == 4) {  // two bytes per group: word 32 k + l, the lane's own
      wa = w[k] & 0xFFFFu;
      wb = w[k] >> 16;
    } else {                 // a word per group: words 64 k + 2 l and the next, held by lanes 2 l mod 32 and the next
      const uint32_t sl = (2u * lane) & 31u;
      const uint32_t a0 = __shfl_sync(full, w[2 * k], sl), a1 = __shfl_sync(full, w[2 * k + 1], sl);
      const uint32_t b0 = __shfl_sync(full, w[2 * k], sl + 1u), b1 = __shfl_sync(full, w[2 * k + 1], sl + 1u);
      wa = lane < 16u ? a0 : a1;
      wb = lane < 16u ? b0 : b1;
    }
    uint4 v;
    v.x = f32x2_to_bf16x2(dequant(wa & L, scale, lo), dequant((wa >> BITS) & L, scale, lo));
    v.y = f32x2_to_bf16x2(dequant((wa >> (2 * BITS)) & L, scale, lo), dequant((wa >> (3 * BITS)) & L, scale, lo));
    v.z = f32x2_to_bf16x2(dequant(wb & L, scale, lo), dequant((wb >> BITS) & L, scale, lo));
    v.w = f32x2_to_bf16x2(dequant((wb >> (2 * BITS)) & L, scale, lo), dequant((wb >> (3 * BITS)) & L, scale, lo));
    if (g + 1u < g1) reinterpret_cast<uint4*>(out)[g >> 1] = v;
    else if (g < g1) reinterpret_cast<uint2*>(out)[g] = make_uint2(v.x, v.y);
  }
}

// Normal plane, sub-warp team of TT lanes (planes of at most 8 * TT groups, one chunk).  cw[k] holds the
// code word of group lane + k * TT, requested before the table entry was known.  Whole groups of planes
// that start on a vector boundary leave as one store; everything else (planes that do not, the ragged
// last group) as element stores.
template <int DT, int BITS, int TT>
__device__ __forceinline__ void decode_small(const uint32_t (&cw)[8], uint32_t lane, uint32_t groups, uint32_t nfull,
                                             uint32_t HW, float scale, float lo, uint8_t* out) {
  constexpr uint32_t L = (1u << BITS) - 1u;
#pragma unroll
  for (int k = 0; k < 8; ++k) {
    const uint32_t g = lane + (uint32_t)k * TT, word = cw[k];
    if (g >= groups) break;
    const float v0 = dequant(word & L, scale, lo), v1 = dequant((word >> BITS) & L, scale, lo);
    const float v2 = dequant((word >> (2 * BITS)) & L, scale, lo), v3 = dequant((word >> (3 * BITS)) & L, scale, lo);
    if (g < nfull) {
      store_group<DT>(out, g, v0, v1, v2, v3);
    } else {
      const uint32_t i = 4u * g;
      store_elem<DT>(out, i, v0);
      if (i + 1u < HW) store_elem<DT>(out, i + 1u, v1);
      if (i + 2u < HW) store_elem<DT>(out, i + 2u, v2);
      if (i + 3u < HW) store_elem<DT>(out, i + 3u, v3);
    }
  }
}

constexpr uint32_t kDeferBlocks = 128;  // planes of at least this many 8x8 blocks: outlier-rich ones go to the whole CTA

// DEFER: instantiated for whole-warp teams on planes of at least kDeferBlocks blocks.
template <int DT, int TT, bool DEFER>
__global__ void __launch_bounds__(kThreads, 4) decompress_kernel(const Plan pl, const DecompressArgs a) {
  extern __shared__ __align__(128) uint8_t smem[];
  __shared__ double s_red[kMaxWarps * 5];
  __shared__ uint32_t s_hdr_ok, s_bits;
  __shared__ float s_eps;
  __shared__ unsigned long long s_total;
  __shared__ Plan s_pl;  // copy for the outlined slow path, which takes it by address
  // Outlier-rich planes of many blocks are not restored by the warp that meets them (one lane per block:
  // nblk / 32 rounds of a long serial walk while the CTA's other warps wait at the exit) but put on this list
  // and restored afterwards by the whole CTA, one lane per block.
  constexpr uint32_t kDeferCap = 64;
  __shared__ uint32_t s_defer[kDeferCap];
  __shared__ uint32_t s_ndefer;
  const uint32_t tid = threadIdx.x;
  if (tid == 0) {
    s_pl = pl;
    s_ndefer = 0;
  }
  dep_trigger();  // the next kernel on the stream may become resident as this one drains
  dep_wait();     // the previous kernel on the stream (the one that wrote the container) has completed
  const unsigned long long off_in = a.d_off_in ? *a.d_off_in : 0ull;
  const uint8_t* src = a.src_base + off_in;
  const unsigned long long src_bytes = a.src_bytes > off_in ? a.src_bytes - off_in : 0ull;
  const Team team = make_team(TT, s_red);
  constexpr uint32_t kTeams = kThreads / TT;
  const uint32_t my_team = tid / TT, lane = team.lane;

  // header check (every CTA, it is 64 bytes)
  if (tid == 0) {
    uint32_t bits = 0;
    float eps = 0.0f;
    unsigned long long total = 0;
    s_hdr_ok = check_header(pl, src, src_bytes, bits, eps, total);
    s_bits = bits;
    s_eps = eps;
    s_total = total;
  }
  __syncthreads();
  const bool hdr_ok = s_hdr_ok != 0;
  bool bad = !hdr_ok;
  if (hdr_ok) {
    const uint32_t bits = s_bits;
    const float eps = s_eps;
    const unsigned long long total = s_total;
    const uint32_t npay = a16(4u * ((pl.HW * bits + 31u) / 32u));
    const unsigned long long slots_off = 64ull + 16ull * pl.P, ovf_off = slots_off + pl.P * (unsigned long long)npay;
    const bool vec = (pl.plane_bytes & (DT == kF32 ? 15u : 7u)) == 0u;  // dst base is 16-byte aligned
    const uint32_t nfull = vec ? pl.HW >> 2 : 0u;                       // groups restored with vector stores
    // Work items are (plane, chunk of 8 * TT groups) pairs so that large planes spread over many
    // teams; a salient or raw plane is restored as a whole by the team that draws its first chunk.
    const uint32_t chunk_groups = 8u * TT;
    const uint32_t chunks = (pl.groups + chunk_groups - 1u) / chunk_groups;
    // Team t takes items t, t + stride, ...  The stride is a prime (teams beyond it stay idle), so that a
    // periodic pattern of expensive planes -- every eighth channel outlier-rich, say -- spreads over all
    // teams instead of landing on the few whose index shares a factor with the period.
    const uint64_t items = pl.P * chunks, stride = a.team_stride;
    const uint64_t first = (uint64_t)blockIdx.x * kTeams + my_team;
    for (uint64_t item = first < stride ? first : items; item < items; item += stride) {
      const uint64_t gp = item / chunks;
      const uint32_t ch = (uint32_t)(item - gp * chunks);
      const uint32_t g0 = ch * chunk_groups, g1 = min(nfull, g0 + chunk_groups);
      // whole-warp teams: the chunk's code words are requested before the table entry is known (the slot
      // sits at a closed-form offset; what a salient plane keeps there is read and dropped)
      uint32_t cw[8];
      if (TT == 32) {
        const uint32_t* s32 = reinterpret_cast<const uint32_t*>(src + slots_off + gp * npay);
        const uint32_t nwords = npay >> 2, w0 = (g0 * bits) >> 3, per = bits;  // words per lane: 2, 4 or 8
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const uint32_t i = w0 + (uint32_t)j * 32u + lane;
          cw[j] = ((uint32_t)j < per && i < nwords) ? __ldg(s32 + i) : 0u;
        }
      } else {  // sub-warp teams: one code word (1, 2 or 4 bytes) per group, the plane is one chunk
        const uint8_t* sl = src + slots_off + gp * npay;
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          const uint32_t g = lane + (uint32_t)k * TT;
          uint32_t w = 0;
          if (g < pl.groups)
            w = bits == 2u ? (uint32_t)__ldg(sl + g)
                           : (bits == 4u ? (uint32_t)__ldg(reinterpret_cast<const uint16_t*>(sl) + g)
                                         : __ldg(reinterpret_cast<const uint32_t*>(sl) + g));
          cw[k] = w;
        }
      }
      const uint4 e = __ldg(reinterpret_cast<const uint4*>(src + 64) + gp);
      const unsigned long long off = (unsigned long long)e.x * 16ull;
      const uint32_t cls = e.y & 3u;
      uint8_t* out = a.dst + gp * pl.plane_bytes;
      const uint8_t* slot = src + slots_off + gp * npay;
      if (cls == kClsNormal) {
        if (off != slots_off + gp * npay) { bad = true; continue; }
        const float lo = __uint_as_float(e.z), scale = __uint_as_float(e.w);
        if (TT == 32 && DT == kBF16 && (pl.plane_bytes & 15u) == 0u) {
          if (bits == 2u) decode_chunk32_bf16_pairs<2>(cw, lane, g0, g1, scale, lo, out);
          else if (bits == 4u) decode_chunk32_bf16_pairs<4>(cw, lane, g0, g1, scale, lo, out);
          else decode_chunk32_bf16_pairs<8>(cw, lane, g0, g1, scale, lo, out);
        } else if (TT == 32) {
          if (bits == 2u) decode_chunk32<DT, 2>(cw, lane, g0, g1, scale, lo, out);
          else if (bits == 4u) decode_chunk32<DT, 4>(cw, lane, g0, g1, scale, lo, out);
          else decode_chunk32<DT, 8>(cw, lane, g0, g1, scale, lo, out);
        } else if (bits == 2u) decode_small<DT, 2, TT>(cw, lane, pl.groups, nfull, pl.HW, scale, lo, out);
        else if (bits == 4u) decode_small<DT, 4, TT>(cw, lane, pl.groups, nfull, pl.HW, scale, lo, out);
        else decode_small<DT, 8, TT>(cw, lane, pl.groups, nfull, pl.HW, scale, lo, out);
        if (TT == 32 && ch == chunks - 1u && nfull * 4u < pl.HW) {  // ragged or unaligned rest: element stores
          const uint32_t L = (1u << bits) - 1u;
          for (uint32_t i = nfull * 4u + lane; i < pl.HW; i += TT) {
            const uint32_t bit = i * bits;
            const uint32_t q = (__ldg(reinterpret_cast<const uint32_t*>(slot) + (bit >> 5)) >> (bit & 31u)) & L;
            store_elem<DT>(out, i, dequant(q, scale, lo));
          }
        }
      } else if (cls == kClsRaw || cls == kClsSalient) {
        if (ch != 0) continue;
        // the continuation, when there is one, lies in the overflow region
        if (off != 0 && (off < ovf_off || off > total)) { bad = true; continue; }
        SplitIn in;
        in.slot = slot;
        in.ovf = src + off;
        in.npay = npay;
        const unsigned long long ovf_avail = off ? total - off : 0ull;
        if (cls == kClsRaw) {
          if (pl.plane_bytes > npay && pl.plane_bytes - npay > ovf_avail) { bad = true; continue; }
          for (uint32_t i = lane; i < (uint32_t)(pl.plane_bytes >> 1); i += TT)
            reinterpret_cast<uint16_t*>(out)[i] = (uint16_t)in.ld16(2u * i);
        } else {
          if (DEFER) {
            uint32_t at = 0;
            if (lane == 0) at = atomicAdd(&s_ndefer, 1u);
            at = __shfl_sync(0xFFFFFFFFu, at, 0);
            if (at < kDeferCap) {
              if (lane == 0) s_defer[at] = (uint32_t)gp;
              continue;
            }
          }
          uint32_t* scr = reinterpret_cast<uint32_t*>(smem + (uint64_t)my_team * pl.sal_stride);
          if (!decode_salient<DT>(team, s_pl, in, ovf_avail, eps, out, scr, s_hdr_ok)) bad = true;
        }
      } else {
        bad = true;
      }
    }
  }
  if (DEFER && hdr_ok) {  // (uniform over the CTA)
    __syncthreads();
    const uint32_t n = min(s_ndefer, kDeferCap);
    const Team cta = make_team(kThreads, s_red);
    const uint32_t bits = s_bits;
    const uint32_t npay = a16(4u * ((pl.HW * bits + 31u) / 32u));
    const unsigned long long total = s_total;
    const unsigned long long slots_off = 64ull + 16ull * pl.P, ovf_off = slots_off + pl.P * (unsigned long long)npay;
    for (uint32_t q = 0; q < n; ++q) {
      const uint64_t gp = s_defer[q];
      const uint4 e = __ldg(reinterpret_cast<const uint4*>(src + 64) + gp);
      const unsigned long long off = (unsigned long long)e.x * 16ull;
      if (off != 0 && (off < ovf_off || off > total)) {  // (the same for every thread)
        bad = true;
        continue;
      }
      SplitIn in;
      in.slot = src + slots_off + gp * npay;
      in.ovf = src + off;
      in.npay = npay;
      if (!decode_salient<DT>(cta, s_pl, in, off ? total - off : 0ull, s_eps, a.dst + gp * pl.plane_bytes,
                              reinterpret_cast<uint32_t*>(smem), s_hdr_ok))
        bad = true;
      __syncthreads();  // the scratch is reused
    }
  }
  decompress_exit(a, bad);
}

// -------------------------------------------------------------------------------------------------
// Small planes (at most 128 groups: 7x7, 14x14, 16x16, ...).  Such planes rarely start on 16-byte boundaries,
// and a team of a few lanes that stores its plane element by element scatters 4-byte stores over many
// sectors.  Here a CTA restores a tile of consecutive planes into shared memory -- a team of lanes per
// normal plane, the whole warp for an outlier-rich one -- and the tile leaves as one bulk (TMA) store.
// Tiles (256 / team planes) start on 16-byte boundaries; two buffers alternate.
// -------------------------------------------------------------------------------------------------

// Outlier-rich plane of at most four blocks and fewer than 32 rows, restored by one warp: CSR scatter, then per
// dense block the inverse of the Lorenzo prediction as a two-dimensional prefix sum of the residuals over the
// warp's lanes (lane l holds raster positions l and l + 32), corrected in raster order for every verbatim
// element, whose k follows from its stored value.  The result is that of the raster walk in decode_salient.
// A payload copied to shared memory as one piece.
struct FlatIn {
  const uint8_t* p;
  uint32_t npay;  // (kept for the size check: bytes of the payload that came from the slot)
  __device__ __forceinline__ uint32_t ld32(uint32_t o) const { return *reinterpret_cast<const uint32_t*>(p + o); }
  __device__ __forceinline__ uint32_t ld16(uint32_t o) const { return *reinterpret_cast<const uint16_t*>(p + o); }
};

template <int DT, typename In>
__device__ __forceinline__ bool small_decode(const Plan& pl, const In& in, uint64_t ovf_avail, float eps, uint8_t* out) {
  const uint32_t lane = threadIdx.x & 31u, full = 0xFFFFFFFFu;
  const uint32_t H = (uint32_t)pl.H, W = (uint32_t)pl.W, nblk = pl.nblk, nbx = pl.nbx, e = (uint32_t)pl.esize, HW = pl.HW;
  const uint32_t nnz_s = in.ld32(0), n_dense = in.ld32(4), n_out_d = in.ld32(8);
  if (nnz_s > HW || n_dense > nblk || n_out_d > HW) return false;
  const uint64_t size = 16ull + 4ull * pl.nbm + 4ull * ((uint64_t)H + 1) + a4(2u * nnz_s) + a4(e * nnz_s) +
                        64ull * n_dense + a4(e * n_out_d);
  if (size > in.npay && size - in.npay > ovf_avail) return false;
  const uint32_t o_bm = 16u, o_rp = o_bm + 4u * pl.nbm, o_col = o_rp + 4u * (H + 1u);
  const uint32_t o_val = o_col + a4(2u * nnz_s), o_codes = o_val + a4(e * nnz_s), o_outl = o_codes + 64u * n_dense;
  const uint32_t bitmap = in.ld32(o_bm) & ((1u << nblk) - 1u);
  if ((uint32_t)__popc(bitmap) != n_dense) return false;
  bool ok = true;
  for (uint32_t i = lane; i < (uint32_t)(pl.plane_bytes >> 1); i += 32u) reinterpret_cast<uint16_t*>(out)[i] = 0;
  __syncwarp();
  if (lane < H) {  // CSR scatter, a lane per row
    const uint32_t r0 = in.ld32(o_rp + 4u * lane), r1 = in.ld32(o_rp + 4u * lane + 4u);
    if (r0 > r1 || r1 > nnz_s) {
      ok = false;
    } else {
      for (uint32_t k = r0; k < r1; ++k) {
        const uint32_t col = in.ld16(o_col + 2u * k);
        if (col >= W) {
          ok = false;
          continue;
        }
        const uint32_t idx = lane * W + col;
        if (DT == kF32) reinterpret_cast<uint32_t*>(out)[idx] = in.ld32(o_val + 4u * k);
        else reinterpret_cast<uint16_t*>(out)[idx] = (uint16_t)in.ld16(o_val + 2u * k);
      }
    }
  }
  const float two_eps = __fmul_rn(2.0f, eps), inv2e = __fdiv_rn(1.0f, two_eps);
  const uint32_t c = lane & 7u, r0 = lane >> 3, lt = (1u << lane) - 1u;
  uint32_t oi = 0, rank = 0;
#pragma unroll 1
  for (uint32_t b = 0; b < nblk; ++b) {
    if (!((bitmap >> b) & 1u)) continue;
    const uint32_t oc = o_codes + 64u * rank;
    const uint32_t code0 = (in.ld32(oc + (lane & ~3u)) >> (8u * (lane & 3u))) & 0xFFu;
    const uint32_t code1 = (in.ld32(oc + 32u + (lane & ~3u)) >> (8u * (lane & 3u))) & 0xFFu;
    const uint32_t by = b / nbx, bx = b - by * nbx;
    const uint32_t y0 = by * 8u + r0, x = bx * 8u + c;
    const bool in0 = y0 < H && x < W, in1 = y0 + 4u < H && x < W;
    const bool v0 = in0 && code0 == 0u, v1 = in1 && code1 == 0u;
    int32_t k0 = (in0 && !v0) ? (int32_t)code0 - 128 : 0, k1 = (in1 && !v1) ? (int32_t)code1 - 128 : 0;
#pragma unroll
    for (uint32_t o = 1; o < 8u; o <<= 1) {  // along the rows
      const int32_t t0 = __shfl_up_sync(full, k0, o), t1 = __shfl_up_sync(full, k1, o);
      if (c >= o) {
        k0 += t0;
        k1 += t1;
      }
    }
#pragma unroll
    for (uint32_t o = 8; o < 32u; o <<= 1) {  // down the columns, within each half
      const int32_t t0 = __shfl_up_sync(full, k0, o), t1 = __shfl_up_sync(full, k1, o);
      if (lane >= o) {
        k0 += t0;
        k1 += t1;
      }
    }
    k1 += __shfl_sync(full, k0, 24 + (int)c);  // rows 4-7 continue below row 3
    const uint32_t m0 = __ballot_sync(full, v0), m1 = __ballot_sync(full, v1);
    const uint32_t nv = (uint32_t)(__popc(m0) + __popc(m1));
    if (oi + nv > n_out_d) return false;  // (the same for every lane)
    uint32_t raw0 = 0, raw1 = 0;
    int32_t kv0 = 0, kv1 = 0;
    if (v0) {
      const uint32_t at = oi + (uint32_t)__popc(m0 & lt);
      raw0 = DT == kF32 ? in.ld32(o_outl + 4u * at) : in.ld16(o_outl + 2u * at);
      bool big;
      kv0 = dense_k(DT == kF32 ? __uint_as_float(raw0) : bf16_bits_to_f32(raw0), inv2e, &big);
    }
    if (v1) {
      const uint32_t at = oi + (uint32_t)__popc(m0) + (uint32_t)__popc(m1 & lt);
      raw1 = DT == kF32 ? in.ld32(o_outl + 4u * at) : in.ld16(o_outl + 2u * at);
      bool big;
      kv1 = dense_k(DT == kF32 ? __uint_as_float(raw1) : bf16_bits_to_f32(raw1), inv2e, &big);
    }
    // a verbatim element replaces its k: the difference moves every k below and to the right of it
    for (uint32_t mm = m0; mm; mm &= mm - 1u) {
      const uint32_t src = (uint32_t)__ffs((int)mm) - 1u, i = src >> 3, j = src & 7u;
      const int32_t diff = __shfl_sync(full, kv0 - k0, (int)src);
      if (c >= j) {
        if (r0 >= i) k0 += diff;
        k1 += diff;
      }
    }
    for (uint32_t mm = m1; mm; mm &= mm - 1u) {
      const uint32_t src = (uint32_t)__ffs((int)mm) - 1u, i = src >> 3, j = src & 7u;
      const int32_t diff = __shfl_sync(full, kv1 - k1, (int)src);
      if (c >= j && r0 >= i) k1 += diff;
    }
    if (in0) {
      const uint32_t idx = y0 * W + x;
      if (v0) {
        if (DT == kF32) reinterpret_cast<uint32_t*>(out)[idx] = raw0;
        else reinterpret_cast<uint16_t*>(out)[idx] = (uint16_t)raw0;
      } else {
        store_elem<DT>(out, idx, __fmul_rn((float)k0, two_eps));
      }
    }
    if (in1) {
      const uint32_t idx = (y0 + 4u) * W + x;
      if (v1) {
        if (DT == kF32) reinterpret_cast<uint32_t*>(out)[idx] = raw1;
        else reinterpret_cast<uint16_t*>(out)[idx] = (uint16_t)raw1;
      } else {
        store_elem<DT>(out, idx, __fmul_rn((float)k1, two_eps));
      }
    }
    oi += nv;
    ++rank;
  }
  return __all_sync(full, ok);
}

template <int DT>
__global__ void __launch_bounds__(kThreads, 4) decompress_small(const Plan pl, const DecompressArgs a) {
  extern __shared__ __align__(128) uint8_t smem[];
  __shared__ double s_red[kMaxWarps * 5];
  __shared__ uint32_t s_hdr_ok, s_bits;
  __shared__ float s_eps;
  __shared__ unsigned long long s_total;
  __shared__ Plan s_pl;  // copy for the outlined slow path, which takes it by address
  const uint32_t tid = threadIdx.x, wlane = tid & 31u;
  if (tid == 0) s_pl = pl;
  dep_trigger();  // the next kernel on the stream may become resident as this one drains
  dep_wait();     // the previous kernel on the stream (the one that wrote the container) has completed
  const unsigned long long off_in = a.d_off_in ? *a.d_off_in : 0ull;
  const uint8_t* src = a.src_base + off_in;
  const unsigned long long src_bytes = a.src_bytes > off_in ? a.src_bytes - off_in : 0ull;
  if (tid == 0) {
    uint32_t bits = 0;
    float eps = 0.0f;
    unsigned long long total = 0;
    s_hdr_ok = check_header(pl, src, src_bytes, bits, eps, total);
    s_bits = bits;
    s_eps = eps;
    s_total = total;
  }
  __syncthreads();
  bool bad = s_hdr_ok == 0;
  if (!bad) {
    const uint32_t bits = s_bits, L = (1u << bits) - 1u;
    const float eps = s_eps;
    const unsigned long long total = s_total;
    const uint32_t npay = a16(4u * ((pl.HW * bits + 31u) / 32u));
    const unsigned long long slots_off = 64ull + 16ull * pl.P, ovf_off = slots_off + pl.P * (unsigned long long)npay;
    const uint32_t tt = pl.team, lane = tid & (tt - 1u), my_team = tid / tt;
    const Team warp_team = make_warp_team(s_red);
    const bool vec = (pl.plane_bytes & (DT == kF32 ? 15u : 7u)) == 0u;  // planes start on vector boundaries in the tile buffer
    const uint32_t tile_bytes_max = pl.stage_bytes;
    const uint32_t pay_stride = pl.sal_stride;  // per-warp scratch: a small plane's payload, or the general path's tables
    uint32_t buf = 0;
    for (uint32_t tile = blockIdx.x; tile < pl.ntiles; tile += gridDim.x, buf ^= 1u) {
      uint8_t* tbuf = smem + (uint64_t)buf * tile_bytes_max;
      if (tid == 0) bulk_wait_read<1>();  // the store that left this buffer two tiles ago has read it
      __syncthreads();
      const uint64_t p0 = (uint64_t)tile * pl.ppt;
      const uint32_t np = (uint32_t)min((uint64_t)pl.ppt, pl.P - p0);
      const uint32_t lp = my_team;
      bool salient = false;
      if (lp < np) {
        const uint64_t gp = p0 + lp;
        const uint4 en = __ldg(reinterpret_cast<const uint4*>(src + 64) + gp);
        const unsigned long long off = (unsigned long long)en.x * 16ull;
        const uint32_t cls = en.y & 3u;
        uint8_t* out = tbuf + (uint64_t)lp * pl.plane_bytes;
        const uint8_t* slot = src + slots_off + gp * npay;
        if (cls == kClsNormal) {
          if (off != slots_off + gp * npay) {
            bad = true;
          } else {
            const float lo = __uint_as_float(en.z), scale = __uint_as_float(en.w);
            for (uint32_t g = lane; g < pl.groups; g += tt) {
              const uint32_t word = bits == 2u ? (uint32_t)__ldg(slot + g)
                                               : (bits == 4u ? (uint32_t)__ldg(reinterpret_cast<const uint16_t*>(slot) + g)
                                                             : __ldg(reinterpret_cast<const uint32_t*>(slot) + g));
              const uint32_t i = 4u * g;
              if (vec && i + 3u < pl.HW) {  // whole group of a plane on a vector boundary: one store
                store_group<DT>(out, g, dequant(word & L, scale, lo), dequant((word >> bits) & L, scale, lo),
                                dequant((word >> (2u * bits)) & L, scale, lo), dequant((word >> (3u * bits)) & L, scale, lo));
              } else {
#pragma unroll
                for (uint32_t k = 0; k < 4u; ++k)
                  if (i + k < pl.HW) store_elem<DT>(out, i + k, dequant((word >> (k * bits)) & L, scale, lo));
              }
            }
          }
        } else if (cls == kClsRaw) {
          if (off != 0 && (off < ovf_off || off > total)) {
            bad = true;
          } else {
            SplitIn in;
            in.slot = slot;
            in.ovf = src + off;
            in.npay = npay;
            const unsigned long long ovf_avail = off ? total - off : 0ull;
            if (pl.plane_bytes > npay && pl.plane_bytes - npay > ovf_avail) bad = true;
            else
              for (uint32_t i = lane; i < (uint32_t)(pl.plane_bytes >> 1); i += tt)
                reinterpret_cast<uint16_t*>(out)[i] = (uint16_t)in.ld16(2u * i);
          }
        } else if (cls == kClsSalient) {
          salient = true;
        } else {
          bad = true;
        }
      }
      // outlier-rich planes of the warp's slice: the whole warp restores them one after the other
      for (uint32_t m = __ballot_sync(0xFFFFFFFFu, salient && lane == 0); m; m &= m - 1u) {
        const uint32_t slp = (tid & ~31u) / tt + ((uint32_t)__ffs((int)m) - 1u) / tt;
        const uint64_t gp = p0 + slp;
        const unsigned long long off = (unsigned long long)__ldg(reinterpret_cast<const uint32_t*>(src + 64 + 16ull * gp)) * 16ull;
        if (off != 0 && (off < ovf_off || off > total)) {
          bad = true;
          continue;
        }
        SplitIn in;
        in.slot = src + slots_off + gp * npay;
        in.ovf = src + off;
        in.npay = npay;
        uint8_t* out = tbuf + (uint64_t)slp * pl.plane_bytes;
        const unsigned long long ovf_avail = off ? total - off : 0ull;
        __syncwarp();
        bool good;
        if (pl.nblk <= 4u && pl.H < 32 && in.ld32(12) == 0u) {  // (a Huffman-coded plane takes the general path)
          // the payload (shorter than the plane, or it would have been stored raw) is fetched in one go into the
          // warp's scratch and decoded from there
          uint8_t* pay = smem + 2ull * tile_bytes_max + (uint64_t)(tid >> 5) * pay_stride;
          const uint32_t nnz_s = in.ld32(0), n_dense = in.ld32(4), n_out_d = in.ld32(8), es = (uint32_t)pl.esize;
          const uint64_t size = 16ull + 4ull * pl.nbm + 4ull * ((uint64_t)pl.H + 1) + a4(2u * nnz_s) + a4(es * nnz_s) +
                                64ull * n_dense + a4(es * n_out_d);
          good = nnz_s <= pl.HW && n_dense <= pl.nblk && n_out_d <= pl.HW && size <= pay_stride &&
                 !(size > npay && size - npay > ovf_avail);
          if (good) {
            for (uint32_t o = 4u * wlane; o < (uint32_t)size; o += 128u) *reinterpret_cast<uint32_t*>(pay + o) = in.ld32(o);
            __syncwarp();
            FlatIn flat;
            flat.p = pay;
            flat.npay = npay;
            good = small_decode<DT>(s_pl, flat, ovf_avail, eps, out);
          }
        } else {
          good = decode_salient<DT>(warp_team, s_pl, in, ovf_avail, eps, out,
                                    reinterpret_cast<uint32_t*>(smem + 2ull * tile_bytes_max + (uint64_t)(tid >> 5) * pl.sal_stride),
                                    s_hdr_ok);
        }
        if (!good) bad = true;
        __syncwarp();
      }
      __syncthreads();
      // the tile leaves: one bulk store when it is whole 16-byte chunks, plain stores otherwise
      const uint32_t bytes = np * (uint32_t)pl.plane_bytes;
      uint8_t* dst = a.dst + p0 * pl.plane_bytes;
      if ((bytes & 15u) == 0u) {
        if (tid == 0) {
          fence_proxy_async();
          bulk_s2g(dst, tbuf, bytes);
          bulk_commit();
        }
      } else {
        for (uint32_t i = tid; i < (bytes >> 1); i += kThreads)
          reinterpret_cast<uint16_t*>(dst)[i] = reinterpret_cast<const uint16_t*>(tbuf)[i];
      }
    }
    if (tid == 0) bulk_wait<0>();  // every store of this CTA is complete
  }
  decompress_exit(a, bad);
}

}  // namespace fh
