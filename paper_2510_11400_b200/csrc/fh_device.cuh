// Device-side building blocks shared by the compress and decompress kernels (sm_100a).
//
// Terminology: a "plane" is one (n, c) feature map of H x W elements; a "group" is four consecutive
// elements of a plane; a "tile" is a run of consecutive planes that one CTA stages in shared memory;
// a "team" is the set of threads that works on one plane: a power-of-two slice of a warp for small
// planes, the whole CTA for large ones.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace fh {

constexpr int kThreads = 256;             // CTA size of every kernel
constexpr int kWarps = kThreads / 32;
constexpr int kMaxWarps = 16;            // largest CTA of any kernel: 512 threads
constexpr uint32_t kMagic = 0x31434846u;  // "FHC1"
constexpr uint32_t kClsNormal = 0, kClsSalient = 1, kClsRaw = 2;
constexpr int kModeAuto = 0, kModeOff = 1, kModeAll = 2, kModeChannel = 3, kModeTensor = 4;
constexpr int kF32 = 0, kBF16 = 1;
constexpr int kMaxStages = 4;
constexpr float kMagicF = 12582912.0f;    // 1.5 * 2^23: fma(v, c, kMagicF) leaves rne(v*c) in the mantissa
constexpr uint32_t kMagicBits = 0x4B400000u;

// Device-side error codes (positive, ordered by priority; status_word() maps them to fh_status).
constexpr uint32_t kErrNone = 0, kErrNonfinite = 1, kErrCapacity = 2, kErrCorrupt = 3, kErrTimeout = 4;

// Everything a kernel needs to know about the tensor, the parameters and the tiling.
struct Plan {
  int32_t dtype, esize, H, W;
  uint32_t N, C;
  uint32_t HW;
  uint32_t groups;       // ceil(HW / 4)
  uint64_t P;            // planes
  uint64_t plane_bytes;  // HW * esize
  uint64_t dense_bytes;  // P * plane_bytes
  double inv_hw;         // 1 / HW in fp64
  int32_t bits, mode;
  int32_t rounding;      // 0: round half to even; 1: random rounding (Philox draws)
  int32_t entropy;       // 1: Huffman stage on the dense-block codes of outlier-rich planes (container version 2)
  uint64_t seed;
  uint32_t rho_num, rho_den, tau_num, tau_den;
  float eps;
  uint64_t tensor_id;
  uint32_t npay;         // slot size: A16(bytes of a normal payload)
  uint64_t slots_off;    // 64 + 16 P
  uint64_t ovf_off;      // slots_off + P * npay: start of the overflow region
  uint32_t nbx, nby, nblk, nbm;  // 8x8 blocks per row / column / plane, bitmap words
  // tiling
  uint32_t ppt;          // planes per tile
  uint32_t ntiles;
  uint32_t team;         // threads per plane: 1..32 (power of two) or kThreads
  uint32_t nstage;       // fast kernels: tiles in flight per CTA
  uint32_t stage_bytes;  // fast kernels: bytes of one stage buffer (ppt * plane_bytes)
  // shared-memory layout (byte offsets into dynamic shared memory)
  uint32_t sm_tile, sm_out, sm_rec, sm_total;
  // block-wise path (outlier-rich planes): measuring scratch of one unit (a warp, or the whole CTA)
  uint32_t sal_words;       // words of measuring scratch per plane: H + 1 + 3 * nblk
  uint32_t sm_sal;          // byte offset of the first measuring area in dynamic shared memory
  uint32_t sal_stride;      // bytes between the areas of consecutive units
};

// Book-keeping scratch, one per stream: a header of counters and three arrays for the plane-ordered
// placement of overflow parts (see "Placement scan" below).  Everything in the header that a call changes
// is returned to zero by the last CTA of its kernel.
struct Scratch {
  unsigned long long ticket[2];  // next tile; consecutive compress calls on a stream alternate between the two
  unsigned long long exited;     // CTAs that have left the running kernel
  unsigned long long status;     // device error code (atomicMax)
  unsigned long long ovf16;      // overflow region size of this call, in 16-byte units
  unsigned long long nsal, nraw;
  unsigned long long reserved;
};
static_assert(sizeof(Scratch) == 64, "Scratch layout");
constexpr uint32_t kScratchHeadBytes = 256;  // the header, padded

// (uint64)(int64) fh_status of a device error code.
__device__ __forceinline__ unsigned long long status_word(uint32_t code) {
  const long long st = code == kErrNonfinite ? -4 : code == kErrCapacity ? -3 : code == kErrCorrupt ? -5
                       : code == kErrTimeout ? -6 : 0;
  return (unsigned long long)st;
}

__device__ __forceinline__ uint32_t a4(uint32_t x) { return (x + 3u) & ~3u; }
__device__ __forceinline__ uint32_t a16(uint32_t x) { return (x + 15u) & ~15u; }
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ unsigned long long ld_acquire(const unsigned long long* p) {
  unsigned long long v;
  asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_release(unsigned long long* p, unsigned long long v) {
  asm volatile("st.release.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}
__device__ __forceinline__ unsigned long long ld_relaxed(const unsigned long long* p) {
  unsigned long long v;
  asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_relaxed(unsigned long long* p, unsigned long long v) {
  asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}

// ---- programmatic dependent launch: a kernel launched with the programmatic-serialisation attribute may
// become resident while its predecessor on the stream is still running; it must pass dep_wait() before it
// touches anything the predecessor reads or writes.  dep_trigger() in the predecessor allows that early start.
__device__ __forceinline__ void dep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void dep_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// ---- shared-memory barriers and bulk (TMA) copies -------------------------------------------------
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void fence_mbar_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
// Bulk copy global -> shared; src, dst and bytes are multiples of 16.  Completion is signalled on `bar`.
__device__ __forceinline__ void bulk_g2s(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                   smem_u32(dst)),
               "l"(src), "r"(bytes), "r"(smem_u32(bar))
               : "memory");
}
// Bulk copy shared -> global (same alignment rules), tracked by bulk async-groups.
__device__ __forceinline__ void bulk_s2g(void* dst, const void* src, uint32_t bytes) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst), "r"(smem_u32(src)), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void bulk_wait_read() { asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory"); }
// ... until all but the N most recent groups are complete (their writes performed).
template <int N>
__device__ __forceinline__ void bulk_wait() { asm volatile("cp.async.bulk.wait_group %0;" ::"n"(N) : "memory"); }
// One wait attempt: the hardware may suspend the thread for up to about `kSuspendNs` nanoseconds
// while the phase is incomplete, so that waiting warps do not burn issue slots polling.
constexpr uint32_t kSuspendNs = 2000;
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3; selp.u32 %0, 1, 0, p; }"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity), "r"(kSuspendNs)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// Bounded wait that also gives up when *abort becomes non-zero (looked at every eighth attempt: an attempt
// ends early whenever anything arrives at the barrier, so a waiting warp makes many of them).
__device__ __forceinline__ bool mbar_wait_abortable(uint64_t* bar, uint32_t parity, uint32_t limit,
                                                    const volatile uint32_t* abort) {
  for (uint32_t i = 0; i < limit; ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((i & 7u) == 7u && *abort) return false;
  }
  return false;
}
// Bounded wait: false when the phase did not complete within `limit` polls.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, uint32_t limit) {
  for (uint32_t i = 0; i < limit; ++i)
    if (mbar_try_wait(bar, parity)) return true;
  return false;
}

// ---- arithmetic helpers --------------------------------------------------------------------------
// min / max that return NaN when any operand is NaN, so that a NaN anywhere in a plane surfaces in
// its minimum and maximum.
__device__ __forceinline__ float min_nan(float a, float b) {
  float r;
  asm("min.NaN.f32 %0, %1, %2;" : "=f"(r) : "f"(a), "f"(b));
  return r;
}
__device__ __forceinline__ float max_nan(float a, float b) {
  float r;
  asm("max.NaN.f32 %0, %1, %2;" : "=f"(r) : "f"(a), "f"(b));
  return r;
}
__device__ __forceinline__ float min3_nan(float a, float b, float c) {
  float r;
  asm("min.NaN.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
  return r;
}
__device__ __forceinline__ float max3_nan(float a, float b, float c) {
  float r;
  asm("max.NaN.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
  return r;
}

__device__ __forceinline__ float bf16_bits_to_f32(uint32_t h) { return __uint_as_float(h << 16); }
// fp32 -> bf16 bits, round half to even (finite inputs).
// fp32 -> bf16, round to nearest even (the hardware conversion; the values converted here are never NaN).
__device__ __forceinline__ uint32_t f32_to_bf16_bits(float f) {
  uint16_t r;
  asm("cvt.rn.bf16.f32 %0, %1;" : "=h"(r) : "f"(f));
  return r;
}
// Two at once: `lo` lands in the low half of the word.
__device__ __forceinline__ uint32_t f32x2_to_bf16x2(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}

template <int DT>
__device__ __forceinline__ float load_elem(const uint8_t* plane, uint32_t i) {
  if (DT == kF32) return reinterpret_cast<const float*>(plane)[i];
  return bf16_bits_to_f32(reinterpret_cast<const uint16_t*>(plane)[i]);
}

// Group g of a plane, elements past HW read as 0.  `vec` says that the plane starts on a 16-byte
// (fp32) / 8-byte (bf16) boundary so that a full group is one load.
template <int DT>
__device__ __forceinline__ void load_group(const uint8_t* plane, uint32_t g, uint32_t HW, bool vec, float v[4]) {
  const uint32_t i0 = g * 4u;
  if (vec && i0 + 3u < HW) {
    if (DT == kF32) {
      const float4 t = reinterpret_cast<const float4*>(plane)[g];
      v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
    } else {
      const uint2 t = reinterpret_cast<const uint2*>(plane)[g];
      v[0] = __uint_as_float(t.x << 16); v[1] = __uint_as_float(t.x & 0xFFFF0000u);
      v[2] = __uint_as_float(t.y << 16); v[3] = __uint_as_float(t.y & 0xFFFF0000u);
    }
  } else {
#pragma unroll
    for (int k = 0; k < 4; ++k) v[k] = (i0 + k < HW) ? load_elem<DT>(plane, i0 + k) : 0.0f;
  }
}

// ---- packed fp32 pairs (sm_100: one instruction, two independent IEEE round-to-nearest results) ----
typedef unsigned long long f32x2;
__device__ __forceinline__ f32x2 pack2(float a, float b) {
  f32x2 r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(a), "f"(b));
  return r;
}
__device__ __forceinline__ void unpack2(f32x2 v, float& a, float& b) { asm("mov.b64 {%0, %1}, %2;" : "=f"(a), "=f"(b) : "l"(v)); }
__device__ __forceinline__ void unpack2u(f32x2 v, uint32_t& a, uint32_t& b) { asm("mov.b64 {%0, %1}, %2;" : "=r"(a), "=r"(b) : "l"(v)); }
__device__ __forceinline__ f32x2 add2(f32x2 a, f32x2 b) {
  f32x2 r;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}
__device__ __forceinline__ f32x2 mul2(f32x2 a, f32x2 b) {
  f32x2 r;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}
__device__ __forceinline__ f32x2 fma2(f32x2 a, f32x2 b, f32x2 c) {
  f32x2 r;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
  return r;
}

// Three-sigma rule: integer moment sums of the distances d = x - lo from the smallest element, scaled by
// the exponent e of the range (2^e <= range < 2^(e+1)): a group of four contributes rne(s * 2^(18-e)) and
// rne(q * 2^(16-2e)), both below 2^22.  The rule is applied for -40 <= e <= 60 only (no product can over-
// or underflow there); a constant plane (range 0, exponent field 0) falls outside like any other.
struct SigmaScale {
  float cs, cq;   // 2^(18-e), 2^(16-2e)
  int32_t e;
  bool applies;
};
__device__ __forceinline__ SigmaScale sigma_scale(float range) {
  SigmaScale s;
  s.e = (int)((__float_as_uint(range) >> 23) & 255u) - 127;
  s.applies = s.e >= -40 && s.e <= 60;
  const int32_t e = s.applies ? s.e : 0;
  s.cs = __uint_as_float((uint32_t)(18 - e + 127) << 23);
  s.cq = __uint_as_float((uint32_t)(16 - 2 * e + 127) << 23);
  return s;
}
// Raw mantissa images of the two addends of one group of distances (d0, d1, d2, d3); the caller sums them
// with wrap-around arithmetic and subtracts kMagicBits once per group at the end.  The group's two pairs
// (d0, d1) and (d2, d3) are combined position by position, s = (d0 + d2) + (d1 + d3) and
// q = fma(d2, d2, d0 * d0) + fma(d3, d3, d1 * d1): with packed two-wide instructions that is one add, one
// multiply and one multiply-add on the pairs as they come out of a 16-byte load, then one add of the halves each.
__device__ __forceinline__ void sigma_addends2(f32x2 p, f32x2 q, const SigmaScale& sc, uint32_t& as, uint32_t& aq) {
  float sa, sb, qa, qb;
  unpack2(add2(p, q), sa, sb);                 // d0 + d2, d1 + d3
  unpack2(fma2(q, q, mul2(p, p)), qa, qb);     // fma(d2, d2, d0 * d0), fma(d3, d3, d1 * d1)
  const f32x2 fixed = fma2(pack2(__fadd_rn(sa, sb), __fadd_rn(qa, qb)), pack2(sc.cs, sc.cq), pack2(kMagicF, kMagicF));
  uint32_t is, iq;
  unpack2u(fixed, is, iq);
  as += is;
  aq += iq;
}
__device__ __forceinline__ void sigma_addends4(float d0, float d1, float d2, float d3, const SigmaScale& sc,
                                               uint32_t& as, uint32_t& aq) {
  sigma_addends2(pack2(d0, d1), pack2(d2, d3), sc, as, aq);
}
__device__ __forceinline__ void sigma_addends(const float d[4], const SigmaScale& sc, uint32_t& as, uint32_t& aq) {
  sigma_addends2(pack2(d[0], d[1]), pack2(d[2], d[3]), sc, as, aq);
}
// Thresholds, as distances from lo, from the exact integer sums: m1 +- 3 sigma.
template <typename I>
__device__ __forceinline__ void sigma_thresholds(I Is, I Iq, const SigmaScale& sc, double inv_count, float& dlo,
                                                 float& dhi) {
  const double ps = __hiloint2double((1023 + sc.e - 18) << 20, 0);      // 2^(e-18)
  const double pq = __hiloint2double((1023 + 2 * sc.e - 16) << 20, 0);  // 2^(2e-16)
  const double m1 = __dmul_rn(__dmul_rn((double)Is, ps), inv_count);
  const double m2 = __dmul_rn(__dmul_rn((double)Iq, pq), inv_count);
  double var = __dsub_rn(m2, __dmul_rn(m1, m1));
  if (!(var > 0.0)) var = 0.0;
  const float m_f = __double2float_rn(m1);
  const float sigma_f = __fsqrt_rn(__double2float_rn(var));
  dhi = __fmaf_rn(3.0f, sigma_f, m_f);
  dlo = __fmaf_rn(-3.0f, sigma_f, m_f);
}

// Quantiser parameters of a normal plane.
__device__ __forceinline__ void quant_params(float range, uint32_t L, float& inv, float& scale) {
  inv = __fdiv_rn((float)L, range);
  scale = __fdiv_rn(range, (float)L);
  if (range == 0.0f || !(fabsf(inv) <= 3.402823466e38f)) {
    inv = 0.0f;
    scale = 0.0f;
  }
}
// Code of one element from its distance d = x - lo: rne of the exact product d * inv, as an integer in the
// mantissa.
__device__ __forceinline__ uint32_t quant_code(float d, float inv, uint32_t L) {
  const float r = __fmaf_rn(d, inv, kMagicF);
  return (__float_as_uint(r) - kMagicBits) & L;
}

// ---- random rounding (rounding = 1) ------------------------------------------------------------------
// Philox-4x32 with 10 rounds (Salmon et al., SC'11): counter-based, so a draw is a pure function of the
// key (seed) and the counter (group within the plane, plane, tensor id).
__device__ __forceinline__ void philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, uint32_t k0, uint32_t k1,
                                              uint32_t (&out)[4]) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const uint32_t h0 = __umulhi(0xD2511F53u, c0), l0 = 0xD2511F53u * c0;
    const uint32_t h1 = __umulhi(0xCD9E8D57u, c2), l1 = 0xCD9E8D57u * c2;
    c0 = h1 ^ c1 ^ k0;
    c1 = l1;
    c2 = h0 ^ c3 ^ k1;
    c3 = l0;
    k0 += 0x9E3779B9u;
    k1 += 0xBB67AE85u;
  }
  out[0] = c0;
  out[1] = c1;
  out[2] = c2;
  out[3] = c3;
}
// Code of one element (distance d = x - lo) under random rounding: t = fp32 product d * inv, n = floor(t), and the code
// goes up iff floor(frac(t) * 2^24) + (word >> 8) reaches 2^24.
__device__ __forceinline__ uint32_t quant_code_random(float d, float inv, uint32_t L, uint32_t word) {
  const float t = __fmul_rn(d, inv);
  const float nf = floorf(t);
  const uint32_t fi = (uint32_t)__fmul_rn(__fsub_rn(t, nf), 16777216.0f);
  const uint32_t up = (fi + (word >> 8)) >> 24;
  const uint32_t n = nf >= (float)L ? L : (uint32_t)nf;
  return min(n + up, L);
}

// Pre-quantisation of dense-block elements (Eq. 9 on integers): k = rne(fp32(x * inv2e)), |k| <= 2^24.
__device__ __forceinline__ int32_t dense_k(float x, float inv2e, bool* big) {
  float kf = rintf(__fmul_rn(x, inv2e));
  *big = fabsf(kf) >= 16777216.0f;
  kf = fminf(fmaxf(kf, -16777216.0f), 16777216.0f);
  return (int32_t)kf;
}

// ------------------------------------------------------------------------------------------------
// Teams
// ------------------------------------------------------------------------------------------------
struct Team {
  uint32_t size;   // threads in the team
  uint32_t lane;   // this thread's index inside the team
  uint32_t mask;   // warp member mask of the team (sub-warp teams)
  bool block;      // the team is the whole CTA
  uint32_t nwarps; // warps of a CTA team
  double* red;     // shared scratch for CTA-wide reductions: kMaxWarps * 5 doubles (see red_half, team_excl_scan)
};

__device__ __forceinline__ Team make_team(uint32_t team_size, double* red) {
  Team t;
  t.size = team_size;
  t.red = red;
  t.nwarps = team_size >> 5;
  if (team_size > 32u) {
    t.block = true;
    t.lane = threadIdx.x;
    t.mask = 0xFFFFFFFFu;
  } else {
    t.block = false;
    t.lane = threadIdx.x & (team_size - 1u);
    const uint32_t wl = threadIdx.x & 31u;
    t.mask = (team_size == 32u) ? 0xFFFFFFFFu : (((1u << team_size) - 1u) << (wl & ~(team_size - 1u)));
  }
  return t;
}
// The warp of this thread as a team (used for the block-wise path of the warp-team kernels).
__device__ __forceinline__ Team make_warp_team(double* red) {
  Team t;
  t.size = 32;
  t.nwarps = 1;
  t.red = red;
  t.block = false;
  t.lane = threadIdx.x & 31u;
  t.mask = 0xFFFFFFFFu;
  return t;
}

__device__ __forceinline__ void team_sync(const Team& t) {
  if (t.block) __syncthreads();
  else __syncwarp(t.mask);
}

// CTA-wide reductions exchange per-warp partials through t.red, which is split in two halves used
// alternately (`rp` counts the reductions of this thread), so that one barrier per reduction
// suffices: a half is rewritten only after the barrier of the reduction in between.
__device__ __forceinline__ double* red_half(const Team& t, uint32_t& rp) {
  double* r = t.red + ((rp++) & 1u) * (kMaxWarps * 2);
  return r;
}

// min / max over the team with NaN propagation (hardware warp reduction for fp32).
__device__ __forceinline__ void team_minmax(const Team& t, float& lo, float& hi, uint32_t& rp) {
  if (!t.block && t.size == 1u) return;
  asm volatile("redux.sync.min.NaN.f32 %0, %0, %1;" : "+f"(lo) : "r"(t.mask));
  asm volatile("redux.sync.max.NaN.f32 %0, %0, %1;" : "+f"(hi) : "r"(t.mask));
  if (t.block) {
    float* r = reinterpret_cast<float*>(red_half(t, rp));
    const uint32_t warp = threadIdx.x >> 5;
    if ((threadIdx.x & 31u) == 0) {
      r[warp * 2] = lo;
      r[warp * 2 + 1] = hi;
    }
    __syncthreads();
    // second stage, lane k takes warp k's pair (a CTA has at most 32 warps): two more warp reductions
    // instead of a walk over all pairs by every thread
    const uint32_t k = min(threadIdx.x & 31u, t.nwarps - 1u);
    const float2 pr = reinterpret_cast<const float2*>(r)[k];
    lo = pr.x;
    hi = pr.y;
    asm volatile("redux.sync.min.NaN.f32 %0, %0, %1;" : "+f"(lo) : "r"(0xFFFFFFFFu));
    asm volatile("redux.sync.max.NaN.f32 %0, %0, %1;" : "+f"(hi) : "r"(0xFFFFFFFFu));
  }
}

// Exact 64-bit sum over the warp of one int32 per lane: high and low halves are summed apart (neither sum
// can overflow 32 bits) and put together again.
__device__ __forceinline__ long long warp_sum_s32_wide(int32_t v) {
  int32_t h = v >> 16;
  uint32_t l = (uint32_t)v & 0xFFFFu;
  asm volatile("redux.sync.add.s32 %0, %0, %1;" : "+r"(h) : "r"(0xFFFFFFFFu));
  asm volatile("redux.sync.add.u32 %0, %0, %1;" : "+r"(l) : "r"(0xFFFFFFFFu));
  return (long long)h * 65536ll + (long long)l;
}

// Sum of two int32 per thread over the team, returned as 64-bit integers.  The sums over one warp
// must fit 32 bits (at most 512 groups per warp, see sigma_addends); warps are combined in 64 bits.
__device__ __forceinline__ void team_sum2(const Team& t, int32_t a, int32_t b, long long& A, long long& B,
                                          uint32_t& rp) {
  if (!t.block && t.size == 1u) {
    A = a;
    B = b;
    return;
  }
  asm volatile("redux.sync.add.s32 %0, %0, %1;" : "+r"(a) : "r"(t.mask));
  asm volatile("redux.sync.add.s32 %0, %0, %1;" : "+r"(b) : "r"(t.mask));
  A = a;
  B = b;
  if (t.block) {
    int2* r = reinterpret_cast<int2*>(red_half(t, rp));
    const uint32_t warp = threadIdx.x >> 5, wl = threadIdx.x & 31u;
    if (wl == 0) r[warp] = make_int2(a, b);
    __syncthreads();
    // second stage: lane k takes warp k's pair, the warp adds them up in 64 bits
    const int2 pr = wl < t.nwarps ? r[wl] : make_int2(0, 0);
    A = warp_sum_s32_wide(pr.x);
    B = warp_sum_s32_wide(pr.y);
  }
}

// The same for per-thread partial sums that may exceed 32 bits once added over a warp (CTA teams on
// very large planes): 64-bit shuffles inside the warp.
__device__ __forceinline__ void team_sum2_wide(const Team& t, long long a, long long b, long long& A, long long& B,
                                               uint32_t& rp) {
  for (uint32_t o = 16; o > 0; o >>= 1) {
    a += __shfl_xor_sync(0xFFFFFFFFu, a, o);
    b += __shfl_xor_sync(0xFFFFFFFFu, b, o);
  }
  long long* r = reinterpret_cast<long long*>(red_half(t, rp));
  const uint32_t warp = threadIdx.x >> 5;
  if ((threadIdx.x & 31u) == 0) {
    r[warp * 2] = a;
    r[warp * 2 + 1] = b;
  }
  __syncthreads();
  A = 0;
  B = 0;
  for (uint32_t k = 0; k < t.nwarps; ++k) {
    A += r[k * 2];
    B += r[k * 2 + 1];
  }
}

__device__ __forceinline__ uint32_t team_sum_u32(const Team& t, uint32_t v, uint32_t& rp) {
  if (!t.block && t.size == 1u) return v;
  asm volatile("redux.sync.add.u32 %0, %0, %1;" : "+r"(v) : "r"(t.mask));
  if (t.block) {
    uint32_t* r = reinterpret_cast<uint32_t*>(red_half(t, rp));
    const uint32_t warp = threadIdx.x >> 5;
    if ((threadIdx.x & 31u) == 0) r[warp] = v;
    __syncthreads();
    v = (threadIdx.x & 31u) < t.nwarps ? r[threadIdx.x & 31u] : 0u;  // second stage: lane k takes warp k's sum
    asm volatile("redux.sync.add.u32 %0, %0, %1;" : "+r"(v) : "r"(0xFFFFFFFFu));
  }
  return v;
}

// In-place exclusive prefix sum of arr[0..n) (shared memory) by the team; returns the total.
// Every lane takes a contiguous chunk; chunk sums are scanned across the team.
__device__ __forceinline__ uint32_t team_excl_scan(const Team& t, uint32_t* arr, uint32_t n) {
  if (!t.block && t.size == 32u && n <= 32u) {  // a warp and at most one element per lane: one shuffle scan
    const uint32_t v = t.lane < n ? arr[t.lane] : 0u;
    uint32_t incl = v;
    for (uint32_t o = 1; o < 32u; o <<= 1) {
      const uint32_t up = __shfl_up_sync(0xFFFFFFFFu, incl, o);
      if (t.lane >= o) incl += up;
    }
    if (t.lane < n) arr[t.lane] = incl - v;
    __syncwarp();
    return __shfl_sync(0xFFFFFFFFu, incl, 31);
  }
  const uint32_t chunk = (n + t.size - 1u) / t.size;
  const uint32_t b = min(t.lane * chunk, n), e = min(b + chunk, n);
  uint32_t local = 0;
  for (uint32_t i = b; i < e; ++i) local += arr[i];
  uint32_t incl = local, total;
  if (!t.block) {
    for (uint32_t o = 1; o < t.size; o <<= 1) {
      const uint32_t up = __shfl_up_sync(t.mask, incl, o, t.size);
      if (t.lane >= o) incl += up;
    }
    total = __shfl_sync(t.mask, incl, t.size - 1u, t.size);
  } else {
    uint32_t* r = reinterpret_cast<uint32_t*>(t.red + kMaxWarps * 4);  // region of its own, behind the two halves
    const uint32_t wl = threadIdx.x & 31u, warp = threadIdx.x >> 5;
    for (uint32_t o = 1; o < 32u; o <<= 1) {
      const uint32_t up = __shfl_up_sync(0xFFFFFFFFu, incl, o);
      if (wl >= o) incl += up;
    }
    __syncthreads();
    if (wl == 31u) r[warp] = incl;
    __syncthreads();
    uint32_t base = 0;
    total = 0;
    for (uint32_t k = 0; k < t.nwarps; ++k) {
      if (k < warp) base += r[k];
      total += r[k];
    }
    incl += base;
  }
  uint32_t run = incl - local;
  team_sync(t);  // all chunk sums are read before anybody overwrites
  for (uint32_t i = b; i < e; ++i) {
    const uint32_t v = arr[i];
    arr[i] = run;
    run += v;
  }
  team_sync(t);
  return total;
}

// ------------------------------------------------------------------------------------------------
// Huffman stage on the residual code bytes of an outlier-rich plane's dense blocks (entropy = 1)
// ------------------------------------------------------------------------------------------------
// One code per plane from the plane's own 256-bin histogram; classical merge of the two least nodes, nodes
// ordered by (weight, id), a leaf's id its symbol, a merged node's 256 + its order of creation; canonical
// code values by (length, symbol); every dense block a chunk of its own that starts on a byte boundary, bits
// most significant first.  Section: u8 len(0) | u8 smin | u8 smax | u8 0 | u8 len(smin..smax) (pad 4) |
// u8 bytes of each chunk (pad 4) | chunks (pad 4).  Lengths stay below 25 (a plane has fewer than 2^17 codes).
constexpr uint32_t kHufMaxLen = 24;
constexpr uint32_t kHufStageWords = 48;  // a chunk has at most 64 * 24 / 8 = 192 bytes

// Encoder scratch of one unit (shared memory).
struct HufEncode {
  uint32_t hist[256];
  uint32_t code[256];
  uint32_t w[512];        // node weights: 0..255 leaves by symbol, 256.. merged nodes
  uint16_t parent[512];
  uint16_t leaf[256];     // symbols that occur, sorted by (weight, symbol)
  uint8_t len[256];
  uint32_t smin, smax, maxlen, nlens;
  uint32_t stage[kMaxWarps][kHufStageWords];  // a chunk's bits while a warp assembles them
};

// One thread: code lengths and canonical codes from h->hist.
__device__ __noinline__ void huffman_build(HufEncode* h) {
  uint32_t n = 0;
  for (uint32_t sym = 0; sym < 256u; ++sym) {
    h->len[sym] = 0;
    h->code[sym] = 0;
    h->w[sym] = h->hist[sym];
    if (h->hist[sym]) h->leaf[n++] = (uint16_t)sym;
  }
  if (n == 1) h->len[h->leaf[0]] = 1;
  if (n > 1) {
    for (uint32_t i = 1; i < n; ++i) {  // insertion sort: equal weights stay in symbol order
      const uint16_t v = h->leaf[i];
      uint32_t j = i;
      while (j > 0 && h->hist[h->leaf[j - 1]] > h->hist[v]) {
        h->leaf[j] = h->leaf[j - 1];
        --j;
      }
      h->leaf[j] = v;
    }
    uint32_t li = 0, mi = 256, mn = 256;  // head of the leaf queue, head and end of the queue of merged nodes
    while ((n - li) + (mn - mi) > 1u) {
      uint32_t pick[2];
      for (int k = 0; k < 2; ++k) {
        bool take_leaf;
        if (li >= n) take_leaf = false;
        else if (mi >= mn) take_leaf = true;
        else take_leaf = h->w[h->leaf[li]] <= h->w[mi];  // equal weights: the leaf has the smaller id
        pick[k] = take_leaf ? h->leaf[li++] : mi++;
      }
      h->w[mn] = h->w[pick[0]] + h->w[pick[1]];
      h->parent[pick[0]] = h->parent[pick[1]] = (uint16_t)mn;
      ++mn;
    }
    const uint32_t root = mn - 1u;
    for (uint32_t i = 0; i < n; ++i) {
      uint32_t d = 0;
      for (uint32_t v = h->leaf[i]; v != root; v = h->parent[v]) ++d;
      h->len[h->leaf[i]] = (uint8_t)min(d, 255u);
    }
  }
  uint32_t next = 0, prev = 0, maxlen = 0, smin = 1, smax = 1;
  bool any = false;
  for (uint32_t l = 1; l <= 32u; ++l)
    for (uint32_t sym = 0; sym < 256u; ++sym)
      if (h->len[sym] == l) {
        next <<= (l - prev);
        prev = l;
        h->code[sym] = next++;
      }
  for (uint32_t sym = 0; sym < 256u; ++sym) {
    maxlen = max(maxlen, (uint32_t)h->len[sym]);
    if (sym && h->len[sym]) {
      if (!any) smin = sym;
      smax = sym;
      any = true;
    }
  }
  h->smin = smin;
  h->smax = smax;
  h->maxlen = maxlen;
  h->nlens = smax - smin + 1u;
}

// Decoder tables of one unit (shared memory), from the lengths stored in a section.
struct HufDecode {
  uint32_t first[kHufMaxLen + 1];   // first code value of every length
  uint16_t count[kHufMaxLen + 1];   // symbols of every length
  uint16_t base[kHufMaxLen + 1];    // index of a length's first symbol in `sorted`
  uint8_t sorted[256];              // symbols by (length, symbol)
  uint8_t len[256];
  uint32_t ok;
};
// One thread: tables from t->len; t->ok = 0 unless the lengths form a complete prefix code (or a single code of any length).
__device__ __noinline__ void huffman_tables(HufDecode* t) {
  for (uint32_t l = 0; l <= kHufMaxLen; ++l) t->count[l] = 0;
  unsigned long long kraft = 0;  // in units of 2^-32
  uint32_t nsym = 0;
  bool bad = false;
  for (uint32_t sym = 0; sym < 256u; ++sym) {
    const uint32_t l = t->len[sym];
    if (l > kHufMaxLen) bad = true;
    else if (l) {
      ++t->count[l];
      kraft += 1ull << (32u - l);
      ++nsym;
    }
  }
  if (nsym == 0 || kraft > (1ull << 32) || (nsym > 1 && kraft != (1ull << 32))) bad = true;
  uint32_t next = 0, prev = 0, idx = 0;
  for (uint32_t l = 1; l <= kHufMaxLen; ++l) {
    t->base[l] = (uint16_t)idx;
    if (t->count[l]) {
      next <<= (l - prev);
      prev = l;
    }
    t->first[l] = next;
    for (uint32_t sym = 0; sym < 256u && !bad; ++sym)
      if (t->len[sym] == l) t->sorted[idx++] = (uint8_t)sym;
    next += t->count[l];
  }
  t->ok = bad ? 0u : 1u;
}

// ------------------------------------------------------------------------------------------------
// Placement scan
// ------------------------------------------------------------------------------------------------
// The overflow parts of outlier-rich and raw planes lie in plane order, so a plane's place is the sum of
// the overflow sizes of all planes before it.  A tile (a run of consecutive planes, handed out in order by
// a ticket) publishes the total U of its planes' overflow sizes as soon as it has measured them -- before
// it waits for anything -- and a tile with U > 0 then needs the sum over all earlier tiles.  Two levels
// keep that look-back short (sizes in units of 16 bytes):
//   tile[t] = epoch << 32 | U_t          written once per call; an entry of another epoch reads as "not yet"
//   grp[g]  = count << 40 | sum of U     over the tiles of group g = t >> 5 that have published (atomic adds).
//                                        Two sets alternate between consecutive calls on a scratch; a call's last
//                                        CTA returns the set of the call BEFORE it to zero (grp_clear): every add
//                                        of that call was performed when its kernel completed, so no fence is
//                                        needed between a tile's add and the clearing store.
//   gpre[g] = epoch << 32 | sum of U     over all tiles of groups 0..g, published by whoever has worked it out
// Progress: tiles are taken in ticket order by CTAs that are running, a CTA works through its tiles in
// increasing order, and a tile publishes before it waits; so the smallest tile that has not published is
// never waiting.  Every wait is bounded all the same and reports a time-out instead of hanging.
struct Scan {
  unsigned long long* tile;
  unsigned long long* grp;
  unsigned long long* gpre;
  unsigned long long* grp_clear;  // group sums the call's last CTA returns to zero (see above)
  uint32_t clear_groups;          // ... and how many
  uint32_t epoch;      // of this call (never 0)
  uint32_t polls;      // limit of every wait, in polls of about 0.1 us
  uint32_t skip_tile;  // this tile never publishes (fault injection for the time-out test; 0xFFFFFFFF: none)
};

// One thread: tile t has measured its planes.
__device__ __forceinline__ void scan_publish(const Scan& s, uint32_t t, uint32_t U) {
  if (t == s.skip_tile) return;
  st_relaxed(&s.tile[t], ((unsigned long long)s.epoch << 32) | U);
  atomicAdd(&s.grp[t >> 5], (1ull << 40) | (unsigned long long)U);
}

__device__ __forceinline__ unsigned long long warp_sum_u64(unsigned long long v) {
  for (uint32_t o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
  return v;
}

// A whole warp: sum of U over the tiles before t.  False when a wait ran out.
__device__ __noinline__ bool scan_prefix(const Scan& s, uint32_t t, uint32_t& prefix) {
  const uint32_t lane = threadIdx.x & 31u, full = 0xFFFFFFFFu;
  const uint32_t g = t >> 5, within = t & 31u;
  // tiles of the own group before t
  unsigned long long u = 0;
  {
    bool ok = lane >= within;
    for (uint32_t k = 0; k < s.polls; ++k) {
      if (!ok) {
        const unsigned long long v = ld_relaxed(&s.tile[g * 32u + lane]);
        if ((uint32_t)(v >> 32) == s.epoch) {
          u = v & 0xFFFFFFFFull;
          ok = true;
        }
      }
      if (__all_sync(full, ok)) break;
      __nanosleep(100);
    }
    if (!__all_sync(full, ok)) return false;
  }
  unsigned long long acc = warp_sum_u64(u);
  // earlier groups, the nearest first, 32 at a time, until a group whose prefix somebody has published
  unsigned long long gsum = 0;
  uint32_t hi = g;
  while (hi > 0) {
    const bool act = lane < hi;
    const uint32_t j = act ? hi - 1u - lane : 0u;
    bool have_pre = false, done = !act;
    unsigned long long val = 0;
    uint32_t first = 32, need = full, dm = 0;
    for (uint32_t k = 0; k < s.polls; ++k) {
      if (act && !have_pre) {
        const unsigned long long v = ld_relaxed(&s.gpre[j]);
        if ((uint32_t)(v >> 32) == s.epoch) {
          have_pre = true;
          done = true;
          val = v & 0xFFFFFFFFull;
        }
      }
      if (act && !done) {
        const unsigned long long v = ld_relaxed(&s.grp[j]);
        if ((v >> 40) == 32ull) {  // every group before another one is a whole group of 32 tiles
          done = true;
          val = v & ((1ull << 40) - 1ull);
        }
      }
      const uint32_t pm = __ballot_sync(full, have_pre);
      first = pm ? (uint32_t)__ffs((int)pm) - 1u : 32u;
      need = first >= 31u ? full : ((2u << first) - 1u);  // lanes 0..first
      dm = __ballot_sync(full, done);
      if ((dm & need) == need) break;
      __nanosleep(100);
    }
    if ((dm & need) != need) return false;
    gsum += warp_sum_u64(lane <= first ? val : 0ull);
    if (first < 32u) break;
    hi = hi > 32u ? hi - 32u : 0u;
  }
  if (g > 0 && lane == 0) st_relaxed(&s.gpre[g - 1u], ((unsigned long long)s.epoch << 32) | (gsum & 0xFFFFFFFFull));
  prefix = (uint32_t)(gsum + acc);
  return true;
}

}  // namespace fh
