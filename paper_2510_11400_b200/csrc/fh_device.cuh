// Device-side building blocks shared by the compress and decompress kernels (sm_100a).
//
// Terminology: a "plane" is one (n, c) feature map of H x W elements; a "tile" is a run of
// consecutive planes that one CTA stages in shared memory; a "team" is the group of threads that
// works on one plane: a power-of-two slice of a warp for small planes, the whole CTA for large ones.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace fh {

constexpr int kThreads = 256;          // CTA size of both kernels
constexpr uint32_t kMagic = 0x31434846u;  // "FHC1"
constexpr uint32_t kClsNormal = 0, kClsSalient = 1, kClsRaw = 2;
constexpr int kModeAuto = 0, kModeOff = 1, kModeAll = 2;
constexpr int kF32 = 0, kBF16 = 1;

// Device-side error codes (positive, ordered by priority; the host maps them to fh_status).
constexpr uint32_t kErrNone = 0, kErrNonfinite = 1, kErrCapacity = 2, kErrCorrupt = 3, kErrTimeout = 4;

// Everything a kernel needs to know about the tensor, the parameters and the tiling.
struct Plan {
  int32_t dtype, esize, H, W;
  uint32_t N, C;
  uint32_t HW;
  uint32_t groups;       // ceil(HW / 4): groups of four consecutive elements
  uint64_t P;            // planes
  uint64_t plane_bytes;  // HW * esize
  uint64_t dense_bytes;  // P * plane_bytes
  int32_t bits, mode;
  uint32_t rho_num, rho_den, tau_num, tau_den;
  float eps;
  uint64_t tensor_id;
  uint32_t ppt;          // planes per tile
  uint32_t ntiles;
  uint32_t team;         // threads per plane: 1..32 (power of two) or kThreads
  uint32_t npay;         // A16(bytes of a normal payload)
  uint32_t nbx, nby, nblk, nbm;  // 8x8 blocks per row / column / plane, bitmap words
  uint32_t sm_tile, sm_tile_bytes;  // shared-memory layout (byte offsets)
  uint32_t sm_out, sm_rec, sm_sal, sm_sal_stride, sm_total;
};

// Scan / bookkeeping scratch, one per stream.  Words carry the call's epoch in their upper half so
// that nothing has to be cleared between calls.
struct TileState {            // 32 bytes per tile
  unsigned long long agg_a;   // epoch << 32 | tile size in 16-byte units
  unsigned long long agg_b;   // n_salient << 32 | n_raw of the tile
  unsigned long long inc_a;   // epoch << 32 | inclusive prefix of sizes
  unsigned long long inc_b;   // inclusive prefix of the counts
};
struct Scratch {
  unsigned long long ticket;  // monotonically increasing tile tickets
  unsigned long long done;    // monotonically increasing count of finished tiles
  unsigned long long status;  // epoch << 32 | device error code (atomicMax)
  unsigned long long total;   // container bytes of the current call
};

// (uint64)(int64) fh_status of a device error code.
__device__ __forceinline__ unsigned long long status_word(uint32_t code) {
  const long long st = code == kErrNonfinite ? -4 : code == kErrCapacity ? -3 : code == kErrCorrupt ? -5
                       : code == kErrTimeout ? -6 : 0;
  return (unsigned long long)st;
}

__device__ __forceinline__ uint32_t a4(uint32_t x) { return (x + 3u) & ~3u; }
__device__ __forceinline__ uint32_t a16(uint32_t x) { return (x + 15u) & ~15u; }

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

// min / max that return NaN when either operand is NaN, so that a NaN anywhere in a plane
// surfaces in its minimum and maximum.
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

__device__ __forceinline__ float bf16_bits_to_f32(uint32_t h) { return __uint_as_float(h << 16); }
// fp32 -> bf16 bits, round half to even (finite inputs).
__device__ __forceinline__ uint32_t f32_to_bf16_bits(float f) {
  uint32_t u = __float_as_uint(f);
  return (u + (((u >> 16) & 1u) + 0x7FFFu)) >> 16;
}

template <int DT>
__device__ __forceinline__ float load_elem(const uint8_t* plane, uint32_t i) {
  if (DT == kF32) return reinterpret_cast<const float*>(plane)[i];
  return bf16_bits_to_f32(reinterpret_cast<const uint16_t*>(plane)[i]);
}

// Four consecutive elements of a plane (group g), elements past HW read as 0.  `vec` says that the
// plane starts on a 16-byte (fp32) / 8-byte (bf16) boundary so that a full group is one load.
template <int DT>
__device__ __forceinline__ void load_group(const uint8_t* plane, uint32_t g, uint32_t HW, bool vec,
                                           float v[4]) {
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

// ------------------------------------------------------------------------------------------------
// Teams
// ------------------------------------------------------------------------------------------------
struct Team {
  uint32_t size;   // threads in the team
  uint32_t lane;   // this thread's index inside the team
  uint32_t mask;   // warp member mask of the team (sub-warp teams)
  bool block;      // the team is the whole CTA
  double* red;     // shared scratch for CTA-wide reductions: (kThreads/32) * 4 doubles + 8
};

__device__ __forceinline__ Team make_team(uint32_t team_size, double* red) {
  Team t;
  t.size = team_size;
  t.red = red;
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

__device__ __forceinline__ void team_sync(const Team& t) {
  if (t.block) __syncthreads();
  else __syncwarp(t.mask);
}

// Plane statistics reduced over the team: lo/hi with NaN propagation, S/Q in fp64.
struct Stats {
  float lo, hi;
  double S, Q;
};

__device__ __forceinline__ Stats team_reduce_stats(const Team& t, Stats s) {
  const uint32_t w = t.block ? 32u : t.size;
  for (uint32_t o = w >> 1; o > 0; o >>= 1) {
    s.lo = min_nan(s.lo, __shfl_xor_sync(t.mask, s.lo, o));
    s.hi = max_nan(s.hi, __shfl_xor_sync(t.mask, s.hi, o));
    s.S += __shfl_xor_sync(t.mask, s.S, o);
    s.Q += __shfl_xor_sync(t.mask, s.Q, o);
  }
  if (t.block) {
    const uint32_t warp = threadIdx.x >> 5, nw = kThreads / 32;
    __syncthreads();
    if ((threadIdx.x & 31u) == 0) {
      t.red[warp * 4 + 0] = (double)s.lo;
      t.red[warp * 4 + 1] = (double)s.hi;
      t.red[warp * 4 + 2] = s.S;
      t.red[warp * 4 + 3] = s.Q;
    }
    __syncthreads();
    s.lo = (float)t.red[0]; s.hi = (float)t.red[1]; s.S = t.red[2]; s.Q = t.red[3];
    for (uint32_t k = 1; k < nw; ++k) {
      s.lo = min_nan(s.lo, (float)t.red[k * 4 + 0]);
      s.hi = max_nan(s.hi, (float)t.red[k * 4 + 1]);
      s.S += t.red[k * 4 + 2];
      s.Q += t.red[k * 4 + 3];
    }
  }
  return s;
}

__device__ __forceinline__ uint32_t team_sum_u32(const Team& t, uint32_t v) {
  const uint32_t w = t.block ? 32u : t.size;
  for (uint32_t o = w >> 1; o > 0; o >>= 1) v += __shfl_xor_sync(t.mask, v, o);
  if (t.block) {
    uint32_t* r = reinterpret_cast<uint32_t*>(t.red);
    const uint32_t warp = threadIdx.x >> 5, nw = kThreads / 32;
    __syncthreads();
    if ((threadIdx.x & 31u) == 0) r[warp] = v;
    __syncthreads();
    v = 0;
    for (uint32_t k = 0; k < nw; ++k) v += r[k];
  }
  return v;
}

// In-place exclusive prefix sum of arr[0..n) (shared memory) by the team; returns the total.
// Every lane takes a contiguous chunk; chunk sums are scanned across the team.
__device__ __forceinline__ uint32_t team_excl_scan(const Team& t, uint32_t* arr, uint32_t n) {
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
    uint32_t* r = reinterpret_cast<uint32_t*>(t.red);  // kThreads/32 + 1 words
    const uint32_t wl = threadIdx.x & 31u, warp = threadIdx.x >> 5, nw = kThreads / 32;
    for (uint32_t o = 1; o < 32u; o <<= 1) {
      const uint32_t up = __shfl_up_sync(0xFFFFFFFFu, incl, o);
      if (wl >= o) incl += up;
    }
    __syncthreads();
    if (wl == 31u) r[warp] = incl;
    __syncthreads();
    uint32_t base = 0;
    total = 0;
    for (uint32_t k = 0; k < nw; ++k) {
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

// Pre-quantisation of dense-block elements (Eq. 9 on integers): k = rne(fp32(x * inv2e)), |k| <= 2^24.
__device__ __forceinline__ int32_t dense_k(float x, float inv2e, bool* big) {
  float kf = rintf(__fmul_rn(x, inv2e));
  *big = fabsf(kf) >= 16777216.0f;
  kf = fminf(fmaxf(kf, -16777216.0f), 16777216.0f);
  return (int32_t)kf;
}

}  // namespace fh
