// Channel-wide three-sigma statistics (salient_mode = CHANNEL): mu, sigma and the outlier count are taken
// over the N planes (n, c) of a channel c together, and the channel as a whole is normal or outlier-rich.
// Tensor-wide statistics (salient_mode = TENSOR) run through the same passes with the whole tensor as the
// one "channel"; a plane's class then follows from its own count.
// Three passes over the tensor, a warp per plane, results gathered per channel with atomics:
//   pass 0: minimum and maximum of the channel (the moments are taken of the distances from the minimum, and the
//           range fixes the scale of the integer sums);
//   pass 1: integer moment sums of the channel (exact, so the order of the atomics is immaterial);
//   pass 2: thresholds from the sums; outliers per plane (kept for the plane table) and per channel.
// The streaming kernel then reads a plane's class from its channel's count.  This mode is not tuned: it
// reads the tensor four times where the per-plane mode reads it once.
#pragma once

#include "fh_device.cuh"

namespace fh {

struct ChanStat {
  unsigned int lo_inv;       // ~key(minimum): atomicMax
  unsigned int hi_key;       // key(maximum): atomicMax
  unsigned long long Is, Iq;  // fixed-point moment sums (two's complement)
  unsigned long long nout;    // three-sigma outliers of the channel
};
static_assert(sizeof(ChanStat) == 32, "ChanStat layout");

// Order-preserving map float -> unsigned (finite values; -0.0 sorts below +0.0, and a distance from either is
// the same number).
__device__ __forceinline__ unsigned int float_key(float f) {
  const unsigned int b = __float_as_uint(f);
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float key_float(unsigned int k) {
  return __uint_as_float((k & 0x80000000u) ? (k & 0x7FFFFFFFu) : ~k);
}

struct ChannelArgs {
  const uint8_t* src;
  ChanStat* chan;        // C entries (one in the tensor-wide mode), zeroed before pass 0
  uint32_t* plane_nout;  // P entries, written by pass 2
  double inv_nhw;        // 1 / (N * HW); tensor-wide: 1 / (N * C * HW)
};

template <int DT>
__device__ __forceinline__ void load_group_global(const uint8_t* plane, uint32_t g, uint32_t HW, float v[4]) {
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const uint32_t i = g * 4u + k;
    float x = 0.0f;
    if (i < HW) x = DT == kF32 ? __ldg(reinterpret_cast<const float*>(plane) + i)
                               : bf16_bits_to_f32(__ldg(reinterpret_cast<const uint16_t*>(plane) + i));
    v[k] = x;
  }
}

template <int DT, int PASS>
__global__ void __launch_bounds__(kThreads) channel_pass(const Plan pl, const ChannelArgs a) {
  const uint32_t lane = threadIdx.x & 31u;
  const uint64_t warps = (uint64_t)gridDim.x * kWarps, first = (uint64_t)blockIdx.x * kWarps + (threadIdx.x >> 5);
  // Tensor-wide statistics have a single destination: a warp gathers over its planes, the CTA's warps are
  // combined in shared memory, and one thread per CTA issues the atomics.
  const bool whole = pl.mode == kModeTensor;
  __shared__ float s_lo[kWarps], s_hi[kWarps];
  __shared__ long long s_s[kWarps], s_q[kWarps];
  float wlo = __int_as_float(0x7F800000), whi = __int_as_float(0xFF800000);
  long long ws = 0, wq = 0;
  for (uint64_t p = first; p < pl.P; p += warps) {
    const uint8_t* plane = a.src + p * pl.plane_bytes;
    ChanStat* cs = a.chan + (pl.mode == kModeTensor ? 0ull : p % pl.C);
    if (PASS == 0) {
      float lo = __int_as_float(0x7F800000), hi = __int_as_float(0xFF800000);
      for (uint32_t i = lane; i < pl.HW; i += 32u) {
        const float x = DT == kF32 ? __ldg(reinterpret_cast<const float*>(plane) + i)
                                   : bf16_bits_to_f32(__ldg(reinterpret_cast<const uint16_t*>(plane) + i));
        lo = fminf(lo, x);   // non-finite input is reported by the streaming kernel; here it only must not trap
        hi = fmaxf(hi, x);
      }
      for (uint32_t o = 16; o > 0; o >>= 1) {
        lo = fminf(lo, __shfl_xor_sync(0xFFFFFFFFu, lo, o));
        hi = fmaxf(hi, __shfl_xor_sync(0xFFFFFFFFu, hi, o));
      }
      if (whole) {
        wlo = fminf(wlo, lo);
        whi = fmaxf(whi, hi);
      } else if (lane == 0) {
        atomicMax(&cs->lo_inv, ~float_key(lo));
        atomicMax(&cs->hi_key, float_key(hi));
      }
    } else {
      const float clo = key_float(~cs->lo_inv), chi = key_float(cs->hi_key);
      const SigmaScale sc = sigma_scale(__fsub_rn(chi, clo));
      if (!sc.applies) {  // constant channel, or a range outside the rule's domain: no outliers
        if (PASS == 2 && lane == 0) a.plane_nout[p] = 0;
        continue;
      }
      if (PASS == 1) {
        long long s = 0, q = 0;
        for (uint32_t g = lane; g < pl.groups; g += 32u) {
          float v[4];
          load_group_global<DT>(plane, g, pl.HW, v);
#pragma unroll
          for (int k = 0; k < 4; ++k) v[k] = (g * 4u + k < pl.HW) ? __fsub_rn(v[k], clo) : 0.0f;
          uint32_t as = 0, aq = 0;
          sigma_addends(v, sc, as, aq);
          s += (int32_t)(as - kMagicBits);
          q += (int32_t)(aq - kMagicBits);
        }
        for (uint32_t o = 16; o > 0; o >>= 1) {
          s += __shfl_xor_sync(0xFFFFFFFFu, s, o);
          q += __shfl_xor_sync(0xFFFFFFFFu, q, o);
        }
        if (whole) {
          ws += s;
          wq += q;
        } else if (lane == 0) {
          atomicAdd(&cs->Is, (unsigned long long)s);
          atomicAdd(&cs->Iq, (unsigned long long)q);
        }
      } else {
        float dlo, dhi;
        sigma_thresholds((long long)cs->Is, (long long)cs->Iq, sc, a.inv_nhw, dlo, dhi);
        uint32_t cnt = 0;
        for (uint32_t i = lane; i < pl.HW; i += 32u) {
          const float x = DT == kF32 ? __ldg(reinterpret_cast<const float*>(plane) + i)
                                     : bf16_bits_to_f32(__ldg(reinterpret_cast<const uint16_t*>(plane) + i));
          const float dd = __fsub_rn(x, clo);
          cnt += (dd > dhi) || (dd < dlo);
        }
        asm volatile("redux.sync.add.u32 %0, %0, %1;" : "+r"(cnt) : "r"(0xFFFFFFFFu));
        if (lane == 0) {
          a.plane_nout[p] = cnt;
          if (cnt && !whole) atomicAdd(&cs->nout, (unsigned long long)cnt);  // the tensor-wide mode classifies by the plane's count
        }
      }
    }
  }
  if (whole && PASS < 2) {
    const uint32_t warp = threadIdx.x >> 5;
    if (lane == 0) {
      s_lo[warp] = wlo;
      s_hi[warp] = whi;
      s_s[warp] = ws;
      s_q[warp] = wq;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
      for (uint32_t k = 1; k < (uint32_t)kWarps; ++k) {
        wlo = fminf(wlo, s_lo[k]);
        whi = fmaxf(whi, s_hi[k]);
        ws += s_s[k];
        wq += s_q[k];
      }
      if (PASS == 0) {  // (every CTA of the grid owns at least one plane, so both values are finite numbers of the input)
        atomicMax(&a.chan->lo_inv, ~float_key(wlo));
        atomicMax(&a.chan->hi_key, float_key(whi));
      } else {
        atomicAdd(&a.chan->Is, (unsigned long long)ws);
        atomicAdd(&a.chan->Iq, (unsigned long long)wq);
      }
    }
  }
}

}  // namespace fh
