// Host side of the C ABI declared in include/fh.h: argument checks, size formulas, tiling plans,
// per-stream scratch, kernel launches, the schedule runner and the host-buffer variants.
#include "../../include/fh.h"

#include <cuda_runtime.h>

#include <atomic>
#include <cmath>
#include <cstring>
#include <map>
#include <mutex>
#include <tuple>
#include <utility>
#include <vector>

#include "fh_channel.cuh"
#include "fh_compress.cuh"
#include "fh_decompress.cuh"

namespace {

using fh::Plan;

constexpr size_t kSmemLimit = 227 * 1024 - 4096;  // dynamic shared memory a CTA may ask for
constexpr size_t kTileTarget = 32 * 1024;         // dense bytes a tile of the generic kernel aims for
constexpr size_t kStageTarget = 72 * 1024;        // shared memory the stages of the CTA-team kernel aim for
constexpr size_t kWarpStageTarget = 72 * 1024;    // ... and those of the warp-team kernel (two CTAs per SM)
constexpr uint32_t kMaxPpt = 2048;

std::atomic<uint64_t> g_launches{0};

inline size_t A16(size_t x) { return (x + 15) & ~(size_t)15; }
inline size_t A256(size_t x) { return (x + 255) & ~(size_t)255; }
inline size_t esize_of(int dtype) { return dtype == FH_F32 ? 4 : 2; }

int check_desc(const fh_tensor_desc* d) {
  if (!d) return FH_ERR_ARG;
  if (d->dtype != FH_F32 && d->dtype != FH_BF16) return FH_ERR_ARG;
  if (d->n < 1 || d->c < 1 || d->h < 1 || d->w < 1) return FH_ERR_ARG;
  if (d->w > 65535) return FH_ERR_UNSUPPORTED;
  return FH_OK;
}

int check_params(const fh_params* p) {
  if (!p) return FH_ERR_ARG;
  if (p->bits != 2 && p->bits != 4 && p->bits != 8) return FH_ERR_UNSUPPORTED;
  if (p->salient_mode < 0 || p->salient_mode > 4) return FH_ERR_ARG;
  if (p->rho_num < 0 || p->rho_den < 1 || p->rho_num > 65535 || p->rho_den > 65535) return FH_ERR_ARG;
  if (p->tau_num < 0 || p->tau_den < 1 || p->tau_num > 65535 || p->tau_den > 65535) return FH_ERR_ARG;
  if (p->block != 8 || p->dense_bits != 8 || (p->rounding != 0 && p->rounding != 1)) return FH_ERR_UNSUPPORTED;
  if (p->entropy != 0 && p->entropy != 1) return FH_ERR_UNSUPPORTED;
  if (!(p->eps >= 1e-30f) || !(p->eps <= 1e30f)) return FH_ERR_ARG;
  return FH_OK;
}

uint32_t pow2_floor(uint32_t x) {
  uint32_t r = 1;
  while (r * 2 <= x) r *= 2;
  return r;
}

uint32_t pow2_ceil(uint32_t x) {
  uint32_t r = 1;
  while (r < x) r *= 2;
  return r;
}

// Which kernel a plan runs on.
struct Variant {
  bool fast = false;  // compress_warp / compress_cta (bulk-copy pipeline) instead of compress_generic
  bool cta = false;   // fast: compress_cta (one plane per CTA) instead of compress_warp (one plane per team of lanes)
  int G = 0;          // fast: groups per thread
};

// Tiling and shared-memory layout.  `compress` selects the compress kernels' layout; the decompress
// kernel only needs the block-wise scratch.
int make_plan(const fh_tensor_desc* d, const fh_params* p, bool compress, Plan* out, Variant* var) {
  Plan pl;
  std::memset(&pl, 0, sizeof(pl));
  pl.dtype = d->dtype;
  pl.esize = (int)esize_of(d->dtype);
  pl.H = d->h;
  pl.W = d->w;
  pl.N = (uint32_t)d->n;
  pl.C = (uint32_t)d->c;
  const uint64_t hw = (uint64_t)d->h * (uint64_t)d->w;
  if (hw * pl.esize > kSmemLimit) return FH_ERR_UNSUPPORTED;
  pl.HW = (uint32_t)hw;
  pl.groups = (pl.HW + 3) / 4;
  pl.P = (uint64_t)d->n * (uint64_t)d->c;
  pl.plane_bytes = hw * pl.esize;
  pl.dense_bytes = pl.P * pl.plane_bytes;
  pl.inv_hw = 1.0 / (double)hw;
  pl.bits = p ? p->bits : 2;
  pl.mode = p ? p->salient_mode : 0;
  pl.rounding = p ? p->rounding : 0;
  pl.entropy = p ? p->entropy : 0;
  pl.seed = p ? p->seed : 0;
  pl.rho_num = p ? p->rho_num : 1;
  pl.rho_den = p ? p->rho_den : 32;
  pl.tau_num = p ? p->tau_num : 1;
  pl.tau_den = p ? p->tau_den : 4;
  pl.eps = p ? p->eps : 0.0625f;
  pl.tensor_id = d->tensor_id;
  pl.npay = (uint32_t)A16(4 * (((uint64_t)pl.HW * pl.bits + 31) / 32));
  pl.slots_off = 64 + 16 * pl.P;
  pl.ovf_off = pl.slots_off + pl.P * pl.npay;
  pl.nbx = (uint32_t)(d->w + 7) / 8;
  pl.nby = (uint32_t)(d->h + 7) / 8;
  pl.nblk = pl.nbx * pl.nby;
  pl.nbm = (pl.nblk + 31) / 32;
  // container offsets are 32-bit counts of 16 bytes
  const long double worst = 64.0L + (long double)pl.P * (16.0L + (long double)A16(pl.plane_bytes));
  if (worst / 16.0L >= 4294967295.0L) return FH_ERR_UNSUPPORTED;
  if (pl.P > 0x7FFFFFFFull) return FH_ERR_UNSUPPORTED;
  // measuring scratch of the block-wise path: row pointers and three words per block; with the Huffman stage two
  // more words per block and the encoder's tables.  Decompress: two words per block and the decoder's tables.
  const size_t sal_words = compress ? (size_t)(pl.H + 1 + 3 * pl.nblk) + (pl.entropy ? 2 * (size_t)pl.nblk + sizeof(fh::HufEncode) / 4 + 4 : 0)
                                    : 2 * (size_t)pl.nblk + sizeof(fh::HufDecode) / 4 + 4;
  pl.sal_words = (uint32_t)sal_words;
  const uint32_t sal_bytes = (uint32_t)A16(4 * sal_words + 16);  // one measuring area of the block-wise path
  const bool blockwise = compress && pl.mode != FH_SALIENT_OFF;

  Variant v;
  // ---- fast compress kernels: planes of whole 16-byte chunks whose groups fit the register budget
  const bool whole16 = pl.HW % 4 == 0 && pl.plane_bytes % 16 == 0;
  // (the Huffman stage runs on the generic kernel; random rounding on the warp-team kernels in the plane-wise
  // three-sigma mode, on the generic kernel otherwise)
  // (a warp-team kernel keeps one measuring area per warp: planes whose area is large -- very tall, narrow
  // ones -- go to the general-purpose kernel)
  const bool rounding_ok = pl.rounding == 0 || (pl.groups <= 256 && pl.mode == FH_SALIENT_AUTO);
  if (compress && rounding_ok && pl.entropy == 0 && ((pl.groups <= 256 && (!blockwise || sal_bytes <= 1024)) || (pl.groups > 256 && whole16))) {
    v.fast = true;
    if (pl.groups <= 256) {
      uint32_t t = pow2_ceil((pl.groups + 7) / 8);
      pl.team = t > 32 ? 32 : t;
      v.G = 8;  // the warp-team kernels keep eight groups per thread
      pl.ppt = fh::kThreads / pl.team;
    } else {
      v.cta = true;  // CTA size by plane size: enough work per thread between barriers
      // (the per-plane reductions and scalar steps cost every warp the same, whatever its share of the plane:
      // fewer, busier threads win as long as enough warps stay resident)
      pl.team = pl.plane_bytes <= 16 * 1024 ? 128 : (pl.plane_bytes <= 64 * 1024 ? 256 : 512);
      v.G = 0;
      // planes of up to 4096 groups: the register variant, with the smallest (threads, groups per thread)
      // that holds the plane
      static const uint32_t kCombo[6][2] = {{128, 7}, {128, 8}, {256, 7}, {256, 8}, {448, 7}, {512, 8}};
      for (int k = 0; k < 6; ++k)
        if (kCombo[k][0] * kCombo[k][1] >= pl.groups) {
          pl.team = kCombo[k][0];
          v.G = (int)kCombo[k][1];
          break;
        }
      pl.ppt = 1;
    }
    if (pl.ppt > pl.P) pl.ppt = (uint32_t)pl.P;
    pl.stage_bytes = (uint32_t)((pl.ppt * pl.plane_bytes + 127) & ~(uint64_t)127);
    uint32_t ns = (uint32_t)((v.cta ? kStageTarget : kWarpStageTarget) / pl.stage_bytes);
    // (CTA-team kernel: two stages; a third buys nothing that more resident CTAs do not give)
    const uint32_t ns_max = v.cta ? 2u : (uint32_t)fh::kMaxStages;
    ns = ns < 2 ? 2 : (ns > ns_max ? ns_max : ns);
    const uint32_t areas = blockwise ? (v.cta ? 1u : (uint32_t)fh::kWarps) : 0u;
    for (;;) {
      pl.nstage = ns;
      pl.sm_tile = 0;
      pl.sm_sal = (uint32_t)A16((size_t)ns * pl.stage_bytes);
      pl.sal_stride = sal_bytes;
      pl.sm_total = pl.sm_sal + areas * sal_bytes;
      if (pl.sm_total <= kSmemLimit) break;
      if (ns == 2) {  // the pipeline needs two stages
        v.fast = false;
        break;
      }
      --ns;
    }
  }
  if (!compress) {
    // decompress: sub-warp teams, planes assigned round-robin (ntiles only bounds the grid)
    uint32_t t = pow2_ceil((pl.groups + 7) / 8);
    pl.team = t > 32 ? 32 : t;
    const uint32_t nteams = fh::kThreads / pl.team;
    pl.sal_stride = sal_bytes;
    pl.sm_total = nteams * sal_bytes + 16;
    if (pl.sm_total > kSmemLimit) return FH_ERR_UNSUPPORTED;
    pl.ppt = nteams;
    {
      const uint64_t chunks = (pl.groups + 8 * pl.team - 1) / (8 * pl.team);
      const uint64_t ctas = (pl.P * chunks + nteams - 1) / nteams;
      pl.ntiles = (uint32_t)(ctas > 0x7FFFFFFFull ? 0x7FFFFFFFull : ctas);
    }
    *out = pl;
    if (var) *var = Variant();
    return FH_OK;
  }
  if (!v.fast) {
    v = Variant();
    if (pl.plane_bytes <= 8192) {
      uint32_t t = pow2_floor(pl.HW / 8 > 0 ? pl.HW / 8 : 1);
      pl.team = t > 32 ? 32 : t;
    } else {
      pl.team = fh::kThreads;
    }
    pl.nstage = 0;
    pl.stage_bytes = 0;
    uint64_t ppt = kTileTarget / pl.plane_bytes;
    if (ppt < 1) ppt = 1;
    if (ppt > kMaxPpt) ppt = kMaxPpt;
    if (ppt > pl.P) ppt = pl.P;
    for (;;) {
      pl.ppt = (uint32_t)ppt;
      pl.sm_tile = 0;
      pl.sm_out = (uint32_t)A16(ppt * pl.plane_bytes + 32);
      pl.sm_rec = pl.sm_out + (uint32_t)(ppt * pl.npay);
      pl.sm_sal = pl.sm_rec + (uint32_t)A16(16 * ppt);
      pl.sal_stride = sal_bytes;
      pl.sm_total = pl.sm_sal + (blockwise ? sal_bytes : 0u);
      if (pl.sm_total <= kSmemLimit) break;
      if (ppt == 1) return FH_ERR_UNSUPPORTED;
      ppt = ppt / 2;
    }
  }
  const uint64_t ntiles = (pl.P + pl.ppt - 1) / pl.ppt;
  if (ntiles > 0x7FFFFFFFull) return FH_ERR_UNSUPPORTED;
  pl.ntiles = (uint32_t)ntiles;
  *out = pl;
  if (var) *var = v;
  return FH_OK;
}

// ---- per-stream scratch ---------------------------------------------------------------------
struct StreamScratch {
  fh::Scratch* sc = nullptr;             // counters
  unsigned long long* scan = nullptr;    // placement scan: tile words, group sums, group prefixes; then the tile links
  size_t tile_cap = 0;                   // tiles the scan arrays hold (groups: tile_cap / 32)
  uint32_t calls = 0;                    // compress calls so far: parity of the ticket counter, epoch of the scan
  uint32_t scan_calls = 0;               // ... those that used the placement scan: which set of group sums is next
  uint32_t prev_groups = 0;              // groups of 32 tiles the last of them used (the next one clears that set)
  uint32_t* plane_nout = nullptr;        // channel-wide three-sigma mode: per-plane counts ...
  size_t pn_cap = 0;
  fh::ChanStat* chan = nullptr;          // ... and per-channel statistics
  size_t chan_cap = 0;
  unsigned long long* sched = nullptr;   // schedule runner: offsets, sizes, statuses
  size_t sched_cap = 0;
};
// tile words | two sets of group sums | group prefixes | tile links (32-bit)
inline size_t scan_words(size_t tile_cap) { return tile_cap + 3 * (tile_cap / 32) + tile_cap / 2; }

std::mutex g_mu;
std::map<std::pair<int, cudaStream_t>, StreamScratch> g_scratch;
int g_sm_count[64] = {0};

// Fault injection for the time-out test (see fh_debug_set in the header): limit of the device-side waits
// of the placement scan, and a tile that never publishes.
uint32_t g_scan_polls = 1u << 22;
uint32_t g_skip_tile = 0xFFFFFFFFu;

// `tiles`: tiles of the compress call that is about to be enqueued (0: none, e.g. for decompress).
int get_scratch(cudaStream_t stream, size_t tiles, StreamScratch** out) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return FH_ERR_CUDA;
  StreamScratch& s = g_scratch[std::make_pair(dev, stream)];
  if (!s.sc) {
    if (cudaMalloc(&s.sc, fh::kScratchHeadBytes) != cudaSuccess) return FH_ERR_CUDA;
    // cleared in the order of the stream that will use it (a non-blocking stream is not ordered with
    // the legacy default stream)
    if (cudaMemsetAsync(s.sc, 0, fh::kScratchHeadBytes, stream) != cudaSuccess) return FH_ERR_CUDA;
  }
  if (tiles > s.tile_cap) {
    size_t cap = s.tile_cap ? s.tile_cap : 16384;
    while (cap < tiles) cap *= 2;
    if (s.scan) {
      cudaDeviceSynchronize();
      cudaFree(s.scan);
      s.scan = nullptr;
      s.tile_cap = 0;
    }
    s.prev_groups = 0;
    if (cudaMalloc(&s.scan, scan_words(cap) * sizeof(unsigned long long)) != cudaSuccess) return FH_ERR_CUDA;
    if (cudaMemsetAsync(s.scan, 0, scan_words(cap) * sizeof(unsigned long long), stream) != cudaSuccess) return FH_ERR_CUDA;
    s.tile_cap = cap;
  }
  *out = &s;
  return FH_OK;
}

// Parity, epoch and scan pointers of the next compress call on a scratch (`scan` may be null when the call
// places nothing).  The epoch never is 0; when the counter wraps, the tagged arrays are cleared.
// `s`: the per-stream scratch, whose two sets of group sums alternate between the calls that use the scan (the
// call returns the other set -- the one its predecessor used -- to zero); null: one set, which the caller
// clears ahead of every call (the fixed scratch of fh_compress_static).
int next_call(uint32_t* calls, unsigned long long* scan, size_t tile_cap, StreamScratch* s, uint32_t groups_now,
              cudaStream_t stream, fh::CompressArgs* a) {
  ++*calls;
  if ((*calls & 0x7FFFFFFFu) == 0u) {  // 2^31 calls later an old tag could pass for a new one: start afresh
    const size_t words = s ? scan_words(tile_cap) : tile_cap + 2 * (tile_cap / 32);
    unsigned long long* all = s ? s->scan : scan;  // (also when this very call places nothing)
    if (all && cudaMemsetAsync(all, 0, words * sizeof(unsigned long long), stream) != cudaSuccess) return FH_ERR_CUDA;
    if (s) s->prev_groups = 0;
    ++*calls;
  }
  const size_t ngrp = tile_cap / 32;
  a->parity = *calls & 1u;
  a->scan.tile = scan;
  a->scan.grp = nullptr;
  a->scan.grp_clear = nullptr;
  a->scan.clear_groups = 0;
  a->scan.gpre = nullptr;
  a->defer_next = nullptr;
  if (scan && s) {
    const uint32_t set = s->scan_calls++ & 1u;
    a->scan.grp = scan + tile_cap + set * ngrp;
    a->scan.grp_clear = scan + tile_cap + (1u - set) * ngrp;
    a->scan.clear_groups = s->prev_groups;
    s->prev_groups = groups_now;
    a->scan.gpre = scan + tile_cap + 2 * ngrp;
    a->defer_next = reinterpret_cast<uint32_t*>(scan + tile_cap + 3 * ngrp);
  } else if (scan) {
    a->scan.grp = scan + tile_cap;
    a->scan.grp_clear = a->scan.grp;
    a->scan.gpre = scan + tile_cap + ngrp;
    a->defer_next = reinterpret_cast<uint32_t*>(scan + tile_cap + 2 * ngrp);
  }
  a->scan.epoch = *calls & 0x7FFFFFFFu;
  a->scan.polls = g_scan_polls;
  a->scan.skip_tile = g_skip_tile;
  return FH_OK;
}

int sm_count();

// Scratch of the channel-wide three-sigma mode (grown on demand like the per-stream scratch).
int get_channel_scratch(StreamScratch* s, size_t planes, size_t channels) {
  if (planes > s->pn_cap) {
    size_t cap = s->pn_cap ? s->pn_cap : 65536;
    while (cap < planes) cap *= 2;
    if (s->plane_nout) {
      cudaDeviceSynchronize();
      cudaFree(s->plane_nout);
      s->plane_nout = nullptr;
      s->pn_cap = 0;
    }
    if (cudaMalloc(&s->plane_nout, cap * sizeof(uint32_t)) != cudaSuccess) return FH_ERR_CUDA;
    s->pn_cap = cap;
  }
  if (channels > s->chan_cap) {
    size_t cap = s->chan_cap ? s->chan_cap : 4096;
    while (cap < channels) cap *= 2;
    if (s->chan) {
      cudaDeviceSynchronize();
      cudaFree(s->chan);
      s->chan = nullptr;
      s->chan_cap = 0;
    }
    if (cudaMalloc(&s->chan, cap * sizeof(fh::ChanStat)) != cudaSuccess) return FH_ERR_CUDA;
    s->chan_cap = cap;
  }
  return FH_OK;
}

template <int DT>
int launch_channel_passes(const Plan& pl, const fh::ChannelArgs& ca, cudaStream_t stream) {
  const int sms = sm_count();
  if (sms < 1) return FH_ERR_CUDA;
  const uint64_t want = (pl.P + fh::kWarps - 1) / fh::kWarps, most = (uint64_t)sms * 8;
  const int grid = (int)(want < most ? want : most);
  if (cudaMemsetAsync(ca.chan, 0, pl.C * sizeof(fh::ChanStat), stream) != cudaSuccess) return FH_ERR_CUDA;
  fh::channel_pass<DT, 0><<<grid, fh::kThreads, 0, stream>>>(pl, ca);
  fh::channel_pass<DT, 1><<<grid, fh::kThreads, 0, stream>>>(pl, ca);
  fh::channel_pass<DT, 2><<<grid, fh::kThreads, 0, stream>>>(pl, ca);
  if (cudaGetLastError() != cudaSuccess) return FH_ERR_CUDA;
  g_launches.fetch_add(3);
  return FH_OK;
}

int sm_count() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 0;
  if (!g_sm_count[dev]) cudaDeviceGetAttribute(&g_sm_count[dev], cudaDevAttrMultiProcessorCount, dev);
  return g_sm_count[dev];
}

template <typename K>
int grid_for(K kernel, size_t smem, uint32_t ntiles, int* grid, int threads = fh::kThreads) {
  static std::map<std::tuple<int, const void*, size_t>, int> cache;  // guarded by g_mu; per device: the attribute is
  int dev = 0;                                                        // set once for every device that runs the kernel
  if (cudaGetDevice(&dev) != cudaSuccess) return FH_ERR_CUDA;
  const auto key = std::make_tuple(dev, (const void*)kernel, (smem << 12) | (size_t)threads);
  auto it = cache.find(key);
  int per_sm;
  if (it == cache.end()) {
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemLimit) != cudaSuccess)
      return FH_ERR_CUDA;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, threads, smem) != cudaSuccess)
      return FH_ERR_CUDA;
    if (per_sm < 1) return FH_ERR_UNSUPPORTED;
    cache[key] = per_sm;
  } else {
    per_sm = it->second;
  }
  const int sms = sm_count();
  if (sms < 1) return FH_ERR_CUDA;
  const uint64_t g = (uint64_t)per_sm * sms;
  *grid = (int)(ntiles < g ? ntiles : g);
  return FH_OK;
}

template <typename K>
int launch_on(K kernel, const Plan& pl, cudaStream_t stream, int* grid) {
  return grid_for(kernel, pl.sm_total, pl.ntiles, grid);
}

// Launch that may overlap the tail of the previous kernel on the stream: every kernel of this library
// passes dep_wait() before it touches global memory, so stream order is kept.
// Tiles a CTA requests at once when it starts: all its stages when every CTA of the grid gets that many, fewer
// when the tensor is small, so that the tiles spread over all CTAs before any CTA takes a second one.
Plan with_first_request(const Plan& pl, int grid, uint32_t least) {
  Plan q = pl;
  const uint32_t each = pl.ntiles / (uint32_t)(grid > 0 ? grid : 1);
  q.nstage = each < least ? least : (each > pl.nstage ? pl.nstage : each);
  return q;
}

template <typename K, typename A>
cudaError_t launch_dependent(K kernel, int grid, int threads, size_t smem, cudaStream_t stream, const Plan& pl,
                             const A& a) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)grid);
  cfg.blockDim = dim3((unsigned)threads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, pl, a);
}

template <int DT, int BITS>
int launch_generic_t(const Plan& pl, const fh::CompressArgs& a, cudaStream_t stream) {
  int grid = 0;
  int rc = grid_for(fh::compress_generic<DT, BITS>, pl.sm_total, pl.ntiles, &grid);
  if (rc != FH_OK) return rc;
  return launch_dependent(fh::compress_generic<DT, BITS>, grid, fh::kThreads, pl.sm_total, stream, pl, a) == cudaSuccess
             ? FH_OK : FH_ERR_CUDA;
}

template <int DT, bool SIGMA, int NT>
int launch_cta_t(const Plan& pl, const fh::CompressArgs& a, cudaStream_t stream) {
  int grid = 0;
  int rc = grid_for(fh::compress_cta<DT, SIGMA, NT>, pl.sm_total, pl.ntiles, &grid, NT);
  if (rc != FH_OK) return rc;
  return launch_dependent(fh::compress_cta<DT, SIGMA, NT>, grid, NT, pl.sm_total, stream, with_first_request(pl, grid, 2), a) == cudaSuccess
             ? FH_OK : FH_ERR_CUDA;
}

template <int DT, bool SIGMA, int NT, int G>
int launch_cta_regs_t(const Plan& pl, const fh::CompressArgs& a, cudaStream_t stream) {
  int grid = 0;
  if (pl.groups == (uint32_t)(NT * G)) {
    int rc = grid_for(fh::compress_cta_regs<DT, SIGMA, NT, G, true>, pl.sm_total, pl.ntiles, &grid, NT);
    if (rc != FH_OK) return rc;
    return launch_dependent(fh::compress_cta_regs<DT, SIGMA, NT, G, true>, grid, NT, pl.sm_total, stream,
                            with_first_request(pl, grid, 2), a) == cudaSuccess ? FH_OK : FH_ERR_CUDA;
  }
  int rc = grid_for(fh::compress_cta_regs<DT, SIGMA, NT, G, false>, pl.sm_total, pl.ntiles, &grid, NT);
  if (rc != FH_OK) return rc;
  return launch_dependent(fh::compress_cta_regs<DT, SIGMA, NT, G, false>, grid, NT, pl.sm_total, stream,
                          with_first_request(pl, grid, 2), a) == cudaSuccess ? FH_OK : FH_ERR_CUDA;
}

template <int DT, int SIGMA, int TT, bool FULLVEC>
int launch_warp_t(const Plan& pl, const fh::CompressArgs& a, cudaStream_t stream) {
  int grid = 0;
  int rc = grid_for(fh::compress_warp<DT, SIGMA, TT, FULLVEC>, pl.sm_total, pl.ntiles, &grid, fh::kWarpKernelThreads);
  if (rc != FH_OK) return rc;
  return launch_dependent(fh::compress_warp<DT, SIGMA, TT, FULLVEC>, grid, fh::kWarpKernelThreads, pl.sm_total, stream,
                          with_first_request(pl, grid, 1), a) == cudaSuccess ? FH_OK : FH_ERR_CUDA;
}

template <int DT, int SIGMA, bool FULLVEC>
int launch_warp_tt(const Plan& pl, const fh::CompressArgs& a, cudaStream_t stream) {
  switch (pl.team) {
    case 1: return launch_warp_t<DT, SIGMA, 1, FULLVEC>(pl, a, stream);
    case 2: return launch_warp_t<DT, SIGMA, 2, FULLVEC>(pl, a, stream);
    case 4: return launch_warp_t<DT, SIGMA, 4, FULLVEC>(pl, a, stream);
    case 8: return launch_warp_t<DT, SIGMA, 8, FULLVEC>(pl, a, stream);
    case 16: return launch_warp_t<DT, SIGMA, 16, FULLVEC>(pl, a, stream);
    case 32: return launch_warp_t<DT, SIGMA, 32, FULLVEC>(pl, a, stream);
  }
  return FH_ERR_UNSUPPORTED;
}

template <int DT, bool SIGMA>
int launch_cta_g(const Plan& pl, const Variant& v, const fh::CompressArgs& a, cudaStream_t stream);

template <int DT, int SIGMA>
int launch_fast_g(const Plan& pl, const Variant& v, const fh::CompressArgs& a, cudaStream_t stream) {
  if (!v.cta) {
    const bool fullvec = pl.plane_bytes % 16 == 0 && pl.HW % 4 == 0 && pl.groups == 8u * pl.team;
    return fullvec ? launch_warp_tt<DT, SIGMA, true>(pl, a, stream) : launch_warp_tt<DT, SIGMA, false>(pl, a, stream);
  }
  if constexpr (SIGMA == 2) return FH_ERR_UNSUPPORTED;  // (make_plan sends random rounding on large planes elsewhere)
  else return launch_cta_g<DT, SIGMA != 0>(pl, v, a, stream);
}

template <int DT, bool SIGMA>
int launch_cta_g(const Plan& pl, const Variant& v, const fh::CompressArgs& a, cudaStream_t stream) {
  if (v.G) {
    switch (pl.team * 16 + v.G) {
      case 128 * 16 + 7: return launch_cta_regs_t<DT, SIGMA, 128, 7>(pl, a, stream);
      case 128 * 16 + 8: return launch_cta_regs_t<DT, SIGMA, 128, 8>(pl, a, stream);
      case 256 * 16 + 7: return launch_cta_regs_t<DT, SIGMA, 256, 7>(pl, a, stream);
      case 256 * 16 + 8: return launch_cta_regs_t<DT, SIGMA, 256, 8>(pl, a, stream);
      case 448 * 16 + 7: return launch_cta_regs_t<DT, SIGMA, 448, 7>(pl, a, stream);
      case 512 * 16 + 8: return launch_cta_regs_t<DT, SIGMA, 512, 8>(pl, a, stream);
    }
    return FH_ERR_UNSUPPORTED;
  }
  switch (pl.team) {
    case 128: return launch_cta_t<DT, SIGMA, 128>(pl, a, stream);
    case 256: return launch_cta_t<DT, SIGMA, 256>(pl, a, stream);
    case 512: return launch_cta_t<DT, SIGMA, 512>(pl, a, stream);
  }
  return FH_ERR_UNSUPPORTED;
}

int launch_compress(const Plan& pl, const Variant& v, const fh::CompressArgs& a, cudaStream_t stream) {
  int rc;
  if (v.fast) {
    const int sigma = pl.mode == FH_SALIENT_AUTO ? (pl.rounding ? 2 : 1) : 0;
    if (pl.dtype == FH_F32)
      rc = sigma == 2 ? launch_fast_g<fh::kF32, 2>(pl, v, a, stream)
           : sigma    ? launch_fast_g<fh::kF32, 1>(pl, v, a, stream) : launch_fast_g<fh::kF32, 0>(pl, v, a, stream);
    else
      rc = sigma == 2 ? launch_fast_g<fh::kBF16, 2>(pl, v, a, stream)
           : sigma    ? launch_fast_g<fh::kBF16, 1>(pl, v, a, stream) : launch_fast_g<fh::kBF16, 0>(pl, v, a, stream);
  } else if (pl.dtype == FH_F32) {
    rc = pl.bits == 2   ? launch_generic_t<fh::kF32, 2>(pl, a, stream)
         : pl.bits == 4 ? launch_generic_t<fh::kF32, 4>(pl, a, stream)
                        : launch_generic_t<fh::kF32, 8>(pl, a, stream);
  } else {
    rc = pl.bits == 2   ? launch_generic_t<fh::kBF16, 2>(pl, a, stream)
         : pl.bits == 4 ? launch_generic_t<fh::kBF16, 4>(pl, a, stream)
                        : launch_generic_t<fh::kBF16, 8>(pl, a, stream);
  }
  if (rc != FH_OK) return rc;
  g_launches.fetch_add(1);
  return FH_OK;
}

// Largest prime <= n (n >= 2), or 1.
uint64_t prime_at_most(uint64_t n) {
  static std::map<uint64_t, uint64_t> cache;  // guarded by g_mu
  auto it = cache.find(n);
  if (it != cache.end()) return it->second;
  for (uint64_t c = n; c >= 2; --c) {
    bool prime = true;
    for (uint64_t f = 2; f * f <= c; ++f)
      if (c % f == 0) {
        prime = false;
        break;
      }
    if (prime) return cache[n] = c;
  }
  return cache[n] = 1;
}

template <int DT, int TT, bool DEFER = false>
int launch_decompress_t(const Plan& pl, const fh::DecompressArgs& a, cudaStream_t stream) {
  if (TT == 32 && !DEFER && pl.nblk >= fh::kDeferBlocks) return launch_decompress_t<DT, TT, TT == 32>(pl, a, stream);
  int grid = 0;
  int rc = grid_for(fh::decompress_kernel<DT, TT, DEFER>, pl.sm_total, pl.ntiles, &grid);
  if (rc != FH_OK) return rc;
  fh::DecompressArgs b = a;
  b.team_stride = prime_at_most((uint64_t)grid * (fh::kThreads / TT));
  if (launch_dependent(fh::decompress_kernel<DT, TT, DEFER>, grid, fh::kThreads, pl.sm_total, stream, pl, b) != cudaSuccess)
    return FH_ERR_CUDA;
  g_launches.fetch_add(1);
  return FH_OK;
}

// Planes of at most 128 groups: tiles of 256 / team planes restored in shared memory, one bulk store per tile.
template <int DT>
int launch_decompress_small(const Plan& pl0, const fh::DecompressArgs& a, cudaStream_t stream) {
  Plan pl = pl0;
  pl.ppt = fh::kThreads / pl.team;
  if (pl.ppt > pl.P) pl.ppt = (uint32_t)pl.P;
  pl.stage_bytes = (uint32_t)((pl.ppt * pl.plane_bytes + 127) & ~(uint64_t)127);
  pl.ntiles = (uint32_t)((pl.P + pl.ppt - 1) / pl.ppt);
  // two tile buffers, then per warp: scratch for a small plane's payload, or the general path's scratch
  const uint32_t pay = (uint32_t)A16(pl.plane_bytes) + 16u;
  if (pl.sal_stride < pay) pl.sal_stride = pay;
  pl.sm_total = 2u * pl.stage_bytes + (uint32_t)fh::kWarps * pl.sal_stride;
  if (pl.sm_total > kSmemLimit) return FH_ERR_UNSUPPORTED;
  int grid = 0;
  int rc = grid_for(fh::decompress_small<DT>, pl.sm_total, pl.ntiles, &grid);
  if (rc != FH_OK) return rc;
  if (launch_dependent(fh::decompress_small<DT>, grid, fh::kThreads, pl.sm_total, stream, pl, a) != cudaSuccess)
    return FH_ERR_CUDA;
  g_launches.fetch_add(1);
  return FH_OK;
}

template <int DT>
int launch_decompress(const Plan& pl, const fh::DecompressArgs& a, cudaStream_t stream) {
  if (pl.groups <= 128 && pl.P <= 0x7FFFFFFFull) return launch_decompress_small<DT>(pl, a, stream);
  switch (pl.team) {
    case 1: return launch_decompress_t<DT, 1>(pl, a, stream);
    case 2: return launch_decompress_t<DT, 2>(pl, a, stream);
    case 4: return launch_decompress_t<DT, 4>(pl, a, stream);
    case 8: return launch_decompress_t<DT, 8>(pl, a, stream);
    case 16: return launch_decompress_t<DT, 16>(pl, a, stream);
    case 32: return launch_decompress_t<DT, 32>(pl, a, stream);
  }
  return FH_ERR_UNSUPPORTED;
}

int enqueue_compress(const fh_tensor_desc* desc, const fh_params* params, const void* d_src, void* d_dst,
                     size_t capacity, const unsigned long long* d_off_in, unsigned long long* d_off_out,
                     unsigned long long* d_out2, cudaStream_t stream) {
  Plan pl;
  Variant v;
  int rc = make_plan(desc, params, true, &pl, &v);
  if (rc != FH_OK) return rc;
  std::lock_guard<std::mutex> lock(g_mu);
  StreamScratch* s = nullptr;
  rc = get_scratch(stream, pl.mode == FH_SALIENT_OFF ? 0 : pl.ntiles, &s);
  if (rc != FH_OK) return rc;
  fh::CompressArgs a = {};
  a.src = (const uint8_t*)d_src;
  a.dst_base = (uint8_t*)d_dst;
  a.capacity = capacity;
  a.d_off_in = d_off_in;
  a.d_off_out = d_off_out;
  a.out2 = d_out2;
  a.sc = s->sc;
  a.early_ticket = 1;
  rc = next_call(&s->calls, pl.mode == FH_SALIENT_OFF ? nullptr : s->scan, s->tile_cap, s, (pl.ntiles + 31u) / 32u, stream, &a);
  if (rc != FH_OK) return rc;
  a.chan_nout = nullptr;
  a.plane_nout = nullptr;
  if (pl.mode >= fh::kModeChannel) {  // statistics per channel over the batch, or over the tensor: three passes ahead of the streaming kernel
    rc = get_channel_scratch(s, pl.P, pl.C);
    if (rc != FH_OK) return rc;
    fh::ChannelArgs ca;
    ca.src = (const uint8_t*)d_src;
    ca.chan = s->chan;
    ca.plane_nout = s->plane_nout;
    ca.inv_nhw = 1.0 / ((double)(pl.mode == fh::kModeTensor ? pl.P : pl.N) * (double)pl.HW);
    rc = pl.dtype == FH_F32 ? launch_channel_passes<fh::kF32>(pl, ca, stream) : launch_channel_passes<fh::kBF16>(pl, ca, stream);
    if (rc != FH_OK) return rc;
    a.chan_nout = reinterpret_cast<const unsigned long long*>(s->chan) + 3;
    a.plane_nout = s->plane_nout;
  }
  return launch_compress(pl, v, a, stream);
}

int enqueue_decompress(const void* d_src, size_t src_bytes, const fh_tensor_desc* expect, void* d_dst,
                       const unsigned long long* d_off_in, unsigned long long* d_status, cudaStream_t stream) {
  Plan pl;
  int rc = make_plan(expect, nullptr, false, &pl, nullptr);
  if (rc != FH_OK) return rc;
  std::lock_guard<std::mutex> lock(g_mu);
  StreamScratch* s = nullptr;
  rc = get_scratch(stream, 0, &s);
  if (rc != FH_OK) return rc;
  fh::DecompressArgs a;
  a.src_base = (const uint8_t*)d_src;
  a.src_bytes = src_bytes;
  a.d_off_in = d_off_in;
  a.dst = (uint8_t*)d_dst;
  a.d_status = d_status;
  a.sc = s->sc;
  if (pl.dtype == FH_F32) return launch_decompress<fh::kF32>(pl, a, stream);
  return launch_decompress<fh::kBF16>(pl, a, stream);
}

bool misaligned(const void* p, size_t a) { return ((uintptr_t)p & (a - 1)) != 0; }

}  // namespace

extern "C" {

void fh_default_params(fh_params* p) {
  if (!p) return;
  p->bits = 2;
  p->salient_mode = FH_SALIENT_AUTO;
  p->rho_num = 1;
  p->rho_den = 32;
  p->block = 8;
  p->tau_num = 1;
  p->tau_den = 4;
  p->eps = 0.0625f;
  p->dense_bits = 8;
  p->rounding = 0;
  p->seed = 0;
  p->entropy = 0;
  p->reserved = 0;
}

int fh_version(void) { return 1; }

int fh_device_count(void) {
  int n = 0;
  if (cudaGetDeviceCount(&n) != cudaSuccess) return FH_ERR_CUDA;
  return n;
}

size_t fh_compressed_bytes(const fh_tensor_desc* desc, const fh_params* params, int which) {
  if (check_desc(desc) != FH_OK || check_params(params) != FH_OK) return 0;
  const size_t P = (size_t)desc->n * (size_t)desc->c, hw = (size_t)desc->h * (size_t)desc->w;
  if (which == 0) return 64 + P * (16 + A16(4 * ((hw * (size_t)params->bits + 31) / 32)));
  return 64 + P * (16 + A16(esize_of(desc->dtype) * hw));
}

int fh_compress(const fh_tensor_desc* desc, const fh_params* params, const void* d_src, void* d_dst,
                size_t dst_capacity, uint64_t* d_out2, void* stream) {
  int rc = check_desc(desc);
  if (rc != FH_OK) return rc;
  rc = check_params(params);
  if (rc != FH_OK) return rc;
  if (!d_src || !d_dst || misaligned(d_src, 16) || misaligned(d_dst, 16) || misaligned(d_out2, 8)) return FH_ERR_ARG;
  const size_t P = (size_t)desc->n * (size_t)desc->c;
  if (dst_capacity < 64 + 16 * P) return FH_ERR_CAPACITY;
  return enqueue_compress(desc, params, d_src, d_dst, dst_capacity, nullptr, nullptr,
                          (unsigned long long*)d_out2, (cudaStream_t)stream);
}

int fh_decompress(const void* d_src, size_t src_bytes, const fh_tensor_desc* expect, void* d_dst,
                  uint64_t* d_status, void* stream) {
  int rc = check_desc(expect);
  if (rc != FH_OK) return rc;
  if (!d_src || !d_dst || misaligned(d_src, 16) || misaligned(d_dst, 16) || misaligned(d_status, 8)) return FH_ERR_ARG;
  return enqueue_decompress(d_src, src_bytes, expect, d_dst, nullptr, (unsigned long long*)d_status,
                            (cudaStream_t)stream);
}

int fh_run_schedule(const fh_sched_entry* entries, int32_t count, const fh_params* params, void* d_arena,
                    size_t arena_bytes, fh_sched_report* report, void* stream_) {
  if (!entries || count < 0 || !report || !d_arena || misaligned(d_arena, 256)) return FH_ERR_ARG;
  int rc = check_params(params);
  if (rc != FH_OK) return rc;
  cudaStream_t stream = (cudaStream_t)stream_;
  std::memset(report, 0, sizeof(*report));
  std::vector<int> idx;
  for (int i = 0; i < count; ++i) {
    if (entries[i].action == FH_COMPRESS) {
      rc = check_desc(&entries[i].desc);
      if (rc != FH_OK) return rc;
      if (!entries[i].d_dense || !entries[i].d_restored || misaligned(entries[i].d_dense, 16) ||
          misaligned(entries[i].d_restored, 16))
        return FH_ERR_ARG;
      Plan pl;
      rc = make_plan(&entries[i].desc, params, true, &pl, nullptr);
      if (rc != FH_OK) return rc;
      idx.push_back(i);
      report->total_dense_bytes += pl.dense_bytes;
    } else if (entries[i].action != FH_KEEP && entries[i].action != FH_EVICT) {
      return FH_ERR_ARG;
    }
  }
  const size_t k = idx.size();
  if (k == 0) return FH_OK;
  // device words: offsets[k+1] | out2[2k] | decode status[k]
  const size_t words = (k + 1) + 2 * k + k;
  unsigned long long* d_words = nullptr;
  {
    std::lock_guard<std::mutex> lock(g_mu);
    StreamScratch* s = nullptr;
    rc = get_scratch(stream, 0, &s);
    if (rc != FH_OK) return rc;
    if (s->sched_cap < words) {
      if (s->sched) {
        cudaDeviceSynchronize();
        cudaFree(s->sched);
        s->sched = nullptr;
      }
      size_t cap = words < 1024 ? 1024 : 2 * words;
      if (cudaMalloc(&s->sched, cap * sizeof(unsigned long long)) != cudaSuccess) return FH_ERR_CUDA;
      s->sched_cap = cap;
    }
    d_words = s->sched;
  }
  unsigned long long* d_off = d_words;
  unsigned long long* d_out2 = d_words + (k + 1);
  unsigned long long* d_dst = d_out2 + 2 * k;
  cudaEvent_t e0, e1, e2;
  if (cudaEventCreate(&e0) != cudaSuccess || cudaEventCreate(&e1) != cudaSuccess ||
      cudaEventCreate(&e2) != cudaSuccess)
    return FH_ERR_CUDA;
  rc = FH_OK;
  if (cudaMemsetAsync(d_words, 0, words * sizeof(unsigned long long), stream) != cudaSuccess) rc = FH_ERR_CUDA;
  cudaEventRecord(e0, stream);
  for (size_t j = 0; j < k && rc == FH_OK; ++j) {  // forward order
    const fh_sched_entry& en = entries[idx[j]];
    rc = enqueue_compress(&en.desc, params, en.d_dense, d_arena, arena_bytes, d_off + j, d_off + j + 1,
                          d_out2 + 2 * j, stream);
  }
  cudaEventRecord(e1, stream);
  for (size_t j = k; j-- > 0 && rc == FH_OK;) {  // reverse order
    const fh_sched_entry& en = entries[idx[j]];
    rc = enqueue_decompress(d_arena, arena_bytes, &en.desc, en.d_restored, d_off + j, d_dst + j, stream);
  }
  cudaEventRecord(e2, stream);
  if (cudaStreamSynchronize(stream) != cudaSuccess) rc = rc == FH_OK ? FH_ERR_CUDA : rc;
  if (rc == FH_OK) {
    std::vector<unsigned long long> h(words);
    if (cudaMemcpy(h.data(), d_words, words * sizeof(unsigned long long), cudaMemcpyDeviceToHost) != cudaSuccess) {
      rc = FH_ERR_CUDA;
    } else {
      cudaEventElapsedTime(&report->ms_forward, e0, e1);
      cudaEventElapsedTime(&report->ms_backward, e1, e2);
      int status = FH_OK;
      uint64_t peak = 0;
      for (size_t j = 0; j < k; ++j) {
        const int cs = (int)(long long)h[(k + 1) + 2 * j + 1];
        if (status == FH_OK && cs != FH_OK) status = cs;
        if (cs == FH_OK) {
          report->total_packed_bytes += h[(k + 1) + 2 * j];
          if (h[j + 1] > peak) peak = h[j + 1];
        }
      }
      for (size_t j = 0; j < k; ++j) {
        const int ds = (int)(long long)h[(k + 1) + 2 * k + j];
        if (status == FH_OK && ds != FH_OK) status = ds;
      }
      report->peak_packed_bytes = peak;
      report->status = status;
    }
  }
  cudaEventDestroy(e0);
  cudaEventDestroy(e1);
  cudaEventDestroy(e2);
  return rc;
}

size_t fh_host_work_bytes(const fh_tensor_desc* desc, const fh_params* params) {
  fh_params def;
  fh_default_params(&def);
  const size_t worst = fh_compressed_bytes(desc, params ? params : &def, 1);
  if (!worst) return 0;
  const size_t dense = (size_t)desc->n * desc->c * desc->h * desc->w * esize_of(desc->dtype);
  return A256(dense) + 256 + A256(worst);
}

int fh_compress_host(const fh_tensor_desc* desc, const fh_params* params, const void* h_src, void* h_dst,
                     size_t dst_capacity, uint64_t* h_out2, void* d_work, size_t work_bytes, void* stream_) {
  int rc = check_desc(desc);
  if (rc != FH_OK) return rc;
  rc = check_params(params);
  if (rc != FH_OK) return rc;
  if (!h_src || !h_dst || !d_work || misaligned(d_work, 256)) return FH_ERR_ARG;
  if (work_bytes < fh_host_work_bytes(desc, params)) return FH_ERR_ARG;
  cudaStream_t stream = (cudaStream_t)stream_;
  const size_t dense = (size_t)desc->n * desc->c * desc->h * desc->w * esize_of(desc->dtype);
  const size_t worst = fh_compressed_bytes(desc, params, 1);
  uint8_t* d_dense = (uint8_t*)d_work;
  unsigned long long* d_out2 = (unsigned long long*)(d_dense + A256(dense));
  uint8_t* d_pack = (uint8_t*)d_out2 + 256;
  const size_t cap = dst_capacity < worst ? dst_capacity : worst;
  if (cudaMemcpyAsync(d_dense, h_src, dense, cudaMemcpyHostToDevice, stream) != cudaSuccess) return FH_ERR_CUDA;
  rc = fh_compress(desc, params, d_dense, d_pack, cap, (uint64_t*)d_out2, stream_);
  if (rc != FH_OK) return rc;
  unsigned long long out2[2] = {0, 0};
  if (cudaMemcpyAsync(out2, d_out2, 16, cudaMemcpyDeviceToHost, stream) != cudaSuccess) return FH_ERR_CUDA;
  if (cudaStreamSynchronize(stream) != cudaSuccess) return FH_ERR_CUDA;
  if (h_out2) {
    h_out2[0] = out2[0];
    h_out2[1] = out2[1];
  }
  const int st = (int)(long long)out2[1];
  if (st != FH_OK) return st;
  if (cudaMemcpyAsync(h_dst, d_pack, out2[0], cudaMemcpyDeviceToHost, stream) != cudaSuccess) return FH_ERR_CUDA;
  if (cudaStreamSynchronize(stream) != cudaSuccess) return FH_ERR_CUDA;
  return FH_OK;
}

int fh_decompress_host(const void* h_src, size_t src_bytes, const fh_tensor_desc* expect, void* h_dst,
                       uint64_t* h_status, void* d_work, size_t work_bytes, void* stream_) {
  int rc = check_desc(expect);
  if (rc != FH_OK) return rc;
  if (!h_src || !h_dst || !d_work || misaligned(d_work, 256)) return FH_ERR_ARG;
  const size_t need = fh_host_work_bytes(expect, nullptr);
  if (work_bytes < need) return FH_ERR_ARG;
  cudaStream_t stream = (cudaStream_t)stream_;
  const size_t dense = (size_t)expect->n * expect->c * expect->h * expect->w * esize_of(expect->dtype);
  uint8_t* d_dense = (uint8_t*)d_work;
  unsigned long long* d_st = (unsigned long long*)(d_dense + A256(dense));
  uint8_t* d_pack = (uint8_t*)d_st + 256;
  if (src_bytes > work_bytes - A256(dense) - 256) return FH_ERR_ARG;
  if (cudaMemcpyAsync(d_pack, h_src, src_bytes, cudaMemcpyHostToDevice, stream) != cudaSuccess) return FH_ERR_CUDA;
  rc = fh_decompress(d_pack, src_bytes, expect, d_dense, (uint64_t*)d_st, stream_);
  if (rc != FH_OK) return rc;
  unsigned long long st = 0;
  if (cudaMemcpyAsync(h_dst, d_dense, dense, cudaMemcpyDeviceToHost, stream) != cudaSuccess) return FH_ERR_CUDA;
  if (cudaMemcpyAsync(&st, d_st, 8, cudaMemcpyDeviceToHost, stream) != cudaSuccess) return FH_ERR_CUDA;
  if (cudaStreamSynchronize(stream) != cudaSuccess) return FH_ERR_CUDA;
  if (h_status) *h_status = st;
  return (int)(long long)st;
}

int fh_plan_measure(const fh_tensor_desc* descs, int32_t n, const fh_params* params, const void* const* d_dense,
                    void* d_work, size_t work_bytes, int32_t repeats, fh_plan_tensor* out, void* stream_) {
  if (!descs || !d_dense || !out || n < 0 || !d_work || misaligned(d_work, 256) || repeats < 1 || repeats > 1000)
    return FH_ERR_ARG;
  int rc = check_params(params);
  if (rc != FH_OK) return rc;
  for (int32_t i = 0; i < n; ++i) {
    rc = check_desc(&descs[i]);
    if (rc != FH_OK) return rc;
    if (!d_dense[i] || misaligned(d_dense[i], 16)) return FH_ERR_ARG;
    if (work_bytes < fh_host_work_bytes(&descs[i], params)) return FH_ERR_ARG;
  }
  cudaStream_t stream = (cudaStream_t)stream_;
  cudaEvent_t e0, e1, e2;
  if (cudaEventCreate(&e0) != cudaSuccess || cudaEventCreate(&e1) != cudaSuccess || cudaEventCreate(&e2) != cudaSuccess)
    return FH_ERR_CUDA;
  rc = FH_OK;
  for (int32_t i = 0; i < n && rc == FH_OK; ++i) {
    const fh_tensor_desc& d = descs[i];
    const size_t dense = (size_t)d.n * d.c * d.h * d.w * esize_of(d.dtype);
    const size_t worst = fh_compressed_bytes(&d, params, 1);
    // work buffer: restored copy | result words | container (the layout of the host-buffer entry points)
    uint8_t* d_rest = (uint8_t*)d_work;
    unsigned long long* d_words = (unsigned long long*)(d_rest + A256(dense));
    uint8_t* d_pack = (uint8_t*)d_words + 256;
    for (int pass = 0; pass < 2 && rc == FH_OK; ++pass) {  // pass 0: the untimed run
      const int reps = pass ? repeats : 1;
      cudaEventRecord(e0, stream);
      for (int r = 0; r < reps && rc == FH_OK; ++r)
        rc = fh_compress(&d, params, d_dense[i], d_pack, worst, (uint64_t*)d_words, stream_);
      cudaEventRecord(e1, stream);
      for (int r = 0; r < reps && rc == FH_OK; ++r)
        rc = fh_decompress(d_pack, worst, &d, d_rest, (uint64_t*)(d_words + 2), stream_);
      cudaEventRecord(e2, stream);
      if (cudaStreamSynchronize(stream) != cudaSuccess) rc = rc == FH_OK ? FH_ERR_CUDA : rc;
      if (rc != FH_OK) break;
      unsigned long long h[3] = {0, 0, 0};
      if (cudaMemcpy(h, d_words, sizeof(h), cudaMemcpyDeviceToHost) != cudaSuccess) {
        rc = FH_ERR_CUDA;
        break;
      }
      if ((int)(long long)h[1] != FH_OK) rc = (int)(long long)h[1];
      else if ((int)(long long)h[2] != FH_OK) rc = (int)(long long)h[2];
      if (pass && rc == FH_OK) {
        float ms_c = 0.0f, ms_d = 0.0f;
        cudaEventElapsedTime(&ms_c, e0, e1);
        cudaEventElapsedTime(&ms_d, e1, e2);
        out[i].bytes = dense;
        out[i].packed_bytes = h[0];
        out[i].t_compress = (double)ms_c * 1e-3 / repeats;
        out[i].t_decompress = (double)ms_d * 1e-3 / repeats;
      }
    }
  }
  cudaEventDestroy(e0);
  cudaEventDestroy(e1);
  cudaEventDestroy(e2);
  return rc;
}

// ---- allocation-free compress -----------------------------------------------------------------
// Scratch compiled into the device image: the counters (padded to 256 bytes), the placement scan's arrays
// and the tile links for FH_STATIC_MAX_PLANES tiles (a tile is at least one plane).  The name is a device symbol: host
// code must not pass it to a kernel, it asks the runtime for the symbol's device address instead (once per
// device).
static __device__ __align__(256) unsigned char g_static_scratch[FH_STATIC_SCRATCH_BYTES];
static_assert(sizeof(fh::Scratch) <= fh::kScratchHeadBytes, "static scratch layout");
static_assert(FH_STATIC_SCRATCH_BYTES ==
                  fh::kScratchHeadBytes + 8 * (FH_STATIC_MAX_PLANES + 2 * (FH_STATIC_MAX_PLANES / 32)) + 4 * FH_STATIC_MAX_PLANES,
              "static scratch layout");

static std::mutex g_static_mu;
static unsigned char* g_static_ptr[64] = {nullptr};
static uint32_t g_static_calls[64] = {0};

int fh_compress_static(const fh_tensor_desc* desc, const fh_params* params, const void* d_src, void* d_dst,
                       size_t dst_capacity, uint64_t* d_out2, void* stream_) {
  int rc = check_desc(desc);
  if (rc != FH_OK) return rc;
  rc = check_params(params);
  if (rc != FH_OK) return rc;
  if (!d_src || !d_dst || misaligned(d_src, 16) || misaligned(d_dst, 16) || misaligned(d_out2, 8)) return FH_ERR_ARG;
  const size_t P = (size_t)desc->n * (size_t)desc->c;
  if (dst_capacity < 64 + 16 * P) return FH_ERR_CAPACITY;
  Plan pl;
  Variant v;
  rc = make_plan(desc, params, true, &pl, &v);
  if (rc != FH_OK) return rc;
  if (pl.P > FH_STATIC_MAX_PLANES) return FH_ERR_UNSUPPORTED;  // beyond the fixed arrays
  if (pl.mode >= fh::kModeChannel) return FH_ERR_UNSUPPORTED;  // its statistics need scratch the fixed array does not hold
  cudaStream_t stream = (cudaStream_t)stream_;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return FH_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_static_mu);
  if (!g_static_ptr[dev]) {  // set-up, once per device, with that device current
    unsigned char* p = nullptr;
    if (cudaGetSymbolAddress((void**)&p, g_static_scratch) != cudaSuccess || !p) return FH_ERR_CUDA;
    g_static_ptr[dev] = p;
  }
  unsigned char* base = g_static_ptr[dev];
  // The array keeps the last call's contents.  The counters and the scan's group sums must start at zero;
  // the scan's other words carry the number of the call that wrote them and need no clearing.
  unsigned long long* scan = reinterpret_cast<unsigned long long*>(base + fh::kScratchHeadBytes);
  const size_t cap = FH_STATIC_MAX_PLANES;
  if (cudaMemsetAsync(base, 0, fh::kScratchHeadBytes, stream) != cudaSuccess) return FH_ERR_CUDA;
  if (cudaMemsetAsync(scan + cap, 0, (cap / 32) * sizeof(unsigned long long), stream) != cudaSuccess) return FH_ERR_CUDA;
  fh::CompressArgs a = {};
  a.src = (const uint8_t*)d_src;
  a.dst_base = (uint8_t*)d_dst;
  a.capacity = dst_capacity;
  a.d_off_in = nullptr;
  a.d_off_out = nullptr;
  a.out2 = (unsigned long long*)d_out2;
  a.sc = reinterpret_cast<fh::Scratch*>(base);
  a.early_ticket = 0;  // the counters are cleared by the memset just enqueued: nothing may touch them before it
  rc = next_call(&g_static_calls[dev], scan, cap, nullptr, 0, stream, &a);
  if (rc != FH_OK) return rc;
  a.chan_nout = nullptr;
  a.plane_nout = nullptr;
  std::lock_guard<std::mutex> lock2(g_mu);  // the launch helpers keep their occupancy cache under g_mu
  return launch_compress(pl, v, a, stream);
}

int fh_debug_set(int what, uint64_t value) {
  std::lock_guard<std::mutex> lock(g_mu);
  if (what == FH_DEBUG_WAIT_POLLS) {
    if (value < 1 || value > 0xFFFFFFFFull) return FH_ERR_ARG;
    g_scan_polls = (uint32_t)value;
  } else if (what == FH_DEBUG_SILENT_TILE) {
    g_skip_tile = value > 0xFFFFFFFEull ? 0xFFFFFFFFu : (uint32_t)value;
  } else {
    return FH_ERR_ARG;
  }
  return FH_OK;
}

uint64_t fh_kernel_launches(void) { return g_launches.load(); }

void fh_shutdown(void) {
  std::lock_guard<std::mutex> lock(g_mu);
  int cur = 0;
  cudaGetDevice(&cur);
  for (auto& kv : g_scratch) {
    cudaSetDevice(kv.first.first);
    cudaDeviceSynchronize();
    if (kv.second.sc) cudaFree(kv.second.sc);
    if (kv.second.scan) cudaFree(kv.second.scan);
    if (kv.second.plane_nout) cudaFree(kv.second.plane_nout);
    if (kv.second.chan) cudaFree(kv.second.chan);
    if (kv.second.sched) cudaFree(kv.second.sched);
  }
  g_scratch.clear();
  cudaSetDevice(cur);
}

}  // extern "C"
