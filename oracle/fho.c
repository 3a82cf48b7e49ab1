/*
 * fho.c -- CPU oracle for Channel-wise Mix Compression (FedHybrid, arXiv 2510.11400, Section 4.4.1).
 *
 * THIS IS TEST INFRASTRUCTURE.  It is a plain, slow, step-by-step statement of what the codec
 * computes, written from the paper, and exists only so that tests, the smoke check and the
 * benchmark's CPU-baseline leg can compare the CUDA library against it.  It shares no code with
 * the CUDA library and must never be used as a fallback for it.
 *
 * The paper fixes the structure of the method (Section 4.4.1):
 *   - outliers are found with the three-sigma rule and channels are classified into outlier-rich
 *     ("salient") and normal;
 *   - normal channels are quantised;
 *   - a salient channel feature map (h x w) is split, through a non-zero mask that is average-pooled
 *     with an n x n window and compared with a threshold tau, into sparse blocks (stored in
 *     Compressed Sparse Row form) and dense blocks (Lorenzo prediction, Eq. 7-8, residuals inside an
 *     error bound eps are quantised, Eq. 9, unpredictable values are kept verbatim, predictions use
 *     decompressed values);
 *   - decompression rebuilds floating-point values from the codes and the prediction.
 * It fixes none of the constants (bit-width, n, tau, eps, ...), the rounding, or a byte layout.
 * Those are parameters here, and every such choice is listed next to the code that takes it.
 *
 * Parity unpinned: the parameter values themselves (bits, rho, block, tau, eps, code width), the
 * per-plane scope of mu and sigma, the rounding mode and the container layout are choices the
 * paper does not fix; tests pin the arithmetic given those choices, not the choices.
 *
 * Arithmetic rules: every float operation below is a single IEEE-754 operation with round to
 * nearest even (compile with -ffp-contract=off, no -ffast-math); fmaf() and fma-free products are
 * written out where the distinction matters.  No flush-to-zero.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define FHO_OK 0
#define FHO_ERR_ARG (-1)
#define FHO_ERR_UNSUPPORTED (-2)
#define FHO_ERR_CAPACITY (-3)
#define FHO_ERR_NONFINITE (-4)
#define FHO_ERR_CORRUPT (-5)

#define FHO_F32 0
#define FHO_BF16 1

#define CLS_NORMAL 0u
#define CLS_SALIENT 1u
#define CLS_RAW 2u

#define MODE_AUTO 0
#define MODE_OFF 1
#define MODE_ALL 2
#define MODE_CHANNEL 3 /* three-sigma rule with mu, sigma and the class taken per channel over the whole batch */
#define MODE_TENSOR 4  /* three-sigma thresholds from mu, sigma of the whole tensor; the class per plane */

typedef struct {
  int32_t dtype;
  int32_t n, c, h, w;
  uint64_t tensor_id;
} fho_desc;

typedef struct {
  int32_t bits;
  int32_t salient_mode;
  int32_t rho_num, rho_den;
  int32_t block;
  int32_t tau_num, tau_den;
  float eps;
  int32_t dense_bits;
  int32_t rounding;
  uint64_t seed;
  int32_t entropy; /* 0: fixed 8-bit residual codes; 1: Huffman stage on the dense-block codes */
  int32_t reserved;
} fho_params;

static int g_threads = 1;

void fho_set_threads(int t) { g_threads = t < 1 ? 1 : t; }
int fho_get_threads(void) { return g_threads; }
int fho_max_threads(void) {
#ifdef _OPENMP
  return omp_get_num_procs();
#else
  return 1;
#endif
}

static size_t a4(size_t x) { return (x + 3) & ~(size_t)3; }
static size_t a16(size_t x) { return (x + 15) & ~(size_t)15; }
static size_t esize(int dtype) { return dtype == FHO_F32 ? 4 : 2; }

static float bf16_to_f32(uint16_t h) {
  uint32_t u = (uint32_t)h << 16;
  float f;
  memcpy(&f, &u, 4);
  return f;
}

/* fp32 -> bf16, round half to even (finite inputs). */
static uint16_t f32_to_bf16(float f) {
  uint32_t u;
  memcpy(&u, &f, 4);
  uint32_t r = ((u >> 16) & 1u) + 0x7FFFu;
  return (uint16_t)((u + r) >> 16);
}

static int check_args(const fho_desc* d, const fho_params* p) {
  if (!d || !p) return FHO_ERR_ARG;
  if (d->dtype != FHO_F32 && d->dtype != FHO_BF16) return FHO_ERR_ARG;
  if (d->n < 1 || d->c < 1 || d->h < 1 || d->w < 1) return FHO_ERR_ARG;
  if (d->w > 65535) return FHO_ERR_UNSUPPORTED;
  if (p->bits != 2 && p->bits != 4 && p->bits != 8) return FHO_ERR_UNSUPPORTED;
  if (p->salient_mode < 0 || p->salient_mode > 4) return FHO_ERR_ARG;
  if (p->rho_num < 0 || p->rho_den < 1 || p->rho_num > 65535 || p->rho_den > 65535) return FHO_ERR_ARG;
  if (p->tau_num < 0 || p->tau_den < 1 || p->tau_num > 65535 || p->tau_den > 65535) return FHO_ERR_ARG;
  if (p->block != 8) return FHO_ERR_UNSUPPORTED;
  if (p->dense_bits != 8) return FHO_ERR_UNSUPPORTED;
  if (p->rounding != 0 && p->rounding != 1) return FHO_ERR_UNSUPPORTED;
  if (p->entropy != 0 && p->entropy != 1) return FHO_ERR_UNSUPPORTED;
  if (!(p->eps >= 1e-30f) || !(p->eps <= 1e30f)) return FHO_ERR_ARG; /* keeps 2*eps and 1/(2*eps) finite */
  return FHO_OK;
}

/* ------------------------------------------------------------------------------------------
 * Sizes.  Container (a layout choice; the paper gives none), little-endian:
 *   [0,64) header | [64, 64+16P) plane table | P fixed slots of npay bytes | overflow region.
 * Every plane owns one slot, npay = A16(4*ceil(HW*bits/32)) bytes, at a closed-form offset.  A
 * normal plane's codes fill its slot.  The payload of a salient or raw plane is laid through its
 * slot first and continues, if longer, in the overflow region (plane order, each part padded to
 * 16 bytes); its table entry holds the offset of that continuation (0 if there is none).
 * ------------------------------------------------------------------------------------------ */
static size_t normal_payload(size_t hw, int bits) { return 4 * ((hw * (size_t)bits + 31) / 32); }

size_t fho_compressed_bytes(const fho_desc* d, const fho_params* p, int which) {
  if (check_args(d, p) != FHO_OK) return 0;
  size_t P = (size_t)d->n * (size_t)d->c, hw = (size_t)d->h * (size_t)d->w;
  if (which == 0) return 64 + P * (16 + a16(normal_payload(hw, p->bits)));
  return 64 + P * (16 + a16(esize(d->dtype) * hw));
}

/* ------------------------------------------------------------------------------------------
 * Three-sigma statistics (Section 4.4.1: outliers are found with the empirical three-sigma rule).
 * mu and sigma are the mean and the population standard deviation of the elements in scope (a plane;
 * a channel over the batch; the whole tensor).
 *
 * The paper does not say how the moments are accumulated.  Two requirements shape the reading taken
 * here: the rule must hold on data with an offset (|mu| much larger than sigma, e.g. a biased
 * pre-activation), so the moments are taken of the distances d = x - lo from the smallest element
 * and never of x itself; and the result must not depend on the order of summation (so that a parallel
 * implementation reproduces it bit for bit), so the sums run over integers:
 *   lo = min x, hi = max x, range = hi - lo (fp32), e = floor(log2(range))
 *   range == 0 (constant data): no outliers.
 *   e < -40 or e > 60 (range below 2^-40 or from 2^61 up): the rule is not applied, no outliers are
 *       counted -- inside [-40, 60] neither d*d nor the scalings below can overflow or underflow.
 *   d_i = x_i - lo (fp32, >= 0); elements are taken in consecutive groups of 4 per plane, the last
 *       group of a plane padded with d = 0; per group, in fp32:
 *     s_g = (d0 + d2) + (d1 + d3),   q_g = fma(d2, d2, d0*d0) + fma(d3, d3, d1*d1)
 *       (elements 0,1 and 2,3 of a group are treated as two pairs that are combined position by position)
 *     i_s = round_half_even(s_g * 2^(18-e)),  i_q = round_half_even(q_g * 2^(16-2e))   (exact products,
 *       integers below 2^22: the sums resolve 2^-18 of the range and 2^-16 of its square per group)
 *   I_s = sum i_s, I_q = sum i_q                                          (exact integers, any order)
 *   r = 1/count (fp64);  m1 = (I_s * 2^(e-18)) * r;  m2 = (I_q * 2^(2e-16)) * r            (fp64)
 *   var = max(m2 - m1*m1, 0) (fp64);  m_f = (float)m1;  sigma_f = sqrtf((float)var)
 *   D_hi = fma(3, sigma_f, m_f),  D_lo = fma(-3, sigma_f, m_f)                             (fp32)
 *   element i is an outlier iff d_i > D_hi or d_i < D_lo                           (fp32 compares)
 * i.e. x_i > mu + 3 sigma or x_i < mu - 3 sigma with mu = lo + m1, written in distances from lo.
 * ------------------------------------------------------------------------------------------ */
typedef struct {
  float lo, range;
  int applies;    /* 0: constant data or range outside [2^-40, 2^61): no outliers are counted */
  int e;
  int64_t Is, Iq; /* the integer sums */
  float d_lo, d_hi;
} sigma_stats;

/* round_half_even(v * 2^k) as an integer; the product of a float with a power of two is exact in fp64 */
static int64_t fixed_point(float v, int k) { return (int64_t)nearbyint(ldexp((double)v, k)); }

/* Integer sums of the distances from lo of n_planes planes of hw elements (plane n at x + n*stride). */
static void sigma_sums(const float* x, int64_t n_planes, int64_t stride, int64_t hw, sigma_stats* st) {
  float lo = x[0], hi = x[0];
  for (int64_t n = 0; n < n_planes; ++n)
    for (int64_t i = 0; i < hw; ++i) {
      float v = x[n * stride + i];
      if (v < lo) lo = v;
      if (v > hi) hi = v;
    }
  memset(st, 0, sizeof(*st));
  st->lo = lo;
  st->range = hi - lo;
  if (!(st->range > 0.0f)) return;
  st->e = ilogbf(st->range);
  if (st->e < -40 || st->e > 60) return;
  st->applies = 1;
  for (int64_t n = 0; n < n_planes; ++n)
    for (int64_t g = 0; g < hw; g += 4) {
      float d[4] = {0.f, 0.f, 0.f, 0.f};
      for (int k = 0; k < 4 && g + k < hw; ++k) d[k] = x[n * stride + g + k] - lo;
      float s02 = d[0] + d[2], s13 = d[1] + d[3];
      float sg = s02 + s13;
      float p0 = d[0] * d[0], p1 = d[1] * d[1];
      float q02 = fmaf(d[2], d[2], p0), q13 = fmaf(d[3], d[3], p1);
      float qg = q02 + q13;
      st->Is += fixed_point(sg, 18 - st->e);
      st->Iq += fixed_point(qg, 16 - 2 * st->e);
    }
}

static void sigma_thresholds(sigma_stats* st, int64_t count) {
  double S = ldexp((double)st->Is, st->e - 18), Q = ldexp((double)st->Iq, 2 * st->e - 16);
  double r = 1.0 / (double)count;
  double m1 = S * r;
  double m2 = Q * r;
  double m1sq = m1 * m1;
  double var = m2 - m1sq;
  if (!(var > 0.0)) var = 0.0;
  float m_f = (float)m1;
  float sigma_f = sqrtf((float)var);
  st->d_hi = fmaf(3.0f, sigma_f, m_f);
  st->d_lo = fmaf(-3.0f, sigma_f, m_f);
}

static int64_t sigma_count(const float* x, int64_t hw, const sigma_stats* st) {
  if (!st->applies) return 0;
  int64_t cnt = 0;
  for (int64_t i = 0; i < hw; ++i) {
    float d = x[i] - st->lo;
    if (d > st->d_hi || d < st->d_lo) ++cnt;
  }
  return cnt;
}

/* Exposed for the tests: the integer sums of one plane and the exponent they are scaled by. */
void fho_plane_sums(const float* x, int64_t hw, int64_t* Is_out, int64_t* Iq_out, int32_t* e_out,
                    int32_t* applies_out) {
  sigma_stats st;
  sigma_sums(x, 1, hw, hw, &st);
  *Is_out = st.Is;
  *Iq_out = st.Iq;
  *e_out = st.e;
  *applies_out = st.applies;
}

/* One plane: lo, the thresholds as distances from lo, and the outlier count. */
void fho_plane_sigma(const float* x, int64_t hw, float* lo_out, float* d_lo, float* d_hi, int64_t* n_out) {
  sigma_stats st;
  sigma_sums(x, 1, hw, hw, &st);
  if (st.applies) sigma_thresholds(&st, hw);
  *lo_out = st.lo;
  *d_lo = st.d_lo;
  *d_hi = st.d_hi;
  *n_out = sigma_count(x, hw, &st);
}

/* ------------------------------------------------------------------------------------------
 * The other readings of "classify channels" (Section 4.4.1): a channel is channel c of the layer, i.e.
 * the N planes (n, c) of the batch together (salient_mode CHANNEL), or what counts as an outlier is
 * fixed once for the whole tensor (TENSOR).  lo, range, the integer sums (every plane cut into its own
 * groups of four) and the divisor then run over all planes in scope.
 * x: n_planes planes, each hw elements, plane n at x + n*stride.
 * ------------------------------------------------------------------------------------------ */
static void scope_sigma(const float* x, int64_t n_planes, int64_t stride, int64_t hw, sigma_stats* st) {
  sigma_sums(x, n_planes, stride, hw, st);
  if (st->applies) sigma_thresholds(st, n_planes * hw);
}

void fho_channel_sigma(const float* x, int64_t n_planes, int64_t stride, int64_t hw, float* lo_out, float* d_lo,
                       float* d_hi, int64_t* n_out) {
  sigma_stats st;
  scope_sigma(x, n_planes, stride, hw, &st);
  int64_t cnt = 0;
  for (int64_t n = 0; n < n_planes; ++n) cnt += sigma_count(x + n * stride, hw, &st);
  *lo_out = st.lo;
  *d_lo = st.d_lo;
  *d_hi = st.d_hi;
  *n_out = cnt;
}

/* ------------------------------------------------------------------------------------------
 * Normal planes "undergo quantization" (Section 4.4.1).  Uniform affine quantiser with one group
 * per plane and the plane's min and max as statistics:
 *   L = 2^b - 1, range = hi - lo, inv = L / range, scale = range / L          (fp32)
 *   range == 0 or inv not finite  ->  inv = scale = 0
 *   q = clamp(round_half_even((x - lo) * inv), 0, L)
 * where (x - lo) is an fp32 subtraction and its product with inv is taken exactly before the
 * rounding to an integer (the fp64 product of two fp32 numbers is exact).
 * ------------------------------------------------------------------------------------------ */
void fho_quant_params(float lo, float hi, int bits, float* inv, float* scale) {
  float L = (float)((1 << bits) - 1);
  float range = hi - lo;
  float i = L / range, s = range / L;
  if (range == 0.0f || !isfinite(i)) {
    i = 0.0f;
    s = 0.0f;
  }
  *inv = i;
  *scale = s;
}

uint32_t fho_quant_code(float x, float lo, float inv, int bits) {
  int L = (1 << bits) - 1;
  float d = x - lo;
  double t = (double)d * (double)inv; /* exact */
  double r = nearbyint(t);            /* default rounding mode: half to even */
  if (r < 0.0) r = 0.0;
  if (r > (double)L) r = (double)L;
  return (uint32_t)r;
}

float fho_dequant(uint32_t q, float lo, float scale) { return fmaf((float)q, scale, lo); }

/* ------------------------------------------------------------------------------------------
 * Random rounding of normal planes (rounding = 1).  The paper is silent on the rounding of its
 * quantiser; the quantisers it builds on (its Section 2.3 citations) round stochastically so that the
 * restored value is unbiased.  Here, with 24-bit integers so that nothing depends on floating-point
 * rounding of a sum:
 *   t = (x - lo) * inv            (fp32 subtraction, fp32 product; t >= 0)
 *   n = floor(t),  f = t - n      (exact)
 *   q = min(n + [ floor(f * 2^24) + r >= 2^24 ], L),   r = a uniform 24-bit integer
 * so the code goes up with probability floor(f * 2^24) / 2^24 and a position that is already an integer
 * never moves.
 *
 * u comes from the counter-based generator Philox-4x32 with 10 rounds (Salmon, Moraes, Dror, Shaw,
 * "Parallel random numbers: as easy as 1, 2, 3", SC'11): multipliers 0xD2511F53 and 0xCD9E8D57, key
 * increments 0x9E3779B9 and 0xBB67AE85.  One call per group of four consecutive elements of a plane:
 *   key     = (seed low word, seed high word)
 *   counter = (group index within the plane, plane index, tensor_id low word, tensor_id high word)
 * and element e of the group takes output word e: r = word >> 8.
 * So the draw of an element depends on (seed, tensor id, element position) and on nothing else.
 * ------------------------------------------------------------------------------------------ */
void fho_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
  uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3], k0 = key[0], k1 = key[1];
  for (int r = 0; r < 10; ++r) {
    uint64_t p0 = (uint64_t)0xD2511F53u * c0, p1 = (uint64_t)0xCD9E8D57u * c2;
    uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0, n1 = (uint32_t)p1;
    uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1, n3 = (uint32_t)p0;
    c0 = n0;
    c1 = n1;
    c2 = n2;
    c3 = n3;
    k0 += 0x9E3779B9u;
    k1 += 0xBB67AE85u;
  }
  out[0] = c0;
  out[1] = c1;
  out[2] = c2;
  out[3] = c3;
}

uint32_t fho_quant_code_random(float x, float lo, float inv, int bits, uint32_t word) {
  uint32_t L = (1u << bits) - 1u;
  float d = x - lo;
  float t = d * inv;
  float nf = floorf(t);
  float f = t - nf;                               /* exact, 0 <= f < 1 */
  uint32_t fi = (uint32_t)(f * 16777216.0f);      /* floor(f * 2^24): the scaling is exact */
  uint32_t up = (fi + (word >> 8)) >> 24;         /* 1 iff fi + r >= 2^24 */
  uint32_t n = nf >= (float)L ? L : (uint32_t)nf; /* t may exceed L by rounding */
  uint32_t q = n + up;
  return q > L ? L : q;
}

/* Pre-quantisation for dense blocks: k = round_half_even(fp32(x * inv2e)), |k| capped at 2^24. */
static int32_t dense_k(float x, float inv2e, int* big) {
  float kf = rintf(x * inv2e);
  *big = fabsf(kf) >= 16777216.0f;
  if (kf > 16777216.0f) kf = 16777216.0f;
  if (kf < -16777216.0f) kf = -16777216.0f;
  return (int32_t)kf;
}

static void put_u32(uint8_t* p, uint32_t v) { memcpy(p, &v, 4); }
static void put_u16(uint8_t* p, uint16_t v) { memcpy(p, &v, 2); }
static uint32_t get_u32(const uint8_t* p) {
  uint32_t v;
  memcpy(&v, p, 4);
  return v;
}
static uint16_t get_u16(const uint8_t* p) {
  uint16_t v;
  memcpy(&v, p, 2);
  return v;
}

/* ------------------------------------------------------------------------------------------
 * Huffman stage (Section 4.4.1: "a Huffman tree is constructed from the quantization array for
 * encoding"; decompression "involves Huffman decoding").  The quantization array is the array of
 * residual code bytes of an outlier-rich plane's dense blocks (64 per block; 0 marks a verbatim value).
 * The paper gives no alphabet, scope, tie-break or stream format; here:
 *   scope      one code per plane, built from that plane's own code bytes (a plane's payload then
 *              depends on nothing but the plane, like everything else in the container)
 *   tree       the classical construction: the two nodes of least weight are merged until one is left.
 *              Nodes are ordered by (weight, id) with id = symbol for a leaf and 256 + order of creation
 *              for a merged node; symbols that do not occur get no code; a single symbol gets length 1
 *   code       canonical: symbols sorted by (length, symbol) take consecutive code values, first code of
 *              a length = (last code of the previous length + 1) << (difference of the lengths)
 *   stream     every dense block's 64 symbols form a chunk of its own that starts on a byte boundary
 *              (chunks decode independently); a code's bits go most significant first, bytes fill from bit 7
 *   section    u8 len(symbol 0) | u8 smin | u8 smax | u8 0 | u8 len(s) for s = smin..smax (pad to 4)
 *              | u8 bytes of chunk b, b = 0..n_dense-1 (pad to 4) | the chunks, concatenated (pad to 4)
 *              where [smin, smax] is the range of symbols 1..255 that occur (1, 1 if none does)
 * The section replaces the plain 64 * n_dense code bytes only if it is smaller; word 3 of the payload
 * header then holds the section's size in bytes, and 0 otherwise.  Code lengths stay below 25: a plane has
 * fewer than 2^17 code bytes and a Huffman code of depth d needs at least Fibonacci(d + 2) of them; a chunk
 * therefore has at most 64 * 24 / 8 = 192 bytes.
 * ------------------------------------------------------------------------------------------ */
void fho_huffman_lengths(const uint32_t hist[256], uint8_t len[256]) {
  /* leaves sorted by (weight, symbol); merged nodes are born in non-decreasing weight order, so two queues
   * (leaves, merged nodes) always have the least node at one of their heads */
  int leaf[256], n = 0;
  for (int sym = 0; sym < 256; ++sym) {
    len[sym] = 0;
    if (hist[sym]) leaf[n++] = sym;
  }
  if (n == 0) return;
  if (n == 1) {
    len[leaf[0]] = 1;
    return;
  }
  for (int i = 1; i < n; ++i) { /* insertion sort: stable, so equal weights stay in symbol order */
    int v = leaf[i], j = i;
    while (j > 0 && hist[leaf[j - 1]] > hist[v]) {
      leaf[j] = leaf[j - 1];
      --j;
    }
    leaf[j] = v;
  }
  uint64_t w[512];   /* weight of node id: ids 0..255 leaves (by symbol), 256.. merged nodes */
  int parent[512];
  for (int sym = 0; sym < 256; ++sym) w[sym] = hist[sym];
  int li = 0, mi = 256, mn = 256; /* head of the leaf queue, head and end of the merged-node queue */
  while ((n - li) + (mn - mi) > 1) {
    int pick[2];
    for (int k = 0; k < 2; ++k) {
      int take_leaf;
      if (li >= n) take_leaf = 0;
      else if (mi >= mn) take_leaf = 1;
      else take_leaf = w[leaf[li]] <= w[mi]; /* equal weights: the leaf has the smaller id */
      pick[k] = take_leaf ? leaf[li++] : mi++;
    }
    w[mn] = w[pick[0]] + w[pick[1]];
    parent[pick[0]] = parent[pick[1]] = mn;
    ++mn;
  }
  int root = mn - 1;
  for (int i = 0; i < n; ++i) {
    int d = 0;
    for (int v = leaf[i]; v != root; v = parent[v]) ++d;
    len[leaf[i]] = (uint8_t)d;
  }
}

/* Canonical code values (right-aligned in `code`) from the lengths alone. */
void fho_canonical_codes(const uint8_t len[256], uint32_t code[256]) {
  uint32_t next = 0;
  int prev = 0;
  for (int l = 1; l <= 32; ++l)
    for (int sym = 0; sym < 256; ++sym)
      if (len[sym] == l) {
        next <<= (l - prev);
        prev = l;
        code[sym] = next++;
      }
}

/* The entropy-coded section for `n_dense` blocks of 64 code bytes; returns its size (a multiple of 4). */
static size_t huffman_section(const uint8_t* codes, uint32_t n_dense, uint8_t** out) {
  uint32_t hist[256] = {0};
  for (size_t i = 0; i < (size_t)n_dense * 64; ++i) ++hist[codes[i]];
  uint8_t len[256];
  uint32_t code[256] = {0};
  fho_huffman_lengths(hist, len);
  for (int sym = 0; sym < 256; ++sym)
    if (len[sym] > 24) { /* cannot happen for planes this library accepts (see above); then the stage is not used */
      *out = NULL;
      return (size_t)-1;
    }
  fho_canonical_codes(len, code);
  int smin = 1, smax = 1, any = 0;
  for (int sym = 1; sym < 256; ++sym)
    if (len[sym]) {
      if (!any) smin = sym;
      smax = sym;
      any = 1;
    }
  size_t nlens = (size_t)(smax - smin + 1);
  size_t head = 4 + a4(nlens) + a4(n_dense);
  uint8_t* buf = (uint8_t*)calloc(head + (size_t)n_dense * 64 * 4 + 8, 1);
  buf[0] = len[0];
  buf[1] = (uint8_t)smin;
  buf[2] = (uint8_t)smax;
  for (int sym = smin; sym <= smax; ++sym) buf[4 + (sym - smin)] = len[sym];
  uint8_t* chunk_bytes = buf + 4 + a4(nlens);
  size_t pos = head; /* byte position of the next chunk */
  for (uint32_t b = 0; b < n_dense; ++b) {
    size_t bit = 0; /* bits written into this chunk */
    for (int i = 0; i < 64; ++i) {
      uint8_t sym = codes[(size_t)b * 64 + i];
      for (int k = len[sym] - 1; k >= 0; --k) { /* most significant bit first */
        if ((code[sym] >> k) & 1u) buf[pos + bit / 8] |= (uint8_t)(0x80u >> (bit % 8));
        ++bit;
      }
    }
    size_t nbytes = (bit + 7) / 8;
    chunk_bytes[b] = (uint8_t)nbytes;
    pos += nbytes;
  }
  *out = buf;
  return a4(pos);
}

/* Decodes the section at `sec` (at most `avail` readable bytes) into n_dense * 64 code bytes; returns the
 * section's size, or 0 if it is inconsistent. */
static size_t huffman_decode_section(const uint8_t* sec, size_t avail, uint32_t n_dense, uint8_t* codes) {
  if (avail < 4) return 0;
  int smin = sec[1], smax = sec[2];
  if (smin < 1 || smax < smin) return 0;
  size_t nlens = (size_t)(smax - smin + 1);
  size_t head = 4 + a4(nlens) + a4(n_dense);
  if (avail < head) return 0;
  uint8_t len[256] = {0};
  len[0] = sec[0];
  for (int sym = smin; sym <= smax; ++sym) len[sym] = sec[4 + (sym - smin)];
  uint64_t kraft = 0; /* in units of 2^-32 */
  int nsym = 0;
  for (int sym = 0; sym < 256; ++sym) {
    if (len[sym] > 32) return 0;
    if (len[sym]) {
      kraft += 1ull << (32 - len[sym]);
      ++nsym;
    }
  }
  if (nsym == 0 || kraft > (1ull << 32) || (nsym > 1 && kraft != (1ull << 32))) return 0;
  uint32_t code[256] = {0};
  fho_canonical_codes(len, code);
  const uint8_t* chunk_bytes = sec + 4 + a4(nlens);
  size_t pos = head;
  for (uint32_t b = 0; b < n_dense; ++b) {
    size_t nbytes = chunk_bytes[b];
    if (pos + nbytes > avail) return 0;
    size_t bit = 0;
    for (int i = 0; i < 64; ++i) {
      uint32_t acc = 0;
      int l = 0, found = -1;
      while (found < 0) {
        if (bit >= nbytes * 8 || l >= 32) return 0;
        acc = (acc << 1) | ((sec[pos + bit / 8] >> (7 - bit % 8)) & 1u);
        ++bit;
        ++l;
        for (int sym = 0; sym < 256; ++sym)
          if (len[sym] == l && code[sym] == acc) found = sym;
      }
      codes[(size_t)b * 64 + i] = (uint8_t)found;
    }
    pos += nbytes;
  }
  return a4(pos);
}

typedef struct {
  uint32_t cls;
  uint32_t n_out;
  float lo, scale;
  uint8_t* payload; /* malloc'd, zero padded to a16(size) */
  size_t size;      /* payload bytes before padding */
  size_t bytes;     /* a16(size) */
  int status;
} plane_result;

/* Salient plane (Section 4.4.1, block-wise path).  Returns payload size before a16 padding, or
 * 0 when buf == NULL is used for sizing only.  Layout:
 *   u32 nnz_s | u32 n_dense | u32 n_out_d | u32 0 | bitmap ceil(nblk/32) u32 (bit=1: dense)
 *   | row_ptr (H+1) u32 | col nnz_s u16 (pad 4) | val nnz_s elems (pad 4)
 *   | codes n_dense*64 bytes | outliers n_out_d elems (pad 4)
 */
static size_t encode_salient(const float* x, const uint8_t* raw, int dtype, int H, int W,
                             const fho_params* p, uint8_t** out_buf) {
  const int B = 8;
  size_t e = esize(dtype);
  int nby = (H + B - 1) / B, nbx = (W + B - 1) / B, nblk = nby * nbx;
  /* mask -> pooled non-zero count per block -> block class.
   * The paper average-pools the 0/1 mask with an n x n window and compares with tau; the mean of
   * the mask over a window is nnz/n^2 (divisor n^2 also at ragged edges: zero padding), so the
   * comparison is nnz/n^2 >= tau, done in integers as nnz * tau_den >= tau_num * n^2. */
  uint8_t* dense = (uint8_t*)calloc((size_t)nblk, 1);
  uint32_t n_dense = 0;
  for (int by = 0; by < nby; ++by)
    for (int bx = 0; bx < nbx; ++bx) {
      int nnz = 0;
      for (int i = 0; i < B; ++i)
        for (int j = 0; j < B; ++j) {
          int y = by * B + i, xx = bx * B + j;
          if (y < H && xx < W && x[(size_t)y * W + xx] != 0.0f) ++nnz;
        }
      int is_dense = (int64_t)nnz * p->tau_den >= (int64_t)p->tau_num * (B * B);
      dense[by * nbx + bx] = (uint8_t)is_dense;
      n_dense += (uint32_t)is_dense;
    }
  /* CSR over non-zeros that lie in sparse blocks. */
  uint32_t* row_ptr = (uint32_t*)calloc((size_t)H + 1, 4);
  uint32_t nnz_s = 0;
  for (int y = 0; y < H; ++y) {
    row_ptr[y] = nnz_s;
    for (int xx = 0; xx < W; ++xx)
      if (x[(size_t)y * W + xx] != 0.0f && !dense[(y / B) * nbx + xx / B]) ++nnz_s;
  }
  row_ptr[H] = nnz_s;
  /* Dense blocks: Lorenzo residuals on pre-quantised integers (Eq. 7-9).
   * First-order 2-D Lorenzo predictor: pred = up + left - upleft (coefficients sum to one);
   * neighbours outside the block count as 0.  Because prediction runs on the integers k, the
   * values the predictor sees are exactly the decoder's reconstruction 2*eps*k. */
  float two_eps = 2.0f * p->eps;
  float inv2e = 1.0f / two_eps;
  uint8_t* codes = (uint8_t*)malloc((size_t)n_dense * 64 + 1);
  uint8_t* outl = (uint8_t*)malloc((size_t)n_dense * 64 * e + 1);
  uint32_t n_out_d = 0, di = 0;
  for (int blk = 0; blk < nblk; ++blk) {
    if (!dense[blk]) continue;
    int by = blk / nbx, bx = blk % nbx;
    int32_t k[8][8];
    int big[8][8], inpl[8][8];
    for (int i = 0; i < B; ++i)
      for (int j = 0; j < B; ++j) {
        int y = by * B + i, xx = bx * B + j;
        inpl[i][j] = (y < H && xx < W);
        float v = inpl[i][j] ? x[(size_t)y * W + xx] : 0.0f;
        k[i][j] = dense_k(v, inv2e, &big[i][j]);
      }
    for (int i = 0; i < B; ++i)
      for (int j = 0; j < B; ++j) {
        uint8_t code;
        if (!inpl[i][j]) {
          code = 128;
        } else {
          int64_t up = i > 0 ? k[i - 1][j] : 0;
          int64_t left = j > 0 ? k[i][j - 1] : 0;
          int64_t ul = (i > 0 && j > 0) ? k[i - 1][j - 1] : 0;
          int64_t delta = (int64_t)k[i][j] - (up + left - ul);
          if (big[i][j] || delta > 127 || delta < -127) {
            code = 0;
            size_t idx = (size_t)(by * B + i) * W + (size_t)(bx * B + j);
            memcpy(outl + (size_t)n_out_d * e, raw + idx * e, e);
            ++n_out_d;
          } else {
            code = (uint8_t)(delta + 128);
          }
        }
        codes[(size_t)di * 64 + i * 8 + j] = code;
      }
    ++di;
  }
  size_t nbm = ((size_t)nblk + 31) / 32;
  /* the dense blocks' code bytes as they are, or through the Huffman stage when that is smaller */
  uint8_t* section = NULL;
  size_t dense_bytes = 64 * (size_t)n_dense;
  int coded = 0;
  if (p->entropy == 1 && n_dense > 0) {
    size_t sz = huffman_section(codes, n_dense, &section);
    if (sz < dense_bytes) {
      dense_bytes = sz;
      coded = 1;
    }
  }
  size_t size = 16 + 4 * nbm + 4 * ((size_t)H + 1) + a4(2 * (size_t)nnz_s) + a4(e * nnz_s) + dense_bytes +
                a4(e * n_out_d);
  uint8_t* buf = (uint8_t*)calloc(a16(size), 1);
  uint8_t* q = buf;
  put_u32(q, nnz_s);
  put_u32(q + 4, n_dense);
  put_u32(q + 8, n_out_d);
  put_u32(q + 12, coded ? (uint32_t)dense_bytes : 0u); /* size of the Huffman-coded section, 0: plain code bytes */
  q += 16;
  for (int blk = 0; blk < nblk; ++blk)
    if (dense[blk]) {
      uint32_t wv = get_u32(q + 4 * (blk / 32));
      put_u32(q + 4 * (blk / 32), wv | (1u << (blk % 32)));
    }
  q += 4 * nbm;
  for (int y = 0; y <= H; ++y) put_u32(q + 4 * y, row_ptr[y]);
  q += 4 * ((size_t)H + 1);
  uint8_t* colp = q;
  uint8_t* valp = q + a4(2 * (size_t)nnz_s);
  uint32_t t = 0;
  for (int y = 0; y < H; ++y)
    for (int xx = 0; xx < W; ++xx)
      if (x[(size_t)y * W + xx] != 0.0f && !dense[(y / B) * nbx + xx / B]) {
        put_u16(colp + 2 * (size_t)t, (uint16_t)xx);
        memcpy(valp + e * t, raw + ((size_t)y * W + xx) * e, e);
        ++t;
      }
  q = valp + a4(e * nnz_s);
  memcpy(q, coded ? section : codes, dense_bytes);
  q += dense_bytes;
  memcpy(q, outl, (size_t)n_out_d * e);
  free(section);
  free(dense);
  free(row_ptr);
  free(codes);
  free(outl);
  *out_buf = buf;
  return size;
}

/* ch: for MODE_CHANNEL the channel's statistics and whether the channel is outlier-rich; for MODE_TENSOR the
 * tensor's {t_lo, t_hi} (a plane is then outlier-rich by its own count against these); NULL otherwise */
typedef struct {
  sigma_stats st;
  int salient;
} channel_info;

static void encode_plane(const uint8_t* raw, int dtype, int H, int W, const fho_params* p,
                         uint64_t plane_index, uint64_t tensor_id, const channel_info* ch, plane_result* r) {
  size_t hw = (size_t)H * W, e = esize(dtype);
  float* x = (float*)malloc(hw * sizeof(float));
  for (size_t i = 0; i < hw; ++i)
    x[i] = dtype == FHO_F32 ? ((const float*)raw)[i] : bf16_to_f32(((const uint16_t*)raw)[i]);
  memset(r, 0, sizeof(*r));
  float lo = x[0], hi = x[0];
  int finite = 1;
  for (size_t i = 0; i < hw; ++i) {
    if (!isfinite(x[i])) finite = 0;
    if (x[i] < lo) lo = x[i];
    if (x[i] > hi) hi = x[i];
  }
  if (!finite || !isfinite(hi - lo)) {
    r->status = FHO_ERR_NONFINITE;
    free(x);
    return;
  }
  uint32_t cls = CLS_NORMAL, n_out = 0;
  if (p->salient_mode == MODE_AUTO) {
    float plo, dlo, dhi;
    int64_t cnt;
    fho_plane_sigma(x, (int64_t)hw, &plo, &dlo, &dhi, &cnt);
    n_out = (uint32_t)cnt;
    /* outlier-rich when the three-sigma outliers exceed the fraction rho of the plane */
    if ((int64_t)cnt * p->rho_den > (int64_t)p->rho_num * (int64_t)hw) cls = CLS_SALIENT;
  } else if (p->salient_mode == MODE_ALL) {
    cls = CLS_SALIENT;
  } else if (p->salient_mode == MODE_CHANNEL) {
    n_out = (uint32_t)sigma_count(x, (int64_t)hw, &ch->st);
    if (ch->salient) cls = CLS_SALIENT;
  } else if (p->salient_mode == MODE_TENSOR) {
    /* Third reading of the three-sigma rule (Section 4.4.1): what counts as an outlier is fixed once for the
     * layer's whole activation tensor (mu and sigma over all N*C*HW elements, the same integer sums with lo and range
     * of the tensor and r = 1/(N*C*HW)); a plane is outlier-rich when its own share of
     * such outliers exceeds rho. */
    n_out = (uint32_t)sigma_count(x, (int64_t)hw, &ch->st);
    if ((int64_t)n_out * p->rho_den > (int64_t)p->rho_num * (int64_t)hw) cls = CLS_SALIENT;
  }
  if (cls == CLS_SALIENT) {
    uint8_t* buf = NULL;
    size_t size = encode_salient(x, raw, dtype, H, W, p, &buf);
    if (a16(size) >= a16(e * hw)) { /* no gain: keep the plane verbatim */
      free(buf);
      cls = CLS_RAW;
      r->size = e * hw;
      r->bytes = a16(e * hw);
      r->payload = (uint8_t*)calloc(r->bytes, 1);
      memcpy(r->payload, raw, e * hw);
    } else {
      r->payload = buf;
      r->size = size;
      r->bytes = a16(size);
    }
  } else {
    float inv, scale;
    fho_quant_params(lo, hi, p->bits, &inv, &scale);
    size_t size = normal_payload(hw, p->bits);
    r->size = size;
    r->bytes = a16(size);
    r->payload = (uint8_t*)calloc(r->bytes, 1);
    for (size_t i = 0; i < hw; ++i) {
      uint32_t qv;
      if (p->rounding == 1) {
        uint32_t ctr[4] = {(uint32_t)(i / 4), (uint32_t)plane_index, (uint32_t)tensor_id, (uint32_t)(tensor_id >> 32)};
        uint32_t key[2] = {(uint32_t)p->seed, (uint32_t)(p->seed >> 32)}, rnd[4];
        fho_philox4x32_10(ctr, key, rnd);
        qv = fho_quant_code_random(x[i], lo, inv, p->bits, rnd[i % 4]);
      } else {
        qv = fho_quant_code(x[i], lo, inv, p->bits);
      }
      size_t bit = i * (size_t)p->bits;
      uint32_t wv = get_u32(r->payload + 4 * (bit / 32));
      put_u32(r->payload + 4 * (bit / 32), wv | (qv << (bit % 32)));
    }
    r->lo = lo;
    r->scale = scale;
  }
  r->cls = cls;
  r->n_out = n_out;
  free(x);
}

/* Compress a whole tensor.  out2[0] = total bytes needed, out2[1] = status (as uint64 of the
 * negative code, 0 when OK).  Returns the status. */
int fho_compress(const fho_desc* d, const fho_params* p, const void* src, void* dst,
                 size_t dst_capacity, uint64_t* out2) {
  int st = check_args(d, p);
  if (st != FHO_OK) return st;
  if (!src || !dst) return FHO_ERR_ARG;
  size_t P = (size_t)d->n * d->c, hw = (size_t)d->h * d->w, e = esize(d->dtype);
  plane_result* res = (plane_result*)calloc(P, sizeof(plane_result));
  channel_info* chan = NULL;
  if (p->salient_mode == MODE_CHANNEL) {
    chan = (channel_info*)calloc((size_t)d->c, sizeof(channel_info));
    int bad = 0;
#ifdef _OPENMP
#pragma omp parallel for schedule(dynamic, 1) num_threads(g_threads)
#endif
    for (int64_t c = 0; c < (int64_t)d->c; ++c) {
      float* x = (float*)malloc((size_t)d->n * hw * sizeof(float));
      int finite = 1;
      for (int64_t n = 0; n < (int64_t)d->n; ++n)
        for (size_t i = 0; i < hw; ++i) {
          size_t idx = ((size_t)n * d->c + (size_t)c) * hw + i;
          float v = d->dtype == FHO_F32 ? ((const float*)src)[idx] : bf16_to_f32(((const uint16_t*)src)[idx]);
          if (!isfinite(v)) finite = 0;
          x[(size_t)n * hw + i] = v;
        }
      if (!finite) {
        bad = 1; /* reported per plane below */
      } else {
        scope_sigma(x, d->n, (int64_t)hw, (int64_t)hw, &chan[c].st);
        int64_t cnt = 0;
        for (int64_t n = 0; n < (int64_t)d->n; ++n) cnt += sigma_count(x + (size_t)n * hw, (int64_t)hw, &chan[c].st);
        chan[c].salient = cnt * (int64_t)p->rho_den > (int64_t)p->rho_num * (int64_t)d->n * (int64_t)hw;
      }
      free(x);
    }
    (void)bad;
  } else if (p->salient_mode == MODE_TENSOR) {
    chan = (channel_info*)calloc(1, sizeof(channel_info));
    float* x = (float*)malloc(P * hw * sizeof(float));
    int finite = 1;
    for (size_t i = 0; i < P * hw; ++i) {
      x[i] = d->dtype == FHO_F32 ? ((const float*)src)[i] : bf16_to_f32(((const uint16_t*)src)[i]);
      if (!isfinite(x[i])) finite = 0;
    }
    if (finite) /* otherwise the planes report the error below */
      scope_sigma(x, (int64_t)P, (int64_t)hw, (int64_t)hw, &chan[0].st);
    free(x);
  }
#ifdef _OPENMP
#pragma omp parallel for schedule(dynamic, 8) num_threads(g_threads)
#endif
  for (int64_t pl = 0; pl < (int64_t)P; ++pl)
    encode_plane((const uint8_t*)src + (size_t)pl * hw * e, d->dtype, d->h, d->w, p, (uint64_t)pl, d->tensor_id,
                 chan ? &chan[p->salient_mode == MODE_TENSOR ? 0 : pl % d->c] : NULL, &res[pl]);
  free(chan);
  const size_t npay = a16(normal_payload(hw, p->bits));
  size_t total = 64 + 16 * P + P * npay;
  uint32_t n_sal = 0, n_raw = 0;
  for (size_t pl = 0; pl < P; ++pl) {
    if (res[pl].status != FHO_OK) st = res[pl].status;
    if (res[pl].bytes > npay) total += res[pl].bytes - npay; /* continuation in the overflow region */
    n_sal += res[pl].cls == CLS_SALIENT;
    n_raw += res[pl].cls == CLS_RAW;
  }
  if (st == FHO_OK && total > dst_capacity) st = FHO_ERR_CAPACITY;
  if (st == FHO_OK && total / 16 > 0xFFFFFFFFull) st = FHO_ERR_UNSUPPORTED;
  if (st == FHO_OK) {
    uint8_t* o = (uint8_t*)dst;
    memset(o, 0, 64);
    put_u32(o + 0, 0x31434846u); /* 'F','H','C','1' */
    put_u16(o + 4, (uint16_t)(p->entropy == 1 ? 2 : 1)); /* version 2: payloads may carry Huffman-coded sections */
    o[6] = (uint8_t)d->dtype;
    o[7] = (uint8_t)p->bits;
    put_u32(o + 8, (uint32_t)d->n);
    put_u32(o + 12, (uint32_t)d->c);
    put_u32(o + 16, (uint32_t)d->h);
    put_u32(o + 20, (uint32_t)d->w);
    o[24] = (uint8_t)p->block;
    o[25] = (uint8_t)p->dense_bits;
    o[26] = (uint8_t)p->rounding;
    o[27] = (uint8_t)p->salient_mode;
    put_u16(o + 28, (uint16_t)p->rho_num);
    put_u16(o + 30, (uint16_t)p->rho_den);
    put_u16(o + 32, (uint16_t)p->tau_num);
    put_u16(o + 34, (uint16_t)p->tau_den);
    memcpy(o + 36, &p->eps, 4);
    put_u32(o + 40, n_sal);
    put_u32(o + 44, n_raw);
    memcpy(o + 48, &d->tensor_id, 8);
    uint64_t tb = total;
    memcpy(o + 56, &tb, 8);
    size_t slots = 64 + 16 * P, ovf = slots + P * npay;
    memset(o + slots, 0, P * npay);
    for (size_t pl = 0; pl < P; ++pl) {
      uint8_t* te = o + 64 + 16 * pl;
      uint8_t* slot = o + slots + pl * npay;
      size_t in_slot = res[pl].bytes < npay ? res[pl].bytes : npay;
      memcpy(slot, res[pl].payload, in_slot);
      uint32_t off16 = (uint32_t)((slots + pl * npay) / 16);
      if (res[pl].cls != CLS_NORMAL) {
        off16 = 0;
        if (res[pl].bytes > npay) {
          off16 = (uint32_t)(ovf / 16);
          memcpy(o + ovf, res[pl].payload + npay, res[pl].bytes - npay);
          ovf += res[pl].bytes - npay;
        }
      }
      put_u32(te, off16);
      put_u32(te + 4, res[pl].cls | (res[pl].n_out << 2));
      memcpy(te + 8, &res[pl].lo, 4);
      memcpy(te + 12, &res[pl].scale, 4);
    }
  }
  for (size_t pl = 0; pl < P; ++pl) free(res[pl].payload);
  free(res);
  if (out2) {
    out2[0] = total;
    out2[1] = (uint64_t)(int64_t)st;
  }
  return st;
}

static void store_elem(uint8_t* dst, int dtype, size_t i, float v) {
  if (dtype == FHO_F32)
    memcpy(dst + 4 * i, &v, 4);
  else {
    uint16_t h = f32_to_bf16(v);
    memcpy(dst + 2 * i, &h, 2);
  }
}

static int decode_salient_payload(const uint8_t* pay, int dtype, int H, int W, float eps, uint32_t nnz_s,
                                  uint32_t n_dense, uint32_t n_out_d, uint32_t coded_bytes, uint8_t* out);

static int decode_plane(const uint8_t* src, size_t src_bytes, size_t pl, size_t P, int dtype, int H,
                        int W, int bits, float eps, int version, uint8_t* out) {
  size_t hw = (size_t)H * W, e = esize(dtype);
  const uint8_t* te = src + 64 + 16 * pl;
  size_t off = (size_t)get_u32(te) * 16;
  uint32_t meta = get_u32(te + 4);
  uint32_t cls = meta & 3u;
  float lo, scale;
  memcpy(&lo, te + 8, 4);
  memcpy(&scale, te + 12, 4);
  const size_t npay = a16(normal_payload(hw, bits));
  const size_t slots = 64 + 16 * P, ovf0 = slots + P * npay;
  if (ovf0 > src_bytes) return FHO_ERR_CORRUPT;
  const uint8_t* slot = src + slots + pl * npay;
  if (cls == CLS_NORMAL) {
    if (off != slots + pl * npay) return FHO_ERR_CORRUPT;
    uint32_t mask = (1u << bits) - 1u;
    for (size_t i = 0; i < hw; ++i) {
      size_t bit = i * (size_t)bits;
      uint32_t q = (get_u32(slot + 4 * (bit / 32)) >> (bit % 32)) & mask;
      store_elem(out, dtype, i, fho_dequant(q, lo, scale));
    }
    return FHO_OK;
  }
  if (cls != CLS_SALIENT && cls != CLS_RAW) return FHO_ERR_CORRUPT;
  const int B = 8;
  int nby = (H + B - 1) / B, nbx = (W + B - 1) / B, nblk = nby * nbx;
  size_t nbm = ((size_t)nblk + 31) / 32;
  uint32_t nnz_s = 0, n_dense = 0, n_out_d = 0, coded_bytes = 0;
  size_t size;
  if (cls == CLS_RAW) {
    size = e * hw;
  } else {
    nnz_s = get_u32(slot);
    n_dense = get_u32(slot + 4);
    n_out_d = get_u32(slot + 8);
    coded_bytes = get_u32(slot + 12);
    if (nnz_s > hw || n_dense > (uint32_t)nblk || n_out_d > hw) return FHO_ERR_CORRUPT;
    if (coded_bytes && (version != 2 || coded_bytes % 4 != 0 || coded_bytes >= 64 * (size_t)n_dense)) return FHO_ERR_CORRUPT;
    size = 16 + 4 * nbm + 4 * ((size_t)H + 1) + a4(2 * (size_t)nnz_s) + a4(e * nnz_s) +
           (coded_bytes ? coded_bytes : 64 * (size_t)n_dense) + a4(e * n_out_d);
  }
  /* the payload runs through the slot and continues at `off` in the overflow region */
  uint8_t* pay = (uint8_t*)calloc(a16(size) + 16, 1);
  memcpy(pay, slot, size < npay ? size : npay);
  if (size > npay) {
    if (off < ovf0 || off > src_bytes || size - npay > src_bytes - off) {
      free(pay);
      return FHO_ERR_CORRUPT;
    }
    memcpy(pay + npay, src + off, size - npay);
  }
  if (cls == CLS_RAW) {
    memcpy(out, pay, e * hw);
    free(pay);
    return FHO_OK;
  }
  int rc = decode_salient_payload(pay, dtype, H, W, eps, nnz_s, n_dense, n_out_d, coded_bytes, out);
  free(pay);
  return rc;
}

static int decode_salient_payload(const uint8_t* pay, int dtype, int H, int W, float eps, uint32_t nnz_s,
                                  uint32_t n_dense, uint32_t n_out_d, uint32_t coded_bytes, uint8_t* out) {
  const int B = 8;
  size_t hw = (size_t)H * W, e = esize(dtype);
  int nby = (H + B - 1) / B, nbx = (W + B - 1) / B, nblk = nby * nbx;
  size_t nbm = ((size_t)nblk + 31) / 32;
  const uint8_t* bm = pay + 16;
  const uint8_t* rp = bm + 4 * nbm;
  const uint8_t* colp = rp + 4 * ((size_t)H + 1);
  const uint8_t* valp = colp + a4(2 * (size_t)nnz_s);
  const uint8_t* codes = valp + a4(e * nnz_s);
  const uint8_t* outl = codes + (coded_bytes ? coded_bytes : 64 * (size_t)n_dense);
  uint8_t* plain = NULL;
  if (coded_bytes) { /* Huffman decoding first (Section 4.4.1, "Decompression involves Huffman decoding") */
    plain = (uint8_t*)malloc((size_t)n_dense * 64 + 1);
    if (huffman_decode_section(codes, coded_bytes, n_dense, plain) != coded_bytes) {
      free(plain);
      return FHO_ERR_CORRUPT;
    }
    codes = plain;
  }
  memset(out, 0, e * hw);
  for (int y = 0; y < H; ++y) {
    uint32_t a = get_u32(rp + 4 * y), b = get_u32(rp + 4 * (y + 1));
    if (a > b || b > nnz_s) { free(plain); return FHO_ERR_CORRUPT; }
    for (uint32_t t = a; t < b; ++t) {
      uint32_t col = get_u16(colp + 2 * (size_t)t);
      if ((int)col >= W) { free(plain); return FHO_ERR_CORRUPT; }
      memcpy(out + ((size_t)y * W + col) * e, valp + e * t, e);
    }
  }
  float two_eps = 2.0f * eps;
  float inv2e = 1.0f / two_eps;
  uint32_t di = 0, oi = 0;
  for (int blk = 0; blk < nblk; ++blk) {
    if (!((get_u32(bm + 4 * (blk / 32)) >> (blk % 32)) & 1u)) continue;
    if (di >= n_dense) { free(plain); return FHO_ERR_CORRUPT; }
    int by = blk / nbx, bx = blk % nbx;
    int64_t k[8][8];
    for (int i = 0; i < B; ++i)
      for (int j = 0; j < B; ++j) {
        int y = by * B + i, xx = bx * B + j;
        int64_t up = i > 0 ? k[i - 1][j] : 0;
        int64_t left = j > 0 ? k[i][j - 1] : 0;
        int64_t ul = (i > 0 && j > 0) ? k[i - 1][j - 1] : 0;
        int64_t pred = up + left - ul;
        uint8_t code = codes[(size_t)di * 64 + i * 8 + j];
        if (!(y < H && xx < W)) {
          k[i][j] = pred; /* padding: never read by an in-plane element */
          continue;
        }
        size_t idx = (size_t)y * W + xx;
        if (code == 0) {
          if (oi >= n_out_d) { free(plain); return FHO_ERR_CORRUPT; }
          memcpy(out + idx * e, outl + (size_t)oi * e, e);
          float v;
          if (dtype == FHO_F32)
            memcpy(&v, outl + (size_t)oi * e, 4);
          else
            v = bf16_to_f32(get_u16(outl + (size_t)oi * e));
          int big;
          k[i][j] = dense_k(v, inv2e, &big);
          ++oi;
        } else {
          k[i][j] = pred + ((int64_t)code - 128);
          float kv = (float)k[i][j];
          store_elem(out, dtype, idx, kv * two_eps);
        }
      }
    ++di;
  }
  free(plain);
  return FHO_OK;
}

int fho_decompress(const void* src, size_t src_bytes, const fho_desc* expect, void* dst) {
  if (!src || !dst || !expect) return FHO_ERR_ARG;
  const uint8_t* s = (const uint8_t*)src;
  if (src_bytes < 64) return FHO_ERR_CORRUPT;
  if (get_u32(s) != 0x31434846u || (get_u16(s + 4) != 1 && get_u16(s + 4) != 2)) return FHO_ERR_CORRUPT;
  int version = get_u16(s + 4);
  int dtype = s[6], bits = s[7];
  uint32_t N = get_u32(s + 8), C = get_u32(s + 12), H = get_u32(s + 16), W = get_u32(s + 20);
  if ((int)N != expect->n || (int)C != expect->c || (int)H != expect->h || (int)W != expect->w ||
      dtype != expect->dtype)
    return FHO_ERR_CORRUPT;
  if (bits != 2 && bits != 4 && bits != 8) return FHO_ERR_CORRUPT;
  if (s[24] != 8 || s[25] != 8) return FHO_ERR_CORRUPT;
  float eps;
  memcpy(&eps, s + 36, 4);
  uint64_t tb;
  memcpy(&tb, s + 56, 8);
  size_t P = (size_t)N * C, hw = (size_t)H * W, e = esize(dtype);
  if (tb > src_bytes || tb < 64 + 16 * P + P * a16(normal_payload(hw, bits))) return FHO_ERR_CORRUPT;
  int st = FHO_OK;
#ifdef _OPENMP
#pragma omp parallel for schedule(dynamic, 8) num_threads(g_threads)
#endif
  for (int64_t pl = 0; pl < (int64_t)P; ++pl) {
    int r = decode_plane(s, (size_t)tb, (size_t)pl, P, dtype, (int)H, (int)W, bits, eps, version,
                         (uint8_t*)dst + (size_t)pl * hw * e);
    if (r != FHO_OK) {
#ifdef _OPENMP
#pragma omp critical
#endif
      st = r;
    }
  }
  return st;
}
