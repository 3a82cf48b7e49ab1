/*
 * fh.h -- C ABI of the B200 activation codec (Channel-wise Mix Compression, FedHybrid,
 * arXiv 2510.11400, Section 4.4.1).
 *
 * Local training compresses the activations its execution plan marks "compress" in the forward
 * pass and restores them when the backward pass needs them (Section 3.2; Algorithm 1, functions
 * Compute and Alloc).  This library is that step for one GPU: a dense, contiguous NCHW tensor
 * goes in, a self-describing packed container comes out, and back.
 *
 * Every plane (one (n, c) feature map of h x w elements) is coded independently:
 *   - three-sigma statistics classify it as normal or outlier-rich (Section 4.4.1);
 *   - a normal plane is quantised to `bits` bits per element between its own minimum and maximum;
 *   - an outlier-rich plane is split into 8 x 8 blocks by its pooled non-zero mask; sparse blocks go
 *     to one CSR structure, dense blocks to 8-bit first-order Lorenzo residual codes within the
 *     absolute error bound eps, unpredictable values verbatim (Eq. 7-9);
 *   - a plane that would not shrink is stored verbatim.
 *
 * Conventions
 *   - All functions return FH_OK (0) or a negative fh_status.  Errors that the host can see
 *     (bad arguments, unsupported shapes) are returned at once and nothing is enqueued.  Errors only
 *     the device can see (non-finite input, capacity, corrupt container, a wait that gave up) are
 *     written to the status word the call names.
 *   - Pointers named d_* are device pointers, h_* host pointers.  The caller owns every buffer.
 *     Dense and packed device buffers must be 16-byte aligned.
 *   - fh_compress and fh_decompress only enqueue work on `stream` (a cudaStream_t passed as
 *     void*; NULL is the legacy default stream) and never synchronise.  Per stream the library keeps
 *     one small scratch allocation (counters, and about 13 bytes per tile of planes of the largest
 *     tensor seen: the words through which tiles tell one another where their payloads go)
 *     that it creates on first use and frees in fh_shutdown(); growing it for a tensor with more
 *     planes synchronises the device once.
 *   - There is no CPU fallback: without a CUDA device every entry point that does work returns
 *     FH_ERR_CUDA.
 *
 * Container (little-endian; a layout of this library, the paper gives none)
 *   [0,64)   header: u32 magic "FHC1" | u16 version (1; 2 with entropy = 1) | u8 dtype | u8 bits | u32 N | u32 C | u32 H |
 *            u32 W | u8 block | u8 dense_bits | u8 rounding | u8 salient_mode | u16 rho_num |
 *            u16 rho_den | u16 tau_num | u16 tau_den | f32 eps | u32 n_salient | u32 n_raw |
 *            u64 tensor_id | u64 total_bytes
 *   [64,64+16P)  plane table, P = N*C entries: u32 offset / 16 (see below) | u32 meta (bits 0-1
 *            class: 0 normal, 1 salient, 2 raw; bits 2-31 three-sigma outlier count) | f32 lo |
 *            f32 scale (lo = scale = 0 unless normal)
 *   [64+16P, 64+16P+P*npay)  one slot per plane, npay = A16(4*ceil(HW*bits/32)) bytes, plane order
 *   [64+16P+P*npay, total)   overflow region
 *   A normal plane's codes fill its slot (zero padded); its table offset is that of the slot.  The
 *   payload of a salient or raw plane is laid through its slot first and, if longer, continues in
 *   the overflow region (continuations in plane order, each zero-padded to a multiple of 16 bytes);
 *   its table offset is that of the continuation, 0 when there is none.  Slots sit at closed-form
 *   offsets, so normal planes are written and read without knowing any other plane's size.
 *     normal : ceil(HW*bits/32) u32 words, element i in bits [(i*bits)%32, +bits) of word i*bits/32
 *     raw    : HW elements verbatim
 *     salient: u32 nnz_s | u32 n_dense | u32 n_out_d | u32 coded | block bitmap ceil(nblk/32) u32
 *              (bit = 1: dense; blocks in raster order) | row_ptr (H+1) u32 | col nnz_s u16 (pad 4) |
 *              val nnz_s elements (pad 4) | codes n_dense*64 u8, or, when coded != 0 (version 2), the
 *              Huffman-coded section of `coded` bytes | verbatim values n_out_d elements (pad 4)
 *     Huffman-coded section (Section 4.4.1; one code per plane from the plane's own code bytes, used only when
 *              smaller than the plain codes): u8 len(symbol 0) | u8 smin | u8 smax | u8 0 | u8 len(s),
 *              s = smin..smax (pad 4) | u8 bytes of chunk b, b = 0..n_dense-1 (pad 4) | chunks (pad 4);
 *              a chunk holds the 64 symbols of one dense block, starts on a byte boundary, code bits most
 *              significant first; codes are canonical (by length, then symbol) from Huffman lengths whose
 *              ties are settled by (weight, id), id = symbol for a leaf, 256 + order of creation for a
 *              merged node
 */
#ifndef FH_H_
#define FH_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  FH_OK = 0,
  FH_ERR_ARG = -1,         /* null pointer, non-positive extent, misaligned buffer, bad enum        */
  FH_ERR_UNSUPPORTED = -2, /* valid but outside what the kernels handle (see fh_compress)          */
  FH_ERR_CAPACITY = -3,    /* packed output does not fit dst_capacity / the arena                  */
  FH_ERR_NONFINITE = -4,   /* NaN or Inf in the input, or max - min overflows                      */
  FH_ERR_CORRUPT = -5,     /* container header/table/payload inconsistent with the expectation    */
  FH_ERR_TIMEOUT = -6,     /* a bounded device-side wait ran out (should never happen)             */
  FH_ERR_CUDA = -7         /* CUDA runtime error or no device                                       */
} fh_status;

typedef enum { FH_F32 = 0, FH_BF16 = 1 } fh_dtype;

/* A dense activation: contiguous NCHW, P = n*c planes of h*w elements; w <= 65535. */
typedef struct {
  int32_t dtype; /* fh_dtype */
  int32_t n, c, h, w;
  uint64_t tensor_id; /* carried in the header; also keys any random rounding */
} fh_tensor_desc;

/* AUTO: three-sigma rule per plane.  OFF: every plane normal.  ALL: every plane takes the block-wise path.
 * CHANNEL: the other reading of "classify channels" (Section 4.4.1) -- mu, sigma and the outlier count are
 * taken over the N planes of channel c together (same fixed-point sums, r = 1/(N*HW)) and the channel as a
 * whole, hence each of its planes, is normal or outlier-rich (n_out*rho_den > rho_num*N*HW); a plane's table
 * entry carries the plane's own count.
 * TENSOR: a third reading -- what counts as an outlier is fixed once for the whole tensor (mu and sigma over
 * all N*C*HW elements, same fixed-point sums, r = 1/(N*C*HW)); a plane is outlier-rich when its own count of
 * such outliers satisfies n_out*rho_den > rho_num*HW.
 * CHANNEL and TENSOR cost three more passes over the tensor and are not available through
 * fh_compress_static. */
typedef enum {
  FH_SALIENT_AUTO = 0, FH_SALIENT_OFF = 1, FH_SALIENT_ALL = 2, FH_SALIENT_CHANNEL = 3, FH_SALIENT_TENSOR = 4
} fh_salient_mode;

/* Codec parameters.  The paper names these quantities but prints no values (Section 4.4.1);
 * fh_default_params() fills the defaults given beside each field. */
typedef struct {
  int32_t bits;             /* code width of normal planes: 2, 4 or 8                      [2]     */
  int32_t salient_mode;     /* fh_salient_mode                                            [AUTO]  */
  int32_t rho_num, rho_den; /* plane is outlier-rich iff n_out*rho_den > rho_num*HW        [1/32]  */
  int32_t block;            /* n: pooling window = block edge; 8 only                      [8]     */
  int32_t tau_num, tau_den; /* block is dense iff nnz*tau_den >= tau_num*n*n               [1/4]   */
  float eps;                /* absolute error bound of dense blocks, 1e-30 <= eps <= 1e30  [1/16]  */
  int32_t dense_bits;       /* residual code width; 8 only                                 [8]     */
  int32_t rounding;         /* 0 = round half to even; 1 = random rounding of normal planes
                               (see fh_compress)                                           [0]     */
  uint64_t seed;            /* key of the random draws (rounding = 1)                      [0]     */
  int32_t entropy;          /* 1 = Huffman stage on the dense-block residual codes (see
                               fh_compress); container version 2                           [0]     */
  int32_t reserved;         /* 0                                                                   */
} fh_params;

typedef enum { FH_KEEP = 0, FH_COMPRESS = 1, FH_EVICT = 2 } fh_action;

/* One saved activation of a training step, in forward order (Algorithm 1's tensor states). */
typedef struct {
  fh_tensor_desc desc;
  int32_t action;      /* fh_action; KEEP and EVICT entries are skipped by the codec               */
  const void* d_dense; /* dense input (device)                                                    */
  void* d_restored;    /* where the backward pass wants it back (device); may equal d_dense       */
} fh_sched_entry;

typedef struct {
  uint64_t total_dense_bytes;  /* dense bytes of the COMPRESS entries                              */
  uint64_t total_packed_bytes; /* sum of their container sizes                                     */
  uint64_t peak_packed_bytes;  /* arena high-water mark (containers start on 256-byte boundaries)  */
  float ms_forward, ms_backward;
  int32_t status; /* first device-side error, FH_OK otherwise */
} fh_sched_report;

void fh_default_params(fh_params* p);

/* Version of the library (1) -- also proves that the shared object loaded. */
int fh_version(void);

/* Number of CUDA devices visible, or a negative fh_status. */
int fh_device_count(void);

/*
 * Size of the container of a tensor (Section 4.4.1 leaves the layout open; sizes follow the
 * container described above).
 *   which = 0: exact size when every plane is normal (always exact for FH_SALIENT_OFF):
 *              64 + P*(16 + A16(4*ceil(HW*bits/32)))
 *   which = 1: worst case, every plane verbatim: 64 + P*(16 + A16(esize*HW)); a dst_capacity of
 *              this many bytes can never overflow.
 * Returns 0 for invalid arguments.  Host-only, no CUDA call.
 */
size_t fh_compressed_bytes(const fh_tensor_desc* desc, const fh_params* params, int which);

/*
 * Compress one tensor (Section 4.4.1; forward pass of a tensor the plan marks "compress").
 *   d_src        dense input, n*c*h*w elements of desc->dtype, device, 16-byte aligned
 *   d_dst        container output, device, 16-byte aligned, dst_capacity bytes; never written past
 *                dst_capacity.  Must hold at least the header and plane table (64 + 16*P bytes).
 *   d_out2       optional, two uint64 in device memory (or pinned host memory mapped to the device):
 *                [0] total container bytes (the size needed, also when it did not fit),
 *                [1] (uint64)(int64) status: FH_OK, FH_ERR_NONFINITE, FH_ERR_CAPACITY, FH_ERR_TIMEOUT.
 *                Written by the kernel; valid once `stream` has reached this point.
 * Limits: one plane plus its working set must fit the shared memory of an SM, i.e. roughly
 * h*w*esize <= 200 KB; larger planes return FH_ERR_UNSUPPORTED.  The container is limited to
 * 64 GiB (32-bit offsets in units of 16 bytes).
 * The packed bytes are a pure function of the input and the parameters.
 *
 * rounding = 1 (the paper does not say how its quantiser rounds; the quantisers it builds on round at
 * random so that the restored value is unbiased): the code of an element of a normal plane is
 * floor(t) + [floor(frac(t) * 2^24) + r >= 2^24] with t = (x - lo) * inv in fp32 and r a uniform 24-bit
 * integer, the top 24 bits of word (i mod 4) of Philox-4x32-10 with key (seed low, seed high) and counter
 * (i / 4, plane index, tensor_id low, tensor_id high), i the element's index within its plane.  The draw
 * thus depends on (seed, tensor id, element position) only and results are reproducible.  Dense-block codes
 * keep round-to-nearest (their error bound needs it).  One generator call per four elements makes this mode
 * about twice as slow as rounding = 0 (planes of at most 1024 elements with salient_mode AUTO; other cases run
 * on the general-purpose kernel and are slower still).
 *
 * entropy = 1 (Section 4.4.1: "a Huffman tree is constructed from the quantization array for encoding"): the
 * residual code bytes of an outlier-rich plane's dense blocks are Huffman-coded, one code per plane (see the
 * container description); the stage is lossless and is skipped for a plane it would not shrink.  The container
 * carries version 2.  This mode runs on the general-purpose kernel and is not tuned.
 */
int fh_compress(const fh_tensor_desc* desc, const fh_params* params, const void* d_src, void* d_dst,
                size_t dst_capacity, uint64_t* d_out2, void* stream);

/*
 * Restore a tensor from its container (Section 4.4.1, "Decompression ..."; Algorithm 1, the
 * COMPRESSED branch of Compute).
 *   d_src, src_bytes   the container and the number of readable bytes
 *   expect             shape and dtype the caller expects; a mismatch with the header is
 *                      FH_ERR_CORRUPT (reported through d_status, the header lives on the device)
 *   d_dst              dense output, device, 16-byte aligned
 *   d_status           optional uint64 in device (or mapped pinned) memory: (uint64)(int64) status
 * Never reads past src_bytes.  Planes whose table entry is corrupt are left unwritten.
 */
int fh_decompress(const void* d_src, size_t src_bytes, const fh_tensor_desc* expect, void* d_dst,
                  uint64_t* d_status, void* stream);

/*
 * One training step's worth of codec work on one stream (Section 3.2; Algorithm 1): entries with
 * action FH_COMPRESS are compressed in forward order into d_arena (bump allocation with a
 * device-side cursor, 256-byte aligned containers, because sizes are only known on the device), then
 * restored in reverse order into their d_restored buffers.  Forward and backward phases are timed
 * with CUDA events.  This call synchronises the stream before it returns and fills *report.
 * An arena too small gives report->status = FH_ERR_CAPACITY (later tensors are skipped, nothing is
 * written outside the arena).
 */
int fh_run_schedule(const fh_sched_entry* entries, int32_t count, const fh_params* params,
                    void* d_arena, size_t arena_bytes, fh_sched_report* report, void* stream);

/*
 * Host-buffer variants: the same codec with host memory on both sides.  The library copies
 * h_src to the device work buffer, runs the kernels, copies the result back and synchronises.
 *   d_work, work_bytes   caller-owned device workspace, 256-byte aligned, at least
 *                        fh_host_work_bytes(desc, params) bytes
 *   h_out2 / h_status    as d_out2 / d_status above, but plain host memory
 * Pinned host buffers give asynchronous copies; pageable ones work but are slower.
 */
size_t fh_host_work_bytes(const fh_tensor_desc* desc, const fh_params* params);
int fh_compress_host(const fh_tensor_desc* desc, const fh_params* params, const void* h_src,
                     void* h_dst, size_t dst_capacity, uint64_t* h_out2, void* d_work,
                     size_t work_bytes, void* stream);
int fh_decompress_host(const void* h_src, size_t src_bytes, const fh_tensor_desc* expect, void* h_dst,
                       uint64_t* h_status, void* d_work, size_t work_bytes, void* stream);

/*
 * fh_compress without any allocation.  (The paper has no counterpart; this exists for callers of this
 * library.)
 *
 * fh_compress keeps its book-keeping (counters and the list of planes that take the block-wise
 * path) in a scratch buffer that it obtains with cudaMalloc on first use and enlarges when a tensor
 * with more planes arrives.  Some callers cannot afford that: the codec is called
 * exactly when device memory is short (a training engine compresses activations because its budget
 * is exhausted, so an allocation inside the codec can fail at the worst moment); a process whose
 * device memory is wholly pre-reserved by a framework pool has nothing left for the driver to hand
 * out; and a latency-bound training loop cannot take the device-wide synchronisation that
 * cudaMalloc / cudaFree may imply.  This variant never calls cudaMalloc, cudaFree or any allocating
 * routine: its scratch is a fixed array compiled into the library's device image
 * (FH_STATIC_SCRATCH_BYTES bytes, resident on every GPU that loads the library until the process
 * exits).
 *
 * Arguments, output, status reporting and the produced bytes are exactly those of fh_compress.
 * Differences:
 *   - the tensor may have at most FH_STATIC_MAX_PLANES planes (n * c); anything larger returns
 *     FH_ERR_UNSUPPORTED and enqueues nothing;
 *   - the first call on a device looks up the device address of the array (once per device, with
 *     that device current).  Make that first call outside any stream capture;
 *   - all calls on a device share the one array, which still holds the previous call's contents, so
 *     each call first clears the counters it uses with a memset on `stream`.  Two calls that overlap
 *     on the GPU (different streams without ordering between them) race on it: order them.
 */
#define FH_STATIC_MAX_PLANES 131072
#define FH_STATIC_SCRATCH_BYTES (256 + 8 * (FH_STATIC_MAX_PLANES + 2 * (FH_STATIC_MAX_PLANES / 32)) + 4 * FH_STATIC_MAX_PLANES)
int fh_compress_static(const fh_tensor_desc* desc, const fh_params* params, const void* d_src, void* d_dst,
                       size_t dst_capacity, uint64_t* d_out2, void* stream);

/*
 * Plan generation (Algorithm 1 with the MPS metric of Eq. 5; host only, no CUDA call).
 *
 * The computation sequence is walked op by op (Main).  Compute(op) makes the op's inputs resident again --
 * a COMPRESSED input gets its dense buffer back (decompress), an EVICTED one is recomputed -- and allocates
 * its outputs.  Every allocation goes through Alloc: while pool_size + size >= memory_budget, the resident
 * tensor with the largest MPS is purged, evicted if MPS_compute > MPS_compress, compressed otherwise.
 *   MPS(d) = SM(d) * FLT(d) / (PC(d) + RC(d))                                                  (Eq. 5)
 *   compress: SM = bytes - packed_bytes, PC = t_compress, RC = t_decompress
 *   evict   : SM = bytes,                PC = 0,          RC = t_recompute  (Eq. 6, supplied by the caller)
 *   FLT(d)  = time from the current op's start to the start of the next op that reads d
 * Readings where the paper is silent: tensors of the current op are locked (never purged); a tensor is
 * dropped from the pool after its last reader; tensors no op produces are resident from the start; only
 * resident tensors with a later reader are candidates; ties go to the lower tensor index; a tensor that
 * cannot shrink (packed_bytes >= bytes) or cannot be recomputed (t_recompute < 0) has MPS 0 for that
 * technique; when nothing can be purged the allocation proceeds over budget and the report says so.
 * t_compress / t_decompress are what this library's fh_compress / fh_decompress take on the target device.
 *
 * actions[t] receives the last purge decision for tensor t (FH_KEEP, FH_COMPRESS or FH_EVICT) -- the action
 * of an fh_sched_entry; events (optional, up to max_events) receive every decision in order:
 * kind FH_COMPRESS / FH_EVICT = purged before op `op`, FH_KEEP = brought back for op `op`.
 * Returns FH_OK, FH_ERR_ARG (null pointers, tensor ids out of range, negative or all-zero costs), or
 * FH_ERR_CAPACITY (plan produced, but some allocation could not be brought under the budget).
 */
typedef struct {
  uint64_t bytes;        /* dense size                                                      */
  uint64_t packed_bytes; /* size once compressed                                            */
  double t_compress;     /* seconds                                                         */
  double t_decompress;   /* seconds                                                         */
  double t_recompute;    /* seconds, Eq. 6; negative: the tensor cannot be recomputed       */
} fh_plan_tensor;

typedef struct {
  double time;            /* OpTime, seconds                                                */
  const int32_t* inputs;  /* tensor ids read                                                */
  int32_t n_inputs;
  const int32_t* outputs; /* tensor ids produced                                            */
  int32_t n_outputs;
} fh_plan_op;

typedef struct {
  int32_t op, tensor, kind;
} fh_plan_event;

typedef struct {
  uint64_t peak_bytes;     /* largest pool size reached                                     */
  double overhead_seconds; /* sum of compress, decompress and recompute times the plan adds  */
  int32_t n_events;        /* decisions taken (may exceed max_events; the rest is not stored) */
  int32_t n_over_budget;   /* allocations that stayed over budget                            */
} fh_plan_report;

int fh_plan_generate(const fh_plan_op* ops, int32_t n_ops, const fh_plan_tensor* tensors, int32_t n_tensors,
                     uint64_t memory_budget, int32_t* actions, fh_plan_event* events, int32_t max_events,
                     fh_plan_report* report);

/*
 * Costs of compression as this library delivers them on the current device, measured: the quantities PC(d)
 * and RC(d) of the compression technique in Eq. 5 and the space it frees (SM(d)), for fh_plan_generate.
 * For every tensor i the call compresses d_dense[i] into the work buffer and restores it again, `repeats`
 * times each after one untimed run, timed with CUDA events on `stream`, and fills
 *   out[i].bytes, out[i].packed_bytes (the container's size), out[i].t_compress, out[i].t_decompress
 * (seconds, mean of the repeats).  out[i].t_recompute is left as the caller set it (Eq. 6 is the caller's).
 *   descs, d_dense   n tensor descriptions and their dense device buffers (16-byte aligned)
 *   d_work           caller-owned device workspace, 256-byte aligned, at least fh_host_work_bytes(desc, params)
 *                    bytes for the largest tensor (it holds the container and the restored copy)
 *   repeats          1..1000
 * The call synchronises the stream.  Returns FH_OK, an argument error, or the first device-side status.
 */
int fh_plan_measure(const fh_tensor_desc* descs, int32_t n, const fh_params* params, const void* const* d_dense,
                    void* d_work, size_t work_bytes, int32_t repeats, fh_plan_tensor* out, void* stream);

/*
 * Fault injection on the host side, for tests of the error path of the device-side waits.  (The paper has no
 * counterpart.)  Compressing places the overflow parts of outlier-rich planes in plane order: a tile of
 * planes waits, with a limit, until every earlier tile has published its size; a wait that runs out ends the
 * call with FH_ERR_TIMEOUT in its status word (no magic in the header) and leaves the library usable.
 *   FH_DEBUG_WAIT_POLLS   limit of those waits in polls of about 0.1 us (default 2^22)
 *   FH_DEBUG_SILENT_TILE  index of a tile that never publishes its size, so that every later tile with
 *                         an outlier-rich plane runs into the limit; UINT64_MAX: none (default)
 * Both apply to calls enqueued afterwards, process-wide.  Returns FH_OK or FH_ERR_ARG.
 */
enum { FH_DEBUG_WAIT_POLLS = 0, FH_DEBUG_SILENT_TILE = 1 };
int fh_debug_set(int what, uint64_t value);

/* Number of kernels this library has launched since it was loaded (for launch accounting). */
uint64_t fh_kernel_launches(void);

/* Free every scratch allocation the library holds on every device.  Synchronises. */
void fh_shutdown(void);

#ifdef __cplusplus
}
#endif
#endif /* FH_H_ */
