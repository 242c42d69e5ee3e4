/*
 * preba.h — C ABI of the fused vision-preprocessing library for B200 (sm_100a).
 *
 * The path is the per-query image preprocessing that runs in front of the model
 * (paper Sec. 2.3 item 1, Fig. 4; Table 1 rows "Resize", "Crop", "Normalize"):
 * every decoded uint8 RGB image of a ragged batch is resized (shorter side to
 * `resize_short`, bilinear, half-pixel centres, edge clamp, no antialias),
 * center-cropped to `out_size` x `out_size`, converted to float with
 * out = (v/255 - mean_c)/std_c, and written as plane c, row k, column j of a
 * dense [n, 3, out_size, out_size] tensor.  As in the paper's pipelined
 * compute unit (Sec. 4.2), the stages are chained on chip: one kernel launch
 * per batch, no intermediate image in device memory.
 *
 * Conventions for every entry point
 *   - Plain C.  Returns PREBA_OK (0) or a negative PREBA_ERR_* code; nothing
 *     is thrown, printed or allocated, and no call synchronises the device.
 *   - Pointers are marked HOST or DEVICE.  The caller owns every buffer; the
 *     library borrows HOST arguments for the duration of the call and DEVICE
 *     buffers until the stream has passed the work the call enqueued.
 *   - Calls keep no state between them and may be made concurrently from
 *     several threads, each on its own stream.
 *   Two entry points depart from this, as their own comments say:
 *   preba_preprocess_host_noalloc keeps the device address of the library's
 *   staging array per device (it does not survive cudaDeviceReset) and every
 *   call shares that array, so its calls must be serialised per device;
 *   preba_preprocess_repeated creates and destroys events and waits for the
 *   stream.
 */
#ifndef PREBA_H_
#define PREBA_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define PREBA_PACK_ALIGN 128u     /* every image offset, and the packed size, is a multiple */
#define PREBA_MAX_DIM 32768u      /* largest accepted image height or width */
#define PREBA_MAX_RESIZE 16384u   /* largest accepted resize_short (and so out_size) */
#define PREBA_SCRATCH_BYTES 256u  /* size of the scheduling scratch a batch may carry */

/* preba_batch_t.flags */
#define PREBA_OVERLAP_PREVIOUS 1u /* the launch need not wait for the kernels before it on the
                                     stream to finish (programmatic dependent launch): as their
                                     warps retire, this one's take their place.  The relaxation
                                     chains: a marked launch may run beside every kernel enqueued
                                     since the last operation on the stream that was not a marked
                                     launch (an unmarked launch, a copy, an event wait), not only
                                     beside the one directly before it.  Set it only if none of
                                     those kernels writes this batch's pixels, table or scratch
                                     or touches its out buffer, e.g. back-to-back batches with
                                     buffers (and scratch) of their own, and put an unmarked
                                     launch where a buffer set comes round again.  Completion
                                     stays ordered: a marked launch does not complete before the
                                     kernels ahead of it have, so whatever is enqueued after it
                                     without the flag (a copy, an event, an unmarked launch)
                                     finds the results of the whole chain. */

#define PREBA_OK 0
#define PREBA_ERR_INVALID_ARG (-1)      /* NULL, zero or out-of-range argument, misaligned buffer */
#define PREBA_ERR_BUFFER_TOO_SMALL (-2) /* a capacity is below what preba_query reports */
#define PREBA_ERR_BAD_TABLE (-3)        /* a table entry is misaligned, out of range or past the pixels */
#define PREBA_ERR_CUDA (-4)             /* a CUDA runtime call failed; see preba_last_cuda_error */
#define PREBA_ERR_TIMEOUT (-5)          /* only in the device status word: a bounded wait ran out */
#define PREBA_ERR_TOO_LARGE (-6)        /* the batch exceeds PREBA_NOALLOC_MAX_BYTES, or an image is
                                           reduced by more than the antialiased kernel can hold */
#define PREBA_ERR_BAD_CROP (-7)         /* a crop window does not lie on its image's resized grid */
#define PREBA_ERR_UNSUPPORTED (-9)      /* a JPEG stream of a kind the decoder does not take
                                           (progressive, arithmetic-coded, 12-bit, CMYK, ...) */
#define PREBA_ERR_BAD_STREAM (-10)      /* a JPEG stream that is malformed or cut short */
#define PREBA_ERR_RANGE (-8)            /* only in the device status word, and only from the checked
                                           build of the library (compiled with PREBA_CHECKED): a
                                           shared-memory offset, a table index or a global address
                                           left its range inside a kernel; the access was skipped */

/* Device memory the library itself carries for preba_preprocess_host_noalloc (64 MiB). */
#define PREBA_NOALLOC_MAX_BYTES (64u << 20)

typedef enum {
  PREBA_F32 = 0,
  PREBA_F16 = 1,
  PREBA_BF16 = 2,
  PREBA_U8 = 3 /* preba_preprocess_ex only: the rounded pixel itself, uint8, HWC */
} preba_dtype_t;

/* One image of the packed batch: `offset` is in bytes from the start of the
 * pixel buffer and a multiple of PREBA_PACK_ALIGN; the image is h rows of w
 * RGB pixels, 3 bytes per pixel, row pitch exactly 3*w bytes. */
typedef struct {
  uint64_t offset;
  uint32_t h;
  uint32_t w;
} preba_img_t;

typedef struct {
  uint64_t packed_bytes; /* size of the packed pixel buffer */
  uint64_t table_bytes;  /* n * sizeof(preba_img_t) */
  uint64_t out_bytes;    /* n * 3 * out_size^2 * sizeof(out element) */
  uint32_t align;        /* PREBA_PACK_ALIGN */
  uint32_t reserved;
} preba_sizes_t;

/* A batch resident in device memory. */
typedef struct {
  const uint8_t* pixels;         /* DEVICE, base aligned to 16 bytes, packed as preba_pack lays out */
  uint64_t pixels_bytes;         /* bytes readable at `pixels` (>= sizes.packed_bytes) */
  const preba_img_t* table;      /* DEVICE, n entries */
  const preba_img_t* table_host; /* HOST copy of the table for checking before launch, or NULL */
  uint32_t n;                    /* images in the batch, >= 1 */
  uint32_t flags;                /* 0 or PREBA_OVERLAP_PREVIOUS */
  void* out;                     /* DEVICE, [n,3,out_size,out_size] contiguous, 16-byte aligned */
  uint64_t out_bytes;            /* bytes writable at `out` (>= sizes.out_bytes) */
  int32_t* status;               /* DEVICE word or NULL: the kernel stores the first PREBA_ERR_*
                                    it meets (bad table entry, wait that ran out); caller zeroes it */
  uint32_t* scratch;             /* DEVICE, PREBA_SCRATCH_BYTES, 16-byte aligned, or NULL.  Task
                                    counters: with it, warps claim slabs as they finish, which
                                    evens out a ragged batch; without it every warp takes a fixed
                                    share.  The caller zeroes it once; each launch leaves it
                                    zeroed again.  Launches that may overlap on the device (other
                                    streams) need scratch of their own; zero it again after a
                                    launch that reported an error status. */
} preba_batch_t;

/* A batch resident in host memory, with the device buffers the call stages it through. */
typedef struct {
  const uint8_t* packed_host;    /* HOST (pinned for an asynchronous copy), packed_bytes bytes */
  uint64_t packed_bytes;
  const preba_img_t* table_host; /* HOST, n entries */
  uint32_t n;
  uint32_t reserved;
  void* out_host;                /* HOST (pinned for an asynchronous copy), out_bytes bytes */
  uint64_t out_bytes;
  uint8_t* dev_pixels;           /* DEVICE staging, >= packed_bytes, 16-byte aligned */
  preba_img_t* dev_table;        /* DEVICE staging, n entries */
  void* dev_out;                 /* DEVICE staging, >= out_bytes, 16-byte aligned */
  int32_t* dev_status;           /* DEVICE word or NULL, as preba_batch_t.status */
  uint32_t* dev_scratch;         /* DEVICE or NULL, as preba_batch_t.scratch */
} preba_host_batch_t;

/* preba_image_batch_t.flags */
#define PREBA_IMAGES_IN_PLACE 1u  /* the kernel reads the images where they lie, in pinned host
                                     memory, across the host-device link: only the bytes the
                                     transform taps cross it, and no copy is enqueued for them.
                                     Every image pointer must then be pinned memory the device
                                     can address (cudaMallocHost / cudaHostAlloc), a multiple of
                                     PREBA_PACK_ALIGN, and readable through the end of the
                                     16-byte block that holds the image's last byte; the
                                     images must not overlap.  dev_pixels is not used. */

#define PREBA_IMAGES_OUT_IN_PLACE 2u /* the kernel stores the result where it is wanted, in pinned
                                        host memory, across the link (streaming 128-byte runs):
                                        no copy is enqueued for it, and with PREBA_IMAGES_IN_PLACE
                                        one kernel moves both directions of the link at once.
                                        out_host must then be pinned memory the device can
                                        address, 16-byte aligned; dev_out is not used. */

/* A batch of separate decoded images in host memory (no packed copy on the host), with the
 * device buffers the call stages it through. */
typedef struct {
  const uint8_t* const* images;  /* HOST array of n HOST pointers; image i is h[i] rows of w[i]
                                    RGB pixels, pitch 3*w[i] (pinned for asynchronous copies) */
  const uint32_t* h;             /* HOST, n entries */
  const uint32_t* w;             /* HOST, n entries */
  uint32_t n;
  uint32_t flags;                /* 0, PREBA_IMAGES_IN_PLACE, PREBA_IMAGES_OUT_IN_PLACE or both */
  preba_img_t* table_host;       /* HOST, n entries, WRITTEN by the call (the table preba_pack
                                    would build); pinned; valid until the stream has passed
                                    the call's copies */
  void* out_host;                /* HOST (pinned for an asynchronous copy), out_bytes bytes */
  uint64_t out_bytes;
  uint8_t* dev_pixels;           /* DEVICE staging, 16-byte aligned */
  uint64_t dev_pixels_bytes;     /* capacity of dev_pixels, >= sizes.packed_bytes */
  preba_img_t* dev_table;        /* DEVICE staging, n entries */
  void* dev_out;                 /* DEVICE staging, >= out_bytes, 16-byte aligned */
  int32_t* dev_status;           /* DEVICE word or NULL, as preba_batch_t.status */
  uint32_t* dev_scratch;         /* DEVICE or NULL, as preba_batch_t.scratch */
} preba_image_batch_t;

/*
 * preba_query — sizes of the buffers a batch needs (host arithmetic only).
 * The packed layout is the problem statement's, not the paper's (which handles
 * each single-input request on its own, Sec. 5 "Input query modeling"): images
 * are concatenated in order, each starting at the running byte count rounded
 * up to PREBA_PACK_ALIGN, and the total is rounded up as well.
 *   h, w      HOST, n entries each, every value in [1, PREBA_MAX_DIM]
 *   out_size  side of the square crop, >= 1
 *   out_dtype PREBA_F32, PREBA_F16 or PREBA_BF16
 *   sizes     HOST, written on success
 * Errors: PREBA_ERR_INVALID_ARG.
 */
int preba_query(const uint32_t* h, const uint32_t* w, uint32_t n, uint32_t out_size,
                int out_dtype, preba_sizes_t* sizes);

/*
 * preba_pack — step 0 of the path: builds the packed pixel buffer and the
 * {offset, h, w} table from n separate decoded images (each HWC uint8, row
 * pitch 3*w).  Padding bytes between images and at the tail are written as 0,
 * so the result is a pure function of the inputs.  Batches above a few megabytes
 * are copied by up to 8 short-lived worker threads.
 *   images    HOST array of n HOST pointers
 *   packed    HOST, `capacity` bytes; must hold sizes.packed_bytes
 *   table     HOST, n entries, written
 * Errors: PREBA_ERR_INVALID_ARG, PREBA_ERR_BUFFER_TOO_SMALL.
 */
int preba_pack(const uint8_t* const* images, const uint32_t* h, const uint32_t* w, uint32_t n,
               uint8_t* packed, uint64_t capacity, preba_img_t* table);

/*
 * preba_preprocess — the transform (Resize -> Crop -> Normalize of Table 1,
 * fused as the paper's compute unit chains them, Sec. 4.2), on a device-resident
 * batch.  Enqueues exactly one kernel on `stream` and returns.
 *   out_size      crop side C, 1 <= C <= resize_short
 *   resize_short  target length S of the shorter side, <= PREBA_MAX_RESIZE;
 *                 the longer side becomes floor(S*long/short)
 *   mean, std     HOST, 3 floats each, copied at call time; std finite, non-zero
 *   out_dtype     PREBA_F32, PREBA_F16 or PREBA_BF16 (one rounding to nearest even)
 *   stream        a cudaStream_t (NULL = the default stream)
 * Per image: crop origin floor((R - C)/2) on each axis; output index j samples
 * source coordinate ((j + origin) + 1/2) * in/R - 1/2, clamped to [0, in-1];
 * taps and weights come from exact integer arithmetic, interpolation and the
 * normalising multiply-add run in fp32, with no rounding to uint8 in between.
 * If `table_host` is given, entries are checked before launch
 * (PREBA_ERR_BAD_TABLE).  The kernel checks each entry again on the device: a
 * bad entry is skipped, its output left untouched, and PREBA_ERR_BAD_TABLE is
 * stored in `status`.
 * Errors: PREBA_ERR_INVALID_ARG, PREBA_ERR_BUFFER_TOO_SMALL,
 * PREBA_ERR_BAD_TABLE, PREBA_ERR_CUDA.
 */
int preba_preprocess(const preba_batch_t* batch, uint32_t out_size, uint32_t resize_short,
                     const float mean[3], const float std[3], int out_dtype, void* stream);

/* preba_options_t.flags */
#define PREBA_EX_ROUND_U8 1u /* round the interpolated value to the nearest integer (ties up,
                                decided in exact integer arithmetic) before normalising, as a
                                pipeline that resizes into a uint8 image does */

typedef struct {
  uint32_t out_size;      /* crop side C */
  uint32_t resize_short;  /* resized length S of the shorter side */
  float mean[3];          /* as preba_preprocess (ignored for PREBA_U8) */
  float std[3];
  int32_t out_dtype;      /* PREBA_F32, PREBA_F16, PREBA_BF16: [n,3,C,C] planar;
                             PREBA_U8 (needs PREBA_EX_ROUND_U8): [n,C,C,3] uint8, no normalisation */
  uint32_t flags;         /* 0 or PREBA_EX_ROUND_U8 */
  const uint32_t* crop_origin;      /* DEVICE, 2n values: (top, left) of image i's window on its
                                       resized grid, top + C <= R_h, left + C <= R_w; NULL: the
                                       centre crop floor((R - C)/2) */
  const uint32_t* crop_origin_host; /* HOST copy for checking before launch (with
                                       batch->table_host), or NULL */
} preba_options_t;

/*
 * preba_preprocess_ex — the transform with the adjustments other models ask of the same
 * Resize / Crop / Normalize units (paper Sec. 4.2, "Flexible design based on reconfigurable
 * hardware": preprocessing differs between models only by incremental changes): a crop
 * window per image instead of the centre crop, rounding of the resized pixel to uint8
 * before normalisation, and the rounded uint8 crop itself as output.  Sampling geometry,
 * resized size, batch layout, status word, scratch and flags are those of preba_preprocess;
 * one kernel is enqueued on `stream`.
 * With PREBA_EX_ROUND_U8 the pixel is floor(v + 1/2) of the exact bilinear value v (a ratio
 * of integers), so the uint8 output is reproducible bit for bit; images whose resized size
 * makes 511 * 4 * R_h * R_w reach 2^32 take a slower exact path.
 * A window that does not fit is refused before launch when the host copies are given
 * (PREBA_ERR_BAD_CROP); the kernel checks again, skips such an image and stores
 * PREBA_ERR_BAD_CROP in the status word.
 * Errors: as preba_preprocess, and PREBA_ERR_BAD_CROP.
 */
int preba_preprocess_ex(const preba_batch_t* batch, const preba_options_t* opt, void* stream);

/*
 * preba_preprocess_antialias — the transform with an antialiased Resize unit, for inputs much
 * larger than the model's resolution (paper Table 1's Resize reconfigured, Sec. 4.2 "Flexible
 * design based on reconfigurable hardware"; the paper fixes no filter): a separable triangle
 * filter whose half-width is the reduction factor.  On each axis, with n_in input pixels, R
 * resized pixels (the sizes of preba_preprocess) and M = max(n_in, R), input pixel j weighs
 *     W = max(0, 2M - |(2j+1) R - (2X+1) n_in|)
 * in resized pixel X, normalised by the sum over the pixels 0 <= j < n_in; the value is
 * sum_i sum_j wy_i wx_j p[i][j], then (v/255 - mean)/std.  An axis that is not reduced gets
 * the two-tap interpolation of preba_preprocess.  Integer taps and weights, fp32 sums.
 * `opt` is read as by preba_preprocess_ex (crop windows included) with flags == 0 and a float
 * out_dtype; batch layout, table checks and status word are those of preba_preprocess;
 * batch->scratch is not used and PREBA_OVERLAP_PREVIOUS has no effect.
 * Up to four kernels share the work, each skipping the others' images.  Images whose width is
 * a multiple of 4 and that are reduced more than 2.5 times vertically (and up to about 6.5
 * times horizontally) go to a kernel that runs both passes on the tensor cores: the horizontal
 * one as integer matrix instructions (the input rows as they lie in memory against the integer
 * weights, exact), the vertical one as binary16 matrix instructions on the exact bytes of the
 * horizontal sums against the exact bytes of the integer weights, accumulated in fp32 (two
 * instances: horizontal windows of 96 and of 128 bytes).  Other images whose width is a
 * multiple of 4 and that are reduced or enlarged up to about six times go to a kernel with
 * the horizontal pass on the tensor cores and the vertical pass in fp32.  Every other image
 * goes to a kernel in which a CTA keeps one channel-planar row of the window's footprint and
 * the weight tables in shared memory.  The result of an image does not depend on the batch it
 * is in.  With `table_host` only the kernels that have images are enqueued on `stream`, the
 * last kernel's launch carries what its largest image needs, and an image that needs more
 * than the device allows is refused (PREBA_ERR_TOO_LARGE: reductions beyond about 40 at
 * out_size 224); without it all are enqueued, the last carries all the device allows and
 * skips and reports such an image in the status word.
 * Errors: PREBA_ERR_INVALID_ARG, PREBA_ERR_BUFFER_TOO_SMALL, PREBA_ERR_BAD_TABLE,
 * PREBA_ERR_BAD_CROP, PREBA_ERR_TOO_LARGE, PREBA_ERR_CUDA.
 */
int preba_preprocess_antialias(const preba_batch_t* batch, const preba_options_t* opt,
                               void* stream);

/*
 * preba_preprocess_host — the same transform for a batch held in host memory
 * (the request path of the paper's server: inputs arrive in host memory and
 * results return to it, Sec. 4.2 "Implication of adding DPU").  Enqueues on
 * `stream`: copy of the packed pixels and the table to the device staging
 * buffers, the kernel, and the copy of the result to `out_host`; then returns.
 * The host buffers must stay valid and unchanged until the stream has passed
 * these operations; use pinned memory for the copies to be asynchronous.
 * The table is always checked on the host first.
 * Errors: as preba_preprocess.
 */
int preba_preprocess_host(const preba_host_batch_t* batch, uint32_t out_size,
                          uint32_t resize_short, const float mean[3], const float std[3],
                          int out_dtype, void* stream);

/*
 * preba_preprocess_images — step 0 and the transform in one call, for decoded images that
 * already sit in (pinned) host memory one by one, as a decoder leaves them: each request
 * arrives on its own (paper Sec. 5 "Input query modeling") and crosses the host-device
 * link once (Sec. 4.2 "Implication of adding DPU").  Nothing is packed on the host: the
 * call lays the batch out as preba_pack would (same offsets, written to `table_host`),
 * copies every image straight to its offset in `dev_pixels`, then enqueues the table copy,
 * the kernel and the copy of the result to `out_host`, all on `stream`, and returns.
 * Padding bytes between images stay as the device buffer had them; the transform never
 * gives them weight.  n + 1 host-to-device copies, one kernel, one device-to-host copy.
 * With PREBA_IMAGES_IN_PLACE the image copies are dropped: `table_host` receives each
 * image's distance from the lowest image address, and the kernel fetches the tapped rows
 * from host memory itself (table copy, kernel, result copy).  With PREBA_IMAGES_OUT_IN_PLACE
 * the result copy is dropped too: the kernel writes `out_host` itself (table copy, kernel).
 * Errors: PREBA_ERR_INVALID_ARG, PREBA_ERR_BUFFER_TOO_SMALL (dev_pixels_bytes, out_bytes),
 * PREBA_ERR_CUDA.
 */
int preba_preprocess_images(const preba_image_batch_t* batch, uint32_t out_size,
                            uint32_t resize_short, const float mean[3], const float std[3],
                            int out_dtype, void* stream);

/*
 * preba_preprocess_host_noalloc — preba_preprocess_host for callers that have no way to
 * obtain device memory.  (The paper has no counterpart; this exists for the embedding.)
 *
 * Some hosts of this library may not allocate on the device at all: a plug-in running
 * inside a server that owns the allocator, code on a latency path where cudaMalloc's
 * implicit device synchronisation is forbidden, a process whose memory budget was fixed at
 * start-up.  They still have pinned host buffers and a stream.  This entry point does the
 * whole host-to-host transform with staging space that is part of the library image: a
 * fixed array of PREBA_NOALLOC_MAX_BYTES in device memory, present on every GPU that
 * loads the library for as long as the process lives.  It calls no allocating routine.
 *
 *   packed_host, packed_bytes, table_host, n   the batch as preba_pack wrote it (HOST;
 *                                              pinned for the copies to be asynchronous)
 *   out_host, out_bytes     HOST, receives [n,3,out_size,out_size]
 *   status_host             HOST int32 or NULL: receives the kernel's status word (0 or the
 *                           first PREBA_ERR_* met on the device) once the stream gets there
 *   other arguments         as preba_preprocess
 *
 * The staging space holds, each rounded up to 256 bytes: 512 bytes of bookkeeping, the
 * table, the packed pixels and the result.  A batch that needs more than
 * PREBA_NOALLOC_MAX_BYTES is refused with PREBA_ERR_TOO_LARGE and nothing is enqueued.
 *
 * The first call on a device looks up the array's device address (one runtime query, no
 * allocation) and keeps it; make that first call before any stream capture begins.
 * Every call on a device uses the same array and finds the previous call's bytes in it:
 * the bookkeeping words are cleared on the stream at the start of each call, the rest is
 * overwritten before it is read.  Two calls whose work overlaps on the device (different
 * streams, or several host threads) would therefore race on the array: issue them on one
 * stream, or order them with events.
 * Errors: PREBA_ERR_INVALID_ARG, PREBA_ERR_BUFFER_TOO_SMALL (out_bytes), PREBA_ERR_BAD_TABLE,
 * PREBA_ERR_TOO_LARGE, PREBA_ERR_CUDA.
 */
int preba_preprocess_host_noalloc(const uint8_t* packed_host, uint64_t packed_bytes,
                                  const preba_img_t* table_host, uint32_t n, void* out_host,
                                  uint64_t out_bytes, int32_t* status_host, uint32_t out_size,
                                  uint32_t resize_short, const float mean[3], const float std[3],
                                  int out_dtype, void* stream);

/*
 * preba_preprocess_repeated — a measuring aid for serving-style loops (the paper's several
 * small inference servers sharing one GPU, Sec. 3): launches the same device-resident batch
 * `iterations` times on `stream`, one kernel each, every launch bracketed by a pair of
 * events, then waits for the stream and writes each launch's device time.  Unlike the other
 * entry points it creates (and destroys) CUDA events and synchronises the stream; several
 * host threads may run it at once on streams of their own.
 *   latency_us   HOST, `iterations` floats (microseconds per launch), or NULL
 *   span_ms      HOST float or NULL: device time from the first launch's start to the last
 *                launch's end
 * Errors: as preba_preprocess.
 */
int preba_preprocess_repeated(const preba_batch_t* batch, uint32_t out_size,
                              uint32_t resize_short, const float mean[3], const float std[3],
                              int out_dtype, void* stream, uint32_t iterations,
                              float* latency_us, float* span_ms);

/*
 * preba_selftest_wait_limit — exercises the kernel's bounded wait on the device: one warp
 * waits on a shared-memory barrier that nothing ever completes, gives up after the same poll
 * limit the transform uses, stores PREBA_ERR_TIMEOUT in `status` and returns normally; the
 * context stays usable.  (Every wait in the transform's kernel is of this kind, so a copy
 * that never lands ends in an error status instead of a hang.)
 *   status   DEVICE word, zeroed by the caller
 * Enqueues one small kernel on `stream`.  Errors: PREBA_ERR_INVALID_ARG, PREBA_ERR_CUDA.
 */
int preba_selftest_wait_limit(int32_t* status, void* stream);

/*
 * Batching front-end (host only) — the stage between preprocessing and model execution
 * (paper Sec. 2.3 item 2): single-input requests wait in arrival order and leave as a batch
 * when Batch_max of them are queued or when the oldest has waited Time_queue.  The paper's
 * batching system (Sec. 4.3) sets the two hyper-parameters from a one-time profile:
 * Batch_max = Batch_knee, the batch size at the knee of the latency curve, and
 * Time_queue = Time_knee / number of servers sharing the GPU (Time_knee itself for one big
 * GPU).  For this library's kernel the profile is bench.py's batch-size sweep.
 *
 * preba_batching_params   the two hyper-parameters from the profile (Sec. 4.3).
 * preba_batcher_create    a queue with those parameters (batch_max >= 1); NULL on failure.
 * preba_batcher_push      enqueue request `id` that arrived at `arrival_ns`; arrival times
 *                         must not decrease.  PREBA_ERR_INVALID_ARG otherwise.
 * preba_batcher_poll      at time `now_ns`: if a batch is due, writes its request ids (oldest
 *                         first) to `ids` and returns their count; else returns 0.  A batch is
 *                         due when batch_max requests are queued (it takes the oldest
 *                         batch_max) or when now_ns >= oldest arrival + time_queue_ns (it
 *                         takes everything queued).  `next_deadline_ns`, if not NULL, receives
 *                         the time at which the then-oldest request runs out of waiting time
 *                         (UINT64_MAX when the queue is empty).  `capacity` must be >=
 *                         batch_max (PREBA_ERR_BUFFER_TOO_SMALL).
 * preba_batcher_destroy   frees the queue.
 * Calls on one queue may come from several threads (one lock per queue).
 */
typedef struct preba_batcher preba_batcher_t;
int preba_batching_params(uint32_t batch_knee, uint64_t time_knee_ns, uint32_t n_servers,
                          uint32_t* batch_max, uint64_t* time_queue_ns);
preba_batcher_t* preba_batcher_create(uint32_t batch_max, uint64_t time_queue_ns);
void preba_batcher_destroy(preba_batcher_t* b);
int preba_batcher_push(preba_batcher_t* b, uint64_t id, uint64_t arrival_ns);
int preba_batcher_poll(preba_batcher_t* b, uint64_t now_ns, uint64_t* ids, uint32_t capacity,
                       uint64_t* next_deadline_ns);

/*
 * Batching front-end for variable-length inputs (paper Sec. 4.3, Fig. "dynamic batching system
 * for audio processing workloads"): input lengths are bucketised into non-overlapping windows
 * (2.5 s in the paper), every bucket has a batching queue of its own with its own Batch_max
 * (the Batch_knee profiled for that length), and no request may wait longer than Time_queue.
 * A bucket's batch is due when Batch_max of its requests are queued (it takes the oldest
 * Batch_max) or when its oldest request has waited Time_queue.  In the second case the batch
 * is short, and the paper fills it from adjacent buckets without exceeding the Batch_max of
 * the longest input in the batch.  Readings taken here: "adjacent" means the two neighbouring
 * buckets; the lower one (shorter inputs, which leave the limit unchanged) is drained first,
 * oldest request first, then the upper one, whose own Batch_max caps the batch once one of
 * its requests is in; when several buckets are due, full ones go first (lowest bucket first),
 * then the one whose deadline passed earliest.
 *
 * preba_bucket_batcher_create   n_buckets >= 1 queues; bucket i takes lengths in
 *                               [i*window, (i+1)*window), the last one everything longer;
 *                               batch_max[i] >= 1; NULL on failure.  `window` and the lengths
 *                               passed to push share one unit (samples, milliseconds, ...).
 * preba_bucket_batcher_push     enqueue request `id` of the given length that arrived at
 *                               `arrival_ns`; arrival times must not decrease.
 * preba_bucket_batcher_poll     at time `now_ns`: writes the ids of one due batch (the due
 *                               bucket's requests oldest first, then those merged from the
 *                               lower and the upper neighbour) and returns their count, or 0;
 *                               call again until it returns 0.  `capacity` must be >= the
 *                               largest batch_max.  `next_deadline_ns` as preba_batcher_poll.
 * Calls on one batcher may come from several threads (one lock per batcher).
 */
typedef struct preba_bucket_batcher preba_bucket_batcher_t;
preba_bucket_batcher_t* preba_bucket_batcher_create(uint32_t n_buckets, uint64_t window,
                                                    const uint32_t* batch_max,
                                                    uint64_t time_queue_ns);
void preba_bucket_batcher_destroy(preba_bucket_batcher_t* b);
int preba_bucket_batcher_push(preba_bucket_batcher_t* b, uint64_t id, uint64_t arrival_ns,
                              uint64_t length);
int preba_bucket_batcher_poll(preba_bucket_batcher_t* b, uint64_t now_ns, uint64_t* ids,
                              uint32_t capacity, uint64_t* next_deadline_ns);

/*
 * preba_serve_run — a measuring aid for the whole front-end under load (paper Sec. 5 "Input
 * query modeling": single-input requests whose arrival times follow a Poisson process;
 * Sec. 2.3 item 2 and Sec. 4.3: the batching queue with Batch_max and Time_queue; Sec. 3:
 * several servers sharing one GPU).  Runs in real time: one thread puts request i into a
 * preba_batcher queue when the clock reaches arrival_ns[i]; one thread per server polls the
 * queue, takes the batch that is due, runs it through preba_preprocess_images with
 * PREBA_IMAGES_IN_PLACE on the server's stream, waits for the stream and stamps the batch's
 * requests with the completion time.  Requests leave in arrival order, so every batch is a run
 * of consecutive requests.  Returns when every request has been served.  Unlike the transform's
 * entry points this one creates threads, a queue and blocks; it allocates nothing on the device.
 *   arrival_ns        HOST, n_requests times in ns from the start of the run, non-decreasing
 *   image_index       HOST, n_requests: the pool image request i carries
 *   pool_images/h/w   HOST arrays of pool_size entries: decoded images in pinned memory as
 *                     PREBA_IMAGES_IN_PLACE wants them (128-byte aligned, device-addressable)
 *   batch_max, time_queue_ns   the queue's two hyper-parameters (preba_batching_params)
 *   n_servers         1..64; table_host, out_host, dev_table, dev_out, dev_status, dev_scratch
 *                     and streams are arrays of n_servers pointers, one staging set per server
 *                     as preba_image_batch_t describes them, each sized for batch_max images
 *                     (dev_status and dev_scratch, or single entries of them, may be NULL)
 *   out_arena         HOST pinned, n_requests results, or NULL: with it request i's result is
 *                     kept at i * 3 * out_size^2 * sizeof(element); without it every server
 *                     writes its batches' results to its own out_host again and again
 *   done_ns           HOST, n_requests, written: completion time of each request (ns from start)
 *   batch_size, batch_first, batch_release_ns, batch_server
 *                     HOST, n_requests entries each, written for batches 0 .. *n_batches - 1 (in
 *                     no particular order): images in the batch, its first request, the time
 *                     the queue released it, the server that ran it
 * Errors: PREBA_ERR_INVALID_ARG, and whatever preba_preprocess_images returns.
 */
typedef struct {
  const uint64_t* arrival_ns;
  const uint32_t* image_index;
  uint32_t n_requests;
  uint32_t pool_size;
  const uint8_t* const* pool_images;
  const uint32_t* pool_h;
  const uint32_t* pool_w;
  uint32_t batch_max;
  uint32_t n_servers;
  uint64_t time_queue_ns;
  uint32_t out_size;
  uint32_t resize_short;
  float mean[3];
  float std[3];
  int32_t out_dtype;
  int32_t device;                /* CUDA device the servers' streams and staging belong to */
  preba_img_t* const* table_host;
  void* const* out_host;
  preba_img_t* const* dev_table;
  void* const* dev_out;
  int32_t* const* dev_status;
  uint32_t* const* dev_scratch;
  void* const* streams;
  void* out_arena;
  uint64_t* done_ns;
  uint32_t* batch_size;
  uint32_t* batch_first;
  uint64_t* batch_release_ns;
  uint32_t* batch_server;
} preba_serve_t;
int preba_serve_run(const preba_serve_t* serve, uint32_t* n_batches);

/*
 * Audio path — the paper's second preprocessing pipeline (Table 1 units "Mel spectrogram" and
 * "Normalize"; Sec. 2.3 item 1: a Fourier transform followed by a Mel filterbank;
 * Sec. 4.2: Normalize as three passes, the mean over all samples, the variance from that mean,
 * then the normalisation).  Samples are taken at 16 kHz; preba_audio_resample (below) brings
 * other rates there.  The paper
 * fixes no numerics; the readings are: frames of 400 samples every 160 (no padding, so
 * T = 1 + (L - 400)/160 frames for L >= 400, else 0), periodic Hann window, zero-padding to a
 * 512-point DFT, power spectrum, 80 unit-height triangular filters equally spaced on the HTK
 * mel scale between 0 and 8000 Hz, natural log of (energy + 2^-24), and per utterance and
 * filter (x - mean)/(sqrt(var) + 1e-5) over the utterance's frames, var = mean squared
 * deviation.  fp32 arithmetic on the device.
 *
 * A ragged batch is one float buffer with every utterance starting at a multiple of
 * PREBA_AUDIO_ALIGN samples (padding samples are 0) and a table {offset, length, frames}.
 * The result is [n, 80, t_max] float32, t_max the largest frame count of the batch; frames
 * beyond an utterance's own count are written as 0.
 */
#define PREBA_AUDIO_ALIGN 4u     /* samples: every utterance starts on a 16-byte boundary */
#define PREBA_AUDIO_RATE 16000u
#define PREBA_AUDIO_WIN 400u
#define PREBA_AUDIO_HOP 160u
#define PREBA_AUDIO_NFFT 512u
#define PREBA_AUDIO_MELS 80u
#define PREBA_AUDIO_MAX_SAMPLES (1u << 28) /* per utterance */

typedef struct {
  uint64_t offset; /* in samples from the start of the sample buffer, multiple of PREBA_AUDIO_ALIGN */
  uint32_t length; /* samples */
  uint32_t frames; /* 1 + (length - 400)/160, or 0 when length < 400 */
} preba_utt_t;

typedef struct {
  uint64_t packed_samples; /* floats in the packed sample buffer */
  uint64_t table_bytes;    /* n * sizeof(preba_utt_t) */
  uint64_t out_bytes;      /* n * 80 * t_max * 4 */
  uint32_t t_max;          /* largest frame count of the batch */
  uint32_t reserved;
} preba_audio_sizes_t;

typedef struct {
  const float* samples;          /* DEVICE, 16-byte aligned, packed as preba_audio_pack lays out */
  uint64_t samples_count;        /* floats readable at `samples` */
  const preba_utt_t* table;      /* DEVICE, n entries */
  const preba_utt_t* table_host; /* HOST copy for checking before launch, or NULL */
  uint32_t n;
  uint32_t t_max;                /* frames per utterance in `out` (>= every entry's frames) */
  float* out;                    /* DEVICE, [n, 80, t_max] contiguous */
  uint64_t out_bytes;
  int32_t* status;               /* DEVICE word or NULL: first PREBA_ERR_* the kernels meet */
} preba_audio_batch_t;

/* Sizes for a batch of utterances of the given lengths (host arithmetic).
 * Errors: PREBA_ERR_INVALID_ARG (NULL, n == 0, a length above PREBA_AUDIO_MAX_SAMPLES). */
int preba_audio_query(const uint32_t* lengths, uint32_t n, preba_audio_sizes_t* sizes);

/* Builds the packed sample buffer (padding written as 0) and the table from n separate
 * utterances.  Errors: PREBA_ERR_INVALID_ARG, PREBA_ERR_BUFFER_TOO_SMALL. */
int preba_audio_pack(const float* const* utterances, const uint32_t* lengths, uint32_t n,
                     float* packed, uint64_t capacity_samples, preba_utt_t* table);

/* Bits of the `normalize` argument of preba_audio_logmel.  With PREBA_AUDIO_OVERLAP_PREVIOUS
 * the spectrogram kernel starts without waiting for the kernels before it on the stream
 * (programmatic dependent launch: its CTAs move in while the Normalize kernel of the batch
 * before is still running), under the contract of PREBA_OVERLAP_PREVIOUS: it may run beside
 * every kernel back to the last operation on the stream that was not marked, so it must share
 * no buffer with any of them; completion stays in stream order. */
#define PREBA_AUDIO_NORMALIZE 1
#define PREBA_AUDIO_OVERLAP_PREVIOUS 2

/* Mel spectrogram (+ Normalize when bit PREBA_AUDIO_NORMALIZE of `normalize` is set) of a
 * device-resident batch:
 * enqueues one kernel for the log Mel energies (the frame pairs of the batch are shared out
 * evenly over the warps of a grid that fills the GPU once; a warp transforms two frames with
 * one complex 512-point FFT held in registers) and, when normalising, one more for the three
 * passes over every (utterance, filter) row, launched so that it is scheduled while the first
 * drains and waits for it on the device; then returns.  No allocation, no synchronisation.  A table
 * entry that is misaligned, runs past the samples or whose frame count does not follow from
 * its length is refused on the host when `table_host` is given (PREBA_ERR_BAD_TABLE) and
 * skipped and reported by the kernel otherwise.
 * Errors: PREBA_ERR_INVALID_ARG (also: bits of `normalize` other than the two above),
 * PREBA_ERR_BUFFER_TOO_SMALL, PREBA_ERR_BAD_TABLE, PREBA_ERR_CUDA. */
int preba_audio_logmel(const preba_audio_batch_t* batch, int normalize, void* stream);

/*
 * Resample — the first audio unit of Table 1 ("resampling", Sec. 2.3 item 1), for utterances
 * that do not arrive at the model's rate.  The paper only names it; the reading is the
 * classical bandlimited interpolation with a Hann-windowed sinc, six zero crossings each
 * side, cutoff at 0.99 of the lower Nyquist frequency:
 *   y[m] = sum_n x[n] * h(n - m*rate_in/rate_out),  h(t) = fc*sinc(fc*t)*cos^2(pi*fc*t/12)
 *   for |fc*t| < 6 (else 0),  fc = 0.99*min(1, rate_out/rate_in),
 * M = ceil(L*rate_out/rate_in) outputs per utterance, samples outside the utterance taken
 * as 0; fp32 on the device.
 *
 * preba_audio_layout          the table {offset, length, frames} of a packed buffer for the
 *                             given lengths (offsets as preba_audio_pack lays them out), without
 *                             copying samples.
 * preba_audio_resample_query  the output length of every utterance (HOST arithmetic).
 * preba_audio_resample        enqueues one kernel on `stream`: every utterance of the packed
 *                             input (DEVICE `samples_in`, `table_in`) is resampled into its
 *                             place in the packed output (DEVICE `samples_out`, `table_out`,
 *                             whose lengths must be those of the query; alignment padding is
 *                             written as 0).  `longest_out` is the largest output length.
 *                             Rate pairs whose phase table (rate_out/gcd phases of about
 *                             12*rate_in/rate_out + 4 taps) exceeds 12000 entries are refused.
 *                             A table entry that is misaligned, runs past its buffer or whose
 *                             output length does not follow from its input length is skipped
 *                             and PREBA_ERR_BAD_TABLE stored in `status`.
 * Errors: PREBA_ERR_INVALID_ARG, PREBA_ERR_CUDA.
 */
int preba_audio_layout(const uint32_t* lengths, uint32_t n, preba_utt_t* table);
int preba_audio_resample_query(const uint32_t* lengths_in, uint32_t n, uint32_t rate_in,
                               uint32_t rate_out, uint32_t* lengths_out);
int preba_audio_resample(const float* samples_in, uint64_t samples_in_count,
                         const preba_utt_t* table_in, float* samples_out,
                         uint64_t samples_out_count, const preba_utt_t* table_out, uint32_t n,
                         uint32_t longest_out, uint32_t rate_in, uint32_t rate_out,
                         int32_t* status, void* stream);

/*
 * JPEG Decode -- the first unit of the paper's image pipeline (Table 1 "Decode", the largest
 * image unit of its accelerator; Sec. 2.3 item 1: JPEG to RGB; Sec. 4.2: Decode -> Resize ->
 * Crop -> Normalize chained in one compute unit).  The paper fixes no numerics; the decoder
 * follows ITU-T T.81 for baseline sequential DCT streams (SOF0, 8-bit samples, Huffman coding,
 * one interleaved scan, restart intervals; one component, or three with the luma sampled 1 or 2
 * times the chroma on each axis).  Readings where the standard leaves a choice (it only bounds
 * the accuracy of the inverse transform): the inverse DCT of A.3.3 in exact integers -- the basis
 * as round(2^20 (C_u / 2) cos((2x+1) u pi / 16)), dequantised coefficients limited to +-16383,
 * horizontal sums first, reduced to floor((t + 2^8) / 2^9), vertical sums, level shift and one
 * rounding floor((s + 128 * 2^31 + 2^30) / 2^31), clamp -- within one of the rounded real-valued
 * transform; chroma enlarged by pixel replication; YCbCr -> RGB by the JFIF equations on the
 * 8-bit samples with the coefficients as round(2^16 c) (91881, 22553, 46802, 116130) and one
 * rounding floor((x + 2^15) / 2^16), clamp.  Every decoder that follows these steps produces the
 * same bytes.  Other streams are refused with PREBA_ERR_UNSUPPORTED.
 *
 * preba_jpeg_query   reads the headers of n streams (HOST pointers and sizes): writes every
 *                    image's height and width (h, w: HOST, n entries, or NULL) and the sizes
 *                    of the buffers preba_jpeg_decode needs.
 * preba_jpeg_decode  decodes the batch into the packed pixel buffer and {offset, h, w} table
 *                    that preba_preprocess reads (the layout of preba_pack), so the transform
 *                    can follow on the same stream.  The host writes one descriptor per image
 *                    (sizes, tables) and the entropy-coded bytes into `stage_host`; enqueued on
 *                    `stream`: the copy of the staging buffer and of the table, the clearing of
 *                    the coefficient buffer, and three kernels (restart markers found per
 *                    image; a thread per restart interval decodes its Huffman codes into
 *                    quantised coefficients; a block per MCU dequantises, transforms,
 *                    converts and stores).  Streams without restart intervals decode on one
 *                    thread each.  A stream that turns out damaged while decoding (a code that
 *                    does not exist, restart markers that do not match the header) leaves its
 *                    remaining blocks grey and PREBA_ERR_BAD_STREAM in `status`.
 * Ownership: everything is the caller's; stage_host and table_host must stay valid until the
 * stream has passed the copies (pinned memory for them to be asynchronous).
 * Errors: PREBA_ERR_INVALID_ARG, PREBA_ERR_BAD_STREAM, PREBA_ERR_UNSUPPORTED,
 * PREBA_ERR_BUFFER_TOO_SMALL, PREBA_ERR_CUDA.
 */
typedef struct {
  uint64_t stage_bytes;  /* staging, host and device: descriptors, segment tables, scans */
  uint64_t coef_bytes;   /* device: the int16 coefficients of every block */
  uint64_t packed_bytes; /* device: the decoded pixels, packed as preba_pack lays them out */
  uint64_t table_bytes;  /* n * sizeof(preba_img_t) */
} preba_jpeg_sizes_t;

typedef struct {
  const uint8_t* const* jpegs; /* HOST array of n HOST pointers: the streams */
  const uint64_t* bytes;       /* HOST, n entries: their sizes */
  uint32_t n;                  /* 1 .. 65535 */
  uint32_t reserved;
  uint8_t* stage_host;         /* HOST (pinned), stage_bytes, 16-byte aligned: written by the call */
  uint8_t* stage_dev;          /* DEVICE, stage_bytes, 16-byte aligned */
  uint64_t stage_bytes;
  int16_t* coef;               /* DEVICE, coef_bytes, 16-byte aligned */
  uint64_t coef_bytes;
  uint8_t* pixels;             /* DEVICE, 16-byte aligned: receives the packed pixels */
  uint64_t pixels_bytes;
  preba_img_t* table;          /* DEVICE, n entries: receives the table */
  preba_img_t* table_host;     /* HOST (pinned), n entries: receives the same table */
  int32_t* status;             /* DEVICE word or NULL, as preba_batch_t.status */
} preba_jpeg_batch_t;

int preba_jpeg_query(const uint8_t* const* jpegs, const uint64_t* bytes, uint32_t n, uint32_t* h,
                     uint32_t* w, preba_jpeg_sizes_t* sizes);
int preba_jpeg_decode(const preba_jpeg_batch_t* batch, void* stream);

/* Text for a PREBA_* code (static storage, never NULL). */
const char* preba_strerror(int code);

/* The cudaError_t value behind the calling thread's last PREBA_ERR_CUDA, else 0. */
int preba_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* PREBA_H_ */
