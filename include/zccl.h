/*
 * zccl.h -- C boundary of the B200 (sm_100a) implementation of ZCCL's data-parallel hot path:
 * the fZ-light error-bounded lossy codec, the fused decompress-reduce-recompress hop of the ring
 * reduce-scatter, and N-rank ring collectives emulated on N buffers in one GPU's memory.
 *
 * Conventions that hold for every entry point unless its comment says otherwise
 *   - Pointers marked [device] are device pointers owned by the caller; [host] are host pointers.  The library
 *     owns only what zccl_ctx_create allocates and never allocates, frees or synchronises on the hot path.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).  Calls only enqueue work;
 *     they return before it has run.  Operations that share one context must be ordered on one stream (the
 *     context's scan workspace is shared); use one context per concurrently used stream.
 *   - Return value: ZCCL_OK, or a negative ZCCL_E_* for what the host can see at once (bad arguments, capacity
 *     below the fixed part of a stream, CUDA launch failure).  What only the device can see (capacity overrun,
 *     values out of range, malformed stream, degenerate range, scan time-out, precision warning) is recorded in
 *     a device status word that zccl_status() reads and clears.  No kernel ever writes outside the capacities it
 *     was given; after a device-side error the contents of the output are unspecified.
 *   - fp32 data only.  Arithmetic is IEEE binary32, round to nearest even, no fused multiply-add, so that
 *     streams and reconstructions are reproducible bit for bit.
 *
 * Stream layout (little endian; the paper, Section 3.3 and Section 3.5.2, fixes the ingredients: per-unit 4-byte
 * outlier, per-block sign bits and one-byte code length, fixed-length bits, constant blocks stored as the code
 * length alone, 4-byte per-chunk sizes gathered at the front of the buffer.  Their order and the header are this
 * library's choice):
 *   header 32 B : u32 magic "ZCL1"; u32 0x05000001; u64 n; f32 eb_abs; f32 s (step); u32 T = 4096; u32 nT
 *   index 4*nT B: u32 per tile, inclusive prefix sum of tile blob sizes in 4-byte words
 *   blobs       : per tile [i32 quantised first value][code-length byte per 32-element block, padded to 4 B]
 *                 [per block with code length L > 0: u32 sign word, then L bit-plane words of |delta|]
 */
#ifndef ZCCL_H
#define ZCCL_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct zccl_ctx zccl_ctx;

/* How `eb` is read.  The paper's tables quote value-range-relative bounds ("REL", Tables 1-4). */
enum { ZCCL_EB_ABS = 0,    /* eb is the absolute bound eb_abs */
       ZCCL_EB_REL = 1,    /* eb_abs = eb * (max - min) of the input (of all ranks' inputs in zccl_sim_*) */
       ZCCL_EB_RESOLVED = 2 };  /* the bound zccl_resolve_range left in the context, on the device; eb is ignored */

enum { ZCCL_OK = 0,
       ZCCL_E_ARG = -1,         /* NULL pointer, size beyond the context's limits, eb not positive and finite */
       ZCCL_E_CUDA = -2,        /* a CUDA runtime call failed */
       ZCCL_E_CAPACITY = -3,    /* an output buffer is too small */
       ZCCL_E_RANGE = -4,       /* some |x / s| >= 2^30: codes do not fit 32-bit deltas */
       ZCCL_E_BAD_STREAM = -5,  /* magic, version, sizes or index of a compressed stream are inconsistent */
       ZCCL_E_TIMEOUT = -6,     /* a bounded device-side wait in the placement scan expired */
       ZCCL_E_DEGENERATE = -7,  /* REL bound on an input whose range is zero (use ZCCL_EB_ABS) */
       ZCCL_E_TOO_LARGE = -8,   /* more elements than the fixed scratch of zccl_compress_noalloc can place */
       ZCCL_W_PRECISION = 1 };  /* some |code| > 2^15: fp32 rounding may exceed eb_abs by about |x| * 1.8e-7 */

/* Flags of the reduce hop and of zccl_sim_allreduce. */
enum { ZCCL_CONSISTENT_OWNER = 1u };  /* owner's copy of a reduced chunk = dequantised value, not the raw sum */
/* Reduce operation of the collective computation framework (Section 3.2: Sum, Average, Max, Min), or-ed into `flags`.
 * Max and Min keep the decoded operand when the two compare equal.  Average is a Sum on every hop; the Allreduce
 * divides every rank's result by the number of ranks at the end (one fp32 division per element). */
enum { ZCCL_OP_SUM = 0u, ZCCL_OP_MAX = 2u, ZCCL_OP_MIN = 4u, ZCCL_OP_AVG = 6u, ZCCL_OP_MASK = 6u };

enum { ZCCL_TILE = 4096, ZCCL_BLOCK = 32, ZCCL_HEADER_BYTES = 32, ZCCL_MAX_RANKS = 64,
       ZCCL_NOALLOC_MAX_ELEMS = 1 << 26 };  /* element limit of zccl_compress_noalloc (256 MiB of fp32) */

/*
 * Context: placement workspace for streams of up to `max_elems` elements (a slot of 4128 bytes per 1024 elements, in
 * which an encoded round waits for its place in the stream: about 1.01 times the size of the largest input, plus a
 * few words per tile), the device status word, the resolved-bound block and, when max_ranks >= 2, an arena of compressed-chunk slots for zccl_sim_* sized for
 * max_ranks ranks exchanging max_elems elements in total per rank buffer (about (max_ranks + 2) *
 * zccl_compress_bound(max_elems) bytes).  Allocates on the current device; the only allocating call.
 * Returns ZCCL_E_ARG for max_elems == 0 or max_ranks outside [0, ZCCL_MAX_RANKS], ZCCL_E_CUDA if allocation fails.
 */
int zccl_ctx_create(zccl_ctx** ctx /*[host] out*/, size_t max_elems, int max_ranks);

/* Frees everything the context owns (synchronises the device first).  NULL is allowed. */
void zccl_ctx_destroy(zccl_ctx* ctx);

/* Worst-case stream size in bytes for n elements (every block at code length 31).  Pure host function. */
size_t zccl_compress_bound(size_t n);

/*
 * Synchronises `stream`, returns the most severe condition recorded on the device since the last call
 * (TIMEOUT, DEGENERATE, BAD_STREAM, RANGE, CAPACITY in that order, then the warning, ZCCL_OK if none) and clears
 * the record.
 */
int zccl_status(zccl_ctx* ctx, void* stream);

/* Number of kernels this library has launched in this process so far (for launch accounting in benchmarks;
 * no paper counterpart).  Pure host function. */
unsigned long long zccl_launch_count(void);

/*
 * Test hook for the bounded waits of the single-pass encoder (failure detection; no paper counterpart).  That
 * encoder, which zccl_compress_noalloc always uses, places tiles by a decoupled look-back: a warp waits, with a
 * poll limit, for the sizes of the tiles in front of its own.  While the hook is set, zccl_compress takes the same
 * encoder instead of its two wait-free launches and does not publish the size of tile number `tile` of a launch,
 * so the tiles after it find nothing to wait for: their look-back gives up after its poll limit (a fraction of a
 * second), writes nothing for those tiles and records ZCCL_E_TIMEOUT; the context stays usable.  tile < 0 switches
 * the hook off (the default).
 */
int zccl_debug_skip_publish(zccl_ctx* ctx, long long tile);

/*
 * Test hook for the launch counter that validates the scan states (no paper counterpart): sets it to `value`
 * (1 .. 2^31 - 1) on `stream`, so that a test can run the launches on both sides of its wrap-around, where every
 * scan state is cleared.  Must not overlap with other work on the context.  Returns ZCCL_E_ARG for a value
 * outside the range, ZCCL_E_CUDA if the copy cannot be queued.
 */
int zccl_debug_set_launch_counter(zccl_ctx* ctx, unsigned int value, void* stream);

/* Static description of a status code. */
const char* zccl_strerror(int code);

/*
 * fZ-light compression (Section 3.3; stream with the chunk-size index of Section 3.5.2).
 * Per 4096-element tile: q_i = rint(x_i * r), r = 1/s, s = 2 * (eb_abs * (1 - 2^-6)); 1-D Lorenzo deltas with the
 * tile's first code kept as a 4-byte outlier; per 32-element block the code length L = bit length of the largest
 * |delta| and, if L > 0, sign bits and L bit planes.  Two launches, neither of which has a block waiting for
 * another: rounds of 1024 elements are encoded into fixed slots of the context's workspace, then placed in the
 * stream from the prefix sums of their sizes.
 *   x [device]          n floats (finite values); may be NULL only if n == 0
 *   out [device]        receives the stream; 4-byte aligned; out_capacity bytes writable
 *   out_bytes [device]  one size_t, receives the stream length in bytes (readable after the stream has run)
 * Host-side errors: ZCCL_E_ARG (NULLs, n > max_elems, eb <= 0 or not finite, bad mode),
 * ZCCL_E_CAPACITY (out_capacity < 32 + 4 * ceil(n / 4096)).  Device-side: CAPACITY (a tile would pass
 * out_capacity; nothing is written beyond it), RANGE, DEGENERATE (REL with max == min), W_PRECISION.
 */
int zccl_compress(zccl_ctx* ctx, const float* x, size_t n, int eb_mode, float eb,
                  void* out, size_t out_capacity, size_t* out_bytes, void* stream);

/*
 * fZ-light decompression (Section 3.3, Section 3.5.2): tile starts come from the index at the front; per block the
 * magnitudes are rebuilt from the bit planes, signs applied, the Lorenzo recurrence undone by a running integer
 * sum from the tile's outlier, and x'_i = float(q_i) * s.
 *   in [device]   the stream; at most in_bytes_max bytes are read; 4-byte aligned
 *   y [device]    receives n floats, n taken from the stream's header; y_capacity_elems must be >= n
 * Host-side errors: ZCCL_E_ARG, ZCCL_E_CAPACITY (in_bytes_max < 32).  Device-side: BAD_STREAM (nothing outside
 * in_bytes_max is read, inconsistent tiles are skipped), CAPACITY (n > y_capacity_elems: nothing is written).
 */
int zccl_decompress(zccl_ctx* ctx, const void* in, size_t in_bytes_max,
                    float* y, size_t y_capacity_elems, void* stream);

/*
 * One reduce-scatter hop of the collective computation framework (Section 3.1.2; error chain of Eq. 2):
 * out_c = compress( decompress(in_c) + local ): decoding, reduction and encoding happen in one kernel, round by
 * round in shared memory, with no uncompressed intermediate in global memory; a second, small launch places the
 * encoded rounds in the stream, as for zccl_compress.  No block of either launch waits for another block, so
 * hops of several contexts may run side by side on one device whatever share of it each gets.
 * y_i = fl32( fl32(float(q_i) * s) + local_i ), the decoded operand on the left; bound and step are in_c's.
 * With ZCCL_OP_MAX / ZCCL_OP_MIN in flags the addition becomes the larger / the smaller of the two operands.
 *   in_c [device]      received compressed chunk (at most in_bytes_max bytes are read)
 *   local [device]     this rank's uncompressed chunk, n floats (the paper's form), or NULL
 *   local_c [device]   instead of `local`: a second compressed chunk of the same n and step (at most
 *                      local_c_bytes_max bytes are read).  Exactly one of local / local_c is non-NULL.
 *   n                  element count; must equal the count in in_c's header (else BAD_STREAM on the device)
 *   out_c, out_capacity, out_bytes [device]  as in zccl_compress
 *   raw_out [device]   NULL, or n floats receiving y (with ZCCL_CONSISTENT_OWNER in flags: float(q(y)) * s)
 * Errors as for zccl_compress and zccl_decompress.
 */
int zccl_decompress_reduce_compress(zccl_ctx* ctx, const void* in_c, size_t in_bytes_max,
                                    const float* local, const void* local_c, size_t local_c_bytes_max, size_t n,
                                    void* out_c, size_t out_capacity, size_t* out_bytes,
                                    float* raw_out, unsigned flags, void* stream);

/*
 * zccl_compress for callers that cannot allocate device memory (the paper has no counterpart: this is an addition
 * of this library).  Work captured into a CUDA graph or running where an allocation would synchronise or is not
 * allowed, plug-ins living inside a host application's fixed memory budget, and out-of-memory or teardown
 * handlers cannot call zccl_ctx_create, because it calls cudaMalloc.  This entry point needs no context: its
 * placement-scan workspace is a fixed array inside the library (about 140 KiB of device memory on every GPU that
 * loads the library, until the process exits), and it calls no cudaMalloc, cudaFree or other allocating routine.
 * Having no room for per-round slots, it compresses in a single pass (a warp per tile, positions by a decoupled
 * look-back with bounded waits) instead of the two launches of zccl_compress.
 *   x, out, out_capacity, out_bytes [device], stream: as in zccl_compress;  eb_abs: absolute error bound
 *   n: at most ZCCL_NOALLOC_MAX_ELEMS, else ZCCL_E_TOO_LARGE is returned and nothing is enqueued
 * Produces the same bytes as zccl_compress(ctx, x, n, ZCCL_EB_ABS, eb_abs, ...).  There is no status word to read:
 * if the device detects an error (capacity overrun, value out of range) *out_bytes is set to 0 and the contents of
 * `out` are unspecified; the precision warning is not reported.
 * The first call on a device looks up the array's device address (a host-side look-up: nothing is enqueued, the
 * array's counters carry their starting values in the module image), so the first call may come from any thread,
 * on any stream, inside a capture or not.  All calls on a device share the array, which keeps the previous call's
 * contents (each call re-arms what it needs): calls whose kernels could overlap on the GPU, for example on two
 * streams, race and must be ordered by the caller.
 */
int zccl_compress_noalloc(const float* x, size_t n, float eb_abs, void* out, size_t out_capacity,
                          size_t* out_bytes, void* stream);

/*
 * Ring Allreduce (sum) over nranks rank buffers in this GPU's memory (Section 3.5: ring reduce-scatter in the
 * collective computation framework, then ring allgather in the data movement framework).
 * Chunk c = elements [c*m, (c+1)*m) of every buffer, m = ceil(n_per_rank / nranks).  Rank r compresses chunk r;
 * on hop k = 0..nranks-2 rank r takes rank r-1's stream of chunk (r-k-1) mod nranks, and runs the fused hop with
 * its own uncompressed chunk; the last hop also leaves the reduced chunk (r+1) mod nranks uncompressed at its
 * owner r.  Then nranks-1 forwarding hops copy compressed chunks between per-rank slots and every rank
 * decompresses the nranks-1 chunks it does not own.  One bound for the whole collective; with ZCCL_EB_REL it is
 * eb times the range over all ranks' inputs.
 *   send [host]  nranks device pointers, each n_per_rank floats (read only)
 *   recv [host]  nranks device pointers, each n_per_rank floats (must not overlap send)
 * Needs a context created with max_ranks >= nranks and max_elems >= n_per_rank.
 */
int zccl_sim_allreduce(zccl_ctx* ctx, const float* const* send, float* const* recv, int nranks,
                       size_t n_per_rank, int eb_mode, float eb, unsigned flags, void* stream);

/*
 * Ring Allgather in the data movement framework (Section 3.1.1, Section 3.5.1): each rank compresses its
 * n_per_rank elements once, compressed bytes are forwarded nranks-1 times, each rank decompresses the nranks-1
 * foreign contributions and copies its own uncompressed.
 *   send [host]  nranks device pointers, each n_per_rank floats
 *   recv [host]  nranks device pointers, each nranks * n_per_rank floats
 * Needs a context with max_ranks >= nranks and max_elems >= nranks * n_per_rank.
 */
int zccl_sim_allgather(zccl_ctx* ctx, const float* const* send, float* const* recv, int nranks,
                       size_t n_per_rank, int eb_mode, float eb, void* stream);

/*
 * Broadcast in the data movement framework (Section 3.1.1): the root compresses once; each of the nsinks
 * receivers gets a copy of the compressed bytes and decompresses it once.
 *   root [device] n floats;  recv [host] nsinks device pointers, each n floats
 * Needs a context with max_ranks >= nsinks and max_elems >= n.
 */
int zccl_sim_bcast(zccl_ctx* ctx, const float* root, float* const* recv, int nsinks, size_t n,
                   int eb_mode, float eb, void* stream);

/*
 * Ring Reduce-scatter (sum) as a collective of its own (Section 3.1.2; the first stage of the Allreduce of
 * Section 3.5 with the ring shifted so that rank r ends with chunk r): chunk c is compressed by rank c+1, travels
 * c+1 -> c+2 -> ... -> c, every receiver runs the fused hop with its own piece of chunk c, and the last one keeps
 * the uncompressed sum.  Chunks as for zccl_sim_allreduce.
 *   send [host]  nranks device pointers, each n_per_rank floats (read only)
 *   recv [host]  nranks device pointers; recv[r] receives the elements of chunk r (at most ceil(n_per_rank / nranks))
 * Needs a context created with max_ranks >= nranks and max_elems >= n_per_rank.
 */
int zccl_sim_reduce_scatter(zccl_ctx* ctx, const float* const* send, float* const* recv, int nranks,
                            size_t n_per_rank, int eb_mode, float eb, void* stream);

/*
 * Scatter over a binomial tree in the data movement framework (Section 4.4): rank 0 holds nranks chunks of
 * n_per_rank elements, compresses chunks 1..nranks-1 once each (one bound for the whole buffer; with ZCCL_EB_REL
 * eb times its range), the tree forwards compressed bytes only (in the round with distance d = the largest power
 * of two below nranks, then d/2, ..., 1, holder h hands the chunks h+d .. h+2d-1 to rank h+d), and every rank
 * decompresses its own chunk; chunk 0 is copied as it is.
 *   root [device] nranks * n_per_rank floats;  recv [host] nranks device pointers, each n_per_rank floats
 * Needs a context with max_ranks >= nranks and max_elems >= nranks * n_per_rank.
 */
int zccl_sim_scatter(zccl_ctx* ctx, const float* root, float* const* recv, int nranks, size_t n_per_rank,
                     int eb_mode, float eb, void* stream);

/*
 * Compressed sizes of the last zccl_sim_* call, for reporting ratios (the paper's compressed_sizes array,
 * Section 3.5.1).  Synchronises `stream`.  sizes [host] receives up to `capacity` entries and the call returns how
 * many there are: allreduce nranks*nranks (entry k*nranks + r = bytes rank r produced at step k, k = 0 the
 * initial compression), allgather nranks, bcast 1, reduce_scatter (nranks-1)*nranks (as for allreduce), scatter
 * nranks (entry c = bytes of chunk c, 0 for the root's own).  Negative on error.
 */
int zccl_sim_sizes(zccl_ctx* ctx, size_t* sizes, int capacity, void* stream);

/*
 * Quality of a reconstruction y of x (Section 4.1: NRMSE and PSNR, reported next to the bit rate 32 / ratio),
 * computed in fp64 on the device.
 *   x, y [device] n floats (n >= 1, n <= max_elems of the context)
 *   out  [device] 6 doubles: max |x - y|, MSE = mean (x - y)^2, NRMSE = sqrt(MSE) / (max x - min x),
 *                 PSNR = 20 log10((max x - min x) / sqrt(MSE)) in dB, min x, max x.
 * A constant x gives NaN for NRMSE and PSNR; an exact reconstruction gives PSNR = +inf.  Sums are formed per
 * thread, per CTA and then over the CTAs in a fixed order, so the result does not vary from run to run.
 * Returns ZCCL_E_ARG for a null pointer, n == 0 or n beyond the context's max_elems.
 */
int zccl_quality(zccl_ctx* ctx, const float* x, const float* y, size_t n, double* out, void* stream);

/*
 * Other tile sizes.  The tile (elements per Lorenzo restart and per index entry) is a header field of the stream;
 * Section 3.5.2 cuts the data into chunks of 5120 points.  The entry points above are built around 4096; these two
 * take any tile size that is a multiple of 32 between 1024 and 8192 and produce and accept exactly the streams the
 * format defines for that tile size: two launches to compress and one to decompress, on kernels of the same design
 * as those for 4096 (a tile is ceil(tile / 1024) rounds of 1024 elements; the context's round slots cover every
 * n <= max_elems when the tile size is a multiple of 1024, and n <= max_elems * 4 * tile / (4096 * ceil(tile / 1024))
 * otherwise; larger inputs are compressed by plain kernels, three launches and several times slower).
 * Arguments, asynchrony and error reporting are those of zccl_compress and zccl_decompress; a stream whose header
 * names another tile size than `tile` sets ZCCL_E_BAD_STREAM.  ZCCL_E_ARG also for a tile size outside the range.
 * zccl_compress_bound_tiled returns 0 for such a tile size.
 */
size_t zccl_compress_bound_tiled(size_t n, unsigned tile);
int zccl_compress_tiled(zccl_ctx* ctx, const float* x, size_t n, int eb_mode, float eb, unsigned tile,
                        void* out, size_t out_capacity, size_t* out_bytes /*device*/, void* stream);
int zccl_decompress_tiled(zccl_ctx* ctx, const void* in, size_t in_bytes_max, unsigned tile,
                          float* y, size_t y_capacity_elems, void* stream);

/*
 * Code-length statistics of a stream (Section 4.1 reports the percentage of constant blocks next to the ratio: a
 * block whose code length is 0 is a constant block and is stored as its one code-length byte).
 *   in   [device] stream, in_bytes_max readable bytes (4-byte aligned)
 *   hist [device] 33 x unsigned long long: hist[L], L = 0..31 = number of 32-element blocks stored with code length
 *        L; hist[32] = number of blocks.  Constant-block share = hist[0] / hist[32]; mean code length =
 *        sum L hist[L] / hist[32].
 * Enqueues on `stream`.  A stream that does not parse (magic, version, tile size, index beyond in_bytes_max, a code
 * length above 31) sets ZCCL_E_BAD_STREAM in the device status and leaves hist incomplete.  ZCCL_E_ARG for null or
 * misaligned pointers, ZCCL_E_CAPACITY when in_bytes_max is smaller than a header.
 */
int zccl_stream_stats(zccl_ctx* ctx, const void* in, size_t in_bytes_max, unsigned long long* hist, void* stream);

/*
 * The per-rank steps of a real ring that are not a codec call (Section 3.2: the error bound is resolved once
 * per collective, over the data of all ranks; Corollary 2: Average = Sum / N).
 *   zccl_range: minmax [device, 2 floats] <- (min, max) of x [device, n floats]; (+inf, -inf) when n == 0.  A
 *               rank combines these with its peers' (min of minima, max of maxima), forms
 *               eb_abs = fl32(eb * fl32(max - min)) and passes it to the codec calls as ZCCL_EB_ABS; that is the
 *               bound a ZCCL_EB_REL call over the concatenated data would resolve.
 *   zccl_resolve_range: the same resolution without the host: minmax [device, 2 floats] is the combined pair
 *               (for example after a Min/Max all-reduce of the ranks' pairs); the bound
 *               eb_abs = fl32(eb_rel * fl32(max - min)), its step and reciprocal go into the context's resolved-bound
 *               block, where zccl_compress and the zccl_*_host forms find them when called with ZCCL_EB_RESOLVED;
 *               eb_abs_out [device, 1 float, or NULL] also receives eb_abs (0 when the range is degenerate).  The
 *               block keeps its contents until the next zccl_resolve_range or ZCCL_EB_REL call on the context.
 *               Device-side: DEGENERATE when max - min is zero, negative, infinite or not a number; codec calls
 *               that use the block then write a header-less, empty stream (length 0).
 *   zccl_scale: y [device, n floats] <- y / divisor, one IEEE fp32 division per element.
 * All enqueue on `stream` and return at once.  ZCCL_E_ARG for null or misaligned pointers, n beyond the
 * context's max_elems (range), a bound or divisor that is not a positive finite number (resolve_range, scale).
 */
int zccl_range(zccl_ctx* ctx, const float* x, size_t n, float* minmax, void* stream);
int zccl_resolve_range(zccl_ctx* ctx, const float* minmax, float eb_rel, float* eb_abs_out, void* stream);

/*
 * The same resolution as a pure host function (no context, no device): from the combined minimum and maximum of the
 * data and the relative bound, eb_abs = fl32(eb_rel * fl32(mx - mn)), the quantisation step s = 2 * fl32(eb_abs *
 * (1 - 2^-6)) and its reciprocal r = fl32(1 / s), each by one IEEE fp32 operation, as the device computes them
 * (Section 3.2: one bound per collective).  Any of the three outputs [host] may be NULL.  Returns ZCCL_E_ARG for a
 * bound that is not a positive finite number, ZCCL_E_DEGENERATE when mx - mn is zero, negative, infinite or not a
 * number, or when step or reciprocal leave the finite range.
 */
int zccl_resolve_range_host(float mn, float mx, float eb_rel, float* eb_abs, float* step, float* reciprocal);
int zccl_scale(zccl_ctx* ctx, float* y, size_t n, float divisor, void* stream);

/*
 * fZ-light for binary64 input (Section 3.3 read for double precision; the paper's data sets are single precision and
 * it states no width).  Everything behind the quantisation is the codec above: 32-bit codes, 1-D Lorenzo deltas per
 * 4096-element tile, code length per 32-element block, sign word and bit planes, the index at the front.
 *   bound     eb_abs = eb (ZCCL_EB_ABS) or fl64(eb * fl64(max - min)) over the array (ZCCL_EB_REL)
 *   step      s = 2 * fl64(eb_abs * (1 - 2^-20)), r = fl64(1 / s)
 *   codes     q_i = nearest integer, ties to even, of fl64(x_i * r); RANGE unless every |x_i * r| < 2^30
 *   values    x'_i = fl64((double)q_i * s); |x_i - x'_i| <= eb_abs for every code in range (no precision warning)
 * The stream's version word carries data type 1 and header bytes 16..23 hold the step as one binary64; binary32
 * entry points reject such a stream and the other way round (BAD_STREAM).  Two launches to compress (rounds into the
 * context's slots, then the placement) and one to decompress, on kernels of the same design as the binary32 ones; an
 * array that does not start on a 16-byte boundary is read or written with plain accesses instead of the copy engine.
 *   x [device] n doubles, 8-byte aligned; y [device] receives n doubles; the rest as for zccl_compress / zccl_decompress.
 * Errors as for those two; ZCCL_E_DEGENERATE at once for a relative bound with n == 0.
 */
int zccl_compress_f64(zccl_ctx* ctx, const double* x, size_t n, int eb_mode, double eb,
                      void* out, size_t out_capacity, size_t* out_bytes, void* stream);
int zccl_decompress_f64(zccl_ctx* ctx, const void* in, size_t in_bytes_max, double* y, size_t y_capacity_elems, void* stream);

/*
 * Host-buffer convenience forms: copy the input from host memory into a staging area of the context, run the
 * device path, copy the result back, all enqueued on `stream` (pinned host memory makes the copies asynchronous).
 * They exist so that end-to-end cost including PCIe transfers can be measured through this boundary.
 *   zccl_compress_host:   x_host n floats -> out_host (out_capacity bytes) and *out_bytes_host; synchronises `stream`
 *                         (the length has to reach the host before the stream can be copied), so both are valid when
 *                         the call returns
 *   zccl_decompress_host: in_host in_bytes bytes -> y_host (y_capacity_elems floats), valid once `stream` has run; the
 *                         element count is read from in_host's header on the host when the call is made, so in_host
 *                         must hold the stream by then
 * Need max_elems >= n.  Errors as for the device forms.
 */
int zccl_compress_host(zccl_ctx* ctx, const float* x_host, size_t n, int eb_mode, float eb,
                       void* out_host, size_t out_capacity, size_t* out_bytes_host, void* stream);
int zccl_decompress_host(zccl_ctx* ctx, const void* in_host, size_t in_bytes,
                         float* y_host, size_t y_capacity_elems, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* ZCCL_H */
