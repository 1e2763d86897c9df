/*
 * mmv.h -- C ABI of the segmented scan / segmented sum / CSR SpMV library for
 * NVIDIA B200 (sm_100a).
 *
 * The library implements the data-parallel hot path of "Segmented Operations
 * using Matrix Multiplications" (MMV-RAM): the prefix sums inside each tile are
 * a tensor-core product of the data tile with a constant triangular all-ones
 * matrix (Section 1.2 "Notation": z = MATMUL(x, U_s); Algorithm A.1,
 * BlockSegScan), vector operations revert the speculation at segment
 * boundaries (Lemma A.1), and the per-block recursion of Section 4.2 is
 * replaced by a single-pass chained carry between tiles.
 *
 * Conventions for every entry point
 *   - All data pointers are DEVICE pointers unless a parameter says "host".
 *     The caller owns every buffer; the library allocates and frees no device
 *     memory and keeps no pointer after the call returns.  Two entry points
 *     hold resources of their own, each described at its declaration:
 *     mmv_seg_scan_static (a fixed buffer inside the library's device image)
 *     and mmv_seg_scan_host (three streams and nine events per device, made
 *     at its first call and kept until the process exits).
 *   - `workspace` is caller-provided device scratch of at least
 *     mmv_workspace_bytes(...) bytes, 256-byte aligned; its content on entry is
 *     irrelevant (the call initialises what it needs on the stream) and it must
 *     not be shared by calls that may overlap on the GPU.
 *   - Calls may overlap on the GPU (different streams, a workspace each).  The
 *     tensor-core kernels (scan, segmented sum, SpMV) need every thread block
 *     of their grid resident at once and are launched cooperatively: two such
 *     calls that meet on the GPU run one after the other rather than side by
 *     side, and where the process may use fewer SMs than the device reports
 *     (an MPS thread limit, a green context) the launch is refused with
 *     MMV_ERR_CUDA instead of stalling.
 *   - Work is enqueued on `cuda_stream` (a cudaStream_t passed as void*, NULL =
 *     the default stream); the call does not synchronise with the host.
 *     mmv_seg_scan, mmv_seg_sum and mmv_spmv_csr enqueue nothing but a memset
 *     and kernels, so they can be captured in a CUDA graph and replayed,
 *     provided one call was made on the device before the capture (the first
 *     call sets the kernels' attributes).
 *   - x, seg and out must be 16-byte aligned and must not overlap each other.
 *   - Argument errors are reported synchronously and nothing is enqueued.
 *     Conditions only the device can detect (a wait that ran out of its time
 *     budget, segment offsets that are not monotone) set a status word inside
 *     the workspace; outputs are then unspecified and
 *     mmv_last_async_status() reports the code.  No device trap, no unbounded
 *     wait.
 *   - n == 0 (nnz == 0, rows == 0) is valid: nothing is read; seg-sum / SpMV
 *     still write their (empty-segment) zeros.
 *
 * Segment encodings
 *   MMV_SEG_FLAGS_U8     n bytes; any non-zero byte marks the first element of a
 *                        segment.  Byte 0 is never consulted: element 0 always
 *                        opens a segment (Problem 2.1, Eq. 1: "i = 0 or f(i) = 1").
 *   MMV_SEG_OFFSETS_I32  nseg+1 int32 values, non-decreasing, the CSR row-pointer
 *                        convention: segment r covers [off[r], off[r+1]) and may
 *                        be empty (Section 4.3, remark after Algorithm 4.4;
 *                        Algorithm A.4 for empty rows).
 *
 * Arithmetic
 *   MMV_F16_TO_F32  fp16 values, fp32 accumulation and output.  Results satisfy
 *                   |out - exact| <= 2e-3 * (sum of |x| over the summed range) + 1e-6.
 *                   The scans (mmv_seg_scan, mmv_seg_scan_exclusive, the static and
 *                   the host-vector form) hold this for any finite values whose
 *                   sums stay finite in fp32: no result is ever formed as a
 *                   difference of two prefixes, so a segment of tiny values
 *                   behind a segment of huge ones keeps its own small bound.
 *                   For mmv_seg_sum and mmv_spmv_csr see their comments.
 *                   Floating-point results are not bit-reproducible from run
 *                   to run because the grouping of the cross-tile carry chain
 *                   depends on timing.
 *   MMV_I8_TO_I32   int8 values, exact int32 result modulo 2^32 (bit-exact and
 *                   deterministic).
 *   MMV_BF16_TO_F32 bfloat16 values, otherwise as MMV_F16_TO_F32.  Accepted by
 *                   mmv_seg_scan, mmv_seg_scan_exclusive and mmv_seg_sum;
 *                   the other entry points answer MMV_ERR_INVALID_ARG.
 */
#ifndef MMV_H_
#define MMV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    MMV_OK = 0,
    MMV_ERR_INVALID_ARG = 1,         /* null/misaligned pointer, negative size, bad enum      */
    MMV_ERR_UNSUPPORTED = 2,         /* combination not implemented                           */
    MMV_ERR_WORKSPACE_TOO_SMALL = 3,
    MMV_ERR_BAD_SEGMENTS = 4,        /* offsets not monotone / out of range (device-detected) */
    MMV_ERR_TIMEOUT = 5,             /* a bounded device-side wait gave up                    */
    MMV_ERR_CUDA = 6                 /* a CUDA runtime / driver call failed                   */
} mmv_status;

typedef enum { MMV_F16_TO_F32 = 0, MMV_I8_TO_I32 = 1, MMV_BF16_TO_F32 = 2 } mmv_dtype;
typedef enum { MMV_SEG_FLAGS_U8 = 0, MMV_SEG_OFFSETS_I32 = 1 } mmv_segfmt;
typedef enum {
    MMV_OP_SEG_SCAN = 0, MMV_OP_SEG_SUM = 1, MMV_OP_SPMV_CSR = 2, MMV_OP_COMPRESS = 3, MMV_OP_SEG_SCAN_MINMAX = 4,
    MMV_OP_SEG_SCAN_WIDE = 5, MMV_OP_MULT = 6
} mmv_op;

/*
 * Bytes of device workspace the given call needs (a pure host computation).
 * n = number of values (nnz for SpMV), nseg = number of segments (rows); nseg is
 * ignored for flag-encoded segments.  Returns 0 for invalid arguments.
 */
size_t mmv_workspace_bytes(mmv_op op, mmv_dtype dt, mmv_segfmt sf, int64_t n, int64_t nseg);

/*
 * Segmented inclusive scan (Problem 2.1, Eq. 1):
 *     out[i] = x[i]               if i == 0 or i starts a segment
 *     out[i] = out[i-1] + x[i]    otherwise
 * x: n values (fp16 or int8 per dt).  seg: n flag bytes, or nseg+1 offsets with
 * off[0] == 0 and off[nseg] == n (empty segments allowed, they start nothing).
 * With sf == MMV_SEG_FLAGS_U8, seg may be NULL: the whole vector is one segment
 * (the plain inclusive scan, the case Algorithm 4.1 treats) and no flag bytes
 * are read.  out: n values (fp32 or int32).  Elements past n are never written.
 */
mmv_status mmv_seg_scan(const void *x, const void *seg, mmv_segfmt sf, int64_t n, int64_t nseg,
                        mmv_dtype dt, void *out,
                        void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * Segmented EXCLUSIVE scan, the companion of Eq. 1: every element receives the
 * sum of the elements of its segment in front of it,
 *     out[i] = 0                      if i == 0 or i starts a segment
 *     out[i] = out[i-1] + x[i-1]      otherwise
 * (the inclusive result moved one element to the right inside each segment).
 * Same arguments, layouts, workspace, ownership and errors as mmv_seg_scan.
 */
mmv_status mmv_seg_scan_exclusive(const void *x, const void *seg, mmv_segfmt sf, int64_t n, int64_t nseg,
                                  mmv_dtype dt, void *out,
                                  void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * One vector cut into contiguous shards, one per GPU (Section 4.2, steps 3-6:
 * the blocks' last values and flags are scanned and the result is added to the
 * first segment of every block -- here a shard is the block, and the scan over
 * the handful of shard records is done by every shard for itself).
 *
 * mmv_seg_scan_shard scans one shard as mmv_seg_scan would (flag-encoded
 * segments; flags_u8 may be NULL: no start inside the shard) without the carry
 * from the shards in front of it, and writes a 16-byte record to `summary`
 * (device pointer, 16-byte aligned):
 *     uint32  bits of the running sum at the shard's last element (fp32 / int32)
 *     uint32  1 if a segment starts inside the shard, else 0
 *     int64   index of the shard's first start, n if there is none
 * first_shard != 0: element 0 opens a segment whatever its flag (Eq. 1).
 * first_shard == 0: flag byte 0 counts like any other, and without it element 0
 * continues the segment that reaches it from the shard in front.
 * Workspace as for mmv_seg_scan (MMV_OP_SEG_SCAN, MMV_SEG_FLAGS_U8, n).
 *
 * The caller then gathers the records of all `world` shards, in shard order,
 * into one buffer on every GPU (one all-gather of 16 bytes per shard: the only
 * exchange of the path) and calls mmv_seg_scan_shard_finish on the same
 * stream order: it folds the records of the shards in front of `rank` with
 * (v1, f1) + (v2, f2) = (f2 ? v2 : v1 + v2, f1 | f2) and adds the resulting
 * carry to out[0 .. first start of this shard).  With segment starts in every
 * shard that touches a few elements; a shard without any start is rewritten
 * once.  Both calls are asynchronous on cuda_stream; errors as for
 * mmv_seg_scan (device-side status in the shard's workspace).
 */
#define MMV_SHARD_SUMMARY_BYTES 16
mmv_status mmv_seg_scan_shard(const void *x, const void *flags_u8, int64_t n, mmv_dtype dt, int first_shard,
                              void *out, void *summary,
                              void *workspace, size_t workspace_bytes, void *cuda_stream);
mmv_status mmv_seg_scan_shard_finish(const void *summaries, int rank, int world, void *out, int64_t n,
                                     mmv_dtype dt, void *cuda_stream);

/*
 * Segmented sum (Section 2: the last element of every segment of the
 * segmented scan; Algorithm 4.2 computes the same quantity).
 * Offsets form: out has nseg entries, out[r] = sum of x over [off[r], off[r+1]),
 * exactly 0 for an empty segment; values outside [off[0], off[nseg]) are
 * ignored; requires 0 <= off[0] and off[nseg] <= n.  d_num_segments is ignored
 * (may be NULL).
 * Flags form: out has capacity n; the K = 1 + #{i >= 1 : flag[i] != 0} segment
 * sums are written in segment order, nothing beyond out[K-1] is touched, and K
 * is written to *d_num_segments (device pointer, int64, 8-byte aligned) when it
 * is not NULL.  The start flags are first compacted into K + 1 offsets inside
 * the workspace (COMPRESS, Section 2; the compaction step of Algorithm 4.2),
 * which therefore holds 4 (n + 1) bytes more than for the offsets form; nseg is
 * ignored.  n < 2^31 in both forms, nseg < 2^31 - 1 (MMV_ERR_INVALID_ARG otherwise).
 * Floating point: a sum is formed from differences of prefixes local to
 * 32-element rows.  A segment that lies inside one row or two adjacent rows
 * (in particular every segment of up to 32 elements) holds the bound for any
 * finite values: a difference that came out small against its prefixes is
 * added up again from the values themselves.  A longer segment holds it when
 * the magnitudes inside its 4096-element span are within about 2^10 of each
 * other; beyond that its absolute error is about 2^-22 of the largest prefix
 * of the rows involved.
 */
mmv_status mmv_seg_sum(const void *x, const void *seg, mmv_segfmt sf, int64_t n, int64_t nseg,
                       mmv_dtype dt, void *out, int64_t *d_num_segments,
                       void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * Segmented running maximum (want_min == 0) or minimum (want_min != 0): Eq. 1
 * with max / min in place of the addition,
 *     out[i] = x[i]                  if i == 0 or flags[i] != 0
 *     out[i] = max(out[i-1], x[i])   otherwise.
 * These operators have no inverse, so the matrix-product method (which reverts
 * its speculation by subtracting: Section 2 asks for a group) does not apply;
 * the scan runs on the CUDA cores and is exact.  x: n values, fp16 or bfloat16
 * (MMV_F16_TO_F32, MMV_BF16_TO_F32: out fp32) or int8 (MMV_I8_TO_I32: out int32); flags: n bytes
 * or NULL (one segment); x, flags, out 16-byte aligned.  Workspace:
 * mmv_workspace_bytes(MMV_OP_SEG_SCAN_MINMAX, dt, MMV_SEG_FLAGS_U8, n, 0)
 * (256-byte aligned, owned by the caller, reusable once the call's work on the
 * stream is done).  n < 2^36.  NaN values and the sign of a zero result are
 * unspecified.  Errors and asynchrony as for mmv_seg_scan: argument errors are
 * returned at once, a look-back that exceeds the time budget is reported by
 * mmv_last_async_status (MMV_ERR_TIMEOUT).
 */
mmv_status mmv_seg_scan_minmax(const void *x, const void *flags, int64_t n, mmv_dtype dt, int want_min, void *out,
                               void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * Segmented inclusive scan (Problem 2.1, Eq. 1) of int8 values with int64
 * results: the exact sums, where mmv_seg_scan's int32 results wrap from
 * n = 2^24 on.  Inside a tile of a few thousand elements every sum fits 32
 * bits; the carries between tiles are 64 bits wide.  Runs on the CUDA cores (the tensor-core
 * path chains its tiles through 32-bit payloads).  x: n int8 values; flags: n
 * bytes or NULL (one segment: the plain inclusive scan); out: n int64 values;
 * x, flags, out 16-byte aligned; n < 2^36.  Workspace (256-byte aligned):
 * mmv_workspace_bytes(MMV_OP_SEG_SCAN_WIDE, MMV_I8_TO_I32, MMV_SEG_FLAGS_U8, n, 0).
 * Errors and asynchrony as for mmv_seg_scan.
 */
mmv_status mmv_seg_scan_i8_i64(const void *x, const void *flags, int64_t n, int64_t *out,
                               void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * COMPRESS (Section 2): the values x[i] with flag[i] != 0, in order, copied
 * unchanged to out[0 .. K-1] (same element type as x: 2 bytes for
 * MMV_F16_TO_F32 and MMV_BF16_TO_F32, 1 byte for MMV_I8_TO_I32); nothing
 * beyond out[K-1] is touched.  Unlike the segment encodings above, flag[0] is
 * an ordinary flag here.  K is written to *d_count (device pointer, int64,
 * 8-byte aligned) when it is not NULL.  out needs room for n elements in the
 * worst case; x, flags and out 16-byte aligned; n < 2^31.  Workspace:
 * mmv_workspace_bytes(MMV_OP_COMPRESS, dt, MMV_SEG_FLAGS_U8, n, 0).  Three
 * streaming kernels (counts per 16384-flag chunk, one-block scan, scatter);
 * asynchronous on the stream like the other calls.
 */
mmv_status mmv_compress(const void *x, const void *flags, int64_t n, mmv_dtype dt, void *out, int64_t *d_count,
                        void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * Element-wise product of two int8 vectors through the segmented sum
 * (Section 4.3.1, Lemma 4.4 / Corollary 4.5): out[i] = x[i] * y[i] as int32.
 * Each product is the sum of the eight partial terms of the school method,
 * c_k = (bit k of y[i]) ? x[i] 2^k : 0 with bit 7 weighing -2^7; the terms of all
 * products are written to the workspace as one vector of 8 n fp16 values (every
 * term is exactly representable) and its segments of eight are summed by the
 * tensor-core kernel of mmv_seg_sum; the sums, exact integers in fp32, are
 * rewritten in place as int32.  The result is exact.  The paper gives this
 * construction for machines without a multiplier; here it is a demonstration
 * of the method, far slower than a plain multiply.
 * x, y: n int8 values; out: n int32, 16-byte aligned; n < 2^28.  Workspace:
 * mmv_workspace_bytes(MMV_OP_MULT, MMV_I8_TO_I32, MMV_SEG_OFFSETS_I32, n, 0)
 * (about 28 bytes per element).  Asynchronous on cuda_stream; errors as for
 * mmv_seg_sum.
 */
mmv_status mmv_mult_i8(const int8_t *x, const int8_t *y, int64_t n, int32_t *out,
                       void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * CSR sparse matrix times dense vector built on the segmented sum
 * (Algorithm 4.4; Algorithms A.4-A.6):  y[r] = sum over k in
 * [rowptr[r], rowptr[r+1]) of val[k] * x[col[k]]; an empty row gives exactly
 * 0.  Every product is formed in fp32 and handed to the tensor core as a pair
 * of bfloat16 values (hi = bf16(z), lo = bf16(z - hi): relative error at most
 * 2^-17 per product); the sums are fp32.  Rows of up to 32 non-zeros (and any
 * row inside one or two adjacent 32-element rows of the product vector) hold
 * the bound of "Arithmetic" above for any finite values; a longer row holds it
 * when the magnitudes of the products inside a 4096-product span are within
 * about 2^10 of each other (see mmv_seg_sum).  rowptr: rows+1 int32 with rowptr[0] == 0 and
 * rowptr[rows] == nnz < 2^31 (and rows < 2^31 - 1); col: nnz int32 in [0, cols) (duplicates simply
 * add; an index outside the range is never dereferenced, it contributes 0 and the
 * call records MMV_ERR_INVALID_ARG in the workspace status); val: nnz fp16;
 * x: cols fp32; y: rows fp32.
 */
mmv_status mmv_spmv_csr(const int32_t *rowptr, const int32_t *col, const void *val_f16,
                        const float *x, float *y, int64_t rows, int64_t cols, int64_t nnz,
                        void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * Synchronises `cuda_stream` and returns the device-side status that the last
 * call using `workspace` recorded (MMV_OK if none), or MMV_ERR_CUDA if the
 * stream itself reports an error.  A call that had nothing to do (no elements,
 * no segments, no rows, no non-zeros) and was handed a workspace records
 * MMV_OK in it; a workspace no call has seen yet holds no status.
 */
mmv_status mmv_last_async_status(const void *workspace, void *cuda_stream);

/* Static, human-readable name of a status code. */
const char *mmv_status_string(mmv_status s);

/*
 * Number of kernels the library has launched in this process since it was
 * loaded (host counter; used by the benchmark to report its launch count).
 */
int64_t mmv_kernel_launch_count(void);

/*
 * Segmented inclusive scan for callers that cannot provide a workspace.
 * (The paper has no counterpart: this is a packaging variant of mmv_seg_scan.)
 *
 * Some users of this library may not allocate device memory at the moment they
 * need a scan: a service that handed the whole GPU to its own memory pool at
 * start-up, a plug-in that runs inside another framework's operator and is
 * given only its input and output buffers, a control loop where an allocation's
 * implicit device synchronisation would break its timing.  For them this entry
 * point takes only x, the uint8 start flags and out; the per-unit carry words
 * that mmv_seg_scan keeps in the caller's workspace live in a fixed buffer
 * inside the library's own device image instead (about 0.5 MB, resident on
 * every GPU that loads the library until the process exits).  The call itself
 * performs no cudaMalloc / cudaFree and uses no allocating library routine.
 *
 * Limits and rules
 *   - n <= MMV_STATIC_SCAN_MAX_N; larger inputs are refused with
 *     MMV_ERR_WORKSPACE_TOO_SMALL and nothing is enqueued.
 *   - Flag-encoded segments only; arithmetic, alignment rules, asynchrony and
 *     error reporting are those of mmv_seg_scan.
 *   - The first call on each device looks up the device address of the built-in
 *     buffer (the device must be current); make that first call before starting
 *     any stream capture.
 *   - All calls on a device share the one buffer.  Each call clears the part it
 *     uses on its stream before the kernel runs, so stale contents never leak
 *     into a result, but two calls that overlap on the GPU (different streams)
 *     would overwrite each other's carries: serialise them.
 *   - Device-side status (time-outs) is returned by
 *     mmv_seg_scan_static_last_status().
 */
#define MMV_STATIC_SCAN_MAX_N (1ll << 28)
mmv_status mmv_seg_scan_static(const void *x, const void *flags_u8, int64_t n, mmv_dtype dt, void *out,
                               void *cuda_stream);

/* Synchronises the stream and returns the device-side status of the last mmv_seg_scan_static call
 * on the current device. */
mmv_status mmv_seg_scan_static_last_status(void *cuda_stream);

/*
 * Segmented scan (Problem 2.1) of vectors that live in HOST memory: x_host (n values), flags_host
 * (n start-flag bytes, or NULL for one segment) and out_host (n results) are host pointers.  The vectors are cut into
 * chunks of chunk_elems elements (a positive multiple of 16384); the chunks are copied to the
 * device, scanned and copied back on three internal streams, so that the copy-in, the kernels
 * and the copy-out of neighbouring chunks overlap; the running sum at the end of a chunk is
 * handed to the next chunk's kernel on the device.  Results are identical to mmv_seg_scan on
 * the whole vector.  device_scratch: device memory, 256-byte aligned, at least
 * mmv_seg_scan_host_scratch_bytes(dt, chunk_elems) bytes (two chunk buffers and their carry
 * words).  The work is ordered after everything already in cuda_stream, and cuda_stream
 * continues only when all results are on the host; the call itself returns without waiting, so
 * the host vectors must stay valid and untouched until the stream has drained.  Use pinned
 * (page-locked) host memory: with pageable memory the copies do not overlap.  The internal
 * streams are shared by all calls on a device, which therefore must not overlap in time.
 * Device-side status: mmv_last_async_status(device_scratch, cuda_stream).
 */
size_t mmv_seg_scan_host_scratch_bytes(mmv_dtype dt, int64_t chunk_elems);
mmv_status mmv_seg_scan_host(const void *x_host, const void *flags_host, int64_t n, mmv_dtype dt, void *out_host,
                             int64_t chunk_elems, void *device_scratch, size_t device_scratch_bytes,
                             void *cuda_stream);

/*
 * Test hook.  wait_budget_ns: time after which a device-side wait gives up
 * (<= 0 restores the default of 4 s).  skip_publish_span: index of one
 * 4096-element span of the scan that never publishes its carry, so that its
 * successors exercise the time-out path without any GPU fault (-1 = off).
 * Applies to calls made after it returns.
 */
void mmv_debug_configure(int64_t wait_budget_ns, int64_t skip_publish_span);

/*
 * Test hook.  The segmented-sum kernel exists with two and with three epilogue
 * warpgroups; the library launches the one with three.  groups = 2 makes every
 * later segmented sum and SpMV use the variant with two, 3 or 0 restore the
 * default.
 */
void mmv_debug_force_sum_groups(int groups);

/*
 * Test hook.  The floating-point scan with a flag vector exists in two shapes:
 * 0 = wide tiles (every flag density), 2 = narrow tiles (fast where segment
 * starts are rare, correct everywhere).  shape = 0 or 2 makes every later
 * floating-point scan with a flag vector use that shape; any other value
 * gives the choice back to the library.
 */
void mmv_debug_force_scan_shape(int shape);

#ifdef __cplusplus
}
#endif
#endif /* MMV_H_ */
