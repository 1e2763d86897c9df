// Host side of the C ABI declared in include/mmv.h: argument checks, workspace
// carve-up, tensor-map encoding and kernel launches.  No allocation, no host
// synchronisation (except mmv_last_async_status, whose job it is).
#include <atomic>
#include <cstdint>
#include <cstring>
#include <cuda.h>
#include <cuda_runtime.h>
#include <mutex>
#include <type_traits>

#include "../../include/mmv.h"
#include "common.cuh"
#include "seg_scan.cuh"
#include "seg_sum.cuh"
#include "compress.cuh"
#include "seg_minmax.cuh"
#include "seg_wide.cuh"

namespace mmv {
namespace {

std::atomic<long long> g_launches{0};
std::atomic<unsigned long long> g_budget_ns{WAIT_BUDGET_NS};
std::atomic<long long> g_debug_skip_span{-1};
std::atomic<int> g_force_groups{0};
std::atomic<int> g_force_scan_shape{-1};      // test hook: -1 = the library chooses

constexpr int kMaxDevices = 64;
constexpr long long kScanProbeMinN = 1ll << 28;       // shortest vector for which the scan samples its flag density

struct DeviceInfo {
    std::mutex lock;
    std::atomic<bool> ok{false};
    int sm_count = 0;
    // copy-in / kernel / copy-out streams and their events for mmv_seg_scan_host (made on first use)
    std::once_flag pipe_once;
    bool pipe_ok = false;
    cudaStream_t s_in = nullptr, s_k = nullptr, s_out = nullptr;
    cudaEvent_t ev_start = nullptr, ev_end_k = nullptr, ev_end_out = nullptr;
    cudaEvent_t in_done[2] = {nullptr, nullptr}, k_done[2] = {nullptr, nullptr}, out_done[2] = {nullptr, nullptr};
};
DeviceInfo g_dev[kMaxDevices];

using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                   const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn g_encode = nullptr;
std::once_flag g_encode_once;

EncodeTiledFn get_encode() {
    std::call_once(g_encode_once, [] {
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            g_encode = reinterpret_cast<EncodeTiledFn>(fn);
    });
    return g_encode;
}

template <typename K>
bool set_smem(K kernel, int bytes) {
    return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) == cudaSuccess;
}

// Launch of a tiled tensor-core kernel (scan, segmented sum).  These kernels hand out their tiles in a fixed order
// (tile = block + iteration * grid) and a tile waits for the carries of the tiles in front of it, so every CTA of
// the grid has to be resident at the same time.  A cooperative launch makes the device guarantee that: the grid
// starts only once all its CTAs fit together, whatever else runs on the GPU (another call of this library on a
// second stream simply runs before or after it), and a grid that can never fit (fewer SMs than the device
// reports: an MPS thread limit, a green context) is refused at launch instead of running into its time-out.
// `programmatic`: the kernel may start while the kernel in front of it in the stream still runs (it waits with
// griddepcontrol before it reads that kernel's results).  Measured: beside the cooperative attribute the early start
// no longer happens for a launch made directly (configuration 2: 37.2 -> 39.2 us per call), while a call replayed
// from a CUDA graph keeps it (32.8 vs 33.3 us); the attribute stays for the graph's sake.
template <typename... KP, typename... A>
cudaError_t launch_resident(void (*kernel)(KP...), int grid, int threads, int smem_bytes, cudaStream_t st, bool programmatic,
                            const A&... args) {
    cudaLaunchConfig_t cfg{};
    cudaLaunchAttribute attr[2];
    unsigned na = 0;
    attr[na].id = cudaLaunchAttributeCooperative;
    attr[na].val.cooperative = 1;
    ++na;
    if (programmatic) {
        attr[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[na].val.programmaticStreamSerializationAllowed = 1;
        ++na;
    }
    cfg.gridDim = dim3(static_cast<unsigned>(grid));
    cfg.blockDim = dim3(static_cast<unsigned>(threads));
    cfg.dynamicSmemBytes = static_cast<size_t>(smem_bytes);
    cfg.stream = st;
    cfg.attrs = attr;
    cfg.numAttrs = na;
    const cudaError_t err = cudaLaunchKernelEx(&cfg, kernel, args...);
    return err != cudaSuccess ? err : cudaGetLastError();
}

// Per-device one-time set-up: SM count and the kernels' dynamic shared-memory limits.
DeviceInfo* device_info() {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
    DeviceInfo* d = &g_dev[dev];
    if (d->ok.load(std::memory_order_acquire)) return d;
    // (only success is remembered: after a failed attempt the next call tries again)
    std::lock_guard<std::mutex> guard(d->lock);
    if (d->ok.load(std::memory_order_relaxed)) return d;
    int sm = 0;
    if (cudaDeviceGetAttribute(&sm, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return nullptr;
    d->sm_count = sm;
    bool ok = true;
    ok &= set_smem(seg_scan_kernel<F16Path>, ScanCfg<F16Path>::kSmemBytes);
    ok &= set_smem(seg_scan_kernel<I8Path>, ScanCfg<I8Path>::kSmemBytes);
    ok &= set_smem(seg_scan_kernel<F16Path, true>, ScanCfg<F16Path>::kSmemBytes);
    ok &= set_smem(seg_scan_kernel<I8Path, true>, ScanCfg<I8Path>::kSmemBytes);
    ok &= set_smem(seg_scan_kernel<BF16ValPath>, ScanCfg<BF16ValPath>::kSmemBytes);
    ok &= set_smem(seg_scan_kernel<BF16ValPath, true>, ScanCfg<BF16ValPath>::kSmemBytes);
    ok &= set_smem(seg_scan_kernel<F16Path, false, SCAN_PLAIN>, ScanCfg<F16Path, SCAN_PLAIN>::kSmemBytes);
    ok &= set_smem(seg_scan_kernel<F16Path, true, SCAN_PLAIN>, ScanCfg<F16Path, SCAN_PLAIN>::kSmemBytes);
    ok &= set_smem(seg_scan_kernel<BF16ValPath, false, SCAN_PLAIN>, ScanCfg<BF16ValPath, SCAN_PLAIN>::kSmemBytes);
    ok &= set_smem(seg_scan_kernel<BF16ValPath, true, SCAN_PLAIN>, ScanCfg<BF16ValPath, SCAN_PLAIN>::kSmemBytes);
    ok &= set_smem(seg_scan_kernel<F16Path, false, SCAN_NARROW>, ScanCfg<F16Path, SCAN_NARROW>::kSmemBytes);
    ok &= set_smem(seg_scan_kernel<F16Path, true, SCAN_NARROW>, ScanCfg<F16Path, SCAN_NARROW>::kSmemBytes);
    ok &= set_smem(seg_scan_kernel<BF16ValPath, false, SCAN_NARROW>, ScanCfg<BF16ValPath, SCAN_NARROW>::kSmemBytes);
    ok &= set_smem(seg_scan_kernel<BF16ValPath, true, SCAN_NARROW>, ScanCfg<BF16ValPath, SCAN_NARROW>::kSmemBytes);
    ok &= set_smem(seg_scan_minmax_kernel<0, false>, MM_SMEM_BYTES);
    ok &= set_smem(seg_scan_minmax_kernel<0, true>, MM_SMEM_BYTES);
    ok &= set_smem(seg_scan_minmax_kernel<1, false>, MM_SMEM_BYTES);
    ok &= set_smem(seg_scan_minmax_kernel<1, true>, MM_SMEM_BYTES);
    ok &= set_smem(seg_scan_minmax_kernel<2, false>, MM_SMEM_BYTES);
    ok &= set_smem(seg_scan_minmax_kernel<2, true>, MM_SMEM_BYTES);
    ok &= set_smem(seg_sum_kernel<BF16ValPath, 2>, SumCfg<BF16ValPath, 2>::kSmemBytes);
    ok &= set_smem(seg_sum_kernel<BF16ValPath, 3>, SumCfg<BF16ValPath, 3>::kSmemBytes);
    ok &= set_smem(seg_sum_kernel<F16Path, 2>, SumCfg<F16Path, 2>::kSmemBytes);
    ok &= set_smem(seg_sum_kernel<I8Path, 2>, SumCfg<I8Path, 2>::kSmemBytes);
    ok &= set_smem(seg_sum_kernel<BF16Path, 2>, SumCfg<BF16Path, 2>::kSmemBytes);
    ok &= set_smem(seg_sum_kernel<F16Path, 3>, SumCfg<F16Path, 3>::kSmemBytes);
    ok &= set_smem(seg_sum_kernel<I8Path, 3>, SumCfg<I8Path, 3>::kSmemBytes);
    ok &= set_smem(seg_sum_kernel<BF16Path, 3>, SumCfg<BF16Path, 3>::kSmemBytes);
    if (!ok) {
        cudaGetLastError();
        return nullptr;
    }
    d->ok.store(true, std::memory_order_release);
    return d;
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// The value vector as [spans][4 pieces][32 rows][32 elements] (full spans only); one box =
// piece i of four consecutive spans = the 128 x 32 A operand of one tensor-core product.
bool encode_span_map(CUtensorMap* map, const void* x, long long n, int elem_bytes, int pieces_per_unit) {
    EncodeTiledFn enc = get_encode();
    if (!enc) return false;
    const cuuint64_t spans = static_cast<cuuint64_t>(n / (static_cast<long long>(pieces_per_unit) * PIECE));
    if (spans == 0) {
        std::memset(map, 0, sizeof(*map));
        return true;
    }
    const cuuint64_t rb = static_cast<cuuint64_t>(ROW) * elem_bytes;
    cuuint64_t dims[4] = {ROW, PIECE_ROWS, static_cast<cuuint64_t>(pieces_per_unit), spans};
    cuuint64_t strides[3] = {rb, rb * PIECE_ROWS, rb * PIECE_ROWS * pieces_per_unit};
    cuuint32_t box[4] = {ROW, PIECE_ROWS, 1, SPANS_PER_TILE};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    const CUtensorMapDataType dtp = elem_bytes == 4 ? CU_TENSOR_MAP_DATA_TYPE_UINT32
                                  : elem_bytes == 2 ? CU_TENSOR_MAP_DATA_TYPE_UINT16 : CU_TENSOR_MAP_DATA_TYPE_UINT8;
    const CUtensorMapSwizzle swz = elem_bytes == 4 ? CU_TENSOR_MAP_SWIZZLE_128B
                                 : elem_bytes == 2 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_32B;
    CUresult r = enc(map, dtp, 4,
                     const_cast<void*>(x), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, swz,
                     CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

// The output vector as rows of 32 four-byte values (full rows only); box = one 32 x 32 piece.
bool encode_out_map(CUtensorMap* map, void* out, long long n) {
    EncodeTiledFn enc = get_encode();
    if (!enc) return false;
    const cuuint64_t rows = static_cast<cuuint64_t>(n / ROW);
    if (rows == 0) {
        std::memset(map, 0, sizeof(*map));
        return true;
    }
    cuuint64_t dims[2] = {ROW, rows};
    cuuint64_t strides[1] = {ROW * 4};
    cuuint32_t box[2] = {ROW, PIECE_ROWS};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_UINT32, 2, out, dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

struct WorkspacePlan {
    size_t status_off, status_bytes;
    size_t flags_off, flags_bytes;     // scratch flag bytes (offset-encoded scan only)
    size_t tileq_off, tileq_bytes;     // per-tile first boundary index (seg-sum, SpMV)
    size_t prod_off, prod_bytes;       // bf16 hi/lo halves of the products (SpMV)
    size_t cmp_off, cmp_bytes;         // flag-encoded seg-sum: chunk counts, chunk bases, segment count
    size_t mask_off, mask_bytes;       // flag-encoded seg-sum, COMPRESS: one bit per flag (a 64-bit mask per thread of the count pass)
    size_t off_off, off_bytes;         // flag-encoded seg-sum: the compacted offsets (n + 1 entries at most)
    long long n_eff;                   // elements the tiled kernel runs over
    size_t total;
};

long long num_tiles_of(long long n) { return (n + TILE - 1) / TILE; }
long long num_scan_tiles_of(long long n) { return (n + SCAN_TILE - 1) / SCAN_TILE; }

WorkspacePlan plan_workspace(mmv_op op, mmv_segfmt sf, long long n) {
    WorkspacePlan p{};
    p.n_eff = n;
    const long long tiles = num_tiles_of(p.n_eff);
    const long long units = (op == MMV_OP_SEG_SCAN)          ? num_scan_tiles_of(n) * SCAN_STATUS_STRIDE
                            : (op == MMV_OP_SEG_SCAN_MINMAX) ? (n + MM_TILE - 1) / MM_TILE
                            : (op == MMV_OP_SEG_SCAN_WIDE)   ? (n + WD_TILE - 1) / WD_TILE
                                                             : tiles * SPANS_PER_TILE;
    p.status_off = sizeof(WorkspaceHeader);
    const int stride = (op == MMV_OP_SEG_SCAN_MINMAX) ? MM_STATUS_STRIDE
                       : (op == MMV_OP_SEG_SCAN_WIDE)  ? WD_STATUS_STRIDE
                       : (op == MMV_OP_SEG_SCAN)       ? 1
                                                       : SUM_STATUS_STRIDE;
    p.status_bytes = round_up(static_cast<size_t>(units) * sizeof(uint64_t) * stride, 256);
    p.flags_off = p.status_off + p.status_bytes;
    p.flags_bytes = (op == MMV_OP_SEG_SCAN && sf == MMV_SEG_OFFSETS_I32) ? round_up(static_cast<size_t>(n), 256) : 0;
    p.tileq_off = p.flags_off + p.flags_bytes;
    p.tileq_bytes = (op != MMV_OP_SEG_SCAN && op != MMV_OP_SEG_SCAN_MINMAX && op != MMV_OP_SEG_SCAN_WIDE) ? round_up(static_cast<size_t>(tiles * SPANS_PER_TILE + 1) * sizeof(int32_t), 256) : 0;
    p.prod_off = p.tileq_off + p.tileq_bytes;
    p.prod_bytes = (op == MMV_OP_SPMV_CSR) ? round_up(static_cast<size_t>(n) * 4, 256) : 0;
    const bool flagsum = (op == MMV_OP_SEG_SUM && sf == MMV_SEG_FLAGS_U8) || op == MMV_OP_COMPRESS;
    const long long nchunks = (n + CMP_CHUNK - 1) / CMP_CHUNK;
    p.cmp_off = p.prod_off + p.prod_bytes;
    p.cmp_bytes = flagsum ? round_up(static_cast<size_t>(2 * nchunks + 8) * sizeof(int32_t) + 16, 256) : 0;
    p.mask_off = p.cmp_off + p.cmp_bytes;
    // (+ one int32 per warp of the count pass: the number of set flags of its chunk in front of it)
    p.mask_bytes = flagsum ? round_up(static_cast<size_t>(nchunks) * CMP_THREADS * sizeof(unsigned long long), 256) +
                                 round_up(static_cast<size_t>(nchunks) * CMP_WARPS * sizeof(int32_t), 256) : 0;
    p.off_off = p.mask_off + p.mask_bytes;
    p.off_bytes = (flagsum && op != MMV_OP_COMPRESS) ? round_up(static_cast<size_t>(n + 1) * sizeof(int32_t), 256) : 0;
    p.total = p.off_off + p.off_bytes;
    return p;
}

// z(k) = val(k) * x(col(k)) in fp32 (Algorithm A.5, CsrGather), written as a pair of bf16 values
// (hi = bf16(z), lo = bf16(z - hi); 4 bytes per product) that the segmented sum feeds to the tensor
// core as two K entries of one element.
// A column index outside [0, cols) is never dereferenced: it reads as x = 0 and the call ends with
// MMV_ERR_INVALID_ARG in the workspace status (the check costs nothing, the kernel waits on its loads).
__device__ __forceinline__ float gather_x(const float* __restrict__ x, int c, long long cols, bool& bad) {
    const bool oob = static_cast<unsigned long long>(static_cast<long long>(c)) >= static_cast<unsigned long long>(cols);
    bad |= oob;
    return oob ? 0.f : __ldg(x + c);
}
__device__ __forceinline__ uint32_t split_product(float z) {
    const __nv_bfloat16 hi = __float2bfloat16_rn(z);
    const __nv_bfloat16 lo = __float2bfloat16_rn(z - __bfloat162float(hi));
    return static_cast<uint32_t>(__bfloat16_as_ushort(hi)) | (static_cast<uint32_t>(__bfloat16_as_ushort(lo)) << 16);
}
__global__ void spmv_gather_kernel(const int32_t* __restrict__ col, const __half* __restrict__ val,
                                   const float* __restrict__ x, uint32_t* __restrict__ prod, long long nnz,
                                   long long cols, WorkspaceHeader* hdr) {
    const long long stride = static_cast<long long>(gridDim.x) * blockDim.x;
    const long long nvec = nnz >> 2;
    bool bad = false;
    for (long long v = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; v < nvec; v += stride) {
        const int4 c = __ldg(reinterpret_cast<const int4*>(col) + v);
        const uint2 hv = __ldg(reinterpret_cast<const uint2*>(val) + v);
        const __half2 h01 = *reinterpret_cast<const __half2*>(&hv.x);
        const __half2 h23 = *reinterpret_cast<const __half2*>(&hv.y);
        const float x0 = gather_x(x, c.x, cols, bad), x1 = gather_x(x, c.y, cols, bad);
        const float x2 = gather_x(x, c.z, cols, bad), x3 = gather_x(x, c.w, cols, bad);
        *(reinterpret_cast<uint4*>(prod) + v) =
            make_uint4(split_product(__low2float(h01) * x0), split_product(__high2float(h01) * x1),
                       split_product(__low2float(h23) * x2), split_product(__high2float(h23) * x3));
    }
    // ragged tail (nnz not a multiple of 4)
    const long long k = (nvec << 2) + static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (k < nnz) prod[k] = split_product(__half2float(val[k]) * gather_x(x, col[k], cols, bad));
    if (bad) report_error(hdr, 1u);
    // This kernel is launched so that it may start while the kernel in front of it (the span partition of the row
    // pointers, which it does not depend on) still runs; it ends only after that kernel has ended, so that whoever
    // follows in the stream finds both finished.
    griddep_wait();
}

// The span partition of the offset-encoded segmented sum (and the validation of the offsets, and the zeros of the
// empty segments).  The header must have been cleared on the stream already.
void launch_partition(const int32_t* off, long long nseg, long long n_eff, void* out, uint8_t* ws, const WorkspacePlan& plan,
                      DeviceInfo* dev, cudaStream_t st) {
    const long long spans = num_tiles_of(n_eff) * SPANS_PER_TILE;
    int32_t* span_q = reinterpret_cast<int32_t*>(ws + plan.tileq_off);
    const int threads = 256;
    const int vec = nseg >= (1ll << 20) ? 4 : 1;                           // offsets per thread and round
    long long blocks = (nseg + 1 + vec * threads - 1) / (vec * threads);
    if (blocks > 16ll * dev->sm_count) blocks = 16ll * dev->sm_count;
    WorkspaceHeader* hdr = reinterpret_cast<WorkspaceHeader*>(ws);
    if (vec == 4)
        partition_offsets_kernel<4><<<static_cast<unsigned>(blocks), threads, 0, st>>>(off, nseg, spans, span_q, n_eff, hdr,
                                                                                      static_cast<uint32_t*>(out));
    else
        partition_offsets_kernel<1><<<static_cast<unsigned>(blocks), threads, 0, st>>>(off, nseg, spans, span_q, n_eff, hdr,
                                                                                      static_cast<uint32_t*>(out));
    ++g_launches;
}

// Shared launcher of the tiled segmented-sum kernel.  `values` holds n_eff elements of the
// path's type; boundaries are off[q] << shift.  The header and status words must have been
// cleared on the stream already.  have_partition: span_q is filled already (by the compaction of
// the flag-encoded form, or by launch_partition earlier in the stream).
template <typename P>
mmv_status launch_seg_sum(const void* values, long long n_eff, const int32_t* off, long long nseg, int shift,
                          void* out, uint8_t* ws, const WorkspacePlan& plan, DeviceInfo* dev, cudaStream_t st,
                          const long long* nseg_dev = nullptr, bool have_partition = false, bool fused = false) {
    const int tiles = static_cast<int>(num_tiles_of(n_eff));
    int32_t* span_q = reinterpret_cast<int32_t*>(ws + plan.tileq_off);
    if (!have_partition && !fused) launch_partition(off, nseg, n_eff, out, ws, plan, dev, st);
    CUtensorMap tmap;
    if (!encode_span_map(&tmap, values, n_eff, P::kElemBytes, PIECES_PER_SPAN)) return MMV_ERR_CUDA;
    SumParams prm;
    prm.off = off;
    prm.nseg = nseg;
    prm.n = n_eff;
    (void)shift;
    prm.out = out;
    prm.num_tiles = tiles;
    prm.span_q = span_q;
    prm.hdr = reinterpret_cast<WorkspaceHeader*>(ws);
    prm.status = reinterpret_cast<uint64_t*>(ws + plan.status_off);
    prm.budget_ns = g_budget_ns.load();
    prm.nseg_dev = nseg_dev;
    prm.fused_prologue = fused ? 1 : 0;
    prm.status_words = static_cast<long long>(plan.status_bytes / sizeof(uint64_t));
    const int grid = tiles < dev->sm_count ? tiles : dev->sm_count;
    // Twelve epilogue warps (three warpgroups) measured faster than eight at every segment density;
    // the shape with two warpgroups stays available for tests and measurements.
    // With the partition kernel right in front, the tiled kernel is launched with programmatic
    // serialisation: its set-up (barriers, tensor memory, constant operand) overlaps the partition's end.
    const bool overlap = !have_partition && !fused;
    cudaError_t err;
    if (g_force_groups.load() != 2)
        err = launch_resident(seg_sum_kernel<P, 3>, grid, SumShape<3>::kThreads, SumCfg<P, 3>::kSmemBytes, st, overlap, tmap, values, prm);
    else
        err = launch_resident(seg_sum_kernel<P, 2>, grid, SumShape<2>::kThreads, SumCfg<P, 2>::kSmemBytes, st, overlap, tmap, values, prm);
    ++g_launches;
    return err == cudaSuccess ? MMV_OK : MMV_ERR_CUDA;
}

// f[off[r]] = 1 for every non-empty segment r (scratch flags of the offset-encoded scan).
__global__ void offsets_to_flags_kernel(const int32_t* __restrict__ off, long long nseg, long long n,
                                        uint8_t* __restrict__ f, WorkspaceHeader* hdr) {
    const long long stride = static_cast<long long>(gridDim.x) * blockDim.x;
    for (long long r = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; r < nseg; r += stride) {
        const long long a = off[r], b = off[r + 1];
        if (a > b || a < 0 || b > n || (r == 0 && a != 0) || (r == nseg - 1 && b != n)) {
            report_error(hdr, 4u);
        } else if (a < b) {
            f[a] = 1;
        }
    }
}

// ---------------------------------------------------------------------------
// Built-in scratch of mmv_seg_scan_static: header + the status words (SCAN_STATUS_STRIDE per tile).
// The symbol below is a host-side stand-in in host code; its device address is looked up once per
// device with cudaGetSymbolAddress and only that address is ever handed to a kernel or a memset.
// ---------------------------------------------------------------------------
constexpr long long kStaticScanMaxN = MMV_STATIC_SCAN_MAX_N;
constexpr size_t kStaticScratchBytes =
    sizeof(WorkspaceHeader) + static_cast<size_t>((kStaticScanMaxN + SCAN_TILE - 1) / SCAN_TILE) * SCAN_STATUS_STRIDE * sizeof(uint64_t);
static __device__ __align__(256) unsigned char g_static_scan_scratch[kStaticScratchBytes];

struct StaticScratch {
    std::mutex lock;
    std::atomic<void*> ptr{nullptr};
};
StaticScratch g_static_scratch[kMaxDevices];

// Device address of the built-in scratch on the current device (nullptr on failure).  Only a successful lookup
// is remembered: after a failure (a first call made during stream capture, a transient error) the next call
// tries again.
void* static_scratch_ptr() {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
    StaticScratch* sc = &g_static_scratch[dev];
    void* p = sc->ptr.load(std::memory_order_acquire);
    if (p) return p;
    std::lock_guard<std::mutex> guard(sc->lock);
    p = sc->ptr.load(std::memory_order_relaxed);
    if (p) return p;
    if (cudaGetSymbolAddress(&p, g_static_scan_scratch) != cudaSuccess || !p) {
        cudaGetLastError();            // the failure is reported through the return value, not left as a sticky error
        return nullptr;
    }
    sc->ptr.store(p, std::memory_order_release);
    return p;
}

// ---------------------------------------------------------------------------
// One vector cut into contiguous shards (one per GPU): each shard is scanned by itself and described
// by a 16-byte summary; the summaries of all shards are exchanged once (an all-gather, done by the
// caller), every shard folds the ones in front of it into its carry and adds that carry to its
// elements in front of its first start.  This is the block recursion of Section 4.2, steps 3-6 (scan
// the blocks' last values and flags, then UpdateFirstSegment), with a shard as the block.
// ---------------------------------------------------------------------------
struct ShardSummary {
    uint32_t value_bits;        // running sum at the shard's last element (fp32 or int32 bits), carry not included
    uint32_t has_start;         // 1 if a segment starts inside the shard
    long long first_start;      // index of the shard's first start, n if it has none
};
static_assert(sizeof(ShardSummary) == MMV_SHARD_SUMMARY_BYTES, "summary record is 16 bytes");

__global__ void shard_summary_kernel(const uint32_t* __restrict__ out, long long n, const unsigned long long* __restrict__ first_word,
                                     int first_shard, ShardSummary* __restrict__ summary) {
    const unsigned long long w = *first_word;                   // n - (index of the first start), 0 = none
    long long first = w ? n - static_cast<long long>(w) : n;
    if (first_shard) first = 0;                                 // element 0 of the whole vector opens a segment
    summary->value_bits = out[n - 1];
    summary->has_start = first < n ? 1u : 0u;
    summary->first_start = first;
}

// carry = fold of the summaries in front of `rank` with (v1, f1) + (v2, f2) = (f2 ? v2 : v1 + v2, f1 | f2);
// out[i] += carry for i < first_start(rank)
template <bool FP>
__global__ void shard_finish_kernel(const ShardSummary* __restrict__ all, int rank, uint32_t* __restrict__ out, long long n) {
    uint32_t carry_bits = 0u;
    float cf = 0.f;
    for (int r = 0; r < rank; ++r) {
        const uint32_t v = all[r].value_bits;
        if (FP) cf = all[r].has_start ? __uint_as_float(v) : cf + __uint_as_float(v);
        else carry_bits = all[r].has_start ? v : carry_bits + v;
    }
    long long limit = all[rank].first_start;
    if (limit > n) limit = n;
    if (limit <= 0) return;
    auto add = [&](uint32_t v) -> uint32_t { return FP ? __float_as_uint(cf + __uint_as_float(v)) : carry_bits + v; };
    const long long stride = static_cast<long long>(gridDim.x) * blockDim.x;
    const long long tid = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
    const long long nvec = limit >> 2;
    uint4* o4 = reinterpret_cast<uint4*>(out);
    for (long long v = tid; v < nvec; v += stride) {
        uint4 q = o4[v];
        q.x = add(q.x);
        q.y = add(q.y);
        q.z = add(q.z);
        q.w = add(q.w);
        o4[v] = q;
    }
    const long long k = (nvec << 2) + tid;
    if (k < limit) out[k] = add(out[k]);
}

// ---------------------------------------------------------------------------
// Element-wise integer product through the segmented sum (Section 4.3.1, Lemma 4.4 / Corollary 4.5): the
// product x(i) y(i) is the sum of the partial terms of the school method, c_k = (bit k of y) ? x 2^k : 0 (bit 7
// of a two's-complement byte weighs -2^7); all terms of all products form one vector whose segments of 8 are
// summed by the tensor-core kernel.  Every term (|c_k| <= 2^14, a shifted int8) is exactly an fp16 value and
// every sum (|x y| <= 2^14) exactly an fp32 value, so the result is exact.
// ---------------------------------------------------------------------------
constexpr int MULT_TERMS = 8;
__global__ void mult_expand_kernel(const int8_t* __restrict__ x, const int8_t* __restrict__ y, long long n,
                                   __half* __restrict__ terms, int32_t* __restrict__ off) {
    const long long stride = static_cast<long long>(gridDim.x) * blockDim.x;
    for (long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; i <= n; i += stride) {
        off[i] = static_cast<int32_t>(i * MULT_TERMS);
        if (i == n) break;
        const int xi = x[i];
        const unsigned yi = static_cast<unsigned char>(y[i]);
        __half t[MULT_TERMS];
#pragma unroll
        for (int k = 0; k < MULT_TERMS; ++k) {
            const int w = k == 7 ? -128 : (1 << k);
            t[k] = __int2half_rn(((yi >> k) & 1u) ? xi * w : 0);          // exact: |x 2^k| <= 2^14
        }
        *reinterpret_cast<uint4*>(terms + i * MULT_TERMS) = *reinterpret_cast<const uint4*>(t);
    }
}
// the sums are exact integers in fp32: rewrite them in place as int32
__global__ void mult_to_int_kernel(float* __restrict__ io, long long n) {
    const long long stride = static_cast<long long>(gridDim.x) * blockDim.x;
    for (long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; i < n; i += stride)
        reinterpret_cast<int32_t*>(io)[i] = __float2int_rn(io[i]);
}

struct MultPlan {
    WorkspacePlan sum;          // the segmented sum over 8 n terms in n segments, at the workspace's base
    size_t terms_off, off_off, total;
};
MultPlan plan_mult(long long n) {
    MultPlan p{};
    p.sum = plan_workspace(MMV_OP_SEG_SUM, MMV_SEG_OFFSETS_I32, n * MULT_TERMS);
    p.terms_off = p.sum.total;
    p.off_off = p.terms_off + round_up(static_cast<size_t>(n) * MULT_TERMS * sizeof(__half), 256);
    p.total = p.off_off + round_up(static_cast<size_t>(n + 1) * sizeof(int32_t), 256);
    return p;
}

}  // namespace
}  // namespace mmv

using namespace mmv;

extern "C" {

size_t mmv_workspace_bytes(mmv_op op, mmv_dtype dt, mmv_segfmt sf, int64_t n, int64_t nseg) {
    if (n < 0 || nseg < 0) return 0;
    if (op == MMV_OP_MULT) return n < (1ll << 28) ? plan_mult(n).total : 0;
    if (op != MMV_OP_SEG_SCAN && op != MMV_OP_SEG_SUM && op != MMV_OP_SPMV_CSR && op != MMV_OP_COMPRESS &&
        op != MMV_OP_SEG_SCAN_MINMAX && op != MMV_OP_SEG_SCAN_WIDE)
        return 0;
    if (dt != MMV_F16_TO_F32 && dt != MMV_I8_TO_I32 && dt != MMV_BF16_TO_F32) return 0;
    if (sf != MMV_SEG_FLAGS_U8 && sf != MMV_SEG_OFFSETS_I32) return 0;
    return plan_workspace(op, sf, n).total;
}

namespace {
// shard: 0 = a whole vector; 1 = the first shard of a longer vector, 2 = a later shard (its flag byte 0 counts,
// and without it element 0 continues the segment that reaches it).  For shards `summary` receives the record.
// A call that has nothing to do still leaves MMV_OK for mmv_last_async_status when it is handed a workspace
// (a workspace that was never used would otherwise answer with whatever its memory holds).
mmv_status nothing_to_do(void* workspace, size_t workspace_bytes, void* cuda_stream) {
    if (workspace && !(reinterpret_cast<uintptr_t>(workspace) & 255u) && workspace_bytes >= sizeof(WorkspaceHeader) &&
        cudaMemsetAsync(workspace, 0, sizeof(WorkspaceHeader), static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess)
        return MMV_ERR_CUDA;
    return MMV_OK;
}

mmv_status seg_scan_impl(const void* x, const void* seg, mmv_segfmt sf, int64_t n, int64_t nseg, mmv_dtype dt,
                         void* out, void* workspace, size_t workspace_bytes, void* cuda_stream, bool exclusive,
                         int shard = 0, void* summary = nullptr) {
    if (n < 0 || nseg < 0) return MMV_ERR_INVALID_ARG;
    if (dt != MMV_F16_TO_F32 && dt != MMV_I8_TO_I32 && dt != MMV_BF16_TO_F32) return MMV_ERR_INVALID_ARG;
    if (sf != MMV_SEG_FLAGS_U8 && sf != MMV_SEG_OFFSETS_I32) return MMV_ERR_INVALID_ARG;
    if (n == 0) return nothing_to_do(workspace, workspace_bytes, cuda_stream);
    if (n >= (1ll << 36)) return MMV_ERR_UNSUPPORTED;
    if (sf == MMV_SEG_OFFSETS_I32 && n >= (1ll << 31)) return MMV_ERR_INVALID_ARG;
    if (!x || !out || !workspace) return MMV_ERR_INVALID_ARG;
    if (!seg && sf != MMV_SEG_FLAGS_U8) return MMV_ERR_INVALID_ARG;           // no flags = one segment; offsets must exist
    if (!aligned16(x) || !aligned16(seg) || !aligned16(out) || (reinterpret_cast<uintptr_t>(workspace) & 255u))
        return MMV_ERR_INVALID_ARG;
    if (sf == MMV_SEG_OFFSETS_I32 && nseg == 0) return MMV_ERR_INVALID_ARG;   // n > 0 needs a segment
    const WorkspacePlan plan = plan_workspace(MMV_OP_SEG_SCAN, sf, n);
    if (workspace_bytes < plan.total) return MMV_ERR_WORKSPACE_TOO_SMALL;
    DeviceInfo* dev = device_info();
    if (!dev) return MMV_ERR_CUDA;

    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    WorkspaceHeader* hdr = reinterpret_cast<WorkspaceHeader*>(ws);
    // Where nothing in front of the scan kernel uses the workspace header (no offsets to turn into flags, no
    // density probe, no shard record), the kernel clears its workspace itself in front of a grid-wide barrier
    // and the call is a single launch; otherwise a memset node does it.
    const bool will_probe = seg != nullptr && g_force_scan_shape.load() < 0 && dt != MMV_I8_TO_I32 && n >= kScanProbeMinN;
    const bool self_clear = sf == MMV_SEG_FLAGS_U8 && !will_probe && shard == 0;
    if (!self_clear && cudaMemsetAsync(ws, 0, plan.status_off + plan.status_bytes, st) != cudaSuccess) return MMV_ERR_CUDA;

    const uint8_t* flags = static_cast<const uint8_t*>(seg);
    if (sf == MMV_SEG_OFFSETS_I32) {
        uint8_t* f = ws + plan.flags_off;
        if (cudaMemsetAsync(f, 0, static_cast<size_t>(n), st) != cudaSuccess) return MMV_ERR_CUDA;
        const int threads = 256;
        long long blocks = (nseg + threads - 1) / threads;
        if (blocks > dev->sm_count * 8) blocks = dev->sm_count * 8;
        offsets_to_flags_kernel<<<static_cast<unsigned>(blocks), threads, 0, st>>>(static_cast<const int32_t*>(seg), nseg,
                                                                                n, f, hdr);
        ++g_launches;
        flags = f;
    }

    CUtensorMap tmap, tmap_out;
    if (!encode_span_map(&tmap, x, n, dt == MMV_I8_TO_I32 ? 1 : 2, SCAN_UP)) return MMV_ERR_CUDA;
    if (!encode_out_map(&tmap_out, out, n)) return MMV_ERR_CUDA;

    ScanParams prm;
    prm.x = x;
    prm.flags = flags;
    prm.out = out;
    prm.n = n;
    prm.num_tiles = static_cast<int>(num_scan_tiles_of(n));
    prm.hdr = hdr;
    prm.status = reinterpret_cast<uint64_t*>(ws + plan.status_off);
    prm.budget_ns = g_budget_ns.load();
    prm.debug_skip_span = g_debug_skip_span.load();
    prm.carry_in = nullptr;
    prm.first_start = nullptr;
    prm.probe_count = nullptr;
    prm.probe_narrow_below = 0u;
    prm.clear_words = self_clear ? static_cast<long long>(plan.status_bytes / sizeof(uint64_t)) : 0;
    if (shard) {
        // (header words behind the two counters, cleared with the header: the first-start word and a carry of zero)
        prm.first_start = reinterpret_cast<unsigned long long*>(&hdr->reserved[0]);
        if (shard == 2) prm.carry_in = &hdr->reserved[2];
    }
    const int grid = prm.num_tiles < dev->sm_count ? prm.num_tiles : dev->sm_count;
    // (no flag vector: the floating-point paths run the narrow-tile shape without flag bytes; with a flag vector
    //  the narrow-tile shape is for vectors with few starts -- see the probe below)
    const bool plain = flags == nullptr;
    const int forced = g_force_scan_shape.load();
    bool narrow = !plain && forced == SCAN_NARROW;
    // A long floating-point vector with a flag vector: which shape is faster depends on how many tiles hold a
    // start (n = 2^30: no start 1.37 ms wide / 1.24 narrow, p = 1e-5 1.22 / 1.16, p = 1e-4 1.15 / 1.18,
    // p = 1e-3 1.13 / 1.40), which only the device can see.  A sampling kernel counts the starts in 256 KB of
    // the flags, both shapes are launched, and the one the count does not ask for returns at once (about
    // 6-8 us for the probe and the idle launch together, 0.6 % at n = 2^30 and 2.6 % at n = 2^28, hence only for
    // vectors of 2^28 elements and more).  Fewer than one start per two tiles: narrow.  A vector whose starts all hide between the samples gets the slower shape, never a
    // wrong result.
    const bool probe = will_probe;
    if (probe) {
        unsigned int* cnt = &hdr->reserved[4];                        // cleared with the header
        flag_density_probe_kernel<<<SCAN_PROBE_BLOCKS, SCAN_PROBE_THREADS, 0, st>>>(flags, n, cnt);
        ++g_launches;
        if (cudaGetLastError() != cudaSuccess) return MMV_ERR_CUDA;
        prm.probe_count = cnt;
        prm.probe_narrow_below = SCAN_PROBE_BYTES / SCAN_TILE / 2;    // half a start per tile on average
    }
    cudaError_t err;
#define MMV_LAUNCH_SCAN(PATH, EXCL, PL)                                                                               \
    err = launch_resident(seg_scan_kernel<PATH, EXCL, PL>, grid, ScanCfg<PATH, PL>::kThreads, ScanCfg<PATH, PL>::kSmemBytes, st, \
                          false, tmap, tmap_out, prm)
    if (dt == MMV_I8_TO_I32) {
        if (exclusive) MMV_LAUNCH_SCAN(I8Path, true, SCAN_WIDE);
        else MMV_LAUNCH_SCAN(I8Path, false, SCAN_WIDE);
    } else if (dt == MMV_BF16_TO_F32) {
        if (plain && exclusive) MMV_LAUNCH_SCAN(BF16ValPath, true, SCAN_PLAIN);
        else if (plain) MMV_LAUNCH_SCAN(BF16ValPath, false, SCAN_PLAIN);
        else {
            if ((narrow || probe) && exclusive) MMV_LAUNCH_SCAN(BF16ValPath, true, SCAN_NARROW);
            else if (narrow || probe) MMV_LAUNCH_SCAN(BF16ValPath, false, SCAN_NARROW);
            if (probe) {
                ++g_launches;
                if (err != cudaSuccess) return MMV_ERR_CUDA;
            }
            if ((!narrow || probe) && exclusive) MMV_LAUNCH_SCAN(BF16ValPath, true, SCAN_WIDE);
            else if (!narrow || probe) MMV_LAUNCH_SCAN(BF16ValPath, false, SCAN_WIDE);
        }
    } else {
        if (plain && exclusive) MMV_LAUNCH_SCAN(F16Path, true, SCAN_PLAIN);
        else if (plain) MMV_LAUNCH_SCAN(F16Path, false, SCAN_PLAIN);
        else {
            if ((narrow || probe) && exclusive) MMV_LAUNCH_SCAN(F16Path, true, SCAN_NARROW);
            else if (narrow || probe) MMV_LAUNCH_SCAN(F16Path, false, SCAN_NARROW);
            if (probe) {
                ++g_launches;
                if (err != cudaSuccess) return MMV_ERR_CUDA;
            }
            if ((!narrow || probe) && exclusive) MMV_LAUNCH_SCAN(F16Path, true, SCAN_WIDE);
            else if (!narrow || probe) MMV_LAUNCH_SCAN(F16Path, false, SCAN_WIDE);
        }
    }
#undef MMV_LAUNCH_SCAN
    ++g_launches;
    if (err != cudaSuccess) return MMV_ERR_CUDA;
    if (shard) {
        shard_summary_kernel<<<1, 1, 0, st>>>(static_cast<const uint32_t*>(out), n, prm.first_start, shard == 1 ? 1 : 0,
                                              static_cast<ShardSummary*>(summary));
        ++g_launches;
        if (cudaGetLastError() != cudaSuccess) return MMV_ERR_CUDA;
    }
    return MMV_OK;
}
}  // namespace

mmv_status mmv_seg_scan(const void* x, const void* seg, mmv_segfmt sf, int64_t n, int64_t nseg, mmv_dtype dt,
                        void* out, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    return seg_scan_impl(x, seg, sf, n, nseg, dt, out, workspace, workspace_bytes, cuda_stream, false);
}

mmv_status mmv_seg_scan_exclusive(const void* x, const void* seg, mmv_segfmt sf, int64_t n, int64_t nseg, mmv_dtype dt,
                                  void* out, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    return seg_scan_impl(x, seg, sf, n, nseg, dt, out, workspace, workspace_bytes, cuda_stream, true);
}

mmv_status mmv_seg_scan_shard(const void* x, const void* flags_u8, int64_t n, mmv_dtype dt, int first_shard, void* out,
                              void* summary, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    if (!summary || (reinterpret_cast<uintptr_t>(summary) & 15u)) return MMV_ERR_INVALID_ARG;
    if (n == 0) {
        // an empty shard: no start, nothing summed
        return cudaMemsetAsync(summary, 0, sizeof(ShardSummary), static_cast<cudaStream_t>(cuda_stream)) == cudaSuccess ? MMV_OK : MMV_ERR_CUDA;
    }
    return seg_scan_impl(x, flags_u8, MMV_SEG_FLAGS_U8, n, 0, dt, out, workspace, workspace_bytes, cuda_stream, false,
                         first_shard ? 1 : 2, summary);
}

mmv_status mmv_seg_scan_shard_finish(const void* summaries, int rank, int world, void* out, int64_t n, mmv_dtype dt,
                                     void* cuda_stream) {
    if (n < 0 || world <= 0 || rank < 0 || rank >= world) return MMV_ERR_INVALID_ARG;
    if (dt != MMV_F16_TO_F32 && dt != MMV_I8_TO_I32 && dt != MMV_BF16_TO_F32) return MMV_ERR_INVALID_ARG;
    if (!summaries || (reinterpret_cast<uintptr_t>(summaries) & 15u)) return MMV_ERR_INVALID_ARG;
    if (n == 0 || rank == 0) return MMV_OK;                        // nothing in front of the first shard
    if (!out || !aligned16(out)) return MMV_ERR_INVALID_ARG;
    DeviceInfo* dev = device_info();
    if (!dev) return MMV_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const int threads = 256;
    long long blocks = ((n >> 2) + threads - 1) / threads;
    const long long cap = static_cast<long long>(dev->sm_count) * 8;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    const ShardSummary* all = static_cast<const ShardSummary*>(summaries);
    if (dt == MMV_I8_TO_I32)
        shard_finish_kernel<false><<<static_cast<unsigned>(blocks), threads, 0, st>>>(all, rank, static_cast<uint32_t*>(out), n);
    else
        shard_finish_kernel<true><<<static_cast<unsigned>(blocks), threads, 0, st>>>(all, rank, static_cast<uint32_t*>(out), n);
    ++g_launches;
    return cudaGetLastError() == cudaSuccess ? MMV_OK : MMV_ERR_CUDA;
}

// ---------------------------------------------------------------------------
// Scan of host-resident vectors: chunks travel host -> device, are scanned, and travel back on
// three streams, so that the copies of neighbouring chunks overlap each other and the kernels.
// Chunk c + 1 continues the open segment of chunk c through the kernel's carry-in word (the last
// output element of chunk c, still in its device buffer).
// ---------------------------------------------------------------------------
namespace {

struct HostScanPlan {
    size_t status_off, status_bytes;      // per buffer
    size_t x_off, f_off, out_off;         // per buffer, relative to the buffer's base
    size_t buf_bytes;
    size_t total;
};

HostScanPlan plan_host_scan(mmv_dtype dt, long long chunk) {
    HostScanPlan p{};
    const size_t eb = dt == MMV_F16_TO_F32 ? 2 : 1;
    p.status_off = 0;
    p.status_bytes = round_up(static_cast<size_t>(num_scan_tiles_of(chunk)) * SCAN_STATUS_STRIDE * sizeof(uint64_t), 256);
    p.x_off = p.status_bytes;
    p.f_off = p.x_off + round_up(static_cast<size_t>(chunk) * eb, 256);
    p.out_off = p.f_off + round_up(static_cast<size_t>(chunk), 256);
    p.buf_bytes = p.out_off + round_up(static_cast<size_t>(chunk) * 4, 256);
    p.total = sizeof(WorkspaceHeader) + 2 * p.buf_bytes;
    return p;
}

bool pipe_streams(DeviceInfo* d) {
    std::call_once(d->pipe_once, [d] {
        bool ok = true;
        ok &= cudaStreamCreateWithFlags(&d->s_in, cudaStreamNonBlocking) == cudaSuccess;
        ok &= cudaStreamCreateWithFlags(&d->s_k, cudaStreamNonBlocking) == cudaSuccess;
        ok &= cudaStreamCreateWithFlags(&d->s_out, cudaStreamNonBlocking) == cudaSuccess;
        cudaEvent_t* evs[] = {&d->ev_start, &d->ev_end_k, &d->ev_end_out, &d->in_done[0], &d->in_done[1],
                              &d->k_done[0], &d->k_done[1], &d->out_done[0], &d->out_done[1]};
        for (cudaEvent_t* e : evs) ok &= cudaEventCreateWithFlags(e, cudaEventDisableTiming) == cudaSuccess;
        d->pipe_ok = ok;
    });
    return d->pipe_ok;
}

}  // namespace

size_t mmv_seg_scan_host_scratch_bytes(mmv_dtype dt, int64_t chunk_elems) {
    if (dt != MMV_F16_TO_F32 && dt != MMV_I8_TO_I32) return 0;
    if (chunk_elems <= 0 || chunk_elems % SCAN_TILE != 0 || chunk_elems >= (1ll << 36)) return 0;
    return plan_host_scan(dt, chunk_elems).total;
}

mmv_status mmv_seg_scan_host(const void* x_host, const void* flags_host, int64_t n, mmv_dtype dt, void* out_host,
                             int64_t chunk_elems, void* device_scratch, size_t device_scratch_bytes, void* cuda_stream) {
    if (n < 0) return MMV_ERR_INVALID_ARG;
    if (dt != MMV_F16_TO_F32 && dt != MMV_I8_TO_I32) return MMV_ERR_INVALID_ARG;
    if (chunk_elems <= 0 || chunk_elems % SCAN_TILE != 0 || chunk_elems >= (1ll << 36)) return MMV_ERR_INVALID_ARG;
    if (n == 0) return MMV_OK;
    if (!x_host || !out_host || !device_scratch) return MMV_ERR_INVALID_ARG;      // flags_host may be null: one segment
    if (reinterpret_cast<uintptr_t>(device_scratch) & 255u) return MMV_ERR_INVALID_ARG;
    const HostScanPlan plan = plan_host_scan(dt, chunk_elems);
    if (device_scratch_bytes < plan.total) return MMV_ERR_WORKSPACE_TOO_SMALL;
    DeviceInfo* dev = device_info();
    if (!dev || !pipe_streams(dev)) return MMV_ERR_CUDA;

    const bool f16 = dt == MMV_F16_TO_F32;
    const size_t eb = f16 ? 2 : 1;
    cudaStream_t user = static_cast<cudaStream_t>(cuda_stream);
    uint8_t* base = static_cast<uint8_t*>(device_scratch);
    WorkspaceHeader* hdr = reinterpret_cast<WorkspaceHeader*>(base);
    uint8_t* buf[2] = {base + sizeof(WorkspaceHeader), base + sizeof(WorkspaceHeader) + plan.buf_bytes};
    bool ok = true;
    ok &= cudaMemsetAsync(hdr, 0, sizeof(WorkspaceHeader), user) == cudaSuccess;
    ok &= cudaEventRecord(dev->ev_start, user) == cudaSuccess;
    ok &= cudaStreamWaitEvent(dev->s_in, dev->ev_start, 0) == cudaSuccess;
    ok &= cudaStreamWaitEvent(dev->s_k, dev->ev_start, 0) == cudaSuccess;
    ok &= cudaStreamWaitEvent(dev->s_out, dev->ev_start, 0) == cudaSuccess;
    if (!ok) return MMV_ERR_CUDA;

    const long long nchunks = (n + chunk_elems - 1) / chunk_elems;
    const void* carry = nullptr;
    for (long long c = 0; c < nchunks; ++c) {
        const int b = static_cast<int>(c & 1);
        const long long o = c * chunk_elems;
        const long long m = n - o < chunk_elems ? n - o : chunk_elems;
        uint8_t* xd = buf[b] + plan.x_off;
        uint8_t* fd = buf[b] + plan.f_off;
        uint8_t* od = buf[b] + plan.out_off;
        // copy in: the buffer's previous kernel (chunk c - 2) must be done with it
        if (c >= 2) ok &= cudaStreamWaitEvent(dev->s_in, dev->k_done[b], 0) == cudaSuccess;
        ok &= cudaMemcpyAsync(xd, static_cast<const uint8_t*>(x_host) + static_cast<size_t>(o) * eb, static_cast<size_t>(m) * eb,
                              cudaMemcpyHostToDevice, dev->s_in) == cudaSuccess;
        if (flags_host)
            ok &= cudaMemcpyAsync(fd, static_cast<const uint8_t*>(flags_host) + o, static_cast<size_t>(m),
                                  cudaMemcpyHostToDevice, dev->s_in) == cudaSuccess;
        ok &= cudaEventRecord(dev->in_done[b], dev->s_in) == cudaSuccess;
        // scan: needs the inputs, and the buffer's previous output (chunk c - 2) copied out
        ok &= cudaStreamWaitEvent(dev->s_k, dev->in_done[b], 0) == cudaSuccess;
        if (c >= 2) ok &= cudaStreamWaitEvent(dev->s_k, dev->out_done[b], 0) == cudaSuccess;
        ok &= cudaMemsetAsync(buf[b] + plan.status_off, 0, plan.status_bytes, dev->s_k) == cudaSuccess;
        if (!ok) return MMV_ERR_CUDA;
        CUtensorMap tmap, tmap_out;
        if (!encode_span_map(&tmap, xd, m, f16 ? 2 : 1, SCAN_UP)) return MMV_ERR_CUDA;
        if (!encode_out_map(&tmap_out, od, m)) return MMV_ERR_CUDA;
        ScanParams prm;
        prm.x = xd;
        prm.flags = flags_host ? fd : nullptr;
        prm.out = od;
        prm.n = m;
        prm.num_tiles = static_cast<int>(num_scan_tiles_of(m));
        prm.hdr = hdr;
        prm.status = reinterpret_cast<uint64_t*>(buf[b] + plan.status_off);
        prm.budget_ns = g_budget_ns.load();
        prm.debug_skip_span = -1;
        prm.carry_in = carry;
        prm.first_start = nullptr;
        prm.probe_count = nullptr;
        prm.probe_narrow_below = 0u;
        prm.clear_words = 0;
        const int grid = prm.num_tiles < dev->sm_count ? prm.num_tiles : dev->sm_count;
        if (f16)
            ok &= launch_resident(seg_scan_kernel<F16Path>, grid, ScanCfg<F16Path>::kThreads, ScanCfg<F16Path>::kSmemBytes, dev->s_k,
                                  false, tmap, tmap_out, prm) == cudaSuccess;
        else
            ok &= launch_resident(seg_scan_kernel<I8Path>, grid, ScanCfg<I8Path>::kThreads, ScanCfg<I8Path>::kSmemBytes, dev->s_k,
                                  false, tmap, tmap_out, prm) == cudaSuccess;
        ++g_launches;
        ok &= cudaEventRecord(dev->k_done[b], dev->s_k) == cudaSuccess;
        carry = od + static_cast<size_t>(m - 1) * 4;           // the running sum at the end of this chunk
        // copy out
        ok &= cudaStreamWaitEvent(dev->s_out, dev->k_done[b], 0) == cudaSuccess;
        ok &= cudaMemcpyAsync(static_cast<uint8_t*>(out_host) + static_cast<size_t>(o) * 4, od, static_cast<size_t>(m) * 4,
                              cudaMemcpyDeviceToHost, dev->s_out) == cudaSuccess;
        ok &= cudaEventRecord(dev->out_done[b], dev->s_out) == cudaSuccess;
        if (!ok) return MMV_ERR_CUDA;
    }
    // the caller's stream continues when everything is back on the host
    ok &= cudaEventRecord(dev->ev_end_k, dev->s_k) == cudaSuccess;
    ok &= cudaEventRecord(dev->ev_end_out, dev->s_out) == cudaSuccess;
    ok &= cudaStreamWaitEvent(user, dev->ev_end_k, 0) == cudaSuccess;
    ok &= cudaStreamWaitEvent(user, dev->ev_end_out, 0) == cudaSuccess;
    return ok ? MMV_OK : MMV_ERR_CUDA;
}

mmv_status mmv_seg_sum(const void* x, const void* seg, mmv_segfmt sf, int64_t n, int64_t nseg, mmv_dtype dt,
                       void* out, int64_t* d_num_segments, void* workspace, size_t workspace_bytes,
                       void* cuda_stream) {
    if (n < 0 || nseg < 0) return MMV_ERR_INVALID_ARG;
    if (dt != MMV_F16_TO_F32 && dt != MMV_I8_TO_I32 && dt != MMV_BF16_TO_F32) return MMV_ERR_INVALID_ARG;
    if (sf != MMV_SEG_FLAGS_U8 && sf != MMV_SEG_OFFSETS_I32) return MMV_ERR_INVALID_ARG;
    if (n >= (1ll << 31)) return MMV_ERR_INVALID_ARG;            // int32 offsets cannot address more
    if (nseg >= (1ll << 31) - 1) return MMV_ERR_INVALID_ARG;     // offset indices are kept in 32 bits (empty segments may outnumber n)
    if (sf == MMV_SEG_FLAGS_U8) {
        // COMPRESS the start flags into offsets (in the workspace), then the offset-encoded kernel with
        // the segment count read on the device.
        cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
        if (n == 0) {
            if (d_num_segments && cudaMemsetAsync(d_num_segments, 0, sizeof(int64_t), st) != cudaSuccess) return MMV_ERR_CUDA;
            return nothing_to_do(workspace, workspace_bytes, cuda_stream);
        }
        if (!x || !seg || !out || !workspace) return MMV_ERR_INVALID_ARG;
        if (!aligned16(x) || !aligned16(seg) || !aligned16(out) || (reinterpret_cast<uintptr_t>(workspace) & 255u))
            return MMV_ERR_INVALID_ARG;
        if (d_num_segments && (reinterpret_cast<uintptr_t>(d_num_segments) & 7u)) return MMV_ERR_INVALID_ARG;
        const WorkspacePlan plan = plan_workspace(MMV_OP_SEG_SUM, sf, n);
        if (workspace_bytes < plan.total) return MMV_ERR_WORKSPACE_TOO_SMALL;
        DeviceInfo* dev = device_info();
        if (!dev) return MMV_ERR_CUDA;
        uint8_t* ws = static_cast<uint8_t*>(workspace);
        if (cudaMemsetAsync(ws, 0, plan.status_off + plan.status_bytes, st) != cudaSuccess) return MMV_ERR_CUDA;
        const long long nchunks = (n + CMP_CHUNK - 1) / CMP_CHUNK;
        long long* nseg_dev = reinterpret_cast<long long*>(ws + plan.cmp_off);
        int32_t* chunk_count = reinterpret_cast<int32_t*>(ws + plan.cmp_off + 16);
        int32_t* chunk_base = chunk_count + ((nchunks + 3) & ~3ll);      // 16-byte aligned: it is written as vectors
        int32_t* off = reinterpret_cast<int32_t*>(ws + plan.off_off);
        const uint8_t* f = static_cast<const uint8_t*>(seg);
        const long long cap = static_cast<long long>(dev->sm_count) * 8;
        const unsigned blocks = static_cast<unsigned>(nchunks < cap ? nchunks : cap);
        unsigned long long* masks = reinterpret_cast<unsigned long long*>(ws + plan.mask_off);
        int32_t* warp_off = reinterpret_cast<int32_t*>(ws + plan.mask_off + round_up(static_cast<size_t>(nchunks) * CMP_THREADS * sizeof(unsigned long long), 256));
        flag_count_kernel<<<blocks, CMP_THREADS, 0, st>>>(f, n, nchunks, chunk_count, masks, warp_off);
        chunk_scan_kernel<<<CMP_SCAN_BLOCKS, 1024, 0, st>>>(chunk_count, nchunks, chunk_base, nseg_dev,
                                              reinterpret_cast<long long*>(d_num_segments), off, n);
        static_assert(CMP_CHUNK == TILE && SPAN == 4096, "a compaction chunk is one tile of four spans");
        flag_scatter_kernel<<<blocks, CMP_THREADS, 0, st>>>(masks, n, nchunks, chunk_base, warp_off, off,
                                                            reinterpret_cast<int32_t*>(ws + plan.tileq_off), nseg_dev);
        g_launches += 3;
        if (cudaGetLastError() != cudaSuccess) return MMV_ERR_CUDA;
        if (dt == MMV_F16_TO_F32) return launch_seg_sum<F16Path>(x, n, off, 0, 0, out, ws, plan, dev, st, nseg_dev, true);
        if (dt == MMV_BF16_TO_F32) return launch_seg_sum<BF16ValPath>(x, n, off, 0, 0, out, ws, plan, dev, st, nseg_dev, true);
        return launch_seg_sum<I8Path>(x, n, off, 0, 0, out, ws, plan, dev, st, nseg_dev, true);
    }
    if (nseg == 0) return nothing_to_do(workspace, workspace_bytes, cuda_stream);
    if (!seg || !out) return MMV_ERR_INVALID_ARG;
    if (!aligned16(seg) || !aligned16(out)) return MMV_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    if (n == 0) {                                                // every segment is empty
        if (cudaMemsetAsync(out, 0, static_cast<size_t>(nseg) * 4, st) != cudaSuccess) return MMV_ERR_CUDA;
        return nothing_to_do(workspace, workspace_bytes, cuda_stream);
    }
    if (!x || !workspace) return MMV_ERR_INVALID_ARG;
    if (!aligned16(x) || (reinterpret_cast<uintptr_t>(workspace) & 255u)) return MMV_ERR_INVALID_ARG;
    const WorkspacePlan plan = plan_workspace(MMV_OP_SEG_SUM, sf, n);
    if (workspace_bytes < plan.total) return MMV_ERR_WORKSPACE_TOO_SMALL;
    DeviceInfo* dev = device_info();
    if (!dev) return MMV_ERR_CUDA;
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    // Up to 2^18 segments, one launch: the tiled kernel clears the header and the status words and partitions the
    // offsets itself, in front of a grid-wide barrier (it is launched cooperatively anyway).  Configuration 2:
    // 39.5 -> 35.9 us per call (a memset, the partition kernel and the tiled kernel were three enqueues), n = 2^28
    // 106 -> 104 us.  With millions of offsets the partition wants more threads than the tiled grid has (11.4 M
    // offsets: 188 -> 210 us fused), so those calls keep the memset and the kernel of its own.
    const bool fused = nseg <= (1ll << 18);
    if (!fused && cudaMemsetAsync(ws, 0, plan.status_off + plan.status_bytes, st) != cudaSuccess) return MMV_ERR_CUDA;
    const int32_t* off = static_cast<const int32_t*>(seg);
    if (dt == MMV_F16_TO_F32) return launch_seg_sum<F16Path>(x, n, off, nseg, 0, out, ws, plan, dev, st, nullptr, false, fused);
    if (dt == MMV_BF16_TO_F32) return launch_seg_sum<BF16ValPath>(x, n, off, nseg, 0, out, ws, plan, dev, st, nullptr, false, fused);
    return launch_seg_sum<I8Path>(x, n, off, nseg, 0, out, ws, plan, dev, st, nullptr, false, fused);
}

mmv_status mmv_seg_scan_minmax(const void* x, const void* flags, int64_t n, mmv_dtype dt, int want_min, void* out,
                               void* workspace, size_t workspace_bytes, void* cuda_stream) {
    if (n < 0) return MMV_ERR_INVALID_ARG;
    if (dt != MMV_F16_TO_F32 && dt != MMV_I8_TO_I32 && dt != MMV_BF16_TO_F32) return MMV_ERR_INVALID_ARG;
    if (n == 0) return nothing_to_do(workspace, workspace_bytes, cuda_stream);
    if (n >= (1ll << 36)) return MMV_ERR_UNSUPPORTED;
    if (!x || !out || !workspace) return MMV_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(flags) || !aligned16(out) || (reinterpret_cast<uintptr_t>(workspace) & 255u))
        return MMV_ERR_INVALID_ARG;
    const WorkspacePlan plan = plan_workspace(MMV_OP_SEG_SCAN_MINMAX, MMV_SEG_FLAGS_U8, n);
    if (workspace_bytes < plan.total) return MMV_ERR_WORKSPACE_TOO_SMALL;
    DeviceInfo* dev = device_info();
    if (!dev) return MMV_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    if (cudaMemsetAsync(ws, 0, plan.status_off + plan.status_bytes, st) != cudaSuccess) return MMV_ERR_CUDA;
    MinMaxParams prm;
    prm.x = x;
    prm.flags = static_cast<const uint8_t*>(flags);
    prm.out = out;
    prm.n = n;
    prm.num_tiles = (n + MM_TILE - 1) / MM_TILE;
    prm.hdr = reinterpret_cast<WorkspaceHeader*>(ws);
    prm.status = reinterpret_cast<uint64_t*>(ws + plan.status_off);
    prm.budget_ns = g_budget_ns.load();
    const long long skip = g_debug_skip_span.load();
    prm.debug_skip_run = skip >= 0 ? skip * SCAN_UNIT / MM_TILE : -1;        // the hook counts 4096-element spans
    const long long cap = static_cast<long long>(dev->sm_count) * MM_CTAS_PER_SM;
    const unsigned blocks = static_cast<unsigned>(prm.num_tiles < cap ? prm.num_tiles : cap);
    if (dt == MMV_F16_TO_F32) {
        if (want_min) seg_scan_minmax_kernel<0, true><<<blocks, MM_THREADS, MM_SMEM_BYTES, st>>>(prm);
        else seg_scan_minmax_kernel<0, false><<<blocks, MM_THREADS, MM_SMEM_BYTES, st>>>(prm);
    } else if (dt == MMV_I8_TO_I32) {
        if (want_min) seg_scan_minmax_kernel<1, true><<<blocks, MM_THREADS, MM_SMEM_BYTES, st>>>(prm);
        else seg_scan_minmax_kernel<1, false><<<blocks, MM_THREADS, MM_SMEM_BYTES, st>>>(prm);
    } else {
        if (want_min) seg_scan_minmax_kernel<2, true><<<blocks, MM_THREADS, MM_SMEM_BYTES, st>>>(prm);
        else seg_scan_minmax_kernel<2, false><<<blocks, MM_THREADS, MM_SMEM_BYTES, st>>>(prm);
    }
    ++g_launches;
    return cudaGetLastError() == cudaSuccess ? MMV_OK : MMV_ERR_CUDA;
}

mmv_status mmv_seg_scan_i8_i64(const void* x, const void* flags, int64_t n, int64_t* out, void* workspace,
                               size_t workspace_bytes, void* cuda_stream) {
    if (n < 0) return MMV_ERR_INVALID_ARG;
    if (n == 0) return nothing_to_do(workspace, workspace_bytes, cuda_stream);
    if (n >= (1ll << 36)) return MMV_ERR_UNSUPPORTED;
    if (!x || !out || !workspace) return MMV_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(flags) || !aligned16(out) || (reinterpret_cast<uintptr_t>(workspace) & 255u))
        return MMV_ERR_INVALID_ARG;
    const WorkspacePlan plan = plan_workspace(MMV_OP_SEG_SCAN_WIDE, MMV_SEG_FLAGS_U8, n);
    if (workspace_bytes < plan.total) return MMV_ERR_WORKSPACE_TOO_SMALL;
    DeviceInfo* dev = device_info();
    if (!dev) return MMV_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    if (cudaMemsetAsync(ws, 0, plan.status_off + plan.status_bytes, st) != cudaSuccess) return MMV_ERR_CUDA;
    WideParams prm;
    prm.x = static_cast<const int8_t*>(x);
    prm.flags = static_cast<const uint8_t*>(flags);
    prm.out = reinterpret_cast<long long*>(out);
    prm.n = n;
    prm.num_tiles = (n + WD_TILE - 1) / WD_TILE;
    prm.hdr = reinterpret_cast<WorkspaceHeader*>(ws);
    prm.status = reinterpret_cast<uint64_t*>(ws + plan.status_off);
    prm.budget_ns = g_budget_ns.load();
    const long long skip = g_debug_skip_span.load();
    prm.debug_skip_tile = skip >= 0 ? skip * SCAN_UNIT / WD_TILE : -1;         // the hook counts 4096-element spans
    const long long cap = static_cast<long long>(dev->sm_count) * WD_CTAS_PER_SM;
    const unsigned blocks = static_cast<unsigned>(prm.num_tiles < cap ? prm.num_tiles : cap);
    seg_scan_wide_kernel<<<blocks, WD_THREADS, 0, st>>>(prm);
    ++g_launches;
    return cudaGetLastError() == cudaSuccess ? MMV_OK : MMV_ERR_CUDA;
}

mmv_status mmv_compress(const void* x, const void* flags, int64_t n, mmv_dtype dt, void* out, int64_t* d_count,
                        void* workspace, size_t workspace_bytes, void* cuda_stream) {
    if (n < 0 || n >= (1ll << 31)) return MMV_ERR_INVALID_ARG;
    if (dt != MMV_F16_TO_F32 && dt != MMV_I8_TO_I32 && dt != MMV_BF16_TO_F32) return MMV_ERR_INVALID_ARG;
    if (d_count && (reinterpret_cast<uintptr_t>(d_count) & 7u)) return MMV_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    if (n == 0) {
        if (d_count && cudaMemsetAsync(d_count, 0, sizeof(int64_t), st) != cudaSuccess) return MMV_ERR_CUDA;
        return nothing_to_do(workspace, workspace_bytes, cuda_stream);
    }
    if (!x || !flags || !out || !workspace) return MMV_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(flags) || !aligned16(out) || (reinterpret_cast<uintptr_t>(workspace) & 255u))
        return MMV_ERR_INVALID_ARG;
    const WorkspacePlan plan = plan_workspace(MMV_OP_COMPRESS, MMV_SEG_FLAGS_U8, n);
    if (workspace_bytes < plan.total) return MMV_ERR_WORKSPACE_TOO_SMALL;
    DeviceInfo* dev = device_info();
    if (!dev) return MMV_ERR_CUDA;
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    if (cudaMemsetAsync(ws, 0, sizeof(WorkspaceHeader), st) != cudaSuccess) return MMV_ERR_CUDA;
    const long long nchunks = (n + CMP_CHUNK - 1) / CMP_CHUNK;
    long long* count_dev = reinterpret_cast<long long*>(ws + plan.cmp_off);
    int32_t* chunk_count = reinterpret_cast<int32_t*>(ws + plan.cmp_off + 16);
    int32_t* chunk_base = chunk_count + ((nchunks + 3) & ~3ll);
    const uint8_t* f = static_cast<const uint8_t*>(flags);
    const long long cap = static_cast<long long>(dev->sm_count) * 8;
    const unsigned blocks = static_cast<unsigned>(nchunks < cap ? nchunks : cap);
    unsigned long long* masks = reinterpret_cast<unsigned long long*>(ws + plan.mask_off);
    int32_t* warp_off = reinterpret_cast<int32_t*>(ws + plan.mask_off + round_up(static_cast<size_t>(nchunks) * CMP_THREADS * sizeof(unsigned long long), 256));
    flag_count_kernel<<<blocks, CMP_THREADS, 0, st>>>(f, n, nchunks, chunk_count, masks, warp_off, false);
    chunk_scan_kernel<<<CMP_SCAN_BLOCKS, 1024, 0, st>>>(chunk_count, nchunks, chunk_base, count_dev, reinterpret_cast<long long*>(d_count),
                                          nullptr, n);
    if (dt == MMV_I8_TO_I32)
        compress_values_kernel<uint8_t><<<blocks, CMP_THREADS, 0, st>>>(static_cast<const uint8_t*>(x), masks, n, nchunks, chunk_base,
                                                                       warp_off, static_cast<uint8_t*>(out));
    else
        compress_values_kernel<unsigned short><<<blocks, CMP_THREADS, 0, st>>>(static_cast<const unsigned short*>(x), masks, n, nchunks,
                                                                              chunk_base, warp_off, static_cast<unsigned short*>(out));
    g_launches += 3;
    return cudaGetLastError() == cudaSuccess ? MMV_OK : MMV_ERR_CUDA;
}

mmv_status mmv_mult_i8(const int8_t* x, const int8_t* y, int64_t n, int32_t* out, void* workspace, size_t workspace_bytes,
                       void* cuda_stream) {
    if (n < 0 || n >= (1ll << 28)) return MMV_ERR_INVALID_ARG;          // 8 n terms are addressed by int32 offsets
    if (n == 0) return nothing_to_do(workspace, workspace_bytes, cuda_stream);
    if (!x || !y || !out || !workspace) return MMV_ERR_INVALID_ARG;
    if (!aligned16(out) || (reinterpret_cast<uintptr_t>(workspace) & 255u)) return MMV_ERR_INVALID_ARG;
    const MultPlan plan = plan_mult(n);
    if (workspace_bytes < plan.total) return MMV_ERR_WORKSPACE_TOO_SMALL;
    DeviceInfo* dev = device_info();
    if (!dev) return MMV_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    __half* terms = reinterpret_cast<__half*>(ws + plan.terms_off);
    int32_t* off = reinterpret_cast<int32_t*>(ws + plan.off_off);
    const int threads = 256;
    long long blocks = (n + threads) / threads;
    const long long cap = static_cast<long long>(dev->sm_count) * 16;
    if (blocks > cap) blocks = cap;
    mult_expand_kernel<<<static_cast<unsigned>(blocks), threads, 0, st>>>(x, y, n, terms, off);
    ++g_launches;
    if (cudaGetLastError() != cudaSuccess) return MMV_ERR_CUDA;
    if (cudaMemsetAsync(ws, 0, plan.sum.status_off + plan.sum.status_bytes, st) != cudaSuccess) return MMV_ERR_CUDA;
    const mmv_status rc = launch_seg_sum<F16Path>(terms, n * MULT_TERMS, off, n, 0, out, ws, plan.sum, dev, st);
    if (rc != MMV_OK) return rc;
    mult_to_int_kernel<<<static_cast<unsigned>(blocks), threads, 0, st>>>(reinterpret_cast<float*>(out), n);
    ++g_launches;
    return cudaGetLastError() == cudaSuccess ? MMV_OK : MMV_ERR_CUDA;
}

mmv_status mmv_spmv_csr(const int32_t* rowptr, const int32_t* col, const void* val_f16, const float* x, float* y,
                        int64_t rows, int64_t cols, int64_t nnz, void* workspace, size_t workspace_bytes,
                        void* cuda_stream) {
    if (rows < 0 || cols < 0 || nnz < 0) return MMV_ERR_INVALID_ARG;
    if (nnz >= (1ll << 31)) return MMV_ERR_INVALID_ARG;          // int32 offsets cannot address more
    if (rows >= (1ll << 31) - 1) return MMV_ERR_INVALID_ARG;     // row indices are kept in 32 bits (empty rows may outnumber nnz)
    if (rows == 0) return nothing_to_do(workspace, workspace_bytes, cuda_stream);
    if (!rowptr || !y) return MMV_ERR_INVALID_ARG;
    if (!aligned16(rowptr) || !aligned16(y)) return MMV_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    if (nnz == 0) {
        if (cudaMemsetAsync(y, 0, static_cast<size_t>(rows) * 4, st) != cudaSuccess) return MMV_ERR_CUDA;
        return nothing_to_do(workspace, workspace_bytes, cuda_stream);
    }
    if (!col || !val_f16 || !x || !workspace || cols == 0) return MMV_ERR_INVALID_ARG;
    if (!aligned16(col) || !aligned16(val_f16) || !aligned16(x) || (reinterpret_cast<uintptr_t>(workspace) & 255u))
        return MMV_ERR_INVALID_ARG;
    const WorkspacePlan plan = plan_workspace(MMV_OP_SPMV_CSR, MMV_SEG_OFFSETS_I32, nnz);
    if (workspace_bytes < plan.total) return MMV_ERR_WORKSPACE_TOO_SMALL;
    DeviceInfo* dev = device_info();
    if (!dev) return MMV_ERR_CUDA;
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    if (cudaMemsetAsync(ws, 0, plan.status_off + plan.status_bytes, st) != cudaSuccess) return MMV_ERR_CUDA;
    uint32_t* prod = reinterpret_cast<uint32_t*>(ws + plan.prod_off);
    // The span partition of the row pointers first: the gather does not depend on it and is launched so that it
    // may start at once (the partition is bound by its few loads in flight, 28 us for 2^20 rows, and leaves the
    // GPU nearly empty); the tiled kernel behind the gather needs both.
    launch_partition(rowptr, rows, nnz, y, ws, plan, dev, st);
    {
        const int threads = 256;
        long long blocks = ((nnz >> 2) + threads - 1) / threads;
        const long long cap = static_cast<long long>(dev->sm_count) * 16;
        if (blocks > cap) blocks = cap;
        if (blocks < 1) blocks = 1;
        cudaLaunchConfig_t cfg{};
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.gridDim = dim3(static_cast<unsigned>(blocks));
        cfg.blockDim = dim3(threads);
        cfg.stream = st;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        const cudaError_t err = cudaLaunchKernelEx(&cfg, spmv_gather_kernel, col, static_cast<const __half*>(val_f16), x, prod,
                                                   static_cast<long long>(nnz), static_cast<long long>(cols),
                                                   reinterpret_cast<WorkspaceHeader*>(ws));
        ++g_launches;
        if (err != cudaSuccess) return MMV_ERR_CUDA;
    }
    return launch_seg_sum<BF16Path>(prod, nnz, rowptr, rows, 0, y, ws, plan, dev, st, nullptr, true);
}

mmv_status mmv_last_async_status(const void* workspace, void* cuda_stream) {
    if (!workspace) return MMV_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    if (cudaStreamSynchronize(st) != cudaSuccess) return MMV_ERR_CUDA;
    WorkspaceHeader h;
    if (cudaMemcpy(&h, workspace, sizeof(unsigned int) * 2, cudaMemcpyDeviceToHost) != cudaSuccess) return MMV_ERR_CUDA;
    return h.error <= 6u ? static_cast<mmv_status>(h.error) : MMV_ERR_CUDA;
}

mmv_status mmv_seg_scan_static(const void* x, const void* flags_u8, int64_t n, mmv_dtype dt, void* out,
                               void* cuda_stream) {
    if (n < 0) return MMV_ERR_INVALID_ARG;
    if (dt != MMV_F16_TO_F32 && dt != MMV_I8_TO_I32) return MMV_ERR_INVALID_ARG;
    if (n == 0) return MMV_OK;
    if (n > kStaticScanMaxN) return MMV_ERR_WORKSPACE_TOO_SMALL;      // the built-in buffer covers 2^28 elements
    if (!x || !flags_u8 || !out) return MMV_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(flags_u8) || !aligned16(out)) return MMV_ERR_INVALID_ARG;
    DeviceInfo* dev = device_info();
    if (!dev) return MMV_ERR_CUDA;
    uint8_t* ws = static_cast<uint8_t*>(static_scratch_ptr());        // device address, never the host symbol
    if (!ws) return MMV_ERR_CUDA;

    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const long long tiles = num_scan_tiles_of(n);
    const size_t used = sizeof(WorkspaceHeader) + static_cast<size_t>(tiles) * SCAN_STATUS_STRIDE * sizeof(uint64_t);
    // the buffer keeps the previous call's words: everything this call reads must start at zero
    if (cudaMemsetAsync(ws, 0, used, st) != cudaSuccess) return MMV_ERR_CUDA;

    const bool f16 = dt == MMV_F16_TO_F32;
    CUtensorMap tmap, tmap_out;
    if (!encode_span_map(&tmap, x, n, f16 ? 2 : 1, SCAN_UP)) return MMV_ERR_CUDA;
    if (!encode_out_map(&tmap_out, out, n)) return MMV_ERR_CUDA;
    ScanParams prm;
    prm.x = x;
    prm.flags = static_cast<const uint8_t*>(flags_u8);
    prm.out = out;
    prm.n = n;
    prm.num_tiles = static_cast<int>(tiles);
    prm.hdr = reinterpret_cast<WorkspaceHeader*>(ws);
    prm.status = reinterpret_cast<uint64_t*>(ws + sizeof(WorkspaceHeader));
    prm.budget_ns = g_budget_ns.load();
    prm.debug_skip_span = g_debug_skip_span.load();
    prm.carry_in = nullptr;
    prm.first_start = nullptr;
    prm.probe_count = nullptr;
    prm.probe_narrow_below = 0u;
    prm.clear_words = 0;
    const int grid = prm.num_tiles < dev->sm_count ? prm.num_tiles : dev->sm_count;
    cudaError_t err;
    if (f16)
        err = launch_resident(seg_scan_kernel<F16Path>, grid, ScanCfg<F16Path>::kThreads, ScanCfg<F16Path>::kSmemBytes, st, false,
                              tmap, tmap_out, prm);
    else
        err = launch_resident(seg_scan_kernel<I8Path>, grid, ScanCfg<I8Path>::kThreads, ScanCfg<I8Path>::kSmemBytes, st, false,
                              tmap, tmap_out, prm);
    ++g_launches;
    return err == cudaSuccess ? MMV_OK : MMV_ERR_CUDA;
}

mmv_status mmv_seg_scan_static_last_status(void* cuda_stream) {
    void* ws = static_scratch_ptr();
    if (!ws) return MMV_ERR_CUDA;
    return mmv_last_async_status(ws, cuda_stream);
}

const char* mmv_status_string(mmv_status s) {
    switch (s) {
        case MMV_OK: return "ok";
        case MMV_ERR_INVALID_ARG: return "invalid argument";
        case MMV_ERR_UNSUPPORTED: return "unsupported combination";
        case MMV_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
        case MMV_ERR_BAD_SEGMENTS: return "segment offsets not monotone or out of range";
        case MMV_ERR_TIMEOUT: return "device-side wait timed out";
        case MMV_ERR_CUDA: return "CUDA call failed";
    }
    return "unknown status";
}

int64_t mmv_kernel_launch_count(void) { return g_launches.load(); }

#ifdef MMV_PHASE_TIMERS
// Development aid: reads and clears the phase-cycle counters of the scan kernel.
void mmv_debug_phase_cycles(unsigned long long* host16) {
    cudaDeviceSynchronize();
    cudaMemcpyFromSymbol(host16, g_phase_cycles, 16 * sizeof(unsigned long long));
    unsigned long long z[16] = {0};
    cudaMemcpyToSymbol(g_phase_cycles, z, sizeof(z));
}
#endif

void mmv_debug_force_scan_shape(int shape) { g_force_scan_shape.store(shape == SCAN_WIDE || shape == SCAN_NARROW ? shape : -1); }

void mmv_debug_force_sum_groups(int groups) { g_force_groups.store(groups == 2 || groups == 3 ? groups : 0); }

void mmv_debug_configure(int64_t wait_budget_ns, int64_t skip_publish_span) {
    g_budget_ns.store(wait_budget_ns > 0 ? static_cast<unsigned long long>(wait_budget_ns) : WAIT_BUDGET_NS);
    g_debug_skip_span.store(skip_publish_span);
}

}  // extern "C"
