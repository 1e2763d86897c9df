// Shared constants and small helpers of the segmented-operation kernels.
#pragma once
#include <cstdint>
#include <cuda_fp16.h>
#include "ptx.cuh"

namespace mmv {

// Phase timers, a supported build flag for performance work (MMV_NVCC_FLAGS=-DMMV_PHASE_TIMERS python
// paper_2506_23906_b200/build.py --force): every epilogue warp adds the cycles it spends between the
// MMV_T_MARK points of the scan and segmented-sum kernels to 16 global counters, which the extra export
// mmv_debug_phase_cycles reads and clears.  Without the flag the macros are empty and nothing is compiled in.
#ifdef MMV_PHASE_TIMERS
__device__ unsigned long long g_phase_cycles[16];
#define MMV_T_DECL long long t_prev = clock64(); unsigned long long t_acc[16] = {0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0};
#define MMV_T_MARK(k) { const long long t_now = clock64(); t_acc[k] += static_cast<unsigned long long>(t_now - t_prev); t_prev = t_now; }
#define MMV_T_FLUSH() { if (lane == 0) { for (int k = 0; k < 16; ++k) atomicAdd(&g_phase_cycles[k], t_acc[k]); } }
#else
#define MMV_T_DECL
#define MMV_T_MARK(k)
#define MMV_T_FLUSH()
#endif

// Geometry.  The value vector is viewed as rows of ROW consecutive elements (the paper's
// ceil(n/s) x s matrix view of MATMUL(x, U_s), with s = ROW).  A warp owns a SPAN of 128
// consecutive rows in four PIECES of 32 rows (one row per lane); a TILE is the four spans
// handled by the four warps of one epilogue warpgroup.  Tensor-core product i of a tile
// multiplies the 128 x 32 matrix made of piece i of the four spans.
constexpr int ROW = 32;
constexpr int PIECE_ROWS = 32;
constexpr int PIECE = ROW * PIECE_ROWS;        // 1024 elements
constexpr int PIECES_PER_SPAN = 4;
constexpr int SPAN = PIECES_PER_SPAN * PIECE;  // 4096 elements
constexpr int SPANS_PER_TILE = 4;
constexpr int TILE = SPANS_PER_TILE * SPAN;    // 16384 elements
constexpr int OPERAND_ROWS = SPANS_PER_TILE * PIECE_ROWS;   // 128 = M of one product
constexpr int FLAG_TILE_BYTES = TILE;

// Every device-side wait (mbarrier, look-back) gives up after this long.
constexpr uint64_t WAIT_BUDGET_NS = 4000000000ull;

// Workspace header (first 256 bytes of the caller's workspace).
struct WorkspaceHeader {
    unsigned int tile_counter;    // next tile to hand out
    unsigned int error;           // first device-detected mmv_status, 0 = none
    unsigned int reserved[62];
};
static_assert(sizeof(WorkspaceHeader) == 256, "header is 256 bytes");

// Look-back status word: bits [0,32) payload, bits [32,34) state.
constexpr uint64_t ST_NONE = 0, ST_AGG = 1, ST_PREFIX = 2, ST_ABORT = 3;
__device__ __forceinline__ uint64_t pack_status(uint64_t state, uint32_t payload) {
    return (state << 32) | static_cast<uint64_t>(payload);
}

// Value-type traits: VIn = element type in memory, Acc = accumulator/output type.
struct F16Path {
    using Acc = float;
    static constexpr int kElemBytes = 2;
    static constexpr bool kIsFloat = true;
    static constexpr int kRowBytes = ROW * 2;            // 64-byte rows -> 64-byte swizzle
    static constexpr int kSlabBytes = OPERAND_ROWS * kRowBytes;    // one K-slab of an operand: 8 KB
    static constexpr int kMmaPerSlab = 2;                  // K = 16 per instruction
    static constexpr int kKStepBytes = 32;
    static constexpr uint32_t kLayoutType = 4;             // SWIZZLE_64B
    static constexpr uint32_t kSbo = 8 * kRowBytes;        // 512
    static constexpr uint32_t kOneBits = 0x3C00u;          // 1.0 in fp16
    static constexpr uint32_t kFmtBits = 0u;               // instruction-descriptor A/B format: f16
    __device__ static __forceinline__ Acc from_bits(uint32_t b) { return __uint_as_float(b); }
    __device__ static __forceinline__ uint32_t to_bits(Acc v) { return __float_as_uint(v); }
    __device__ static __forceinline__ Acc add(Acc a, Acc b) { return a + b; }
    __device__ static __forceinline__ Acc sub(Acc a, Acc b) { return a - b; }
    // two packed input values -> fp32 (low half first), and one value from memory
    __device__ static __forceinline__ void unpack2(uint32_t w, float& lo, float& hi) {
        const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&w));
        lo = f.x;
        hi = f.y;
    }
    __device__ static __forceinline__ float load_elem(const void* x, long long idx) {
        return __half2float(static_cast<const __half*>(x)[idx]);
    }
};
// bfloat16 input values, fp32 results: the layout and arithmetic of the fp16 path, with the tensor-core
// operands declared bf16 (the products with the 0/1 matrix stay exact, the accumulator is fp32).
struct BF16ValPath : F16Path {
    static constexpr uint32_t kOneBits = 0x3F80u;                       // 1.0 in bf16
    static constexpr uint32_t kFmtBits = (1u << 7) | (1u << 10);        // A and B are bf16
    __device__ static __forceinline__ void unpack2(uint32_t w, float& lo, float& hi) {
        lo = __uint_as_float(w << 16);
        hi = __uint_as_float(w & 0xffff0000u);
    }
    __device__ static __forceinline__ float load_elem(const void* x, long long idx) {
        return __uint_as_float(static_cast<uint32_t>(static_cast<const unsigned short*>(x)[idx]) << 16);
    }
};
struct I8Path {
    using Acc = uint32_t;                                  // wrap-around arithmetic on unsigned
    static constexpr int kElemBytes = 1;
    static constexpr bool kIsFloat = false;
    static constexpr int kRowBytes = ROW;                  // 32-byte rows -> 32-byte swizzle
    static constexpr int kSlabBytes = OPERAND_ROWS * kRowBytes;    // 4 KB
    static constexpr int kMmaPerSlab = 1;                  // K = 32 per instruction
    static constexpr int kKStepBytes = 32;
    static constexpr uint32_t kLayoutType = 6;             // SWIZZLE_32B
    static constexpr uint32_t kSbo = 8 * kRowBytes;        // 256
    static constexpr uint32_t kOneBits = 1u;
    static constexpr uint32_t kFmtBits = 0u;
    __device__ static __forceinline__ Acc from_bits(uint32_t b) { return b; }
    __device__ static __forceinline__ uint32_t to_bits(Acc v) { return v; }
    __device__ static __forceinline__ Acc add(Acc a, Acc b) { return a + b; }
    __device__ static __forceinline__ Acc sub(Acc a, Acc b) { return a - b; }
};

// Byte offset of (row, byte-in-row) inside a K-major slab with rows of RowBytes
// bytes stored with the matching TMA/UMMA swizzle (16-byte chunk index XOR a
// function of the row).
template <int RowBytes>
__device__ __forceinline__ uint32_t swz_offset(uint32_t row, uint32_t byte_in_row) {
    uint32_t chunk = byte_in_row >> 4;
    if (RowBytes == 128) chunk ^= (row & 7u);
    else if (RowBytes == 64) chunk ^= ((row >> 1) & 3u);
    else if (RowBytes == 32) chunk ^= ((row >> 2) & 1u);
    return row * RowBytes + (chunk << 4) + (byte_in_row & 15u);
}

// Shared-memory matrix descriptor of a K-major swizzled slab: rows of RowBytes bytes, groups of 8 rows contiguous,
// the 16-byte chunk index XOR-ed with a function of the row (swz_offset above).  `addr` = shared address of the
// first row plus the byte offset of the K slice inside the row.
__device__ __forceinline__ uint64_t make_desc(uint32_t addr, uint32_t sbo_bytes, uint32_t layout_type) {
    uint64_t d = 0;
    d |= static_cast<uint64_t>((addr & 0x3FFFFu) >> 4);        // start address, bits [0,14)
    d |= static_cast<uint64_t>(1) << 16;                       // leading byte offset (unused for swizzled K-major)
    d |= static_cast<uint64_t>(sbo_bytes >> 4) << 32;          // stride byte offset: 8 rows
    d |= static_cast<uint64_t>(1) << 46;                       // descriptor version (sm_100)
    d |= static_cast<uint64_t>(layout_type) << 61;             // 2 = 128-byte, 4 = 64-byte, 6 = 32-byte swizzle
    return d;
}

__device__ __forceinline__ void report_error(WorkspaceHeader* hdr, unsigned int code) {
    atomicCAS(&hdr->error, 0u, code);
}

// Bounded mbarrier wait that also gives up when another role of the CTA has aborted.
__device__ __noinline__ bool wait_bar_slow(uint64_t* bar, uint32_t parity, volatile int* abort_flag, uint64_t budget_ns) {
    const uint64_t t0 = global_timer_ns();
    uint32_t polls = 0;
    while (!mbar_try_wait(bar, parity)) {
        if ((++polls & 31u) == 0u) {
            if (*abort_flag) return false;
            if (global_timer_ns() - t0 > budget_ns) return false;
        }
    }
    return true;
}
// (The polling loop is out of line: there are dozens of wait sites and the epilogues have to
// stay inside the instruction cache.)
__device__ __forceinline__ bool wait_bar(uint64_t* bar, uint32_t parity, volatile int* abort_flag,
                                         uint64_t budget_ns) {
    if (mbar_try_wait(bar, parity)) return true;
    return wait_bar_slow(bar, parity, abort_flag, budget_ns);
}

template <typename P>
__device__ __forceinline__ typename P::Acc warp_sum(typename P::Acc v) {
    if constexpr (P::kIsFloat) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
        return v;
    } else {
        return __reduce_add_sync(0xffffffffu, v);
    }
}

// ---------------------------------------------------------------------------
// Decoupled look-back over per-span status words.
//
// Span s publishes either its aggregate (ST_AGG: sum of all its elements, it holds no segment
// start) or an inclusive prefix (ST_PREFIX: sum of the segment that is open at its end).  The
// carry into span s is the sum of the aggregates of s-1, s-2, ... down to and including the
// first one that published a prefix.  A window is 32 * W consecutive predecessors, W per lane,
// nearest first: lane l holds positions W*l .. W*l + W-1.
// ---------------------------------------------------------------------------
// W = words per lane: a window is 32 * W consecutive predecessors.
template <int W>
struct LookbackWindow {
    uint64_t w[W];
};

// Issues the loads of the window whose nearest predecessor is `idx` (no wait on the data).
// Positions before word 0 read as an inclusive prefix of `base_bits`: zero, or the carry that an
// earlier call hands in when a long input is processed chunk by chunk.
// STRIDE: distance in words between the status words of consecutive positions (1: a dense array).
template <int W, int STRIDE = 1>
__device__ __forceinline__ void lookback_load(const uint64_t* status, long long idx, LookbackWindow<W>& win,
                                              uint32_t base_bits = 0u) {
    const long long first = idx - static_cast<long long>(W) * lane_id();
#pragma unroll
    for (int q = 0; q < W; ++q) {
        const long long my = first - q;
        win.w[q] = (my >= 0) ? ld_relaxed_gpu_u64(status + my * STRIDE) : pack_status(ST_PREFIX, base_bits);
    }
}

// Returns the carry into position s.  `win` may hold a window loaded earlier with lookback_load
// (preloaded = true) so that the first round trip overlaps the caller's work.  Bounded: returns
// false on time-out, when another role of the CTA aborted, or when a predecessor aborted.
template <typename P, int W, int STRIDE = 1>
__device__ __forceinline__ bool lookback(const uint64_t* status, long long s, typename P::Acc& carry,
                                         volatile int* abort_flag, uint64_t budget_ns, LookbackWindow<W>& win,
                                         bool preloaded, uint32_t base_bits = 0u) {
    using Acc = typename P::Acc;
    const uint32_t lane = lane_id();
    Acc acc = Acc(0);
    long long idx = s - 1;
    uint64_t t0 = global_timer_ns();
    uint32_t polls = 0;
    if (!preloaded) lookback_load<W, STRIDE>(status, idx, win, base_bits);
    while (true) {
        uint32_t tmask = 0u, rmask = 0u, xmask = 0u;
#pragma unroll
        for (int q = 0; q < W; ++q) {
            const uint32_t st = static_cast<uint32_t>(win.w[q] >> 32);
            rmask |= (st != ST_NONE) ? (1u << q) : 0u;
            tmask |= (st == ST_PREFIX || st == ST_ABORT) ? (1u << q) : 0u;
            xmask |= (st == ST_ABORT) ? (1u << q) : 0u;
        }
        const uint32_t lanes_t = __ballot_sync(0xffffffffu, tmask != 0u);
        const int L = lanes_t ? (__ffs(lanes_t) - 1) : 32;            // first lane that holds a terminal word
        const int qt = tmask ? (__ffs(tmask) - 1) : W;                // this lane's first terminal word
        // words this lane must contribute: all of them before lane L, up to its terminal in lane L
        const int need = (static_cast<int>(lane) < L) ? W : ((static_cast<int>(lane) == L) ? qt + 1 : 0);
        const uint32_t need_mask = (1u << need) - 1u;
        const bool lane_ready = (rmask & need_mask) == need_mask;
        bool reload = true;                   // after a step back every lane loads; on a retry only the lanes that wait
        if (__all_sync(0xffffffffu, lane_ready)) {
            if (__any_sync(0xffffffffu, (xmask & need_mask) != 0u)) return false;
            Acc v = Acc(0);
#pragma unroll
            for (int q = W - 1; q >= 0; --q)
                if (q < need) v = P::add(P::from_bits(static_cast<uint32_t>(win.w[q])), v);
            v = warp_sum<P>(v);
            acc = P::add(v, acc);
            if (L < 32) {
                carry = acc;
                return true;
            }
            idx -= 32 * W;
            t0 = global_timer_ns();
#ifdef MMV_PHASE_TIMERS
            if (lane == 0) atomicAdd(&g_phase_cycles[14], 1ull);  // windows walked past
#endif
        } else {
            if ((++polls & 7u) == 0u) {
                if (*abort_flag) return false;
                if (global_timer_ns() - t0 > budget_ns) return false;
            }
            __nanosleep(40);        // keep the polling traffic in L2 small
            reload = !lane_ready;
        }
#ifdef MMV_PHASE_TIMERS
        if (lane == 0) atomicAdd(&g_phase_cycles[13], 1ull);      // polls after the first window
#endif
        if (reload) lookback_load<W, STRIDE>(status, idx, win, base_bits);
    }
}

}  // namespace mmv
