// Segmented sum over CSR offsets (Section 2; Algorithm 4.2 computes the same
// quantity; Section 4.3 remark after Algorithm 4.4 for the offset encoding) and
// CSR SpMV built on it (Algorithm 4.4, Algorithms A.4-A.6), single pass, sm_100a.
//
// Layout (the paper's ceil(n/s) x s row-major matrix view, s = ROW = 32):
//   a warp owns a SPAN of 128 consecutive rows (4096 elements) in four PIECES of
//   32 rows; a TILE is four spans.  Tensor-core product i of a tile multiplies the
//   [128 rows x 32] matrix made of piece i of each span (A operand, brought by one
//   4-D TMA box, K-major, hardware swizzle) with the constant upper-triangular
//   all-ones U_32 (B operand): TMEM lane 32w+l, column j = inclusive prefix at
//   position j of row l of piece i of span w  --  z = MATMUL(x, U_s).
//   With two epilogue warpgroups the MMA warp runs one tile ahead (two TMEM buffers per group);
//   the shape with three groups has one buffer per group.
//   Epilogue warps (lane = row).  partition_offsets_kernel has stored, per span, the index of its
//   first offset; a warp requests that index and the span's first 128 offsets one tile ahead.
//     pre-pass     row totals (TMEM column 31) and the one prefix in front of the span's last
//                  segment start give the span's aggregate, published at once.
//     few boundaries (<= 8): each boundary's prefix is read straight from TMEM (one column, it
//                  sits in the lane of its row), the 128 row totals are scanned with four
//                  interleaved warp scans, and lane j emits the segment that ends at boundary j.
//     general path every boundary of the span marks, in a per-warp bit table in shared memory, the
//                  element it ends behind (one lane per boundary, 128 at a time); then, piece by
//                  piece, the 32 x 32 prefixes go to shared memory and every lane walks the marked
//                  elements of ITS row: a segment end emits  prefix(end) - prefix(previous end)
//                  (the DIFF of Algorithm 4.2 applied to the COMPRESSed speculative scan, with
//                  prefixes local to the row so that magnitudes stay small); a row's first end adds
//                  what is open from the rows before it (segmented warp scan of row totals and
//                  tails).  The output index of a row's first sum is the number of boundaries in
//                  front of the row, so nothing is searched or sorted; only rows that contain
//                  empty segments look their indices up in the offsets.
//     Floating point: a difference of prefixes loses a small sum next to large values.  In the
//     few-boundaries path segments of at most 32 elements are therefore summed from the input
//     values themselves (up to four: from two words requested ahead; more: one element per lane,
//     such segments are rare there); in the general path any segment inside one row or two adjacent rows whose
//     sum came out below 2^-10 of those rows' largest prefix is added up again from its values, and
//     so is the segment of at most 32 elements that reaches back across the span's first element.
//     The one segment per span that began before it (and is longer) takes the carry of the sibling
//     spans (shared memory) or of a decoupled look-back over per-span status words.  Pieces
//     without a boundary only add their total.
#pragma once
#include <cooperative_groups.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include "../../include/mmv.h"
#include "common.cuh"

namespace mmv {

// The kernel comes with G = 2 or 3 epilogue warpgroups (4 G epilogue warps, then the TMA producer
// warp and the MMA warp).  The epilogue is a chain of dependent instructions per span, so its
// throughput grows with the number of warps: G = 3 (12 epilogue warps, 128 registers, one TMEM
// buffer per group) measured faster than G = 2 (8 warps, 168 registers, the MMA warp one tile
// ahead) at every segment density and is what the library launches; G = 2 is kept for tests.
// (G = 4 compiles too but measured no better than 3.)
constexpr int SUM_BUFS = 4;                                        // TMEM tile buffers, shared out among the warpgroups
constexpr int SUM_TMEM_COLS = SUM_BUFS * PIECES_PER_SPAN * ROW;    // 512
template <int G>
struct SumShape {
    static_assert(G == 2 || G == 3 || G == 4, "two to four epilogue warpgroups");
    static constexpr int kEpiWarps = 4 * G;
    static constexpr int kProducerWarp = 4 * G;
    static constexpr int kMmaWarp = 4 * G + 1;
    static constexpr int kThreads = (4 * G + 2) * 32;
};
constexpr int SUM_SPARSE_MAX = 8;                                  // spans with at most this many boundaries read single prefixes from TMEM
constexpr int SUM_DIRECT_LEN = 4;                                  // few-boundaries path: segments this short are summed from the inputs
constexpr float SUM_CANCEL = 1.0f / 1024.0f;                       // general path: a sum this small against its prefixes is added up again
constexpr int SUM_CHUNK = 128;                                     // boundaries a warp handles at a time (four per lane)
constexpr int SUM_MARK_BYTES = 2 * (SPAN / ROW) * 4 + 16;          // per warp: marked elements and boundary counts of 128 rows, one counter

// The fp32 products of SpMV, each stored as a pair of bf16 values (hi = bf16(z), lo = bf16(z - hi),
// 4 bytes).  An ELEMENT of this path is one product; a row of 32 products is a 128-byte operand
// row of 64 bf16 values (K = 64), and the constant operand adds both halves of every product into
// the prefix:  B[k][j] = 1 iff floor(k / 2) <= j.  So the epilogue sees nnz elements, not 2 nnz.
struct BF16Path {
    using Acc = float;
    static constexpr int kElemBytes = 4;
    static constexpr bool kIsFloat = true;
    static constexpr int kRowBytes = ROW * 4;              // 128-byte rows -> 128-byte swizzle
    static constexpr int kSlabBytes = OPERAND_ROWS * kRowBytes;    // 16 KB
    static constexpr int kMmaPerSlab = 4;                  // K = 16 bf16 values per instruction
    static constexpr int kKStepBytes = 32;
    static constexpr uint32_t kLayoutType = 2;             // SWIZZLE_128B
    static constexpr uint32_t kSbo = 8 * kRowBytes;        // 1024
    static constexpr uint32_t kOneBits = 0x3F80u;          // 1.0 in bf16
    static constexpr uint32_t kFmtBits = (1u << 7) | (1u << 10);        // A and B are bf16
    __device__ static __forceinline__ Acc from_bits(uint32_t b) { return __uint_as_float(b); }
    __device__ static __forceinline__ uint32_t to_bits(Acc v) { return __float_as_uint(v); }
    __device__ static __forceinline__ Acc add(Acc a, Acc b) { return a + b; }
    __device__ static __forceinline__ Acc sub(Acc a, Acc b) { return a - b; }
};
// one product = hi + lo, added in the order the tensor core sees them
__device__ __forceinline__ float pair_value(uint32_t bits) {
    return __uint_as_float(bits << 16) + __uint_as_float(bits & 0xffff0000u);
}

template <typename P>
__device__ __forceinline__ typename P::Acc load_value(const void* base, long long idx);
template <>
__device__ __forceinline__ float load_value<F16Path>(const void* base, long long idx) {
    return __half2float(static_cast<const __half*>(base)[idx]);
}
template <>
__device__ __forceinline__ float load_value<BF16ValPath>(const void* base, long long idx) {
    return __uint_as_float(static_cast<uint32_t>(static_cast<const unsigned short*>(base)[idx]) << 16);
}
template <>
__device__ __forceinline__ float load_value<BF16Path>(const void* base, long long idx) {
    return pair_value(static_cast<const uint32_t*>(base)[idx]);
}
template <>
__device__ __forceinline__ uint32_t load_value<I8Path>(const void* base, long long idx) {
    return static_cast<uint32_t>(static_cast<int32_t>(static_cast<const int8_t*>(base)[idx]));
}

// One input element given as its bit pattern in the low bits of a word.
template <typename P>
__device__ __forceinline__ typename P::Acc elem_bits_to_acc(uint32_t bits);
template <>
__device__ __forceinline__ float elem_bits_to_acc<F16Path>(uint32_t bits) {
    return __half2float(__ushort_as_half(static_cast<unsigned short>(bits)));
}
template <>
__device__ __forceinline__ float elem_bits_to_acc<BF16ValPath>(uint32_t bits) {
    return __uint_as_float((bits & 0xffffu) << 16);
}
template <>
__device__ __forceinline__ float elem_bits_to_acc<BF16Path>(uint32_t bits) {
    return pair_value(bits);
}
template <>
__device__ __forceinline__ uint32_t elem_bits_to_acc<I8Path>(uint32_t bits) {
    return static_cast<uint32_t>(static_cast<int32_t>(static_cast<int8_t>(bits)));
}

// Sum of the elements [sb, cb) of a very short segment, taken from the input values themselves.
// (Not inlined: it is the rare path, and the epilogue has to stay inside the instruction cache.)
template <typename P>
__device__ __noinline__ typename P::Acc direct_sum(const void* xg, long long sb, long long cb) {
    typename P::Acc val = typename P::Acc(0);
    for (long long e = sb; e < cb; ++e) val = P::add(val, load_value<P>(xg, e));
    return val;
}

// The same sum in two steps, so that the loads can be in flight while other work is done:
// window_load fetches the two aligned words of four elements each that hold [sb, sb + 4) (no
// arithmetic on them), window_sum adds up the first `len` elements once they are needed.
// Falls back to element loads where an aligned word would reach past the n input values.
struct ValueWindow {
    uint32_t r[4];
    bool wide;
};
template <typename P>
__device__ __forceinline__ void window_load(const void* xg, long long sb, int len, long long n, ValueWindow& win) {
    constexpr int EB = P::kElemBytes;                   // 2 or 1: a word of four elements is 8 or 4 bytes
    if constexpr (EB == 4) {
        // 4-byte elements: one load per element, nothing to align
        win.wide = true;
#pragma unroll
        for (int i = 0; i < 4; ++i) win.r[i] = (i < len && sb + i < n) ? static_cast<const uint32_t*>(xg)[sb + i] : 0u;
        return;
    }
    const long long base = sb & ~3ll;
    const int sh = static_cast<int>(sb & 3);
    win.r[0] = win.r[1] = win.r[2] = win.r[3] = 0u;
    win.wide = (base + 4 <= n) && (sh + len <= 4 || base + 8 <= n);
    if (!win.wide) return;
    const uint8_t* p = static_cast<const uint8_t*>(xg) + base * EB;
    if constexpr (EB == 2) {
        const uint2 a = *reinterpret_cast<const uint2*>(p);
        win.r[0] = a.x;
        win.r[1] = a.y;
        if (sh + len > 4) {
            const uint2 b = *reinterpret_cast<const uint2*>(p + 8);
            win.r[2] = b.x;
            win.r[3] = b.y;
        }
    } else {
        win.r[0] = *reinterpret_cast<const uint32_t*>(p);
        if (sh + len > 4) win.r[1] = *reinterpret_cast<const uint32_t*>(p + 4);
    }
}
template <typename P>
__device__ __forceinline__ typename P::Acc window_sum(const void* xg, long long sb, int len, const ValueWindow& win) {
    using Acc = typename P::Acc;
    if (!win.wide) return direct_sum<P>(xg, sb, sb + len);
    constexpr int EB = P::kElemBytes;
    const int sh = static_cast<int>(sb & 3);
    Acc val = Acc(0);
    if constexpr (EB == 4) {
#pragma unroll
        for (int i = 0; i < 4; ++i)
            if (i < len) val = P::add(val, elem_bits_to_acc<P>(win.r[i]));
        return val;
    }
    if constexpr (EB == 2) {
        const int bits = sh * 16;
        const uint32_t a0 = bits >= 32 ? win.r[1] : win.r[0];
        const uint32_t a1 = bits >= 32 ? win.r[2] : win.r[1];
        const uint32_t a2 = bits >= 32 ? win.r[3] : win.r[2];
        const uint32_t o0 = __funnelshift_r(a0, a1, bits & 31), o1 = __funnelshift_r(a1, a2, bits & 31);
        const uint32_t e[4] = {o0 & 0xffffu, o0 >> 16, o1 & 0xffffu, o1 >> 16};
#pragma unroll
        for (int i = 0; i < 4; ++i)
            if (i < len) val = P::add(val, elem_bits_to_acc<P>(e[i]));
    } else {
        const uint32_t o = __funnelshift_r(win.r[0], win.r[1], sh * 8);
#pragma unroll
        for (int i = 0; i < 4; ++i)
            if (i < len) val = P::add(val, elem_bits_to_acc<P>((o >> (8 * i)) & 0xffu));
    }
    return val;
}

#ifndef MMV_SUM_STATUS_STRIDE
#define MMV_SUM_STATUS_STRIDE 1
#endif
// Span s publishes word s * SUM_STATUS_STRIDE of the status area.  The scans spread their words over 32-byte
// sectors and gain by it; here nearly every span holds a boundary and a look-back ends at its first word, and
// a stride of 4 or 8 measured the same or slightly worse (a larger area to clear), so the array stays dense.
constexpr int SUM_STATUS_STRIDE = MMV_SUM_STATUS_STRIDE;

// The look-back of the segmented sum behind one signature for its three call sites.
template <typename P>
__device__ __forceinline__ bool sum_lookback(const uint64_t* status, long long s, typename P::Acc* carry,
                                          volatile int* abort_flag, uint64_t budget_ns, uint64_t window, bool preloaded) {
    LookbackWindow<1> win;
    win.w[0] = window;
    typename P::Acc c = typename P::Acc(0);
    const bool ok = lookback<P, 1, SUM_STATUS_STRIDE>(status, s, c, abort_flag, budget_ns, win, preloaded);
    *carry = c;
    return ok;
}

template <typename P, int G>
struct SumCfg {
    static constexpr int kStages = P::kElemBytes == 4 ? 2 : 4;      // (the bf16-pair tiles are 64 KB)
    static constexpr int kBBytes = ROW * P::kRowBytes;               // constant operand: 32 rows
    static constexpr int kXBytes = PIECES_PER_SPAN * P::kSlabBytes;  // four [128 x 32] operands
    static constexpr int kDumpRowBytes = ROW * 4 + 16;               // rows of 36 words: 16-byte stores and single-word loads
                                                                     // both spread over the banks, and a prefix is at
                                                                     // row + 4 c (no swizzle to undo per look-up)
    static constexpr int kDumpBytes = PIECE_ROWS * kDumpRowBytes;    // per epilogue warp
    static constexpr int kStageOffset = 4096;                        // after the constant operand
    static constexpr int kDumpOffset = kStageOffset + kStages * kXBytes;
    static constexpr int kMarkOffset = kDumpOffset + SumShape<G>::kEpiWarps * kDumpBytes;
    static constexpr int kBarOffset = kMarkOffset + SumShape<G>::kEpiWarps * SUM_MARK_BYTES;
    static constexpr int kSmemBytes = kBarOffset + 512 + 1024;
    static_assert(kBBytes <= kStageOffset, "constant operand fits its slot");
    static_assert(kSmemBytes <= 227 * 1024, "fits the shared memory of one CTA");
};

struct SumParams {
    const int32_t* off;          // nseg + 1 offsets
    long long nseg;
    long long n;                 // number of values
    void* out;                   // nseg results
    int num_tiles;
    const int32_t* span_q;       // 4 * num_tiles + 1: first q with (off[q] << shift) >= span start
    WorkspaceHeader* hdr;
    uint64_t* status;
    unsigned long long budget_ns;
    const long long* nseg_dev;   // when not null: the number of segments is read from here (flag-encoded
                                 // segments, whose count is only known on the device); nseg is ignored
    int fused_prologue;          // 1: the kernel itself clears the header and the status words and partitions the
                                 // offsets (span_q, validation, zeros of empty segments) before a grid-wide
                                 // barrier -- one launch per call instead of a memset and two kernels
    long long status_words;      // number of 8-byte status words to clear in that case
};

// First index q in [lo, hi) with (off[q] << shift) >= target, hi if none; the offsets are
// non-decreasing.  One warp, 32-ary search (every lane probes the last element of its block).
__device__ __forceinline__ long long first_index_at_least(const int32_t* __restrict__ off, int shift, long long lo, long long hi,
                                                          long long target) {
    const int lane = threadIdx.x & 31;
    while (hi > lo) {
        const long long len = hi - lo;
        const long long step = (len + 31) / 32;
        const long long bstart = lo + lane * step;
        long long bend = bstart + step;
        if (bend > hi) bend = hi;
        bool pred = false;
        if (bstart < hi) pred = (static_cast<long long>(off[bend - 1]) << shift) >= target;
        const unsigned m = __ballot_sync(0xffffffffu, pred);
        if (m == 0u) {
            lo = hi;
        } else {
            const int k = __ffs(m) - 1;
            const long long ks = lo + k * step;
            long long ke = ks + step;
            if (ke > hi) ke = hi;
            lo = ks;
            hi = ke - 1;
        }
    }
    return lo;
}
// The same out of line, for the rare jump over a long run of equal offsets in the epilogue.
__device__ __noinline__ long long first_index_at_least_call(const int32_t* off, int shift, long long lo, long long hi,
                                                            long long target) {
    return first_index_at_least(off, shift, lo, hi, target);
}

// span_q[s] = first index i in [0, nseg] with bnd(i) = off[i] << shift >= s * SPAN, nseg + 1 if none,
// for s = 0 .. num_spans.  Every offset index i is handled by one thread: i is that first index exactly
// for the spans s with bnd(i-1) < s * SPAN <= bnd(i), a range the thread writes itself (ranges of more than 32
// spans, i.e. very long segments, are written by the whole warp).  The same pass validates the
// offsets (non-decreasing, inside [0, n]; MMV_ERR_BAD_SEGMENTS otherwise -- entries may then be
// missing or inconsistent, which the main kernel tolerates: it clamps what it reads and never
// indexes outside its tile) and writes the zero of every EMPTY segment, so that the main kernel
// may jump over long runs of equal offsets instead of visiting them one by one.
// (the work of one thread of `nthreads`, `tid` its index; every warp must come as a whole)
// Returns true if this thread met an offset that is out of order or out of range (the caller reports it).
template <int VEC>       // offsets per lane and round: 4 when there are many (one 16-byte load each), else 1
__device__ __forceinline__ bool partition_offsets(const int32_t* __restrict__ off, long long nseg, long long num_spans,
                                                  int32_t* __restrict__ span_q, long long n,
                                                  uint32_t* __restrict__ out, long long tid, long long nthreads) {
    const int lane = threadIdx.x & 31;
    bool bad = false;
    const long long stride = static_cast<long long>(VEC) * nthreads;
    const int n32 = static_cast<int>(n < 0x7fffffffll ? n : 0x7fffffffll);
    const int last_span = static_cast<int>(num_spans);
    static_assert(SPAN == 4096, "span index = position >> 12");
    // A warp takes 32 VEC consecutive offsets per round; with many offsets four per lane in one 16-byte
    // load (the kernel is bound by the loads it has in flight).  Every warp makes the same number of rounds: the votes below
    // need all its lanes.  Positions and span indices fit 32 bits because the offsets do.
    for (long long wbase = VEC * (tid - lane); wbase <= nseg; wbase += stride) {
        const long long i0 = wbase + VEC * lane;   // my first offset index
        int c[VEC];
#pragma unroll
        for (int e = 0; e < VEC; ++e) c[e] = 0;
        bool vector_load = false;
        if constexpr (VEC == 4) {
            if (i0 + 3 <= nseg) {
                const int4 v = *reinterpret_cast<const int4*>(off + i0);
                c[0] = v.x;
                c[1] = v.y;
                c[2] = v.z;
                c[3] = v.w;
                vector_load = true;
            }
        }
        if (!vector_load) {
#pragma unroll
            for (int e = 0; e < VEC; ++e)
                if (i0 + e <= nseg) c[e] = off[i0 + e];
        }
        int before = __shfl_up_sync(0xffffffffu, c[VEC - 1], 1);
        if (lane == 0) before = wbase >= 1 ? off[wbase - 1] : 0;
        int lo[VEC], hi[VEC];                      // spans [lo, hi] get the offset's index
        bool any = false;
#pragma unroll
        for (int e = 0; e < VEC; ++e) {
            const long long i = i0 + e;
            const int cur = c[e], prev = e ? c[e - 1] : before;
            lo[e] = 0;
            hi[e] = -1;
            if (i <= nseg) {
                if (i >= 1) {
                    if (prev > cur || prev < 0 || cur > n32) bad = true;
                    if (prev == cur) out[i - 1] = 0u;              // segment i - 1 is empty
                    lo[e] = prev < 0 ? 0 : (prev >> 12) + 1;
                } else if (cur < 0 || cur > n32) {
                    bad = true;
                }
                hi[e] = cur < 0 ? -1 : (cur >> 12);
                if (hi[e] > last_span) hi[e] = last_span;
                any |= hi[e] >= lo[e] || i == nseg;
            }
        }
        if (__ballot_sync(0xffffffffu, any) == 0u) continue;       // no span starts between this warp's offsets
#pragma unroll 1
        for (int e = 0; e < VEC; ++e) {
            int l = lo[0], h = hi[0], cur = c[0];
#pragma unroll
            for (int t = 1; t < VEC; ++t)
                if (e == t) { l = lo[t]; h = hi[t]; cur = c[t]; }
            const long long i = i0 + e;
            if (h >= l && h - l < 32) {
                for (int sp = l; sp <= h; ++sp) span_q[sp] = static_cast<int32_t>(i);
                l = h + 1;
            }
            // long ranges, and the range behind the last offset: the whole warp writes them
            unsigned todo = __ballot_sync(0xffffffffu, h >= l);
            while (todo) {
                const int src = __ffs(todo) - 1;
                const int ll = __shfl_sync(0xffffffffu, l, src), hh = __shfl_sync(0xffffffffu, h, src);
                const int v = static_cast<int>(wbase) + VEC * src + e;
                for (int sp = ll + lane; sp <= hh; sp += 32) span_q[sp] = v;
                todo &= todo - 1;
            }
            todo = __ballot_sync(0xffffffffu, i == nseg);
            if (todo) {
                const int src = __ffs(todo) - 1;
                const int h0 = __shfl_sync(0xffffffffu, cur < 0 ? -1 : (cur >> 12), src);
                for (int sp = (h0 > last_span ? last_span : h0) + 1 + lane; sp <= last_span; sp += 32)
                    span_q[sp] = static_cast<int32_t>(nseg + 1);
            }
        }
    }
    return bad;
}

template <int VEC>
__global__ void partition_offsets_kernel(const int32_t* __restrict__ off, long long nseg, long long num_spans,
                                         int32_t* __restrict__ span_q, long long n, WorkspaceHeader* hdr,
                                         uint32_t* __restrict__ out) {
    griddep_launch_dependents();       // the kernel behind may set itself up meanwhile (it waits before it reads)
    if (partition_offsets<VEC>(off, nseg, num_spans, span_q, n, out, static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x,
                               static_cast<long long>(gridDim.x) * blockDim.x))
        report_error(hdr, 4u);
}

template <typename P, int G>
__global__ void __launch_bounds__(SumShape<G>::kThreads, 1)
seg_sum_kernel(const __grid_constant__ CUtensorMap tmap_x, const void* __restrict__ xg, const SumParams prm) {
    using Acc = typename P::Acc;
    using Cfg = SumCfg<P, G>;
    using Shape = SumShape<G>;
    constexpr int S = Cfg::kStages;

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* sB = smem;
    uint8_t* sStage = smem + Cfg::kStageOffset;
    uint64_t* bar_full = reinterpret_cast<uint64_t*>(smem + Cfg::kBarOffset);
    uint64_t* bar_empty = bar_full + S;
    uint64_t* bar_acc_full = bar_empty + S;
    uint64_t* bar_acc_empty = bar_acc_full + SUM_BUFS;
    // per stage: (iteration << 32) | tile, written as one word before the stage's barrier is armed
    uint64_t* bar_agg = bar_acc_empty + SUM_BUFS;          // per warpgroup: its four span aggregates are in agg_slot
    // [group][tile parity][span]: (has start << 32) | open-segment sum.  Two sets, because a warp may
    // write its next tile's aggregate while a sibling still reads this tile's.
    uint64_t* agg_slot = bar_agg + G;
    volatile long long* stage_info = reinterpret_cast<volatile long long*>(agg_slot + G * 2 * SPANS_PER_TILE);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(const_cast<long long*>(stage_info) + S);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5;
    const uint32_t lane = lane_id();
    const uint64_t budget = prm.budget_ns;

    if (threadIdx.x == 0) {
        for (int i = 0; i < S; ++i) {
            mbar_init(&bar_full[i], 1);
            mbar_init(&bar_empty[i], 1);      // released by the MMA warp's commit
            stage_info[i] = -1;
        }
        for (int i = 0; i < G; ++i) mbar_init(&bar_agg[i], SPANS_PER_TILE);
        for (int i = 0; i < SUM_BUFS; ++i) {
            mbar_init(&bar_acc_full[i], 1);
            mbar_init(&bar_acc_empty[i], 4);
        }
        *abort_flag = 0;
        mbar_fence_init();
    }
    if (warp == Shape::kMmaWarp) {
        tmem_alloc(tmem_slot, SUM_TMEM_COLS);
        tmem_relinquish();
    }
    if (warp == Shape::kProducerWarp && lane == 0) tma_prefetch_desc(&tmap_x);
    {
        // constant B = U_32 stored K-major: row nn (output position), element k (input position): 1 iff k <= nn
        // (bf16 pairs: element k is the two K entries 2k and 2k + 1, both set)
        constexpr int kVecPerRow = P::kRowBytes / 16;
        constexpr int kElemPerVec = 16 / P::kElemBytes;
        for (int v = threadIdx.x; v < ROW * kVecPerRow; v += Shape::kThreads) {
            const int nn = v / kVecPerRow, cv = v % kVecPerRow;
            uint32_t words[4] = {0u, 0u, 0u, 0u};
#pragma unroll
            for (int e = 0; e < kElemPerVec; ++e) {
                const int k = cv * kElemPerVec + e;
                if (k <= nn) {
                    if constexpr (P::kElemBytes == 4) words[e] = P::kOneBits | (P::kOneBits << 16);   // both halves of product k
                    else if constexpr (P::kElemBytes == 2) words[e >> 1] |= static_cast<uint32_t>(P::kOneBits) << ((e & 1) * 16);
                    else words[e >> 2] |= 1u << ((e & 3) * 8);
                }
            }
            *reinterpret_cast<uint4*>(sB + swz_offset<P::kRowBytes>(nn, cv * 16)) =
                make_uint4(words[0], words[1], words[2], words[3]);
        }
    }
    fence_proxy_async_smem();
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    // Everything above (barriers, tensor memory, the constant operand) touched nothing a predecessor in the
    // stream writes; from here on the kernel reads the span partition, the status words and the offsets.
    griddep_wait();
    if (prm.fused_prologue) {
        // The whole grid (resident as one: cooperative launch) first does what a memset and the partition kernel
        // would do -- clear the header and the status words, partition and check the offsets, write the zeros of
        // the empty segments -- then meets at one grid-wide barrier.  An error in the offsets is reported behind
        // the barrier, when the header is certainly cleared.
        const long long tid = static_cast<long long>(blockIdx.x) * Shape::kThreads + threadIdx.x;
        const long long nthreads = static_cast<long long>(gridDim.x) * Shape::kThreads;
        for (long long i = tid; i < prm.status_words; i += nthreads) prm.status[i] = 0ull;
        if (tid < static_cast<long long>(sizeof(WorkspaceHeader) / sizeof(unsigned int))) reinterpret_cast<unsigned int*>(prm.hdr)[tid] = 0u;
        const long long spans = static_cast<long long>(prm.num_tiles) * SPANS_PER_TILE;
        bool bad;
        if (prm.nseg >= (1ll << 20))
            bad = partition_offsets<4>(prm.off, prm.nseg, spans, const_cast<int32_t*>(prm.span_q), prm.n, static_cast<uint32_t*>(prm.out), tid, nthreads);
        else
            bad = partition_offsets<1>(prm.off, prm.nseg, spans, const_cast<int32_t*>(prm.span_q), prm.n, static_cast<uint32_t*>(prm.out), tid, nthreads);
        __threadfence();
        cooperative_groups::this_grid().sync();
        if (bad) report_error(prm.hdr, 4u);
    }

    if (warp == Shape::kProducerWarp) {
        // =========================== producer ===========================
        int it = 0, sentinels = 0;
        bool ok = true;
        while (ok) {
            const int stage = it % S;
            if (!wait_bar(&bar_empty[stage], ((it / S) & 1) ^ 1, abort_flag, budget)) { ok = false; break; }
            // static round-robin tile assignment: all CTAs are resident (grid <= SM count, one CTA per
            // SM), so iteration `it` of every CTA runs at about the same time and a tile's predecessors
            // are always in flight or finished
            int tile = static_cast<int>(blockIdx.x) + it * static_cast<int>(gridDim.x);
            if (tile >= prm.num_tiles) tile = -1;
            if (lane == 0)
                stage_info[stage] = (static_cast<long long>(it) << 32) | static_cast<long long>(static_cast<unsigned int>(tile));
            if (tile < 0) {
                __syncwarp();
                if (lane == 0) mbar_arrive(&bar_full[stage]);
                ++it;
                if (++sentinels == 2) break;
                continue;
            }
            uint8_t* xs = sStage + stage * Cfg::kXBytes;
            const long long tbase = static_cast<long long>(tile) * TILE;
            if (tbase + TILE <= prm.n) {
                if (lane == 0) {
                    mbar_arrive_expect_tx(&bar_full[stage], Cfg::kXBytes);
#pragma unroll
                    for (int i = 0; i < PIECES_PER_SPAN; ++i)
                        tma_load_4d(xs + i * P::kSlabBytes, &tmap_x, &bar_full[stage], 0, 0, i, tile * SPANS_PER_TILE);
                }
            } else {
                // ragged last tile: 16-byte asynchronous copies with zero fill past n (MATMUL zero-pads its operand)
                const long long cnt = prm.n - tbase;
                constexpr int kElemPerVec = 16 / P::kElemBytes;
                const uint8_t* xt = static_cast<const uint8_t*>(xg) + tbase * P::kElemBytes;
                for (int v = lane; v < TILE / kElemPerVec; v += 32) {
                    const int e0 = v * kElemPerVec;
                    const int w = e0 / SPAN, i = (e0 % SPAN) / PIECE, l = (e0 % PIECE) / ROW, j0 = e0 % ROW;
                    uint8_t* dst = xs + i * P::kSlabBytes + swz_offset<P::kRowBytes>(w * PIECE_ROWS + l, j0 * P::kElemBytes);
                    if (e0 + kElemPerVec <= cnt) {
                        cp_async_16(dst, xt + static_cast<size_t>(e0) * P::kElemBytes);
                        continue;
                    }
                    uint4 xv = make_uint4(0u, 0u, 0u, 0u);
                    if (e0 < cnt) {
                        __align__(16) uint8_t tmp[16];
                        for (int b = 0; b < 16; ++b)
                            tmp[b] = (e0 + b / P::kElemBytes < cnt) ? xt[static_cast<size_t>(e0) * P::kElemBytes + b] : uint8_t(0);
                        xv = *reinterpret_cast<const uint4*>(tmp);
                    }
                    *reinterpret_cast<uint4*>(dst) = xv;
                }
                cp_async_wait_all();
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) mbar_arrive(&bar_full[stage]);
            }
            ++it;
        }
        if (!ok) {
            *abort_flag = 1;
            if (lane == 0) report_error(prm.hdr, 5u);
        }
        for (int k = (it > S ? it - S : 0); k < it; ++k) mbar_wait(&bar_full[k % S], (k / S) & 1, 2000000ull);
    } else if (warp == Shape::kMmaWarp) {
        // =========================== MMA issuer (one tile ahead of the epilogue) ===========================
        constexpr uint32_t idesc = P::kIsFloat ? (make_idesc_f16_f32(128, ROW) | P::kFmtBits)
                                               : make_idesc_s8_s32(128, ROW);
        int sentinels = 0;
        for (int it = 0;; ++it) {
            const int stage = it % S;
            if (!wait_bar(&bar_full[stage], (it / S) & 1, abort_flag, budget)) {
                *abort_flag = 1;
                if (lane == 0) report_error(prm.hdr, 5u);
                break;
            }
            if (static_cast<int>(stage_info[stage] & 0xffffffffll) < 0) {
                if (++sentinels == 2) break;
                continue;
            }
            // iteration `it` uses buffer it % SUM_BUFS whichever warpgroup takes it: with three groups and four
            // buffers the products of a group's next tile are finished while all groups are still busy
            const int buf = it % SUM_BUFS;
            if (!wait_bar(&bar_acc_empty[buf], ((it / SUM_BUFS) & 1) ^ 1, abort_flag, budget)) {
                *abort_flag = 1;
                if (lane == 0) report_error(prm.hdr, 5u);
                break;
            }
            tc_fence_after_sync();
            if (lane == 0) {
                const uint32_t xs = smem_u32(sStage + stage * Cfg::kXBytes);
                const uint32_t bs = smem_u32(sB);
#pragma unroll
                for (int i = 0; i < PIECES_PER_SPAN; ++i) {
                    const uint32_t d = tmem_base + buf * (PIECES_PER_SPAN * ROW) + i * ROW;
#pragma unroll
                    for (int ks = 0; ks < P::kMmaPerSlab; ++ks) {
                        const uint64_t da = make_desc(xs + i * P::kSlabBytes + ks * P::kKStepBytes, P::kSbo, P::kLayoutType);
                        const uint64_t db = make_desc(bs + ks * P::kKStepBytes, P::kSbo, P::kLayoutType);
                        if constexpr (P::kIsFloat) mma_f16_ss(d, da, db, idesc, ks != 0);
                        else mma_i8_ss(d, da, db, idesc, ks != 0);
                    }
                }
                tc_commit(&bar_empty[stage]);       // operands consumed: the stage may be refilled
                tc_commit(&bar_acc_full[buf]);
            }
            __syncwarp();
        }
    } else {
        // =========================== epilogue ===========================
        const int g = warp >> 2;
        const int w = warp & 3;
        Acc* outp = static_cast<Acc*>(prm.out);
        // per row of the span: marked elements (bits), number of boundaries; boundaries at the span's first element
        uint8_t* dump = smem + Cfg::kDumpOffset + warp * Cfg::kDumpBytes;      // [32 rows][32] prefixes of a piece, rows padded
        uint32_t* emask = reinterpret_cast<uint32_t*>(smem + Cfg::kMarkOffset + warp * SUM_MARK_BYTES);
        uint32_t* ecnt = emask + SPAN / ROW;
        uint32_t* nbase = ecnt + SPAN / ROW;
        constexpr int sh = 0;             // (boundaries are the offsets themselves)
        const long long nq = (prm.nseg_dev ? *prm.nseg_dev : prm.nseg) + 1;
        bool failed = false;
        // The boundaries of the NEXT tile's span are requested one tile ahead (first the span's first
        // offset index, then one offset per lane), so that their two dependent round trips never
        // sit on the critical path.
        auto tile_of = [&](int kk) -> int {
            const int t = static_cast<int>(blockIdx.x) + (g + G * kk) * static_cast<int>(gridDim.x);
            return t < prm.num_tiles ? t : -1;
        };
        constexpr int32_t kNoOffset = 0;
        // offsets q0 + lane + 32 j (j < 4), the one before q0, and the last one below the span's end
        // (No arithmetic may touch a prefetched value before the tile that uses it: even a sign
        // extension would make the warp wait for the load on the spot.  `last_ok` says whether `last`
        // was loaded at all.)
        auto load_offsets = [&](long long q0, long long qe, int32_t (&raw)[4], int32_t& rawp, int32_t& last, bool& last_ok) {
            if (q0 < 0) q0 = 0;
            if (q0 > nq) q0 = nq;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const long long qi = q0 + lane + 32 * j;
                raw[j] = kNoOffset;
                if (qi < nq) raw[j] = prm.off[qi];
            }
            rawp = kNoOffset;
            if (q0 >= 1 && q0 - 1 < nq) rawp = prm.off[q0 - 1];
            last = kNoOffset;
            last_ok = qe > q0 && qe <= nq;
            if (last_ok) last = prm.off[qe - 1];
        };
        auto load_span_q = [&](int t, int32_t& q0, int32_t& qe) {
            const int32_t* sq = prm.span_q + static_cast<long long>(t) * SPANS_PER_TILE + w;
            q0 = sq[0];
            qe = sq[1];
        };
        MMV_T_DECL
        // The boundaries of the NEXT tile's span are prefetched one tile ahead.
        int32_t q_next = 0, qe_next = 0, nlast = kNoOffset;
        bool nlast_ok = false;
        int32_t nraw[4] = {kNoOffset, kNoOffset, kNoOffset, kNoOffset}, nrawp = kNoOffset;
        if (tile_of(0) >= 0) {
            load_span_q(tile_of(0), q_next, qe_next);
            load_offsets(q_next, qe_next, nraw, nrawp, nlast, nlast_ok);
        }
        // a segment that began before an earlier span of this warp and still waits for its carry
        bool pending = false;
        long long pend_s = 0, pend_r = -1;
        Acc pend_val = Acc(0), pend_ex = Acc(0);
        LookbackWindow<1> plw;
        for (int k = 0;; ++k) {
            // the epilogue never reads the operand stage (the MMA warp releases it); with the static
            // tile order it knows its tile without being told
            const int tile = tile_of(k);
            if (tile < 0) break;
            const int it = g + G * k;
            const int buf = it % SUM_BUFS;
            const long long s = static_cast<long long>(tile) * SPANS_PER_TILE + w;
            const long long sbase = s * SPAN;
            const uint32_t taddr = tmem_base + buf * (PIECES_PER_SPAN * ROW) + ((static_cast<uint32_t>(w) * 32u) << 16);

            // ---- the span's boundaries: one offset per lane (requested during the previous tile) ----
            // (clamped: with offsets that are not sorted the partition may hold anything)
            long long q = q_next < 0 ? 0 : (q_next > nq ? nq : q_next);     // first q with bnd(q) >= sbase
            const long long cq = q;                            // index held by lane 0 of the cache
            int32_t raw[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) raw[j] = nraw[j];
            const int32_t rawp = nrawp;
            const int32_t last_raw = nlast;                    // last boundary below the span's end (if nlast_ok)
            const bool last_ok = nlast_ok;
            MMV_T_MARK(8)
            const int tile_n = tile_of(k + 1);
            if (tile_n >= 0) load_span_q(tile_n, q_next, qe_next);
            MMV_T_MARK(10)
            // lane holds boundaries cq + lane + 32 j (j < 4).  The first 32 first: they
            // decides between the path for spans with few boundaries and the general one.
            // (Positions are below 2^31 because the offsets are 32-bit, so what follows is 32-bit arithmetic; the span's
            //  end may be 2^31 itself, so boundaries are compared relative to the span's first element.)
            int cb = -1, csb = -1;                             // my boundary among the first 32, and the one before it; -1: none
            {
                int32_t pr = __shfl_up_sync(0xffffffffu, raw[0], 1);
                if (lane == 0) pr = rawp;
                if (cq + lane < nq) cb = raw[0];
                if (cq + lane >= 1) csb = pr;
            }
            const int sb32i = static_cast<int>(sbase);
            const int n32i = static_cast<int>(prm.n);
            const int crel = static_cast<int>(static_cast<unsigned>(cb) - static_cast<unsigned>(sb32i));      // (meaningful where cb >= 0)
            // the first 32 entries cover the span if they reach past its end (or the end of the offsets)
            const bool covers = __any_sync(0xffffffffu, (q + lane >= nq) || (cb >= 0 && crel > SPAN));
            // number of boundaries with sbase <= bnd <= send (a prefix of the lanes)
            const int nb_span = __popc(__ballot_sync(0xffffffffu, cb >= 0 && crel <= SPAN));
            const bool sparse = covers && nb_span <= SUM_SPARSE_MAX;
            // the last segment start inside the span, or -1
            const int last_d = static_cast<int>(static_cast<unsigned>(last_raw) - static_cast<unsigned>(sb32i));
            const int lastrel = (last_ok && static_cast<unsigned>(last_d) < static_cast<unsigned>(SPAN)) ? last_d : -1;
            const bool seen = lastrel >= 0;   // a segment start lies inside this span
            MMV_T_MARK(9)
            // very short segments that end in this span are summed from the inputs; the loads go out
            // now and return while the accumulators are awaited
            const int seglen = static_cast<int>(static_cast<unsigned>(cb) - static_cast<unsigned>(csb));     // (meaningful where both exist)
            // (one unsigned test each: 1 <= length <= SUM_DIRECT_LEN, and the end inside (sbase, send])
            bool is_direct = csb >= 0 && cb >= 0 && static_cast<unsigned>(seglen - 1) < static_cast<unsigned>(SUM_DIRECT_LEN) &&
                             static_cast<unsigned>(crel - 1) < static_cast<unsigned>(SPAN) && cb <= n32i;
            // (the general path needs only the one that reaches back across the span's first element)
            if (!sparse && !(lane == 0 && csb < sb32i)) is_direct = false;
            ValueWindow win0;
            win0.wide = false;
            if (is_direct) window_load<P>(xg, csb, seglen, prm.n, win0);
            int xlen = 0;
            Acc xval = Acc(0);
            // ---- general path, first step: every boundary marks the element it ends behind.  emask[row] has
            //      bit c set if a segment ends behind element c of that row of the span, ecnt[row] counts the
            //      boundaries there (more than the bits if empty segments follow), nbase those exactly at the
            //      span's first element.  The first 128 boundaries are in registers already. ----
            const uint32_t sb32 = static_cast<uint32_t>(sbase);
            bool tcovers = covers;
            int32_t yraw[4] = {kNoOffset, kNoOffset, kNoOffset, kNoOffset};
            auto mark = [&](int32_t braw) -> bool {          // returns true if the boundary lies behind the span
                // element the boundary ends behind, relative to the span (one unsigned test covers 1 <= rel <= SPAN;
                // a negative offset wraps to a huge value and marks nothing)
                const uint32_t e = static_cast<uint32_t>(braw) - sb32 - 1u;
                if (e < static_cast<uint32_t>(SPAN)) {
                    atomicOr(&emask[e >> 5], 1u << (e & 31u));
                    atomicAdd(&ecnt[e >> 5], 1u);
                } else if (e == 0xffffffffu && braw >= 0) {
                    atomicAdd(nbase, 1u);
                }
                return static_cast<int>(e) >= SPAN;
            };
            if (!sparse) {
#pragma unroll
                for (int j = 0; j < 4; ++j) emask[lane + 32 * j] = 0u;
#pragma unroll
                for (int j = 0; j < 4; ++j) ecnt[lane + 32 * j] = 0u;
                if (lane == 0) *nbase = 0u;
                __syncwarp();
                bool tc = false;
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    if (j == 0 || !covers) {           // (if the first 32 reach past the span the others lie behind it)
                        if (cq + lane + 32 * j < nq) tc |= mark(raw[j]);
                        else tc = true;
                    }
                }
                tcovers = covers || __any_sync(0xffffffffu, tc);
                // General path: the segment that reaches back across the span's first element (it ends at the first
                // boundary): with at most 32 elements its values themselves are added up, one per lane.  Its carry
                // would be a difference of the previous span's prefixes, which loses a small sum next to large values.
                if constexpr (P::kIsFloat) {
                    // (lane 0's boundary and the one before it)
                    const bool crossing = csb >= 0 && cb >= 0 && csb < sb32i && static_cast<unsigned>(crel - 1) < static_cast<unsigned>(SPAN) &&
                                          cb <= n32i && seglen <= 32;
                    xlen = __shfl_sync(0xffffffffu, crossing ? seglen : 0, 0);
                    if (xlen > 0) {
                        const long long xsb = __shfl_sync(0xffffffffu, csb, 0);      // (widened: an element index)
                        if (static_cast<int>(lane) < xlen) xval = load_value<P>(xg, xsb + lane);
                    }
                }
                // the next 128 offsets travel behind the accumulator wait
                if (!tcovers) {
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const long long qi = cq + SUM_CHUNK + lane + 32 * j;
                        if (qi < nq) yraw[j] = prm.off[qi];
                    }
                }
            }

            MMV_T_MARK(0)
            if (!wait_bar(&bar_acc_full[buf], (it / SUM_BUFS) & 1, abort_flag, budget)) { failed = true; break; }
            tc_fence_after_sync();
            MMV_T_MARK(1)
            // request the next tile's offsets (its first index has arrived by now): they travel while this
            // tile's boundaries are worked through
            if (tile_n >= 0) load_offsets(q_next, qe_next, nraw, nrawp, nlast, nlast_ok);

            LookbackWindow<1> lbw;
            Acc tot[PIECES_PER_SPAN];
            Acc run = Acc(0);              // sum of the open segment inside this span so far
            long long def_r = -1;          // segment that began before the span and ends inside it
            Acc def_val = Acc(0);
            // the span's aggregate: published before the boundaries are worked through, kept for the siblings
            auto publish = [&](Acc tail) {
                if (lane == 0) {
                    st_relaxed_gpu_u64(prm.status + s * SUM_STATUS_STRIDE, pack_status((seen || s == 0) ? ST_PREFIX : ST_AGG, P::to_bits(tail)));
                    agg_slot[(g * 2 + (k & 1)) * SPANS_PER_TILE + w] = (static_cast<uint64_t>(seen ? 1u : 0u) << 32) | P::to_bits(tail);
                    mbar_arrive(&bar_agg[g]);
                }
                // the first window beyond the tile travels while the boundaries are processed
                if (tile != 0 && !seen) lookback_load<1, SUM_STATUS_STRIDE>(prm.status, s - w - 1, lbw);
                if (pending) lookback_load<1, SUM_STATUS_STRIDE>(prm.status, pend_s - w - 1, plw);
            };
            if (sparse) {
                // ---- few boundaries (lane j <-> boundary j): the one prefix each boundary needs is read
                //      straight from TMEM (one column; it sits in the lane of its row), together with the
                //      row totals (column 31), with a single wait ----
                // (crel = cb - sbase is 0..SPAN for lanes < nb_span)
                uint32_t vv[SUM_SPARSE_MAX];
#pragma unroll
                for (int i = 0; i < PIECES_PER_SPAN; ++i) tot[i] = P::from_bits(tmem_ld_32x1(taddr + i * ROW + (ROW - 1)));
                // (spans with at most two boundaries -- the usual case with long segments -- skip the other six slots
                //  with one branch instead of issuing their predicated-off instructions: n = 2^28, lengths
                //  U{1..4096}: 104.4 -> 98.9 us.  Replacing the four scans by one masked warp sum per boundary for
                //  such spans measured slower again, 104 us.)
                auto request = [&](int j) {
                    vv[j] = 0u;
                    if (j < nb_span) {
                        const int e = __shfl_sync(0xffffffffu, crel, j) - 1;                 // element before the boundary
                        if (e >= 0) vv[j] = tmem_ld_32x1(taddr + (e >> 10) * ROW + (e & 31));
                    }
                };
                request(0);
                request(1);
                if (nb_span > 2) {
#pragma unroll
                    for (int j = 2; j < SUM_SPARSE_MAX; ++j) request(j);
                } else {
#pragma unroll
                    for (int j = 2; j < SUM_SPARSE_MAX; ++j) vv[j] = 0u;
                }
                tmem_ld_wait();
                MMV_T_MARK(12)
                // exclusive prefix of the 128 row totals of the span (four interleaved warp scans)
                Acc inc[PIECES_PER_SPAN];
#pragma unroll
                for (int i = 0; i < PIECES_PER_SPAN; ++i) inc[i] = tot[i];
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
#pragma unroll
                    for (int i = 0; i < PIECES_PER_SPAN; ++i) {
                        const Acc t = __shfl_up_sync(0xffffffffu, inc[i], o);
                        if (static_cast<int>(lane) >= o) inc[i] = P::add(t, inc[i]);
                    }
                }
                Acc span_total = Acc(0), rowpre_span[PIECES_PER_SPAN];
#pragma unroll
                for (int i = 0; i < PIECES_PER_SPAN; ++i) {
                    rowpre_span[i] = P::add(span_total, P::sub(inc[i], tot[i]));
                    span_total = P::add(span_total, __shfl_sync(0xffffffffu, inc[i], 31));
                }
                MMV_T_MARK(13)
                // lane j fetches, for its boundary: the prefix inside the row and the prefix of the rows before
                const int e = crel - 1;
                const bool have = static_cast<int>(lane) < nb_span && e >= 0;
                const int myrow = have ? (e >> 5) : -1;                  // row inside the span (0..127)
                const int src = have ? (myrow & 31) : 0;
                Acc mylocal = Acc(0), myrp = Acc(0);
                auto fetch = [&](int j) {
                    const uint32_t t = __shfl_sync(0xffffffffu, vv[j], src);
                    if (static_cast<int>(lane) == j) mylocal = P::from_bits(t);
                };
                fetch(0);
                fetch(1);
                if (nb_span > 2) {
#pragma unroll
                    for (int j = 2; j < SUM_SPARSE_MAX; ++j) fetch(j);
                }
#pragma unroll
                for (int i = 0; i < PIECES_PER_SPAN; ++i) {
                    const Acc t = __shfl_sync(0xffffffffu, rowpre_span[i], src);
                    if ((e >> 10) == i) myrp = t;
                }
                if (!have) { mylocal = Acc(0); myrp = Acc(0); }
                // the span's aggregate = sum of the segment open at its end
                Acc tail = span_total;
                if (seen) {
                    // the last start is the last boundary below the span's end: lane jl
                    const int jl = __popc(__ballot_sync(0xffffffffu, static_cast<int>(lane) < nb_span && crel < SPAN)) - 1;
                    const int il = lastrel >> 10, rl = (lastrel >> 5) & 31, pos = lastrel & 31;
                    Acc after = Acc(0), totl = tot[0];
#pragma unroll
                    for (int i = 0; i < PIECES_PER_SPAN; ++i) {
                        if (i > il) after = P::add(after, tot[i]);
                        if (i == il) totl = tot[i];
                    }
                    if (static_cast<int>(lane) > rl) after = P::add(after, totl);
                    after = warp_sum<P>(after);
                    const Acc before = (pos > 0) ? __shfl_sync(0xffffffffu, mylocal, jl & 31) : Acc(0);
                    tail = P::add(P::sub(__shfl_sync(0xffffffffu, totl, rl), before), after);
                }
                publish(tail);
                run = tail;
                MMV_T_MARK(2)
                const Acc dval = is_direct ? window_sum<P>(xg, csb, seglen, win0) : Acc(0);
                const Acc plocal = __shfl_up_sync(0xffffffffu, mylocal, 1);
                const Acc prp = __shfl_up_sync(0xffffffffu, myrp, 1);
                const int prow = __shfl_up_sync(0xffffffffu, myrow, 1);
                const long long qi = cq + lane;
                bool deferred = false;
                bool redo = false;        // a short segment whose sum is taken again from its values, at the end of this path
                Acc val = Acc(0);
                // lane j: boundary j as the END of segment qi-1 (bnd in (sbase, send], or 0 for leading empties)
                if (static_cast<int>(lane) < nb_span && qi >= 1 && (crel > 0 || (sb32i == 0 && cb == 0))) {
                    if (csb > cb || csb < 0 || cb > n32i) {
                        report_error(prm.hdr, 4u);
                    } else {
                        if (cb != csb) {
                            if (seglen <= SUM_DIRECT_LEN) {
                                val = dval;
                            } else if (csb > sb32i) {
                                // the start is the previous boundary (lane - 1), inside this span
                                val = (prow == myrow) ? P::sub(mylocal, plocal)
                                                      : P::sub(P::add(myrp, mylocal), P::add(prp, plocal));
                                if constexpr (P::kIsFloat) redo = seglen <= 32;
                            } else {
                                val = P::add(myrp, mylocal);        // from the span's first element
                                deferred = csb < sb32i;
                                // (short and reaching back across the span's first element: its carry would be a difference
                                //  of the previous span's prefixes)
                                if constexpr (P::kIsFloat) {
                                    if (deferred && seglen <= 32) {
                                        deferred = false;
                                        redo = true;
                                    }
                                }
                            }
                        }
                        if (!deferred) outp[qi - 1] = val;
                    }
                }
                const unsigned dm = __ballot_sync(0xffffffffu, deferred);
                if (dm) {
                    const int srcl = __ffs(dm) - 1;
                    def_r = cq + srcl - 1;
                    def_val = __shfl_sync(0xffffffffu, val, srcl);
                }
                // Floating point: a difference of prefixes loses a small sum next to large values, and this path has no
                // row-wide magnitudes to measure a difference against (the general path has).  Every segment of 5 to 32 elements
                // that starts behind the span's first element or in front of it is therefore added up again from its
                // values, one element per lane (a single round trip to memory; with so few boundaries in the span such
                // segments are rare).
                if constexpr (P::kIsFloat) {
                    unsigned rm = __ballot_sync(0xffffffffu, redo);
                    while (rm) {
                        const int j = __ffs(rm) - 1;
                        rm &= rm - 1;
                        const long long sbj = __shfl_sync(0xffffffffu, csb, j);
                        const int lenj = __shfl_sync(0xffffffffu, seglen, j);
                        Acc v = Acc(0);
                        if (static_cast<int>(lane) < lenj) v = load_value<P>(xg, sbj + lane);
                        v = warp_sum<P>(v);
                        if (static_cast<int>(lane) == j) outp[qi - 1] = v;
                    }
                }
                MMV_T_MARK(5)
            } else {
                // ---- general path: row totals, pre-pass ----
#pragma unroll
                for (int i = 0; i < PIECES_PER_SPAN; ++i) tot[i] = P::from_bits(tmem_ld_32x1(taddr + i * ROW + (ROW - 1)));
                tmem_ld_wait();
                MMV_T_MARK(11)
                Acc tail;
                if (!seen) {
                    tail = warp_sum<P>(P::add(P::add(tot[0], tot[1]), P::add(tot[2], tot[3])));
                } else {
                    const int il = lastrel >> 10, rl = (lastrel >> 5) & 31, pos = lastrel & 31;
                    Acc after = Acc(0), totl = tot[0];
#pragma unroll
                    for (int i = 0; i < PIECES_PER_SPAN; ++i) {
                        if (i > il) after = P::add(after, tot[i]);
                        if (i == il) totl = tot[i];
                    }
                    if (static_cast<int>(lane) > rl) after = P::add(after, totl);
                    after = warp_sum<P>(after);
                    Acc before = Acc(0);
                    if (pos > 0) {
                        before = P::from_bits(tmem_ld_32x1(taddr + il * ROW + (pos - 1)));
                        tmem_ld_wait();
                    }
                    tail = P::add(__shfl_sync(0xffffffffu, P::sub(totl, before), rl), after);
                }
                publish(tail);
                MMV_T_MARK(2)
            }
            if (!sparse) {
                // ---- general path, second step: the boundaries beyond the first 128 mark their elements, 128 at
                //      a time with the next 128 offsets already requested.  128 equal offsets in a row are a run of
                //      empty segments (their zeros were written when the offsets were partitioned): the run is
                //      jumped over with a 32-ary search and only counted. ----
                if (!tcovers) {
                    long long tp = cq + SUM_CHUNK;            // index of yraw's first boundary
                    while (true) {
                        int32_t zraw[4] = {kNoOffset, kNoOffset, kNoOffset, kNoOffset};
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const long long qi = tp + SUM_CHUNK + lane + 32 * j;
                            if (qi < nq) zraw[j] = prm.off[qi];
                        }
                        const int32_t first = __shfl_sync(0xffffffffu, yraw[0], 0);
                        bool beyond = false, same = true;
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            if (tp + lane + 32 * j < nq) beyond |= mark(yraw[j]);
                            else beyond = true;
                            same &= yraw[j] == first;
                        }
                        if (__any_sync(0xffffffffu, beyond)) break;
                        tp += SUM_CHUNK;
#pragma unroll
                        for (int j = 0; j < 4; ++j) yraw[j] = zraw[j];
                        if (__all_sync(0xffffffffu, same)) {
                            const long long u = first_index_at_least_call(prm.off, sh, tp, nq, static_cast<long long>(first) + 1);
                            if (u > tp) {
                                const int rel = static_cast<int>(static_cast<uint32_t>(first) - sb32);
                                if (lane == 0) {
                                    if (rel == 0) atomicAdd(nbase, static_cast<uint32_t>(u - tp));
                                    else if (rel > 0 && rel <= SPAN) atomicAdd(&ecnt[(rel - 1) >> 5], static_cast<uint32_t>(u - tp));
                                }
                                tp = u;
#pragma unroll
                                for (int j = 0; j < 4; ++j) {
                                    const long long qi = tp + lane + 32 * j;
                                    yraw[j] = qi < nq ? prm.off[qi] : kNoOffset;
                                }
                            }
                        }
                    }
                }
                __syncwarp();
                MMV_T_MARK(3)

                // ---- third step, lane = row: the piece's prefixes go to shared memory and every lane visits the
                //      marked elements of its row, one sum each.  Inside the row a sum is the difference of two row
                //      prefixes; the first one of a row adds what is open from the rows before (a segmented warp
                //      scan of row totals and row tails).  A floating-point sum of a segment inside one row or two
                //      adjacent rows that came out small against the prefixes it was taken from (cancellation:
                //      under 2^-10 of the largest prefix of those rows) is added up again from the input values.  Output indices follow from the counts: the r-th row's first sum
                //      belongs to boundary cq + nbase + (number of boundaries in the rows before). ----
                const bool open_at_base = *nbase == 0u;          // the segment open at the span's first element began before it
                long long obase = cq + static_cast<long long>(*nbase) - 1;     // output index of the span's first marked element
                bool span_has_end = false;
                // a very short segment that reaches back across the span's first element: summed from its values
                const bool cross_done = xlen > 0 || __shfl_sync(0xffffffffu, is_direct ? 1 : 0, 0) != 0;
                if (xlen > 0) {
                    const Acc xsum = warp_sum<P>(xval);
                    if (lane == 0) outp[cq - 1] = xsum;
                } else if (lane == 0 && is_direct) {
                    outp[cq - 1] = window_sum<P>(xg, csb, seglen, win0);
                }
                // number of elements open at the end of the previous piece's last row (64: too many to matter),
                // and the largest prefix magnitude of that row
                int pc_len = open_at_base ? 64 : 0;
                float pc_scale = 0.f;
#pragma unroll 1
                for (int i = 0; i < PIECES_PER_SPAN; ++i) {
                    const long long pbase = sbase + i * PIECE;
                    Acc toti = tot[0];
#pragma unroll
                    for (int t = 1; t < PIECES_PER_SPAN; ++t)
                        if (i == t) toti = tot[t];
                    const uint32_t m = emask[i * PIECE_ROWS + lane];
                    const uint32_t cn = ecnt[i * PIECE_ROWS + lane];
                    const unsigned hb = __ballot_sync(0xffffffffu, m != 0u);
                    // output index of the row's first sum: exclusive scan of the boundary counts
                    uint32_t cinc = cn;
#pragma unroll
                    for (int o = 1; o < 32; o <<= 1) {
                        const uint32_t t = __shfl_up_sync(0xffffffffu, cinc, o);
                        if (static_cast<int>(lane) >= o) cinc += t;
                    }
                    const long long orow = obase + (cinc - cn);
                    obase += __shfl_sync(0xffffffffu, cinc, 31);
                    if (hb == 0u) {
                        run = P::add(run, warp_sum<P>(toti));
                        pc_len = 64;
                        continue;
                    }
                    float scale = 0.f;             // largest prefix magnitude of my row
                    {
                        uint32_t r[32];
                        tmem_ld_32x32(taddr + i * ROW, r);
                        tmem_ld_wait();
#pragma unroll
                        for (int c4 = 0; c4 < 8; ++c4)
                            *reinterpret_cast<uint4*>(dump + lane * Cfg::kDumpRowBytes + (c4 << 4)) =
                                make_uint4(r[4 * c4], r[4 * c4 + 1], r[4 * c4 + 2], r[4 * c4 + 3]);
                        if constexpr (P::kIsFloat) {
                            // (two chains of three-operand maxima)
                            float s0 = 0.f, s1 = 0.f;
#pragma unroll
                            for (int c = 0; c < 32; c += 4) {
                                s0 = fmaxf(fmaxf(s0, fabsf(__uint_as_float(r[c]))), fabsf(__uint_as_float(r[c + 1])));
                                s1 = fmaxf(fmaxf(s1, fabsf(__uint_as_float(r[c + 2]))), fabsf(__uint_as_float(r[c + 3])));
                            }
                            scale = fmaxf(s0, s1);
                        }
                    }
                    __syncwarp();
                    MMV_T_MARK(4)

                    // rows with empty segments among their boundaries look their output indices up in the offsets
                    const bool dirty = cn != static_cast<uint32_t>(__popc(m));
                    long long bp = orow + 1;                       // boundary index the next sum is looked for at
                    const long long bend = bp + cn;
                    const long long rowpos = pbase + lane * ROW;   // position of my row's first element
                    Acc pv = Acc(0), first_pref = Acc(0);
                    int cprev = -1, nend = 0, first_len = 0;
                    long long first_oi = -1;
                    uint32_t mm = m;
                    const uint8_t* drow = dump + lane * Cfg::kDumpRowBytes;       // my row of the prefixes
                    auto prefix_at = [&](int c) -> Acc { return *reinterpret_cast<const Acc*>(drow + (c << 2)); };
                    auto index_of = [&](int c, int k) -> long long {          // output index of my k-th sum, which ends behind column c
                        if (!dirty) return orow + k;
                        const int32_t bpos = static_cast<int32_t>(rowpos + c + 1);
                        while (bp + 1 < bend && prm.off[bp] < bpos) ++bp;
                        return (bp++) - 1;
                    };
                    if (mm) {                                      // the row's first marked element: finished below
                        const int c = __ffs(mm) - 1;
                        mm &= mm - 1;
                        first_pref = pv = prefix_at(c);
                        first_len = c + 1;
                        first_oi = index_of(c, 0);
                        cprev = c;
                        nend = 1;
                    }
                    float cancel_below = 0.f;
                    if constexpr (P::kIsFloat) cancel_below = scale * SUM_CANCEL;
                    Acc* po = outp + orow;                          // (rows without empty segments: sums at consecutive indices)
                    while (mm) {                                   // (lanes differ in the number of marked elements)
                        const int c = __ffs(mm) - 1;
                        mm &= mm - 1;
                        const Acc pc = prefix_at(c);
                        Acc val = P::sub(pc, pv);
                        if constexpr (P::kIsFloat) {
                            if (fabsf(val) < cancel_below) val = direct_sum<P>(xg, rowpos + cprev + 1, rowpos + c + 1);
                        }
                        if (dirty) outp[index_of(c, nend)] = val;
                        else po[nend] = val;
                        pv = pc;
                        cprev = c;
                        ++nend;
                    }
                    // what is open at the end of each row: the part behind its last marked element, or all of it
                    const bool has_end = nend > 0;
                    Acc v = has_end ? P::sub(toti, pv) : toti;
                    // rows back to (not including) the nearest one at or before mine that has a marked element: the
                    // open part reaches that far back
                    const uint32_t heads = hb & (0xffffffffu >> (31 - lane));
                    const int reach = heads ? static_cast<int>(lane) - (31 - __clz(heads)) : static_cast<int>(lane);
#pragma unroll
                    for (int o = 1; o < 32; o <<= 1) {
                        const Acc t = __shfl_up_sync(0xffffffffu, v, o);
                        if (o <= reach) v = P::add(t, v);
                    }
                    // open sum at the START of my row: the inclusive value of the row before (plus the piece's carry
                    // if no row before me has a marked element)
                    Acc open = __shfl_up_sync(0xffffffffu, v, 1);
                    if (lane == 0) open = Acc(0);
                    const bool none_before = (hb & ((1u << lane) - 1u)) == 0u;
                    if (none_before) open = P::add(run, open);
                    // the previous row's open elements, if it has a marked element itself
                    const int my_open = has_end ? 31 - cprev : 64;
                    int c_len = __shfl_up_sync(0xffffffffu, my_open, 1);
                    float c_scale = __shfl_up_sync(0xffffffffu, scale, 1);
                    if (lane == 0) {
                        c_len = pc_len;
                        c_scale = pc_scale;
                    }
                    bool deferred = false;
                    Acc fval = Acc(0);
                    if (has_end) {
                        fval = P::add(open, first_pref);
                        const bool first_of_span = !span_has_end && none_before;
                        if (first_of_span && open_at_base) {
                            deferred = !cross_done;           // waits for the carry (or was summed from its values)
                        } else {
                            if constexpr (P::kIsFloat) {
                                if (c_len < 64 && fabsf(fval) < fmaxf(scale, c_scale) * SUM_CANCEL)
                                    fval = direct_sum<P>(xg, rowpos - c_len, rowpos + first_len);
                            }
                            if (first_oi >= 0) outp[first_oi] = fval;
                        }
                    }
                    const unsigned dm = __ballot_sync(0xffffffffu, deferred);
                    if (dm) {
                        const int src = __ffs(dm) - 1;
                        def_r = __shfl_sync(0xffffffffu, first_oi, src);
                        def_val = __shfl_sync(0xffffffffu, fval, src);
                    }
                    span_has_end = true;
                    // carries into the next piece
                    run = __shfl_sync(0xffffffffu, v, 31);
                    pc_len = __shfl_sync(0xffffffffu, my_open, 31);
                    pc_scale = __shfl_sync(0xffffffffu, scale, 31);
                    __syncwarp();
                    MMV_T_MARK(5)
                }
            }

            // ---- the TMEM buffer is free; publish, look back, emit the segment that began before this span ----
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(&bar_acc_empty[buf]);
            MMV_T_MARK(6)
            // Every warp waits on every phase of bar_agg (parity waits must not skip phases).  The carry
            // into this span is first sought among the tile's earlier spans (shared memory); only if
            // none of them holds a segment start does the look-back go out to the other CTAs' words.
            if (!wait_bar(&bar_agg[g], k & 1, abort_flag, budget)) { failed = true; break; }
            MMV_T_MARK(14)
            // the segment parked at this warp's previous tile: its look-back window was requested during
            // this tile's pre-pass, so the predecessor's word has normally arrived
            if (pending) {
                Acc carry_out = Acc(0);
                if (!sum_lookback<P>(prm.status, pend_s - w, &carry_out, abort_flag, budget, plw.w[0], true)) { failed = true; break; }
                if (lane == 0) outp[pend_r] = P::add(P::add(carry_out, pend_ex), pend_val);
                pending = false;
            }
            MMV_T_MARK(15)
            if (s == 0) {
                if (def_r >= 0 && lane == 0) outp[def_r] = def_val;
            } else if (!seen || def_r >= 0) {
                Acc ex = Acc(0);
                bool exflag = false;
#pragma unroll
                for (int j = 0; j < SPANS_PER_TILE; ++j) {
                    if (j < w) {
                        const uint64_t a = agg_slot[(g * 2 + (k & 1)) * SPANS_PER_TILE + j];
                        const Acc tj = P::from_bits(static_cast<uint32_t>(a));
                        if ((a >> 32) != 0u) { ex = tj; exflag = true; }
                        else ex = P::add(ex, tj);
                    }
                }
                if (exflag || tile == 0) {
                    // the carry is complete inside the tile
                    if (!seen && lane == 0)
                        st_relaxed_gpu_u64(prm.status + s * SUM_STATUS_STRIDE, pack_status(ST_PREFIX, P::to_bits(P::add(ex, run))));
                    if (def_r >= 0 && lane == 0) outp[def_r] = P::add(ex, def_val);
                } else if (seen) {
                    // The span's own word is final already; only the segment that ends here waits for the
                    // carry from the other CTAs.  It is parked until this warp's next tile is done, which
                    // keeps the CTAs from falling into step with their slowest neighbour.
                    pending = true;
                    pend_s = s;
                    pend_r = def_r;
                    pend_val = def_val;
                    pend_ex = ex;
                } else {
                    Acc carry_out = Acc(0);
                    if (!sum_lookback<P>(prm.status, s - w, &carry_out, abort_flag, budget, lbw.w[0], true)) {
                        if (lane == 0) st_relaxed_gpu_u64(prm.status + s * SUM_STATUS_STRIDE, pack_status(ST_ABORT, 0u));
                        failed = true;
                        break;
                    }
                    const Acc carry = P::add(carry_out, ex);
                    if (lane == 0) st_relaxed_gpu_u64(prm.status + s * SUM_STATUS_STRIDE, pack_status(ST_PREFIX, P::to_bits(P::add(carry, run))));
                    if (def_r >= 0 && lane == 0) outp[def_r] = P::add(carry, def_val);
                }
            }
            MMV_T_MARK(7)
        }
        if (pending && !failed) {
            Acc carry_out = Acc(0);
            if (!sum_lookback<P>(prm.status, pend_s - w, &carry_out, abort_flag, budget, 0ull, false)) failed = true;
            else if (lane == 0) outp[pend_r] = P::add(P::add(carry_out, pend_ex), pend_val);
        }
        MMV_T_FLUSH()
        if (failed) {
            *abort_flag = 1;
            if (lane == 0) report_error(prm.hdr, 5u);
        }
    }

    tc_fence_before_sync();
    __syncthreads();
    if (warp == Shape::kMmaWarp) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, SUM_TMEM_COLS);
    }
}

}  // namespace mmv
