// Single-pass segmented inclusive scan (Problem 2.1, Eq. 1) for sm_100a, row-major layout.
//
// The value vector is the paper's ceil(n/s) x s matrix with s = ROW = 32.  A warp owns a
// SPAN of 128 consecutive rows (4096 elements) in four PIECES of 32 rows; a TILE is four
// spans.  For each tile:
//   producer warp  one 4-D TMA box per piece index i (the [128 rows x 32] matrix made of
//                  piece i of the four spans, K-major, hardware swizzle) and one bulk copy
//                  of the tile's 16 KB of flag bytes, several tiles ahead.
//   tensor core    tcgen05.mma issued by the leader of the warpgroup that takes the tile:
//                  A = that matrix, B = the constant [U_32 | I_32] (fp16) or U_32 (int8):
//                  TMEM lane 32w+l, column j (< 32) = inclusive prefix at position j of row l
//                  of piece i of span w, the speculative block scan z = MATMUL(x, U_s) of
//                  Algorithm A.1 (BlockSegScan); columns 32..63 (fp16) return the row itself
//                  converted exactly to fp32.
//   epilogue warps (lane = row; two warpgroups for fp16, three for int8, taking tiles in turn)
//     pre-pass     flag bytes -> one 32-bit start mask per row; row totals (TMEM column 31);
//                  from these each span's aggregate (sum of its open tail segment, any flag) is
//                  formed with a handful of shuffles; the four spans of a tile exchange theirs
//                  through shared memory and the tile's first warp publishes ONE status word
//                  for the tile.
//     main pass    per piece: revert the speculation inside each row (Lemma A.1).  int8: subtract the
//                  prefix just before the element's segment start, exact modulo 2^32.  Floating
//                  point, where addition has no inverse: a piece that holds a start takes the rows
//                  themselves (identity half) and forms the running sum since the last start, so
//                  no prefix is ever subtracted from another.  Then a segmented scan of the 32 row tails
//                  with shuffles, add the row carries (UpdateFirstSegment inside the span),
//                  stage the 32 x 32 results in shared memory and write them with one TMA
//                  store.  Pieces without any flag skip the revert.  Pieces that reach back
//                  to the start of the span (up to and including the first flagged one) are
//                  parked in TMEM instead.
//     look-back    the tile's first warp runs the decoupled look-back over the earlier tiles'
//                  status words (this replaces the recursion of Section 4.2 / Algorithm A.1's
//                  Recurse) and hands the carry to its siblings through shared memory; its
//                  latency is covered by the main pass.  The parked pieces then receive the
//                  carry on the elements before the span's first flag and are stored.
#pragma once
#include <cooperative_groups.h>
#include "common.cuh"

namespace mmv {

struct ScanParams {
    const void* x;
    const uint8_t* flags;        // start flags, or null: one segment (the plain scan of Algorithm 4.1; no flag traffic)
    void* out;
    long long n;
    int num_tiles;
    WorkspaceHeader* hdr;
    uint64_t* status;            // one word per span
    unsigned long long budget_ns;
    long long debug_skip_span;   // test hook: this span never publishes (-1 = off)
    const void* carry_in;        // device pointer to one fp32 / int32, or null: the running sum that
                                 // reaches element 0 from an earlier chunk of the same vector (element 0
                                 // then continues that segment unless its flag is set)
    const unsigned int* probe_count;   // device word, or null: number of starts a sampling kernel found in
    unsigned int probe_narrow_below;   // SCAN_PROBE_BYTES flag bytes; the narrow shape runs iff it is below this,
                                       // the wide shape iff it is not (the other launch returns at once)
    long long clear_words;             // > 0: the kernel itself clears the header and this many 8-byte status words in
                                       // front of a grid-wide barrier (no memset node in front of the launch)
    unsigned long long* first_start;   // device word, or null: receives n - (index of the vector's first start)
                                 // by atomicMax (it begins at 0 = no start); used when the vector is one
                                 // shard of a longer one, whose carry belongs in front of that index
};

// Scan geometry: a warp owns a UNIT of SCAN_UP consecutive pieces (the grain of the carry
// chain: one status word per unit); a scan tile is four units and SCAN_UP tensor-core products.
// The warpgroups of the epilogue (two for fp16, three for int8) take tiles in turn; with two TMEM
// buffers per warpgroup (int8 built with two groups) the products of a group's next tile are
// finished before it gets there.
constexpr int SCAN_UP = 4;
constexpr int SCAN_UNIT = SCAN_UP * PIECE;                  // 4096 elements
constexpr int SCAN_TILE = SPANS_PER_TILE * SCAN_UNIT;       // 16384 elements
#ifndef MMV_SCAN_LB_WORDS
#define MMV_SCAN_LB_WORDS 1
#endif
#ifndef MMV_SCAN_STATUS_STRIDE
#define MMV_SCAN_STATUS_STRIDE 4
#endif
#ifndef MMV_SCAN_LB_DENSE_ROWS
#define MMV_SCAN_LB_DENSE_ROWS 4
#endif
constexpr int SCAN_LB_DENSE_ROWS = MMV_SCAN_LB_DENSE_ROWS;  // rows with a start, of the 32 of a piece, above which the look-back is requested early
constexpr int SCAN_LB_WORDS = MMV_SCAN_LB_WORDS;            // look-back window: 32 tiles per poll and word
// A tile publishes one status word; tile t uses word t * SCAN_STATUS_STRIDE of the workspace, so that every
// word sits in a 32-byte sector of its own: the tiles in flight poll and write neighbouring words all the
// time, and in a dense array those accesses queue at one sector.  Measured at n = 2^30 (fp16), dense array
// -> stride 4: no start at all 1.53 -> 1.36 ms, p = 1e-3 1.19 -> 1.15 ms, no flag vector 1.26 -> 1.10 ms,
// but p >= 0.1 1.20 -> 1.27 ms; a stride of 8 moves each of these a little further in the same direction.
constexpr int SCAN_STATUS_STRIDE = MMV_SCAN_STATUS_STRIDE;
#ifndef MMV_SCAN_I8_GROUPS
#define MMV_SCAN_I8_GROUPS 3
#endif

// The kernel comes in three shapes.
//   SCAN_WIDE    the product also returns the rows themselves ([U | I], 256 TMEM columns per fp16 tile), two
//                warpgroups (int8: U only, 128 columns, three warpgroups).  Every flag density.
//   SCAN_PLAIN   the call has no flag vector (one segment): no row ever needs its own values back, so the
//                floating-point paths drop the identity half: narrow tiles (128 TMEM columns), four warpgroups
//                with one tile each, four 32 KB stages without flag bytes, one staging buffer per warp.
//   SCAN_NARROW  floating point with a flag vector in which starts are RARE: the narrow tiles and four
//                warpgroups of SCAN_PLAIN, three 48 KB stages; the rare piece that holds a start fetches its
//                rows from global memory instead of from identity columns.  Correct for every flag vector,
//                fast only where few pieces hold a start (a tile can then wait for its carry in a quarter
//                of the tensor memory while three others are worked on).
constexpr int SCAN_WIDE = 0, SCAN_PLAIN = 1, SCAN_NARROW = 2;
template <typename P, int MODE = SCAN_WIDE>
struct ScanCfg {
    static constexpr bool kWide = P::kIsFloat && MODE == SCAN_WIDE;      // [U | I] product
    static constexpr int kN = kWide ? 2 * ROW : ROW;                     // accumulator columns per product
    static constexpr int kGroups = kWide ? 2 : (P::kIsFloat ? 4 : MMV_SCAN_I8_GROUPS);
    static constexpr int kTmemCols = 512;
    // TMEM tile buffers: as many as fit.  Iteration `it` of the CTA uses buffer it % kBufs, whichever warpgroup
    // takes it, so with more buffers than warpgroups (int8 with three groups: four) the products of a group's
    // next tile are finished while all groups are still busy with their current ones
    // (int8, n = 2^28: every second element a start 274 -> 266 us, p = 1e-3 280 -> 278 us).
    static constexpr int kBufs = kTmemCols / (SCAN_UP * kN);
    static constexpr int kEpiWarps = 4 * kGroups;
    static constexpr int kProducerWarp = kEpiWarps;
    static constexpr int kMmaWarp = kEpiWarps + 1;
    static constexpr int kThreads = (kEpiWarps + 2) * 32;
    static constexpr int kStages = (P::kIsFloat && MODE == SCAN_PLAIN) ? 4 : 3;
    static_assert(kBufs >= kGroups && kBufs * SCAN_UP * kN <= kTmemCols, "a tile buffer per warpgroup, all inside the tensor memory");
    static constexpr int kBBytes = kN * P::kRowBytes;                    // constant operand [U_32 | I_32] / U_32
    static constexpr int kBSlot = 4096;
    static constexpr int kXBytes = SCAN_UP * P::kSlabBytes;
    static constexpr int kFlagBytes = MODE == SCAN_PLAIN ? 0 : SCAN_TILE;
    static constexpr int kStageBytes = kXBytes + kFlagBytes;
    static constexpr int kStageOffset = kBSlot;
    static constexpr int kOutOffset = kStageOffset + kStages * kStageBytes;
    static constexpr int kOutBufBytes = PIECE * 4;                       // 32 rows x 128 B
    static constexpr int kOutBufs = kGroups >= 4 ? 1 : 2;                // staging buffers per warp
    static constexpr int kOutBytes = kEpiWarps * kOutBufs * kOutBufBytes;
    static constexpr int kBarOffset = kOutOffset + kOutBytes;
    static constexpr int kSmemBytes = kBarOffset + 640 + 1024;        // barriers and small slots, alignment slack
    static_assert(kSmemBytes <= 227 * 1024, "fits the shared memory of one CTA");
    static_assert(kBBytes <= kBSlot, "constant operand fits its slot");
    static_assert(kStageOffset % 1024 == 0 && kStageBytes % 1024 == 0 && kOutOffset % 1024 == 0, "swizzle atoms");
};

// 32 flag bytes (8 words) -> bit j set iff byte j is non-zero.
__device__ __forceinline__ uint32_t flag_bytes_to_mask(const uint4& a, const uint4& b) {
    const uint32_t w[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
    uint32_t m = 0u;
#pragma unroll
    for (int k = 0; k < 8; ++k) {
        // bit 7 of every byte := byte != 0, then gather the four bits
        const uint32_t t = (((w[k] & 0x7F7F7F7Fu) + 0x7F7F7F7Fu) | w[k]) & 0x80808080u;
        m |= ((t * 0x00204081u) >> 28) << (4 * k);
    }
    return m;
}

// Waits until shared-memory stage `stage` holds iteration `it` (the producer writes the iteration
// number before it arms the barrier) and its bytes have landed.  Checking the iteration number
// first makes the parity wait unambiguous even for a waiter that does not see every phase.
__device__ __forceinline__ bool wait_stage(const volatile int* stage_iter, int it, uint64_t* bar, uint32_t parity,
                                           volatile int* abort_flag, uint64_t budget_ns) {
    if (*stage_iter != it) {
        const uint64_t t0 = global_timer_ns();
        uint32_t polls = 0;
        while (*stage_iter != it) {
            if ((++polls & 31u) == 0u) {
                if (*abort_flag) return false;
                if (global_timer_ns() - t0 > budget_ns) return false;
            }
        }
    }
    return wait_bar(bar, parity, abort_flag, budget_ns);
}

// Flag density probe: SCAN_PROBE_BLOCKS blocks of 1 KB, spread evenly over the flag vector, are counted for
// non-zero bytes (one 16-byte load per thread); the total goes to *count, which the caller has cleared.
constexpr int SCAN_PROBE_BLOCKS = 256;
constexpr int SCAN_PROBE_THREADS = 64;
constexpr int SCAN_PROBE_BYTES = SCAN_PROBE_BLOCKS * SCAN_PROBE_THREADS * 16;     // 256 KB
__global__ void __launch_bounds__(SCAN_PROBE_THREADS)
flag_density_probe_kernel(const uint8_t* __restrict__ flags, long long n, unsigned int* __restrict__ count) {
    const long long base = (static_cast<long long>(blockIdx.x) * (n / SCAN_PROBE_BLOCKS)) & ~15ll;
    const long long p = base + threadIdx.x * 16;
    unsigned int c = 0u;
    if (p + 16 <= n) {
        const uint4 q = *reinterpret_cast<const uint4*>(flags + p);
        const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
        for (int k = 0; k < 4; ++k) c += __popc((((w[k] & 0x7F7F7F7Fu) + 0x7F7F7F7Fu) | w[k]) & 0x80808080u);
    }
    c = __reduce_add_sync(0xffffffffu, c);
    if ((threadIdx.x & 31) == 0 && c) atomicAdd(count, c);
}

// SCAN_NARROW only.  The 32 values of one row (elements e0 .. e0 + 31 of the vector, zero past n) as fp32 bit
// patterns, fetched from global memory: that shape has no identity columns to take them from.
template <typename P>
__device__ __forceinline__ void load_row_from_memory(const void* x, long long e0, long long n, uint32_t (&r)[32]) {
    if (e0 + ROW <= n) {
        const uint4* p = reinterpret_cast<const uint4*>(static_cast<const uint8_t*>(x) + e0 * 2);
#pragma unroll
        for (int v = 0; v < 4; ++v) {
            const uint4 q = __ldg(p + v);
            const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                float a, b;
                P::unpack2(w[k], a, b);
                r[8 * v + 2 * k] = __float_as_uint(a);
                r[8 * v + 2 * k + 1] = __float_as_uint(b);
            }
        }
    } else {
#pragma unroll 1
        for (int j = 0; j < ROW; ++j) {
            const float v = (e0 + j < n) ? P::load_elem(x, e0 + j) : 0.f;
#pragma unroll
            for (int q = 0; q < ROW; ++q)
                if (q == j) r[q] = __float_as_uint(v);
        }
    }
}
// Sum of the elements pl .. 31 of the row that starts at element e0 (the tail behind a row's last start).
template <typename P>
__device__ __noinline__ float row_tail_from_memory(const void* x, long long e0, int pl, long long n) {
    float t = 0.f;
    for (int j = pl; j < ROW && e0 + j < n; ++j) t += P::load_elem(x, e0 + j);
    return t;
}

// EX = true gives the exclusive variant: every element receives the sum of the elements of its
// segment in FRONT of it (0 at a segment start), i.e. the inclusive result moved one element to
// the right inside each segment.  The shift happens in registers just before a piece is staged for
// its store; everything else is the same kernel.
template <typename P, bool EX = false, int MODE = SCAN_WIDE>
__global__ void __launch_bounds__(ScanCfg<P, MODE>::kThreads, 1)
seg_scan_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_out,
                 const ScanParams prm) {
    using Acc = typename P::Acc;
    using Cfg = ScanCfg<P, MODE>;
    constexpr bool PLAIN = MODE == SCAN_PLAIN;
    constexpr int S = Cfg::kStages;
    constexpr int N = Cfg::kN;

    // Two shapes of this kernel may have been launched for one call (wide and narrow tiles); the one the sampled
    // flag density does not ask for returns before it touches anything.
    if (prm.probe_count != nullptr && ((*prm.probe_count < prm.probe_narrow_below) != (MODE == SCAN_NARROW))) return;

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* sB = smem;
    uint8_t* sStage = smem + Cfg::kStageOffset;
    uint64_t* bar_full = reinterpret_cast<uint64_t*>(smem + Cfg::kBarOffset);
    uint64_t* bar_empty = bar_full + S;
    uint64_t* bar_acc_full = bar_empty + S;                // per TMEM buffer: the tile's products are in it
    uint64_t* bar_acc_empty = bar_acc_full + Cfg::kBufs;    // per TMEM buffer: the four warps are done with it
    uint64_t* bar_agg = bar_acc_empty + Cfg::kBufs;          // per warpgroup: its four unit aggregates are in agg_slot
    uint64_t* bar_carry = bar_agg + Cfg::kGroups;           // per warpgroup: the tile's carry is in carry_slot
    // [group][tile parity][unit]: (flag << 32) | payload; two sets so that a warp's next-tile write
    // can never meet a sibling's read of this tile's values
    uint64_t* agg_slot = bar_carry + Cfg::kGroups;
    uint32_t* carry_slot = reinterpret_cast<uint32_t*>(agg_slot + Cfg::kGroups * 2 * SPANS_PER_TILE);   // [group]
    int* tile_slot = reinterpret_cast<int*>(carry_slot + Cfg::kGroups);
    volatile int* stage_iter = tile_slot + S;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tile_slot + 2 * S);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    // smallest index of a start that this CTA has reported so far (its tiles come in ascending order, so only its
    // first few units with a start ever go to the global word)
    volatile long long* cta_first = reinterpret_cast<volatile long long*>((reinterpret_cast<uintptr_t>(tmem_slot + 2) + 7) & ~uintptr_t(7));

    const int warp = threadIdx.x >> 5;
    const uint32_t lane = lane_id();
    const uint64_t budget = prm.budget_ns;

    if (threadIdx.x == 0) {
        *cta_first = 0x7fffffffffffffffll;
        for (int i = 0; i < S; ++i) {
            mbar_init(&bar_full[i], 1);
            mbar_init(&bar_empty[i], 4);      // the group's four warps, once their flag bytes are read
            stage_iter[i] = -1;
        }
        for (int i = 0; i < Cfg::kGroups; ++i) {
            mbar_init(&bar_agg[i], SPANS_PER_TILE);
            mbar_init(&bar_carry[i], 1);
        }
        for (int i = 0; i < Cfg::kBufs; ++i) {
            mbar_init(&bar_acc_full[i], 1);
            mbar_init(&bar_acc_empty[i], 4);
        }
        *abort_flag = 0;
        mbar_fence_init();
    }
    if (warp == Cfg::kMmaWarp) {
        tmem_alloc(tmem_slot, Cfg::kTmemCols);
        tmem_relinquish();
    }
    if (warp == Cfg::kProducerWarp && lane == 0) {
        tma_prefetch_desc(&tmap_x);
        tma_prefetch_desc(&tmap_out);
    }
    {
        // constant B, K-major: row nn = output column, element k = input position.
        // nn < 32: 1 iff k <= nn (U_32);  nn >= 32 (fp16 only): 1 iff k == nn - 32 (identity).
        constexpr int kVecPerRow = P::kRowBytes / 16;
        constexpr int kElemPerVec = 16 / P::kElemBytes;
#pragma unroll 1
        for (int v = threadIdx.x; v < N * kVecPerRow; v += Cfg::kThreads) {
            const int nn = v / kVecPerRow, cv = v % kVecPerRow;
            uint32_t words[4] = {0u, 0u, 0u, 0u};
#pragma unroll
            for (int e = 0; e < kElemPerVec; ++e) {
                const int k = cv * kElemPerVec + e;
                const bool one = (nn < ROW) ? (k <= nn) : (k == nn - ROW);
                if (one) {
                    if constexpr (P::kElemBytes == 2) words[e >> 1] |= static_cast<uint32_t>(P::kOneBits) << ((e & 1) * 16);
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
    if (prm.clear_words > 0) {
        // the whole grid is resident (cooperative launch): it clears its own workspace and meets at a barrier
        const long long tid = static_cast<long long>(blockIdx.x) * Cfg::kThreads + threadIdx.x;
        const long long nthreads = static_cast<long long>(gridDim.x) * Cfg::kThreads;
        for (long long i = tid; i < prm.clear_words; i += nthreads) prm.status[i] = 0ull;
        if (tid < static_cast<long long>(sizeof(WorkspaceHeader) / sizeof(unsigned int))) reinterpret_cast<unsigned int*>(prm.hdr)[tid] = 0u;
        __threadfence();
        cooperative_groups::this_grid().sync();
    }

    if (warp == Cfg::kProducerWarp) {
        // =========================== producer ===========================
        int it = 0;
        bool ok = true;
        while (ok) {
            // static round-robin tile assignment: all CTAs are resident (cooperative launch, one CTA per
            // SM), so iteration `it` of every CTA runs at about the same time and a tile's predecessors
            // are always in flight or finished.  Every role of the CTA derives its tiles from the same
            // formula, so the end of the work needs no message.
            const int tile = static_cast<int>(blockIdx.x) + it * static_cast<int>(gridDim.x);
            if (tile >= prm.num_tiles) break;
            const int stage = it % S;
            if (!wait_bar(&bar_empty[stage], ((it / S) & 1) ^ 1, abort_flag, budget)) { ok = false; break; }
            if (lane == 0) {
                tile_slot[stage] = tile;
                stage_iter[stage] = it;
            }
            uint8_t* xs = sStage + stage * Cfg::kStageBytes;
            uint8_t* fs = xs + Cfg::kXBytes;
            const long long tbase = static_cast<long long>(tile) * SCAN_TILE;
            if (tbase + SCAN_TILE <= prm.n) {
                if (lane == 0) {
                    mbar_arrive_expect_tx(&bar_full[stage], prm.flags ? Cfg::kStageBytes : Cfg::kXBytes);
#pragma unroll
                    for (int i = 0; i < SCAN_UP; ++i)
                        tma_load_4d(xs + i * P::kSlabBytes, &tmap_x, &bar_full[stage], 0, 0, i, tile * SPANS_PER_TILE);
                    if (prm.flags) tma_load_1d(fs, prm.flags + tbase, Cfg::kFlagBytes, &bar_full[stage]);
                }
            } else {
                // ragged last tile: 16-byte asynchronous copies, zero fill past n (MATMUL zero-pads its operand)
                const long long cnt = prm.n - tbase;
#pragma unroll 1
                for (int v = lane; v < (prm.flags ? SCAN_TILE / 16 : 0); v += 32) {
                    const int e0 = v * 16;
                    if (e0 + 16 <= cnt) {
                        cp_async_16(fs + e0, prm.flags + tbase + e0);
                        continue;
                    }
                    uint4 fv = make_uint4(0u, 0u, 0u, 0u);
                    if (e0 < cnt) {
                        __align__(16) uint8_t tmp[16];
#pragma unroll 1
                        for (int e = 0; e < 16; ++e) tmp[e] = (e0 + e < cnt) ? prm.flags[tbase + e0 + e] : uint8_t(0);
                        fv = *reinterpret_cast<const uint4*>(tmp);
                    }
                    *reinterpret_cast<uint4*>(fs + e0) = fv;
                }
                constexpr int kElemPerVec = 16 / P::kElemBytes;
                const uint8_t* xt = static_cast<const uint8_t*>(prm.x) + tbase * P::kElemBytes;
#pragma unroll 1
                for (int v = lane; v < SCAN_TILE / kElemPerVec; v += 32) {
                    const int e0 = v * kElemPerVec;
                    const int w = e0 / SCAN_UNIT, i = (e0 % SCAN_UNIT) / PIECE, l = (e0 % PIECE) / ROW, j0 = e0 % ROW;
                    uint8_t* dst = xs + i * P::kSlabBytes + swz_offset<P::kRowBytes>(w * PIECE_ROWS + l, j0 * P::kElemBytes);
                    if (e0 + kElemPerVec <= cnt) {
                        cp_async_16(dst, xt + static_cast<size_t>(e0) * P::kElemBytes);
                        continue;
                    }
                    uint4 xv = make_uint4(0u, 0u, 0u, 0u);
                    if (e0 < cnt) {
                        __align__(16) uint8_t tmp[16];
#pragma unroll 1
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
    } else if (warp == Cfg::kMmaWarp) {
        // =========================== MMA issuer ===========================
        // Runs ahead of the epilogue: the products of a warpgroup's next tile go to its other buffer.
        constexpr uint32_t idesc = P::kIsFloat ? (make_idesc_f16_f32(128, N) | P::kFmtBits) : make_idesc_s8_s32(128, N);
        for (int it = 0; static_cast<int>(blockIdx.x) + it * static_cast<int>(gridDim.x) < prm.num_tiles; ++it) {
            const int stage = it % S;
            if (!wait_bar(&bar_full[stage], (it / S) & 1, abort_flag, budget)) {
                *abort_flag = 1;
                if (lane == 0) report_error(prm.hdr, 5u);
                break;
            }
            const int buf = it % Cfg::kBufs;
            if (!wait_bar(&bar_acc_empty[buf], ((it / Cfg::kBufs) & 1) ^ 1, abort_flag, budget)) {
                *abort_flag = 1;
                if (lane == 0) report_error(prm.hdr, 5u);
                break;
            }
            tc_fence_after_sync();
            if (lane == 0) {
                const uint32_t xs = smem_u32(sStage + stage * Cfg::kStageBytes);
                const uint32_t bs = smem_u32(sB);
#pragma unroll
                for (int i = 0; i < SCAN_UP; ++i) {
                    const uint32_t d = tmem_base + buf * (SCAN_UP * N) + i * N;
#pragma unroll
                    for (int ks = 0; ks < P::kMmaPerSlab; ++ks) {
                        const uint64_t da = make_desc(xs + i * P::kSlabBytes + ks * P::kKStepBytes, P::kSbo, P::kLayoutType);
                        const uint64_t db = make_desc(bs + ks * P::kKStepBytes, P::kSbo, P::kLayoutType);
                        if constexpr (P::kIsFloat) mma_f16_ss(d, da, db, idesc, ks != 0);
                        else mma_i8_ss(d, da, db, idesc, ks != 0);
                    }
                }
                tc_commit(&bar_acc_full[buf]);
            }
            __syncwarp();
        }
    } else {
        // =========================== epilogue ===========================
        constexpr int UP = SCAN_UP;
        const int g = warp >> 2;            // warpgroup: iterations g, g + Cfg::kGroups, ...
        const int w = warp & 3;             // unit inside the tile = TMEM lane quarter
        Acc* outp = static_cast<Acc*>(prm.out);
        uint8_t* stg = smem + Cfg::kOutOffset + warp * Cfg::kOutBufs * Cfg::kOutBufBytes;
        const long long nrows_full = prm.n / ROW;
        // first accumulator column of this warp's unit, in its lane quarter
        int obuf = 0;
        bool failed = false;
        // carry handed in by the caller (null: none); only read here, used much later
        const bool has_in = prm.carry_in != nullptr;
        uint32_t base_bits = 0u;
        if (has_in) base_bits = *static_cast<const uint32_t*>(prm.carry_in);

        MMV_T_DECL
        // stages the 32 x 32 block held in r (lane = row) and stores it with one TMA store
        // (exclusive variant: `fmask` = start flags of this lane's row, `prev_last` = inclusive value of the
        //  element in front of the piece)
        auto store_piece = [&](uint32_t (&r)[32], long long prow, uint32_t fmask, Acc prev_last) {
            if constexpr (EX) {
                uint32_t up = __shfl_up_sync(0xffffffffu, r[31], 1);
                if (lane == 0) up = P::to_bits(prev_last);
#pragma unroll
                for (int j = 31; j >= 1; --j) r[j] = ((fmask >> j) & 1u) ? 0u : r[j - 1];
                r[0] = (fmask & 1u) ? 0u : up;
            }
            uint8_t* ob = stg + obuf * Cfg::kOutBufBytes;
            if (lane == 0) tma_store_wait_read<Cfg::kOutBufs - 1>();   // the buffer about to be reused is free again
            __syncwarp();
            MMV_T_MARK(6)
#pragma unroll
            for (int c4 = 0; c4 < 8; ++c4)
                *reinterpret_cast<uint4*>(ob + lane * 128 + ((c4 ^ (lane & 7)) << 4)) =
                    make_uint4(r[4 * c4], r[4 * c4 + 1], r[4 * c4 + 2], r[4 * c4 + 3]);
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0 && prow < nrows_full) {
                tma_store_2d(&tmap_out, ob, 0, static_cast<int>(prow));
                tma_store_commit();
            }
            // the one row that straddles n (n not a multiple of 32) is written with plain stores,
            // read back from the staging buffer
            if (prow + lane == nrows_full) {
                const int cnt = static_cast<int>(prm.n - nrows_full * ROW);
#pragma unroll 1
                for (int j = 0; j < cnt; ++j)
                    reinterpret_cast<uint32_t*>(outp)[nrows_full * ROW + j] =
                        *reinterpret_cast<const uint32_t*>(ob + lane * 128 + ((((j >> 2) ^ (lane & 7)) << 4) | ((j & 3) << 2)));
            }
            obuf = (obuf + 1) % Cfg::kOutBufs;
        };

        for (int k = 0;; ++k) {
            const int it = g + Cfg::kGroups * k;
            if (static_cast<int>(blockIdx.x) + it * static_cast<int>(gridDim.x) >= prm.num_tiles) break;
            const int stage = it % S;
            if (!wait_stage(&stage_iter[stage], it, &bar_full[stage], (it / S) & 1, abort_flag, budget)) { failed = true; break; }
            const int tile = tile_slot[stage];
            MMV_T_MARK(0)

            const int buf = it % Cfg::kBufs;
            const uint32_t taddr = tmem_base + buf * (UP * N) + ((static_cast<uint32_t>(w) * 32u) << 16);
            const long long s = static_cast<long long>(tile) * SPANS_PER_TILE + w;      // this warp's unit

            // ---- flag bytes -> one start mask per row (registers) ----
            uint32_t fm[UP];
            uint32_t pm[UP];
            {
                const uint8_t* fs = sStage + stage * Cfg::kStageBytes + Cfg::kXBytes + w * SCAN_UNIT + lane * ROW;
#pragma unroll
                for (int i = 0; i < UP; ++i) {
                    fm[i] = 0u;
                    if (prm.flags) {
                        const uint4 a = *reinterpret_cast<const uint4*>(fs + i * PIECE);
                        const uint4 b = *reinterpret_cast<const uint4*>(fs + i * PIECE + 16);
                        const uint32_t any = a.x | a.y | a.z | a.w | b.x | b.y | b.z | b.w;
                        fm[i] = any ? flag_bytes_to_mask(a, b) : 0u;
                    }
                    pm[i] = __ballot_sync(0xffffffffu, fm[i] != 0u);
                }
            }
            MMV_T_MARK(1)
            if (!wait_bar(&bar_acc_full[buf], (it / Cfg::kBufs) & 1, abort_flag, budget)) { failed = true; break; }
            MMV_T_MARK(2)
            __syncwarp();
            if (lane == 0) mbar_arrive(&bar_empty[stage]);      // operands consumed, flags in registers
            tc_fence_after_sync();

            // ---- pre-pass: row totals, unit aggregate, publish ----
            uint32_t anyp = 0u;
            int i0 = UP;                    // first piece with a flag
            int istar = 0;                  // ... and the last one
#pragma unroll
            for (int i = UP - 1; i >= 0; --i) {
                anyp |= pm[i];
                if (pm[i]) i0 = i;
            }
#pragma unroll
            for (int i = 0; i < UP; ++i)
                if (pm[i]) istar = i;
            const bool flagged = anyp != 0u;
            // the unit's last start: row lstar of piece istar, position pl in that row (known from the masks alone)
            int lstar = 0, pl = 0;
            if (flagged) {
                uint32_t pms = pm[0], fms = fm[0];
#pragma unroll
                for (int i = 1; i < UP; ++i)
                    if (istar == i) { pms = pm[i]; fms = fm[i]; }
                lstar = 31 - __clz(pms);
                pl = 31 - __clz(__shfl_sync(0xffffffffu, fms, lstar));
            }
            Acc tot[UP];
#pragma unroll
            for (int i = 0; i < UP; ++i) tot[i] = P::from_bits(tmem_ld_32x1(taddr + i * N + (ROW - 1)));
            // What the tail behind the unit's last start needs travels with the same wait.  Floating point: the rows
            // of the last flagged piece themselves (the identity half of the product).  Integers: the prefix in
            // front of that start.
            uint32_t xr[Cfg::kWide ? 32 : 1];
            uint32_t before_bits = 0u;
            if constexpr (Cfg::kWide) {
                if (flagged) tmem_ld_32x32(taddr + istar * N + ROW, xr);
            } else if constexpr (!P::kIsFloat) {
                if (flagged && pl > 0) before_bits = tmem_ld_32x1(taddr + istar * N + (pl - 1));
            }
            tmem_ld_wait();
            Acc tail_unit;
            if (!flagged) {
                Acc t = tot[0];
#pragma unroll
                for (int i = 1; i < UP; ++i) t = P::add(t, tot[i]);
                tail_unit = warp_sum<P>(t);
            } else {
                Acc tots = tot[0];
#pragma unroll
                for (int i = 1; i < UP; ++i)
                    if (istar == i) tots = tot[i];
                Acc after = Acc(0);                            // totals of the rows behind it
#pragma unroll
                for (int i = 0; i < UP; ++i)
                    if (i > istar) after = P::add(after, tot[i]);
                if (static_cast<int>(lane) > lstar) after = P::add(after, tots);
                after = warp_sum<P>(after);
                Acc row_tail;
                if constexpr (Cfg::kWide) {
                    // Floating point addition has no inverse (Section 2 asks for a group): total - prefix(pl - 1)
                    // would leave a small tail behind large values in the rounding of the two prefixes.  The
                    // tail is the sum of the row's own values from its last start on (four partial sums, so
                    // that the 32 additions are not one dependent chain).
                    Acc part[4] = {Acc(0), Acc(0), Acc(0), Acc(0)};
#pragma unroll
                    for (int j = 0; j < 32; ++j)
                        if (j >= pl) part[j & 3] = P::add(part[j & 3], P::from_bits(xr[j]));
                    row_tail = P::add(P::add(part[0], part[1]), P::add(part[2], part[3]));
                } else if constexpr (P::kIsFloat) {
                    // narrow tiles: the same sum, the row's values fetched from memory (only the lane of that row)
                    row_tail = Acc(0);
                    if (static_cast<int>(lane) == lstar)
                        row_tail = row_tail_from_memory<P>(prm.x, s * SCAN_UNIT + istar * PIECE + lstar * ROW, pl, prm.n);
                } else {
                    row_tail = P::sub(tots, P::from_bits(before_bits));      // exact: integer arithmetic modulo 2^32 is a group
                }
                tail_unit = P::add(__shfl_sync(0xffffffffu, row_tail, lstar), after);
            }
            // ---- the four units of the tile exchange their aggregates through shared memory; the carry
            //      chain between CTAs runs over one status word per TILE, published by the first warp ----
            if (lane == 0) {
                agg_slot[(g * 2 + (k & 1)) * SPANS_PER_TILE + w] = (static_cast<uint64_t>(flagged ? 1u : 0u) << 32) | P::to_bits(tail_unit);
                mbar_arrive(&bar_agg[g]);
            }
            if (!wait_bar(&bar_agg[g], k & 1, abort_flag, budget)) { failed = true; break; }
            Acc ex = Acc(0);                  // open-segment sum of the tile's units before this one
            bool exflag = false;              // ... and whether one of them holds a flag
            Acc tail_tile = Acc(0);
            bool flag_tile = false;
#pragma unroll
            for (int j = 0; j < SPANS_PER_TILE; ++j) {
                const uint64_t a = agg_slot[(g * 2 + (k & 1)) * SPANS_PER_TILE + j];
                const bool fj = (a >> 32) != 0u;
                const Acc tj = P::from_bits(static_cast<uint32_t>(a));
                if (j == w) { ex = tail_tile; exflag = flag_tile; }
                tail_tile = fj ? tj : P::add(tail_tile, tj);
                flag_tile = flag_tile || fj;
            }
            const bool need_global = !exflag && (tile != 0 || has_in);      // the carry reaches back past the tile
            const bool skip_publish = (prm.debug_skip_span >= 0) && ((prm.debug_skip_span >> 2) == tile);
            if (w == 0 && lane == 0 && !skip_publish)
                st_relaxed_gpu_u64(prm.status + tile * SCAN_STATUS_STRIDE,
                                   pack_status((flag_tile || (tile == 0 && !has_in)) ? ST_PREFIX : ST_AGG, P::to_bits(tail_tile)));
            MMV_T_MARK(3)

            // ---- main pass: everything that does not need the carry of earlier units ----
            const long long row0 = s * (SCAN_UNIT / ROW);
            Acc run = Acc(0);                 // sum of the open segment inside this unit so far
            Acc last_incl = Acc(0);           // exclusive variant: inclusive value of the last element of the piece before
            uint32_t fm0 = 0u, pm0 = 0u;      // masks of the first flagged piece
            LookbackWindow<SCAN_LB_WORDS> lbw;
            // The first look-back window is requested during the last piece of the main pass: earlier, the
            // predecessor has often not published yet and the poll has to be repeated.  Where most rows hold a
            // segment start, a piece takes less time than the load and the request goes out one piece earlier
            // (n = 2^30, p >= 0.1: 1.27 -> 1.22 ms; done for every tile it costs 1 % at p = 1e-3, 3 % at p = 0).
            const int lb_piece = (UP >= 2 && __popc(pm[0]) > SCAN_LB_DENSE_ROWS) ? UP - 2 : UP - 1;
            // (not unrolled: the body is large and the instruction cache is the scarcer resource)
#pragma unroll 1
            for (int i = 0; i < UP; ++i) {
                // the first look-back window travels while the last piece is processed
                if (i == lb_piece && need_global && w == 0 && tile != 0)
                    lookback_load<SCAN_LB_WORDS, SCAN_STATUS_STRIDE>(prm.status, tile - 1, lbw, base_bits);
                uint32_t fmi = fm[0], pmi = pm[0];
                Acc toti = tot[0];
#pragma unroll
                for (int q = 1; q < UP; ++q)
                    if (i == q) { fmi = fm[q]; pmi = pm[q]; toti = tot[q]; }
                if (i == i0) { fm0 = fmi; pm0 = pmi; }
                uint32_t r[32];
                // a floating-point piece with a start takes its rows themselves (the identity half of the
                // product), every other piece the speculative row prefixes
                if constexpr (Cfg::kWide) tmem_ld_32x32(taddr + i * N + (pmi != 0u ? ROW : 0), r);
                else tmem_ld_32x32(taddr + i * N, r);
                tmem_ld_wait();
                MMV_T_MARK(4)
                if (PLAIN || pmi == 0u) {
                    // no flag in the piece: plain prefix of the row totals, one add per element
                    Acc inc = toti;
#pragma unroll
                    for (int o = 1; o < 32; o <<= 1) {
                        const Acc t = __shfl_up_sync(0xffffffffu, inc, o);
                        if (static_cast<int>(lane) >= o) inc = P::add(t, inc);
                    }
                    // (the exclusive value comes from the lane below, not as inc - toti: no subtraction in floating point)
                    Acc exc = __shfl_up_sync(0xffffffffu, inc, 1);
                    if (lane == 0) exc = Acc(0);
                    const Acc carry_row = P::add(run, exc);
#pragma unroll
                    for (int j = 0; j < 32; ++j) r[j] = P::to_bits(P::add(carry_row, P::from_bits(r[j])));
                    run = P::add(run, __shfl_sync(0xffffffffu, inc, 31));
                } else {
                    if constexpr (P::kIsFloat) {
                        // Reverting the speculation (Lemma A.1: z = prefix(j) - prefix(last start - 1)) is exact only in
                        // a group, and a difference of two fp32 prefixes errs relative to the prefixes, not to the
                        // segment behind them.  The same quantity is therefore formed without a subtraction, as the
                        // running sum of the row's own values since the last start (since the row's beginning in
                        // front of its first start).  One chain of 32 additions: splitting the row into two or four
                        // independent chains measured slower (n = 2^30, every element a start: 1.17 / 1.19 / 1.22 ms),
                        // the elements that continue the part before them cost more than the latency saved.
                        if constexpr (!Cfg::kWide) load_row_from_memory<P>(prm.x, (row0 + i * PIECE_ROWS + lane) * ROW, prm.n, r);
                        Acc since = Acc(0);
#pragma unroll
                        for (int j = 0; j < 32; ++j) {
                            const Acc xj = P::from_bits(r[j]);
                            since = ((fmi >> j) & 1u) ? xj : P::add(since, xj);
                            r[j] = P::to_bits(since);
                        }
                    } else {
                        // revert the speculation inside each row (Lemma A.1); exact modulo 2^32
                        Acc base = Acc(0);
                        uint32_t prev = 0u;
#pragma unroll
                        for (int j = 0; j < 32; ++j) {
                            const bool pj = (fmi >> j) & 1u;
                            if (j > 0) base = pj ? prev : base;
                            prev = r[j];
                            r[j] = P::sub(r[j], base);
                        }
                    }
                    // segmented scan of the row tails across the 32 rows
                    const bool rowflag = fmi != 0u;
                    Acc val = P::from_bits(r[31]);
                    if (lane == 0 && !rowflag) val = P::add(run, val);
                    uint32_t flg = rowflag ? 1u : 0u;
#pragma unroll
                    for (int o = 1; o < 32; o <<= 1) {
                        const Acc tv = __shfl_up_sync(0xffffffffu, val, o);
                        const uint32_t tf = __shfl_up_sync(0xffffffffu, flg, o);
                        if (static_cast<int>(lane) >= o) {
                            if (!flg) val = P::add(tv, val);
                            flg |= tf;
                        }
                    }
                    Acc carry_row = __shfl_up_sync(0xffffffffu, val, 1);
                    if (lane == 0) carry_row = run;
                    run = __shfl_sync(0xffffffffu, val, 31);
                    const int f0 = rowflag ? (__ffs(fmi) - 1) : 32;
#pragma unroll
                    for (int j = 0; j < 32; ++j)
                        if (j < f0) r[j] = P::to_bits(P::add(carry_row, P::from_bits(r[j])));
                }
                MMV_T_MARK(5)
                Acc last_i = Acc(0);
                if constexpr (EX) last_i = P::from_bits(__shfl_sync(0xffffffffu, r[31], 31));
                if (i > i0) {
                    store_piece(r, row0 + i * PIECE_ROWS, fmi, last_incl);       // complete: no element reaches back past a flag
                } else {
                    tmem_st_32x32(taddr + i * N, r);             // parked until the carry is known
                }
                last_incl = last_i;            // (of piece i0 it is final already: its last element lies behind the flag)
                MMV_T_MARK(4)
            }
            tmem_st_wait();

            // ---- look back (most of its latency has been covered by the main pass) ----
            // Only the tile's first warp polls the other CTAs' status words; it hands the tile's carry to
            // its siblings through shared memory (they have passed bar_agg of this tile, so the previous
            // phase of bar_carry is complete and the parity wait cannot alias).
            Acc carry = ex;
            MMV_T_MARK(8)
            if (w == 0) {
                Acc carry_tile = Acc(0);
                if (tile != 0) {
                    if (!lookback<P, SCAN_LB_WORDS, SCAN_STATUS_STRIDE>(prm.status, tile, carry_tile, abort_flag, budget, lbw, true, base_bits)) {
                        if (lane == 0) st_relaxed_gpu_u64(prm.status + tile * SCAN_STATUS_STRIDE, pack_status(ST_ABORT, 0u));
                        failed = true;
                        break;
                    }
                    if (!flag_tile && lane == 0 && !skip_publish)
                        st_relaxed_gpu_u64(prm.status + tile * SCAN_STATUS_STRIDE, pack_status(ST_PREFIX, P::to_bits(P::add(carry_tile, tail_tile))));
                } else if (has_in) {
                    carry_tile = P::from_bits(base_bits);           // the first tile of a later chunk
                    if (!flag_tile && lane == 0 && !skip_publish)
                        st_relaxed_gpu_u64(prm.status + tile * SCAN_STATUS_STRIDE, pack_status(ST_PREFIX, P::to_bits(P::add(carry_tile, tail_tile))));
                }
                if (lane == 0) {
                    carry_slot[g] = P::to_bits(carry_tile);
                    mbar_arrive(&bar_carry[g]);
                }
                carry = carry_tile;
                MMV_T_MARK(10)
            } else if (need_global) {
                if (!wait_bar(&bar_carry[g], k & 1, abort_flag, budget)) { failed = true; break; }
                carry = P::add(P::from_bits(carry_slot[g]), ex);
                MMV_T_MARK(9)
            }

            // ---- parked pieces: add the carry in front of the unit's first flag, store ----
            const int l0 = pm0 ? (__ffs(pm0) - 1) : 32;                       // first flagged row of piece i0
            const int fpos = __ffs(__shfl_sync(0xffffffffu, fm0, l0 & 31)) - 1;  // its first flag
            if (prm.first_start != nullptr && flagged && lane == 0) {
                const long long gidx = s * SCAN_UNIT + i0 * PIECE + l0 * ROW + fpos;       // this unit's first start
                if (gidx < *cta_first) {
                    *cta_first = gidx;
                    atomicMax(prm.first_start, static_cast<unsigned long long>(prm.n - gidx));
                }
            }
            Acc prev_parked = carry;           // exclusive variant: what stands in front of the unit's first element
#pragma unroll 1
            for (int i = 0; i <= i0 && i < UP; ++i) {
                uint32_t r[32];
                tmem_ld_32x32(taddr + i * N, r);
                int limit = 32;
                if (i == i0) limit = (static_cast<int>(lane) < l0) ? 32 : ((static_cast<int>(lane) == l0) ? fpos : 0);
                tmem_ld_wait();
#pragma unroll
                for (int j = 0; j < 32; ++j)
                    if (j < limit) r[j] = P::to_bits(P::add(carry, P::from_bits(r[j])));
                Acc last_p = Acc(0);
                if constexpr (EX) last_p = P::from_bits(__shfl_sync(0xffffffffu, r[31], 31));
                store_piece(r, row0 + i * PIECE_ROWS, i == i0 ? fm0 : 0u, prev_parked);
                prev_parked = last_p;
            }
            MMV_T_MARK(7)

            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(&bar_acc_empty[buf]);
        }
        if (failed) {
            *abort_flag = 1;
            if (lane == 0) report_error(prm.hdr, 5u);
        }
        if (lane == 0) tma_store_wait_all<0>();
        MMV_T_FLUSH()
    }

    tc_fence_before_sync();
    __syncthreads();
    if (warp == Cfg::kMmaWarp) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, Cfg::kTmemCols);
    }
}

}  // namespace mmv
