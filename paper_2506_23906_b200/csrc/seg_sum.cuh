// Segmented sum over CSR offsets (Section 2; Algorithm 4.2 computes the same
// quantity; Section 4.3 remark after Algorithm 4.4 for the offset encoding) and
// CSR SpMV built on it (Algorithm 4.4, Algorithms A.4-A.6), single pass, sm_100a.
//
// Layout ("row-major" view of the paper: x as a ceil(n/s) x s matrix, s = ROW = 32):
//   a warp owns a SPAN of 128 consecutive rows (4096 elements) in four PIECES of
//   32 rows; a TILE is four spans.  Tensor-core product i of a tile multiplies the
//   [128 rows x 32] matrix made of piece i of each span (A operand, brought by one
//   4-D TMA box, K-major, hardware swizzle) with the constant upper-triangular
//   all-ones U_32 (B operand): TMEM lane 32w+l, column j = inclusive prefix at
//   position j of row l of piece i of span w  --  z = MATMUL(x, U_s).
//   Epilogue warps copy their 32 x 32 prefixes to shared memory, scan the 32 row
//   totals with shuffles, and then only touch the segment boundaries: every segment
//   end inside the piece emits  prefix(end) - prefix(start-1)  (the DIFF of
//   Algorithm 4.2 applied to the COMPRESSed speculative scan, but with prefixes that
//   are local to the row or the piece so that magnitudes stay small), segments that
//   cross pieces take the running sum of the open segment, and segments that cross
//   spans take the carry of a decoupled look-back over per-span status words.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include "../../include/mmv.h"
#include "common.cuh"

namespace mmv {

constexpr int SUM_EPI_WARPS = 8;
constexpr int SUM_PRODUCER_WARP = 8;
constexpr int SUM_MMA_WARP = 9;
constexpr int SUM_THREADS = 320;
constexpr int SUM_TMEM_COLS = 256;             // 2 buffers x 4 products x 32 columns

// bf16 values (used for the hi/lo halves of the fp32 products of SpMV): same geometry as fp16.
struct BF16Path : F16Path {
    static constexpr uint32_t kOneBits = 0x3F80u;                       // 1.0 in bf16
    static constexpr uint32_t kFmtBits = (1u << 7) | (1u << 10);        // A and B are bf16
};

template <typename P>
struct SumCfg {
    static constexpr int kStages = 4;
    static constexpr int kBBytes = ROW * P::kRowBytes;               // constant U_32: 32 rows
    static constexpr int kXBytes = PIECES_PER_SPAN * P::kSlabBytes;  // four [128 x 32] operands
    static constexpr int kDumpBytes = PIECE * 4;                     // per epilogue warp
    static constexpr int kStageOffset = 2048;                        // after the constant operand
    static constexpr int kDumpOffset = kStageOffset + kStages * kXBytes;
    static constexpr int kRowpreOffset = kDumpOffset + SUM_EPI_WARPS * kDumpBytes;
    static constexpr int kBarOffset = kRowpreOffset + SUM_EPI_WARPS * PIECE_ROWS * 4;
    static constexpr int kSmemBytes = kBarOffset + 512 + 1024;
    static_assert(kBBytes <= 2048, "constant operand fits its slot");
};

struct SumParams {
    const int32_t* off;          // nseg + 1 offsets
    long long nseg;
    long long n;                 // number of values
    int off_shift;               // boundaries are off[q] << off_shift (1 for the hi/lo pairs of SpMV)
    void* out;                   // nseg results
    int num_tiles;
    const int32_t* tile_q;       // num_tiles + 1: first q with (off[q] << shift) >= tile start
    WorkspaceHeader* hdr;
    uint64_t* status;
    unsigned long long budget_ns;
};

// tile_q[t] = first index q in [0, nseg] with (off[q] << shift) >= t * TILE, nseg + 1 if none.
// One warp per tile boundary, 32-ary search.
// The same launch validates the offsets (non-decreasing, inside [0, n]) and records
// MMV_ERR_BAD_SEGMENTS otherwise; the main kernel never indexes outside its tile whatever they hold.
__global__ void partition_offsets_kernel(const int32_t* __restrict__ off, long long nseg, int shift, int num_tiles,
                                         int32_t* __restrict__ tile_q, long long n, WorkspaceHeader* hdr) {
    {
        const long long stride = static_cast<long long>(gridDim.x) * blockDim.x;
        bool bad = false;
        for (long long q = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; q < nseg; q += stride) {
            const long long a = static_cast<long long>(off[q]) << shift, b = static_cast<long long>(off[q + 1]) << shift;
            bad |= (a > b) || (a < 0) || (b > n);
        }
        if (bad) report_error(hdr, 4u);
    }
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (warp > num_tiles) return;
    const long long target = static_cast<long long>(warp) * TILE;
    long long lo = 0, hi = nseg + 1;
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
    if (lane == 0) tile_q[warp] = static_cast<int32_t>(lo);
}

template <typename P>
__global__ void __launch_bounds__(SUM_THREADS, 1)
seg_sum_kernel(const __grid_constant__ CUtensorMap tmap_x, const void* __restrict__ xg, const SumParams prm) {
    using Acc = typename P::Acc;
    using Cfg = SumCfg<P>;
    constexpr int S = Cfg::kStages;

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* sB = smem;
    uint8_t* sStage = smem + Cfg::kStageOffset;
    uint64_t* bar_full = reinterpret_cast<uint64_t*>(smem + Cfg::kBarOffset);
    uint64_t* bar_empty = bar_full + S;
    uint64_t* bar_acc_full = bar_empty + S;
    uint64_t* bar_acc_empty = bar_acc_full + 2;
    int* tile_slot = reinterpret_cast<int*>(bar_acc_empty + 2);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tile_slot + S);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5;
    const uint32_t lane = lane_id();
    const uint64_t budget = prm.budget_ns;

    if (threadIdx.x == 0) {
        for (int i = 0; i < S; ++i) {
            mbar_init(&bar_full[i], 1);
            mbar_init(&bar_empty[i], 1);      // released by the MMA warp's commit
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(&bar_acc_full[i], 1);
            mbar_init(&bar_acc_empty[i], 4);
        }
        *abort_flag = 0;
        mbar_fence_init();
    }
    if (warp == SUM_MMA_WARP) {
        tmem_alloc(tmem_slot, SUM_TMEM_COLS);
        tmem_relinquish();
    }
    if (warp == SUM_PRODUCER_WARP && lane == 0) tma_prefetch_desc(&tmap_x);
    {
        // constant B = U_32 stored K-major: row nn (output position), element k (input position): 1 iff k <= nn
        constexpr int kVecPerRow = P::kRowBytes / 16;
        constexpr int kElemPerVec = 16 / P::kElemBytes;
        for (int v = threadIdx.x; v < ROW * kVecPerRow; v += SUM_THREADS) {
            const int nn = v / kVecPerRow, cv = v % kVecPerRow;
            uint32_t words[4] = {0u, 0u, 0u, 0u};
#pragma unroll
            for (int e = 0; e < kElemPerVec; ++e) {
                const int k = cv * kElemPerVec + e;
                if (k <= nn) {
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

    if (warp == SUM_PRODUCER_WARP) {
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
            if (lane == 0) tile_slot[stage] = tile;
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
                // ragged last tile: plain loads with zero fill past n (MATMUL zero-pads its operand)
                const long long cnt = prm.n - tbase;
                constexpr int kElemPerVec = 16 / P::kElemBytes;
                const uint8_t* xt = static_cast<const uint8_t*>(xg) + tbase * P::kElemBytes;
                for (int v = lane; v < TILE / kElemPerVec; v += 32) {
                    const int e0 = v * kElemPerVec;
                    uint4 xv = make_uint4(0u, 0u, 0u, 0u);
                    if (e0 + kElemPerVec <= cnt) {
                        xv = *reinterpret_cast<const uint4*>(xt + static_cast<size_t>(e0) * P::kElemBytes);
                    } else if (e0 < cnt) {
                        __align__(16) uint8_t tmp[16];
                        for (int b = 0; b < 16; ++b)
                            tmp[b] = (e0 + b / P::kElemBytes < cnt) ? xt[static_cast<size_t>(e0) * P::kElemBytes + b] : uint8_t(0);
                        xv = *reinterpret_cast<const uint4*>(tmp);
                    }
                    const int w = e0 / SPAN, i = (e0 % SPAN) / PIECE, l = (e0 % PIECE) / ROW, j0 = e0 % ROW;
                    *reinterpret_cast<uint4*>(xs + i * P::kSlabBytes +
                                              swz_offset<P::kRowBytes>(w * PIECE_ROWS + l, j0 * P::kElemBytes)) = xv;
                }
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
    } else if (warp == SUM_MMA_WARP) {
        // =========================== MMA issuer ===========================
        constexpr uint32_t idesc = P::kIsFloat ? (make_idesc_f16_f32(128, ROW) | P::kFmtBits)
                                               : make_idesc_s8_s32(128, ROW);
        for (int it = 0;; ++it) {
            const int stage = it % S;
            if (!wait_bar(&bar_full[stage], (it / S) & 1, abort_flag, budget)) {
                *abort_flag = 1;
                if (lane == 0) report_error(prm.hdr, 5u);
                break;
            }
            if (tile_slot[stage] < 0) break;
            const int acc = it & 1;
            if (!wait_bar(&bar_acc_empty[acc], ((it >> 1) & 1) ^ 1, abort_flag, budget)) {
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
                    const uint32_t d = tmem_base + acc * (PIECES_PER_SPAN * ROW) + i * ROW;
#pragma unroll
                    for (int ks = 0; ks < P::kMmaPerSlab; ++ks) {
                        const uint64_t da = make_desc(xs + i * P::kSlabBytes + ks * P::kKStepBytes, P::kSbo, P::kLayoutType);
                        const uint64_t db = make_desc(bs + ks * P::kKStepBytes, P::kSbo, P::kLayoutType);
                        if constexpr (P::kIsFloat) mma_f16_ss(d, da, db, idesc, ks != 0);
                        else mma_i8_ss(d, da, db, idesc, ks != 0);
                    }
                }
                tc_commit(&bar_empty[stage]);       // operands consumed: the stage may be refilled
                tc_commit(&bar_acc_full[acc]);
            }
            __syncwarp();
        }
    } else {
        // =========================== epilogue ===========================
        const int g = warp >> 2;
        const int w = warp & 3;
        Acc* outp = static_cast<Acc*>(prm.out);
        uint8_t* dump = smem + Cfg::kDumpOffset + warp * Cfg::kDumpBytes;      // [32 rows][32] swizzled by row
        Acc* rowpre = reinterpret_cast<Acc*>(smem + Cfg::kRowpreOffset) + warp * PIECE_ROWS;
        const int sh = prm.off_shift;
        const long long nq = prm.nseg + 1;
        // inclusive prefix inside the piece at element offset j (0..1023); j = -1 gives 0
        auto piece_prefix = [&](int j, Acc& rowpart, int& row) -> Acc {
            row = j >> 5;
            const int pos = j & 31;
            rowpart = *reinterpret_cast<const Acc*>(dump + row * 128 + ((((pos >> 2) ^ (row & 7)) << 4) | ((pos & 3) << 2)));
            return P::add(rowpre[row], rowpart);
        };
        for (int it = g;; it += 2) {
            const int stage = it % S;
            if (!wait_bar(&bar_full[stage], (it / S) & 1, abort_flag, budget)) {
                *abort_flag = 1;
                if (lane == 0) report_error(prm.hdr, 5u);
                break;
            }
            const int tile = tile_slot[stage];
            if (tile < 0) break;
            if (!wait_bar(&bar_acc_full[g], (it >> 1) & 1, abort_flag, budget)) {
                *abort_flag = 1;
                if (lane == 0) report_error(prm.hdr, 5u);
                break;
            }
            tc_fence_after_sync();

            const long long s = static_cast<long long>(tile) * SPANS_PER_TILE + w;
            const long long sbase = s * SPAN;
            const uint32_t taddr = tmem_base + g * (PIECES_PER_SPAN * ROW) + ((static_cast<uint32_t>(w) * 32u) << 16);

            // first boundary index of this span: first q in the tile's range with bnd(q) >= sbase
            long long q;
            {
                long long lo = prm.tile_q[tile], hi = prm.tile_q[tile + 1];
                while (hi > lo) {
                    const long long len = hi - lo, step = (len + 31) / 32;
                    const long long bstart = lo + lane * step;
                    long long bend = bstart + step;
                    if (bend > hi) bend = hi;
                    bool pred = false;
                    if (bstart < hi) pred = (static_cast<long long>(prm.off[bend - 1]) << sh) >= sbase;
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
                q = lo;
            }

            Acc run = Acc(0);              // sum of the open segment inside this span so far
            bool seen = false;             // a segment start lies inside this span
            long long def_r = -1;          // segment that began before the span and ends inside it
            Acc def_val = Acc(0);
            uint32_t r[32];
#pragma unroll 1
            for (int i = 0; i < PIECES_PER_SPAN; ++i) {
                const long long pbase = sbase + i * PIECE;
                tmem_ld_32x32(taddr + i * ROW, r);
                tmem_ld_wait();
                // row prefixes -> shared memory (16-byte chunks rotated by the row to avoid bank conflicts)
#pragma unroll
                for (int c4 = 0; c4 < 8; ++c4)
                    *reinterpret_cast<uint4*>(dump + lane * 128 + ((c4 ^ (lane & 7)) << 4)) =
                        make_uint4(r[4 * c4], r[4 * c4 + 1], r[4 * c4 + 2], r[4 * c4 + 3]);
                // exclusive scan of the 32 row totals
                const Acc tot = P::from_bits(r[31]);
                Acc inc = tot;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const Acc t = __shfl_up_sync(0xffffffffu, inc, o);
                    if (static_cast<int>(lane) >= o) inc = P::add(t, inc);
                }
                rowpre[lane] = P::sub(inc, tot);
                const Acc piece_total = __shfl_sync(0xffffffffu, inc, 31);
                __syncwarp();

                // boundaries with pbase <= bnd(q) <= pbase + PIECE, 32 at a time (sorted, so the
                // ones of this piece are a prefix of every batch)
                const long long pend = pbase + PIECE;
                bool piece_has_start = false;
                long long last_start = -1;
                long long qp = q;              // batch pointer
                int advance = 0;               // boundaries strictly before pend: consumed for good
                while (true) {
                    const long long qi = qp + lane;
                    long long b = -1;
                    if (qi < nq) b = static_cast<long long>(prm.off[qi]) << sh;
                    const bool in_piece = (qi < nq) && (b <= pend);
                    const unsigned inm = __ballot_sync(0xffffffffu, in_piece);
                    const int cnt = (inm == 0xffffffffu) ? 32 : (__ffs(~inm) - 1);
                    const bool mine = static_cast<int>(lane) < cnt;
                    bool deferred = false;
                    Acc val = Acc(0);
                    // as the END of segment qi-1: bnd in (pbase, pend], or 0 for leading empty segments
                    if (mine && qi >= 1 && (b > pbase || (pbase == 0 && b == 0))) {
                        const long long sb = static_cast<long long>(prm.off[qi - 1]) << sh;
                        if (sb > b || sb < 0 || b > prm.n) {
                            report_error(prm.hdr, 4u);
                        } else {
                            if (b != sb) {
                                Acc ep, sp = Acc(0);
                                int erow, srow;
                                const Acc e_full = piece_prefix(static_cast<int>(b - 1 - pbase), ep, erow);
                                if (sb >= pbase) {
                                    Acc s_full = Acc(0);
                                    if (sb > pbase) s_full = piece_prefix(static_cast<int>(sb - 1 - pbase), sp, srow);
                                    if (static_cast<int>((sb - pbase) >> 5) == erow)
                                        val = ((sb - pbase) & 31) ? P::sub(ep, sp) : ep;   // inside one row
                                    else
                                        val = P::sub(e_full, s_full);
                                } else {
                                    val = P::add(run, e_full);
                                    deferred = sb < sbase;
                                }
                            }
                            if (!deferred) outp[qi - 1] = val;
                        }
                    }
                    const unsigned dm = __ballot_sync(0xffffffffu, deferred);
                    if (dm) {
                        const int src = __ffs(dm) - 1;
                        def_r = __shfl_sync(0xffffffffu, qi, src) - 1;
                        def_val = __shfl_sync(0xffffffffu, val, src);
                    }
                    // as a START: bnd in [pbase, pend)
                    const bool is_start = mine && (b >= pbase) && (b < pend);
                    const unsigned sm = __ballot_sync(0xffffffffu, is_start);
                    if (sm) {
                        piece_has_start = true;
                        last_start = __shfl_sync(0xffffffffu, b, 31 - __clz(sm));
                    }
                    advance += __popc(__ballot_sync(0xffffffffu, mine && (b < pend)));
                    qp += cnt;
                    if (cnt < 32) break;
                }
                q += advance;
                if (piece_has_start) {
                    Acc sp2;
                    int srow2;
                    Acc before = Acc(0);
                    if (last_start > pbase) before = piece_prefix(static_cast<int>(last_start - 1 - pbase), sp2, srow2);
                    run = P::sub(piece_total, before);
                    seen = true;
                } else {
                    run = P::add(run, piece_total);
                }
                __syncwarp();
            }

            // ---- publish, look back, emit the segment that began before this span ----
            if (s == 0) {
                if (lane == 0) st_relaxed_gpu_u64(prm.status + s, pack_status(ST_PREFIX, P::to_bits(run)));
                if (def_r >= 0 && lane == 0) outp[def_r] = def_val;
            } else {
                if (lane == 0) st_relaxed_gpu_u64(prm.status + s, pack_status(seen ? ST_PREFIX : ST_AGG, P::to_bits(run)));
                Acc carry = Acc(0);
                if (!seen || def_r >= 0) {
                    LookbackWindow lbw;
                    if (!lookback<P>(prm.status, s, carry, abort_flag, budget, lbw, false)) {
                        *abort_flag = 1;
                        if (lane == 0) {
                            report_error(prm.hdr, 5u);
                            st_relaxed_gpu_u64(prm.status + s, pack_status(ST_ABORT, 0u));
                        }
                        break;
                    }
                    if (!seen && lane == 0)
                        st_relaxed_gpu_u64(prm.status + s, pack_status(ST_PREFIX, P::to_bits(P::add(carry, run))));
                    if (def_r >= 0 && lane == 0) outp[def_r] = P::add(carry, def_val);
                }
            }

            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(&bar_acc_empty[g]);
        }
    }

    tc_fence_before_sync();
    __syncthreads();
    if (warp == SUM_MMA_WARP) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, SUM_TMEM_COLS);
    }
}

}  // namespace mmv
