// Single-pass segmented inclusive scan (Problem 2.1, Eq. 1) for sm_100a.
//
// Per tile of TILE = 4 x 128 x 32 elements:
//   producer warp   TMA: four [128 rows x 32 elements] boxes of x (one per span,
//                   K-major, hardware swizzle) and the tile's flag bytes.
//   MMA warp        tcgen05.mma  D[128 x 128] = A . B^T  with B the x boxes and A the
//                   constant block-diagonal lower-triangular all-ones matrix
//                   (I_4 (x) L_32): TMEM lane 32w+l, column c holds the inclusive
//                   prefix at position l of row c of span w -- the speculative
//                   block scan MATMUL(x, U_s) of Algorithm A.1 (BlockSegScan),
//                   transposed so that a warp's lanes are consecutive elements.
//   epilogue warps  (two warpgroups on alternating tiles) per row: ballot of the flag
//                   bytes -> boundary mask; revert the speculation by subtracting the
//                   prefix just before the element's segment start (Lemma A.1), one
//                   shuffle; chain the row tails through the span; publish the span's
//                   aggregate, look back over earlier spans (decoupled look-back:
//                   the recursion of Section 4.2 folded into one pass), add the carry
//                   to the elements before the span's first flag (UpdateFirstSegment of
//                   Algorithm A.1) and store with 128-byte coalesced warp stores.
#pragma once
#include "common.cuh"

namespace mmv {

constexpr int SCAN_EPI_WARPS = 8;
constexpr int SCAN_PRODUCER_WARP = 8;
constexpr int SCAN_MMA_WARP = 9;
constexpr int SCAN_THREADS = 320;
constexpr int SCAN_TMEM_COLS = 256;          // two 128-column accumulators

template <typename P>
struct ScanCfg {
    static constexpr int kStages = P::kIsFloat ? 4 : 6;
    static constexpr int kABytes = 4 * P::kSlabBytes;
    static constexpr int kXBytes = 4 * P::kSlabBytes;
    static constexpr int kStageBytes = kXBytes + FLAG_TILE_BYTES;
    static constexpr int kBarOffset = kABytes + kStages * kStageBytes;
    static constexpr int kSmemBytes = kBarOffset + 512 + 1024;   // + barriers/slots + alignment slack
};

struct ScanParams {
    const void* x;
    const uint8_t* flags;
    void* out;
    long long n;
    int num_tiles;
    WorkspaceHeader* hdr;
    uint64_t* status;            // one word per span
    unsigned long long budget_ns;
    long long debug_skip_span;   // test hook: this span never publishes (-1 = off)
};

// Bounded mbarrier wait that also gives up when another role of the CTA has aborted.
__device__ __forceinline__ bool wait_bar(uint64_t* bar, uint32_t parity, volatile int* abort_flag,
                                         uint64_t budget_ns) {
    if (mbar_try_wait(bar, parity)) return true;
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

// Decoupled look-back: exclusive carry of span s = running sum of the open segment at the
// end of span s-1.  Walks predecessor status words, 32 per step, adding aggregates until it
// meets a span that published an inclusive prefix.  Bounded: returns false on time-out or if
// a predecessor aborted.
template <typename P>
__device__ __forceinline__ bool lookback(const uint64_t* status, long long s, typename P::Acc& carry,
                                         volatile int* abort_flag, uint64_t budget_ns) {
    using Acc = typename P::Acc;
    const uint32_t lane = lane_id();
    Acc acc = Acc(0);
    long long idx = s - 1;
    uint64_t t0 = global_timer_ns();
    uint32_t polls = 0;
    while (true) {
        const long long my = idx - lane;
        const uint64_t wv = (my >= 0) ? ld_relaxed_gpu_u64(status + my) : pack_status(ST_PREFIX, 0u);
        const uint32_t st = static_cast<uint32_t>(wv >> 32);
        const uint32_t rdy = __ballot_sync(0xffffffffu, st != ST_NONE);
        const uint32_t pm = __ballot_sync(0xffffffffu, st == ST_PREFIX);
        const uint32_t xm = __ballot_sync(0xffffffffu, st == ST_ABORT);
        const uint32_t term = pm | xm;
        uint32_t need = 0xffffffffu;
        int t = 32;
        if (term) {
            t = __ffs(term) - 1;
            need = (t == 31) ? 0xffffffffu : ((2u << t) - 1u);
        }
        if ((rdy & need) == need) {
            if (term && ((xm >> t) & 1u)) return false;
            Acc v = ((need >> lane) & 1u) ? P::from_bits(static_cast<uint32_t>(wv)) : Acc(0);
            v = warp_sum<P>(v);
            acc = P::add(v, acc);
            if (term) {
                carry = acc;
                return true;
            }
            idx -= 32;
            t0 = global_timer_ns();
            continue;
        }
        if ((++polls & 7u) == 0u) {
            if (*abort_flag) return false;
            if (global_timer_ns() - t0 > budget_ns) return false;
        }
    }
}

template <typename P>
__global__ void __launch_bounds__(SCAN_THREADS, 1)
seg_scan_kernel(const __grid_constant__ CUtensorMap tmap_x, const ScanParams prm) {
    using Acc = typename P::Acc;
    using Cfg = ScanCfg<P>;
    constexpr int S = Cfg::kStages;

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* sA = smem;
    uint8_t* sStage = smem + Cfg::kABytes;
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

    // ---- set-up: barriers, TMEM, the constant operand A = I_4 (x) L_32 ----
    if (threadIdx.x == 0) {
        for (int i = 0; i < S; ++i) {
            mbar_init(&bar_full[i], 1);
            mbar_init(&bar_empty[i], 4);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(&bar_acc_full[i], 1);
            mbar_init(&bar_acc_empty[i], 4);
        }
        *abort_flag = 0;
        mbar_fence_init();
    }
    if (warp == SCAN_MMA_WARP) {
        tmem_alloc(tmem_slot, SCAN_TMEM_COLS);
        tmem_relinquish();
    }
    if (warp == SCAN_PRODUCER_WARP && lane == 0) tma_prefetch_desc(&tmap_x);
    {
        // slab w, row m, element k of the row: 1 iff m belongs to block w and k <= m mod 32
        constexpr int kVecPerRow = P::kRowBytes / 16;
        constexpr int kElemPerVec = 16 / P::kElemBytes;
        for (int v = threadIdx.x; v < 4 * NCOL * kVecPerRow; v += SCAN_THREADS) {
            const int w = v / (NCOL * kVecPerRow);
            const int m = (v / kVecPerRow) % NCOL;
            const int cv = v % kVecPerRow;
            uint32_t words[4] = {0u, 0u, 0u, 0u};
            if ((m >> 5) == w) {
#pragma unroll
                for (int e = 0; e < kElemPerVec; ++e) {
                    const int k = cv * kElemPerVec + e;
                    if (k <= (m & 31)) {
                        if constexpr (P::kIsFloat) words[e >> 1] |= 0x3C00u << ((e & 1) * 16);   // fp16 1.0
                        else words[e >> 2] |= 1u << ((e & 3) * 8);
                    }
                }
            }
            uint4* dst = reinterpret_cast<uint4*>(sA + w * P::kSlabBytes + swz_offset<P::kRowBytes>(m, cv * 16));
            *dst = make_uint4(words[0], words[1], words[2], words[3]);
        }
    }
    fence_proxy_async_smem();
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == SCAN_PRODUCER_WARP) {
        // =========================== producer ===========================
        int it = 0, sentinels = 0;
        bool ok = true;
        while (ok) {
            const int stage = it % S;
            if (!wait_bar(&bar_empty[stage], ((it / S) & 1) ^ 1, abort_flag, budget)) { ok = false; break; }
            int tile = 0;
            if (lane == 0) tile = static_cast<int>(atomicAdd(&prm.hdr->tile_counter, 1u));
            tile = __shfl_sync(0xffffffffu, tile, 0);
            if (tile >= prm.num_tiles) tile = -1;
            if (lane == 0) tile_slot[stage] = tile;
            if (tile < 0) {
                __syncwarp();
                if (lane == 0) mbar_arrive(&bar_full[stage]);
                ++it;
                if (++sentinels == 2) break;
                continue;
            }
            uint8_t* xs = sStage + stage * Cfg::kStageBytes;
            uint8_t* fs = xs + Cfg::kXBytes;
            const long long tbase = static_cast<long long>(tile) * TILE;
            if (tbase + TILE <= prm.n) {
                if (lane == 0) {
                    mbar_arrive_expect_tx(&bar_full[stage], Cfg::kXBytes + FLAG_TILE_BYTES);
#pragma unroll
                    for (int w = 0; w < 4; ++w)
                        tma_load_2d(xs + w * P::kSlabBytes, &tmap_x, &bar_full[stage], 0, tile * (TILE / CHUNK) + w * NCOL);
                    tma_load_1d(fs, prm.flags + tbase, FLAG_TILE_BYTES, &bar_full[stage]);
                }
            } else {
                // ragged last tile: plain loads, zero fill past n (the paper zero-pads MATMUL's operand)
                const long long cnt = prm.n - tbase;
                for (int v = lane; v < TILE / 16; v += 32) {
                    const int e0 = v * 16;
                    uint4 fv = make_uint4(0u, 0u, 0u, 0u);
                    if (e0 + 16 <= cnt) {
                        fv = *reinterpret_cast<const uint4*>(prm.flags + tbase + e0);
                    } else if (e0 < cnt) {
                        uint8_t tmp[16];
                        for (int e = 0; e < 16; ++e) tmp[e] = (e0 + e < cnt) ? prm.flags[tbase + e0 + e] : uint8_t(0);
                        fv = *reinterpret_cast<const uint4*>(tmp);
                    }
                    *reinterpret_cast<uint4*>(fs + e0) = fv;
                }
                constexpr int kElemPerVec = 16 / P::kElemBytes;
                const uint8_t* xg = static_cast<const uint8_t*>(prm.x) + tbase * P::kElemBytes;
                for (int v = lane; v < TILE / kElemPerVec; v += 32) {
                    const int e0 = v * kElemPerVec;
                    uint4 xv = make_uint4(0u, 0u, 0u, 0u);
                    if (e0 + kElemPerVec <= cnt) {
                        xv = *reinterpret_cast<const uint4*>(xg + static_cast<size_t>(e0) * P::kElemBytes);
                    } else if (e0 < cnt) {
                        __align__(16) uint8_t tmp[16];
                        for (int b = 0; b < 16; ++b)
                            tmp[b] = (e0 + b / P::kElemBytes < cnt) ? xg[static_cast<size_t>(e0) * P::kElemBytes + b] : uint8_t(0);
                        xv = *reinterpret_cast<const uint4*>(tmp);
                    }
                    const int w = e0 / SPAN, c = (e0 % SPAN) / CHUNK, j0 = e0 % CHUNK;
                    *reinterpret_cast<uint4*>(xs + w * P::kSlabBytes + swz_offset<P::kRowBytes>(c, j0 * P::kElemBytes)) = xv;
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
        // wait (bounded) for copies still in flight before the CTA may exit
        for (int k = (it > S ? it - S : 0); k < it; ++k) mbar_wait(&bar_full[k % S], (k / S) & 1, 2000000ull);
    } else if (warp == SCAN_MMA_WARP) {
        // =========================== MMA issuer ===========================
        constexpr uint32_t idesc = P::kIsFloat ? make_idesc_f16_f32(128, NCOL) : make_idesc_s8_s32(128, NCOL);
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
                const uint32_t xs = smem_u32(sStage + stage * Cfg::kStageBytes);
                const uint32_t as = smem_u32(sA);
                const uint32_t d = tmem_base + acc * NCOL;
#pragma unroll
                for (int w = 0; w < 4; ++w) {
#pragma unroll
                    for (int ks = 0; ks < P::kMmaPerSlab; ++ks) {
                        const uint32_t off = w * P::kSlabBytes + ks * P::kKStepBytes;
                        const uint64_t da = make_desc(as + off, P::kSbo, P::kLayoutType);
                        const uint64_t db = make_desc(xs + off, P::kSbo, P::kLayoutType);
                        if constexpr (P::kIsFloat) mma_f16_ss(d, da, db, idesc, (w | ks) != 0);
                        else mma_i8_ss(d, da, db, idesc, (w | ks) != 0);
                    }
                }
                tc_commit(&bar_acc_full[acc]);
            }
            __syncwarp();
        }
    } else {
        // =========================== epilogue ===========================
        const int g = warp >> 2;            // warpgroup: handles iterations it = g, g+2, ...
        const int w = warp & 3;             // span inside the tile = TMEM lane block
        const uint32_t lanemask_le = 0xffffffffu >> (31u - lane);
        Acc* outp = static_cast<Acc*>(prm.out);
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

            const uint8_t* xs = sStage + stage * Cfg::kStageBytes + w * P::kSlabBytes;
            const uint8_t* fs = sStage + stage * Cfg::kStageBytes + Cfg::kXBytes + w * SPAN;
            const long long s = static_cast<long long>(tile) * SPANS_PER_TILE + w;
            const long long base = s * SPAN;
            const long long rem = prm.n - base;           // elements of this span that exist (may be <= 0)
            const int lim = rem >= SPAN ? SPAN : (rem > 0 ? static_cast<int>(rem) : 0);
            const uint32_t taddr = tmem_base + g * NCOL + ((static_cast<uint32_t>(w) * 32u) << 16);

            // ---- pass A: local segmented scan of the span ----
            Acc run = Acc(0);                 // sum of the open segment so far (uniform)
            bool seen = false;                // a flag occurred in this span (uniform)
            int ffc = NCOL;                   // chunk of the span's first flag
            uint32_t ffm = 0u;                // flag mask of that chunk
            int ndef = 0;                     // leading groups whose store waits for the carry
            uint32_t r[32];
#pragma unroll 1
            for (int gg = 0; gg < NCOL / 32; ++gg) {
                tmem_ld_32x32(taddr + gg * 32, r);
                tmem_ld_wait();
                const bool defer = !seen;
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    const int c = gg * 32 + j;
                    const uint32_t fb = fs[c * CHUNK + lane];
                    uint32_t m = __ballot_sync(0xffffffffu, fb != 0u);
                    if (s == 0 && c == 0) m |= 1u;        // element 0 always opens a segment
                    const Acc xb = P::from_bits(r[j]);
                    const uint32_t le = m & lanemask_le;
                    const int p = 31 - __clz(le);         // last flag at or before this lane, -1 if none
                    const Acc v = __shfl_sync(0xffffffffu, xb, (p - 1) & 31);
                    Acc zl = (p > 0) ? P::sub(xb, v) : xb;
                    if constexpr (P::kIsFloat) {
                        // the first element of a segment is the input value itself, exactly
                        if ((m >> lane) & 1u) {
                            const __half hx = *reinterpret_cast<const __half*>(xs + swz_offset<P::kRowBytes>(c, lane * 2));
                            zl = __half2float(hx);
                        }
                    }
                    const Acc tail = __shfl_sync(0xffffffffu, zl, 31);
                    const Acc z = (le == 0u) ? P::add(run, zl) : zl;
                    run = (m != 0u) ? tail : P::add(run, tail);
                    if (m != 0u && !seen) {
                        seen = true;
                        ffc = c;
                        ffm = m;
                    }
                    r[j] = P::to_bits(z);
                    if (!defer) {
                        if (c * CHUNK + static_cast<int>(lane) < lim) outp[base + c * CHUNK + lane] = z;
                    }
                }
                if (defer) {
                    tmem_st_32x32(taddr + gg * 32, r);
                    ndef = gg + 1;
                }
            }
            tmem_st_wait();

            // ---- publish, look back, publish ----
            Acc carry = Acc(0);
            bool ok = true;
            const bool skip_publish = (s == prm.debug_skip_span);
            if (s == 0) {
                if (lane == 0 && !skip_publish) st_relaxed_gpu_u64(prm.status + s, pack_status(ST_PREFIX, P::to_bits(run)));
            } else {
                if (lane == 0 && !skip_publish)
                    st_relaxed_gpu_u64(prm.status + s, pack_status(seen ? ST_PREFIX : ST_AGG, P::to_bits(run)));
                ok = lookback<P>(prm.status, s, carry, abort_flag, budget);
                if (!ok) {
                    *abort_flag = 1;
                    if (lane == 0) {
                        report_error(prm.hdr, 5u);
                        st_relaxed_gpu_u64(prm.status + s, pack_status(ST_ABORT, 0u));
                    }
                    break;
                }
                if (!seen && lane == 0 && !skip_publish)
                    st_relaxed_gpu_u64(prm.status + s, pack_status(ST_PREFIX, P::to_bits(P::add(carry, run))));
            }

            // ---- pass B: add the carry before the span's first flag, store the deferred groups ----
#pragma unroll 1
            for (int gg = 0; gg < ndef; ++gg) {
                tmem_ld_32x32(taddr + gg * 32, r);
                tmem_ld_wait();
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    const int c = gg * 32 + j;
                    Acc z = P::from_bits(r[j]);
                    const bool pre = (c < ffc) || (c == ffc && (ffm & lanemask_le) == 0u);
                    if (pre) z = P::add(carry, z);
                    if (c * CHUNK + static_cast<int>(lane) < lim) outp[base + c * CHUNK + lane] = z;
                }
            }

            // ---- release the accumulator and the shared-memory stage ----
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(&bar_acc_empty[g]);
                mbar_arrive(&bar_empty[stage]);
            }
        }
    }

    tc_fence_before_sync();
    __syncthreads();
    if (warp == SCAN_MMA_WARP) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, SCAN_TMEM_COLS);
    }
}

}  // namespace mmv
