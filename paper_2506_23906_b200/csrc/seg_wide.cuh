// Segmented inclusive scan of int8 values with int64 results: Eq. (1) without the wrap of the int32 path
// (|z| <= 128 n needs more than 32 bits from n = 2^24 on).  The tensor-core scan accumulates in int32 and
// chains its tiles through 32-bit status payloads; this variant keeps 32-bit arithmetic where it is exact --
// inside a 2048-element tile no sum exceeds 2^18 -- and carries 64 bits between tiles.  It runs on the CUDA
// cores with the structure of the running maximum / minimum (seg_minmax.cuh): a thread scans 16 consecutive
// elements, a segmented warp scan whose limits come from one ballot and the same scan over the four warp
// aggregates give the sums inside the tile (CTAs of 128 threads, eight per SM: with 256 threads and 4096-element
// tiles the CTA-wide barriers cost 7 % where segment starts are frequent); tiles are handed out by an atomic counter and chained by a
// single-pass decoupled look-back over one status word per tile (one word per 32-byte sector); only the
// elements in front of the tile's first segment start need the carry, so all others leave while the first warp
// still looks back; inputs arrive by 16-byte asynchronous copies into one of two shared-memory buffers, and a
// tile without a start publishes the aggregate of the tile it has prefetched before it looks back (so that a
// slow look-back never holds up the words that the tiles behind it wait for).  Integer sums: results are exact.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>
#include "common.cuh"
#include "ptx.cuh"

namespace mmv {

#ifndef MMV_WD_THREADS
#define MMV_WD_THREADS 128
#endif
constexpr int WD_THREADS = MMV_WD_THREADS;
constexpr int WD_WARPS = WD_THREADS / 32;
constexpr int WD_PER_THREAD = 16;
constexpr int WD_TILE = WD_THREADS * WD_PER_THREAD;      // 2048 elements: one pass of the CTA, one status word
static_assert(WD_TILE <= 12288, "the buffers are static shared memory");
constexpr int WD_CTAS_PER_SM = 1024 / WD_THREADS;
constexpr int WD_STATUS_STRIDE = 4;                       // status words of consecutive tiles: one per 32-byte sector

struct WideParams {
    const int8_t* x;            // n values
    const uint8_t* flags;       // n start flags, or null: one segment
    long long* out;             // n results
    long long n;
    long long num_tiles;
    WorkspaceHeader* hdr;       // tile_counter and error, cleared by the caller
    uint64_t* status;           // WD_STATUS_STRIDE words per tile, cleared by the caller
    unsigned long long budget_ns;
    long long debug_skip_tile;  // test hook: this tile never publishes a status word (-1: none)
};

// Status word: state in bits 0-1 (ST_NONE = 0: cleared memory), the value in the 62 bits above it.
__device__ __forceinline__ uint64_t wide_pack(uint64_t state, long long v) { return (static_cast<uint64_t>(v) << 2) | state; }
__device__ __forceinline__ uint32_t wide_state(uint64_t w) { return static_cast<uint32_t>(w & 3u); }
__device__ __forceinline__ long long wide_value(uint64_t w) { return static_cast<long long>(w) >> 2; }

// Bit i of the result: byte i of w is not zero.
__device__ __forceinline__ uint32_t wide_nonzero_byte_bits(uint32_t w) {
    const uint32_t t = (((w & 0x7f7f7f7fu) + 0x7f7f7f7fu) | w) >> 7;
    return ((t & 0x01010101u) * 0x01020408u) >> 24 & 0xfu;
}

__global__ void __launch_bounds__(WD_THREADS, WD_CTAS_PER_SM)
seg_scan_wide_kernel(const WideParams prm) {
    __shared__ __align__(16) uint8_t in_x[2][WD_TILE];
    __shared__ __align__(16) uint8_t in_f[2][WD_TILE];
    __shared__ __align__(16) uint4 outb[WD_TILE / 4];      // 16-byte chunk c sits at c ^ ((c >> 3) & 7) inside its group of 8
    __shared__ int warp_val[WD_WARPS];
    __shared__ int warp_first[WD_WARPS];
    __shared__ int early_val[WD_WARPS];
    __shared__ long long s_tile[2];
    __shared__ long long s_carry;
    __shared__ int s_failed;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t lanes_below = (1u << lane) - 1u;

    // Requests tile t into buffer b (nothing for a tile past the end).
    auto stage = [&](long long t, int b) {
        if (t >= prm.num_tiles) return;
        const long long t0 = t * WD_TILE;
        if (t0 + WD_TILE <= prm.n) {
            cp_async_16(&in_x[b][tid * 16], prm.x + t0 + tid * 16);
            if (prm.flags) cp_async_16(&in_f[b][tid * 16], prm.flags + t0 + tid * 16);
        } else {
            // the ragged end of the input: element by element; what lies past n adds nothing and starts nothing
            for (int e = tid; e < WD_TILE; e += WD_THREADS) {
                const bool in = t0 + e < prm.n;
                in_x[b][e] = in ? static_cast<uint8_t>(prm.x[t0 + e]) : uint8_t(0);
                in_f[b][e] = (in && prm.flags) ? prm.flags[t0 + e] : uint8_t(0);
            }
        }
    };

    if (tid == 0) {
        s_tile[0] = static_cast<long long>(atomicAdd(&prm.hdr->tile_counter, 1u));
        s_failed = 0;
    }
    __syncthreads();
    long long tile = s_tile[0];
    int b = 0;
    bool published = false;                                // this tile's aggregate went out ahead of time (below)
    stage(tile, 0);

    while (tile < prm.num_tiles) {
        cp_async_wait_all();
        __syncthreads();                                   // this tile's inputs are in; the previous tile has left outb
        const long long t0 = tile * WD_TILE;

        // ---- my 16 values, my 16 flags as bits ----
        int v[WD_PER_THREAD];
        {
            const uint4 a = *reinterpret_cast<const uint4*>(&in_x[b][tid * 16]);
            const uint32_t w[4] = {a.x, a.y, a.z, a.w};
#pragma unroll
            for (int j = 0; j < WD_PER_THREAD; ++j) v[j] = static_cast<int>(static_cast<int8_t>((w[j >> 2] >> (8 * (j & 3))) & 0xffu));
        }
        uint32_t fmask = 0u;                               // bit j: element j starts a segment
        if (prm.flags) {
            const uint4 f = *reinterpret_cast<const uint4*>(&in_f[b][tid * 16]);
            if (f.x | f.y | f.z | f.w)
                fmask = wide_nonzero_byte_bits(f.x) | wide_nonzero_byte_bits(f.y) << 4 | wide_nonzero_byte_bits(f.z) << 8 |
                        wide_nonzero_byte_bits(f.w) << 12;
        }
        // ---- the recurrence inside the thread ----
        int run = v[0];
        if (fmask == 0u) {
#pragma unroll
            for (int j = 1; j < WD_PER_THREAD; ++j) {
                run += v[j];
                v[j] = run;
            }
        } else {
#pragma unroll
            for (int j = 1; j < WD_PER_THREAD; ++j) {
                run = ((fmask >> j) & 1u) ? v[j] : run + v[j];
                v[j] = run;
            }
        }
        // ---- segmented warp scan of the threads' open tails; the starts are known from one ballot ----
        const unsigned starts = __ballot_sync(0xffffffffu, fmask != 0u);
        const int seg_lane = 31 - __clz((starts & (lanes_below | (1u << lane))) | 1u);   // nearest lane at or below mine with a start (else 0)
        int val = run;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int tv = __shfl_up_sync(0xffffffffu, val, o);
            if (lane - o >= seg_lane) val += tv;
        }
        int ev = __shfl_up_sync(0xffffffffu, val, 1);                     // open sum of the lanes in front of mine
        if (lane == 0) ev = 0;
        const bool ef = (starts & lanes_below) != 0u;
        const int lead = starts ? __ffs(starts) - 1 : 0;
        const uint32_t lead_mask = __shfl_sync(0xffffffffu, fmask, lead);
        if (lane == 31) {
            warp_val[warp] = val;
            warp_first[warp] = starts ? (warp * 32 + lead) * WD_PER_THREAD + __ffs(lead_mask) - 1 : WD_TILE;
        }
        if (tid == 0) s_tile[b ^ 1] = static_cast<long long>(atomicAdd(&prm.hdr->tile_counter, 1u));
        __syncthreads();
        const long long next = s_tile[b ^ 1];
        stage(next, b ^ 1);                                               // the next tile comes in behind everything below

        // ---- across the warps: the same scan over one value per lane ----
        const int wv = lane < WD_WARPS ? warp_val[lane] : 0;
        const int wf = lane < WD_WARPS ? warp_first[lane] : WD_TILE;
        const unsigned wstarts = __ballot_sync(0xffffffffu, wf < WD_TILE);
        const int wseg = 31 - __clz((wstarts & (lanes_below | (1u << lane))) | 1u);
        int wval = wv;
#pragma unroll
        for (int o = 1; o < WD_WARPS; o <<= 1) {
            const int tv = __shfl_up_sync(0xffffffffu, wval, o);
            if (lane - o >= wseg) wval += tv;
        }
        const int tile_val = __shfl_sync(0xffffffffu, wval, WD_WARPS - 1);          // sum of the tile's open tail
        const bool tile_flg = wstarts != 0u;
        const int tile_first = static_cast<int>(__reduce_min_sync(0xffffffffu, static_cast<unsigned>(wf)));
        int pre = __shfl_sync(0xffffffffu, wval, (warp + 31) & 31);                 // open sum of the warps in front of mine
        if (warp == 0) pre = 0;
        const bool first = tile == 0;
        const bool silent = tile == prm.debug_skip_tile;
        if (tid == 0 && !published && !silent)
            st_relaxed_gpu_u64(prm.status + tile * WD_STATUS_STRIDE, wide_pack((tile_flg || first) ? ST_PREFIX : ST_AGG, tile_val));

        // ---- finish my elements up to my first start inside the tile, park the results ----
        const int ex = ef ? ev : pre + ev;
        const int first_flag = fmask ? __ffs(fmask) - 1 : WD_PER_THREAD;
#pragma unroll
        for (int q = 0; q < WD_PER_THREAD / 4; ++q) {
            uint32_t o[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int j = 4 * q + i;
                o[i] = static_cast<uint32_t>(j < first_flag ? ex + v[j] : v[j]);
            }
            const int c = tid * 4 + q;
            outb[c ^ ((c >> 3) & 7)] = make_uint4(o[0], o[1], o[2], o[3]);
        }
        __syncwarp();                                      // a warp stores the results of its own lanes: no CTA-wide barrier

        // ---- where segment starts are rare: the NEXT tile's aggregate, ahead of time ----
        published = false;
        if (!tile_flg && next < prm.num_tiles) {
            cp_async_wait_all();
            __syncthreads();
            int any = 0;
            if (prm.flags) {
                const uint4 f = *reinterpret_cast<const uint4*>(&in_f[b ^ 1][tid * 16]);
                any = (f.x | f.y | f.z | f.w) != 0u;
            }
            if (!__syncthreads_or(any)) {
                const uint4 a = *reinterpret_cast<const uint4*>(&in_x[b ^ 1][tid * 16]);
                int m = __dp4a(static_cast<int>(a.x), 0x01010101, 0);
                m = __dp4a(static_cast<int>(a.y), 0x01010101, m);
                m = __dp4a(static_cast<int>(a.z), 0x01010101, m);
                m = __dp4a(static_cast<int>(a.w), 0x01010101, m);
#pragma unroll
                for (int o = 16; o >= 1; o >>= 1) m += __shfl_xor_sync(0xffffffffu, m, o);
                if (lane == 0) early_val[warp] = m;
                __syncthreads();
                if (tid == 0 && next != prm.debug_skip_tile) {
                    int r = 0;
#pragma unroll
                    for (int q = 0; q < WD_WARPS; ++q) r += early_val[q];
                    st_relaxed_gpu_u64(prm.status + next * WD_STATUS_STRIDE, wide_pack(ST_AGG, r));
                }
                published = true;
            }
        }

        // Results leave as int64, two 16-byte stores per four elements.  late = false: the elements that need no
        // carry (all but those in front of the tile's first start); late = true: the rest, and the first warp's share.
        const bool whole = t0 + WD_TILE <= prm.n;
        auto copy_out = [&](bool late, long long carry) {
#pragma unroll
            for (int k = 0; k < WD_PER_THREAD / 4; ++k) {
                const int c = warp * (32 * WD_PER_THREAD / 4) + k * 32 + lane;      // a chunk of four of my warp's elements
                const int e = 4 * c;
                const bool needs = e < tile_first;
                if (warp == 0 ? !late : needs != late) continue;
                const uint4 r = outb[c ^ ((c >> 3) & 7)];
                long long o[4] = {static_cast<int>(r.x), static_cast<int>(r.y), static_cast<int>(r.z), static_cast<int>(r.w)};
                if (needs) {
#pragma unroll
                    for (int i = 0; i < 4; ++i)
                        if (e + i < tile_first) o[i] += carry;
                }
                long long* dst = prm.out + t0 + e;
                if (whole) {
                    reinterpret_cast<longlong2*>(dst)[0] = make_longlong2(o[0], o[1]);
                    reinterpret_cast<longlong2*>(dst)[1] = make_longlong2(o[2], o[3]);
                } else {
#pragma unroll
                    for (int i = 0; i < 4; ++i)
                        if (t0 + e + i < prm.n) dst[i] = o[i];
                }
            }
        };

        if (warp == 0) {
            // ---- the first warp looks back for the carry ----
            long long carry = 0;
            bool ok = true;
            if (!first) {
                long long idx = tile - 1;
                const uint64_t tstart = global_timer_ns();
                uint32_t polls = 0;
                while (true) {
                    const long long my = idx - lane;
                    const uint64_t w = my >= 0 ? ld_relaxed_gpu_u64(prm.status + my * WD_STATUS_STRIDE) : wide_pack(ST_PREFIX, 0);
                    const uint32_t st = wide_state(w);
                    const unsigned term = __ballot_sync(0xffffffffu, st == ST_PREFIX || st == ST_ABORT);
                    const int L = term ? __ffs(term) - 1 : 32;               // nearest lane with a final word
                    const bool needed = lane <= L;
                    if (__all_sync(0xffffffffu, !needed || st != ST_NONE)) {
                        if (__any_sync(0xffffffffu, needed && st == ST_ABORT)) { ok = false; break; }
                        long long part = needed ? wide_value(w) : 0ll;
#pragma unroll
                        for (int o = 16; o >= 1; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
                        carry += part;
                        if (L < 32) break;
                        idx -= 32;
                    } else {
                        if ((++polls & 7u) == 0u && global_timer_ns() - tstart > prm.budget_ns) { ok = false; break; }
                    }
                }
            }
            if (lane == 0) {
                if (!ok) {
                    st_relaxed_gpu_u64(prm.status + tile * WD_STATUS_STRIDE, wide_pack(ST_ABORT, 0));
                    report_error(prm.hdr, 5u);
                    s_failed = 1;
                } else if (!tile_flg && !first && !silent) {
                    st_relaxed_gpu_u64(prm.status + tile * WD_STATUS_STRIDE, wide_pack(ST_PREFIX, carry + tile_val));
                }
                s_carry = carry;
            }
        } else {
            copy_out(false, 0ll);
        }
        __syncthreads();
        if (s_failed) break;
        copy_out(true, s_carry);
        tile = next;
        b ^= 1;
    }
    cp_async_wait_all();
}

}  // namespace mmv
