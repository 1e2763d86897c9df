// Segmented running maximum / minimum: Eq. (1) with max or min in place of the addition.
// These operators have no inverse, and the matrix-product method of the paper reverts its
// speculation by subtracting (Section 2: the operator has to form a group), so this scan is the
// plain recurrence on the CUDA cores -- no tensor-core product, nothing to revert: every thread
// scans 16 consecutive elements, a segmented warp scan and a short pass over the eight warp
// aggregates give the prefix inside a 4096-element tile, and tiles are chained with a single-pass
// decoupled look-back over one status word per tile (tiles are handed out by an atomic counter,
// so a tile's predecessors have always started).  No arithmetic is involved: results are exact.
//
// Memory side: a tile's values and flags come in by 16-byte asynchronous copies into one of two
// shared-memory buffers (the next tile is requested before this one's look-back, so its latency
// hides behind the wait and the stores); every thread reads its 16 elements from there.  Results
// go through a swizzled shared buffer and leave as coalesced 16-byte stores, and the carry from
// the tiles in front -- which only the elements before the tile's first segment start need -- is
// applied on that way out.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>
#include "common.cuh"
#include "ptx.cuh"

namespace mmv {

constexpr int MM_THREADS = 256;
constexpr int MM_PER_THREAD = 16;
constexpr int MM_TILE = MM_THREADS * MM_PER_THREAD;      // 4096 elements
constexpr int MM_CTAS_PER_SM = 4;                         // 40 KB of shared memory and at most 64 registers each

struct MinMaxParams {
    const void* x;              // n values (fp16 or int8)
    const uint8_t* flags;       // n start flags, or null: one segment
    void* out;                  // n results (fp32 or int32)
    long long n;
    long long num_tiles;
    WorkspaceHeader* hdr;       // tile_counter and error, cleared by the caller
    uint64_t* status;           // one word per tile, cleared by the caller
    unsigned long long budget_ns;
};

// V = float (fp16 input) or int (int8 input); MIN selects the operator.
template <typename V, bool MIN>
struct MinMaxOp {
    __device__ static __forceinline__ V op(V a, V b) {
        if constexpr (MIN) return a < b ? a : b;
        else return a > b ? a : b;
    }
    __device__ static __forceinline__ V identity() {
        if constexpr (sizeof(V) == 4 && V(0.5) != V(0)) return MIN ? V(__int_as_float(0x7f800000)) : V(__int_as_float(0xff800000));
        else return MIN ? V(0x7fffffff) : V(-0x7fffffff - 1);
    }
    __device__ static __forceinline__ uint32_t bits(V v) {
        if constexpr (sizeof(V) == 4 && V(0.5) != V(0)) return __float_as_uint(static_cast<float>(v));
        else return static_cast<uint32_t>(static_cast<int>(v));
    }
    __device__ static __forceinline__ V from_bits(uint32_t b) {
        if constexpr (sizeof(V) == 4 && V(0.5) != V(0)) return V(__uint_as_float(b));
        else return V(static_cast<int>(b));
    }
};

template <typename V, bool MIN>
__global__ void __launch_bounds__(MM_THREADS, MM_CTAS_PER_SM)
seg_scan_minmax_kernel(const MinMaxParams prm) {
    using Op = MinMaxOp<V, MIN>;
    constexpr bool kFloat = V(0.5) != V(0);
    constexpr int kElem = kFloat ? 2 : 1;                  // bytes per input value
    constexpr int kXBytes = MM_TILE * kElem;
    constexpr int kWarps = MM_THREADS / 32;
    __shared__ __align__(16) uint8_t in_x[2][kXBytes];
    __shared__ __align__(16) uint8_t in_f[2][MM_TILE];
    __shared__ __align__(16) uint4 outb[MM_TILE / 4];      // 16-byte chunk c sits at c ^ ((c >> 3) & 7) inside its group of 8
    __shared__ uint32_t warp_val[kWarps];
    __shared__ uint32_t warp_flg[kWarps];
    __shared__ int warp_first[kWarps];
    __shared__ long long s_tile[2];
    __shared__ uint32_t s_carry;
    __shared__ int s_failed;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    uint32_t* outp = static_cast<uint32_t*>(prm.out);

    // Requests tile t into buffer b (nothing for a tile past the end).
    auto stage = [&](long long t, int b) {
        if (t >= prm.num_tiles) return;
        const long long t0 = t * MM_TILE;
        if (t0 + MM_TILE <= prm.n) {
            const uint8_t* gx = static_cast<const uint8_t*>(prm.x) + t0 * kElem;
#pragma unroll
            for (int c = 0; c < kXBytes / 16 / MM_THREADS; ++c)
                cp_async_16(&in_x[b][(c * MM_THREADS + tid) * 16], gx + (c * MM_THREADS + tid) * 16);
            if (prm.flags) cp_async_16(&in_f[b][tid * 16], prm.flags + t0 + tid * 16);
        } else {
            // the ragged end of the input: element by element; what lies past n is neutral and starts nothing
            for (int e = tid; e < MM_TILE; e += MM_THREADS) {
                const bool in = t0 + e < prm.n;
                if constexpr (kFloat)
                    reinterpret_cast<unsigned short*>(in_x[b])[e] =
                        in ? static_cast<const unsigned short*>(prm.x)[t0 + e] : static_cast<unsigned short>(MIN ? 0x7c00u : 0xfc00u);
                else
                    in_x[b][e] = in ? static_cast<const uint8_t*>(prm.x)[t0 + e] : static_cast<uint8_t>(MIN ? 0x7fu : 0x80u);
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
    stage(tile, 0);

    while (tile < prm.num_tiles) {
        cp_async_wait_all();
        __syncthreads();                                   // this tile's inputs are in; the previous tile has left outb
        const long long t0 = tile * MM_TILE;

        // ---- my 16 values and 16 flag bytes ----
        V v[MM_PER_THREAD];
        uint32_t fmask = 0u;                               // bit j: element j starts a segment
        if constexpr (kFloat) {
            const uint4 a = *reinterpret_cast<const uint4*>(&in_x[b][tid * 32]);
            const uint4 c = *reinterpret_cast<const uint4*>(&in_x[b][tid * 32 + 16]);
            const uint32_t w[8] = {a.x, a.y, a.z, a.w, c.x, c.y, c.z, c.w};
#pragma unroll
            for (int j = 0; j < MM_PER_THREAD; ++j)
                v[j] = V(__half2float(__ushort_as_half(static_cast<unsigned short>((w[j >> 1] >> (16 * (j & 1))) & 0xffffu))));
        } else {
            const uint4 a = *reinterpret_cast<const uint4*>(&in_x[b][tid * 16]);
            const uint32_t w[4] = {a.x, a.y, a.z, a.w};
#pragma unroll
            for (int j = 0; j < MM_PER_THREAD; ++j)
                v[j] = V(static_cast<int>(static_cast<int8_t>((w[j >> 2] >> (8 * (j & 3))) & 0xffu)));
        }
        if (prm.flags) {
            const uint4 f = *reinterpret_cast<const uint4*>(&in_f[b][tid * 16]);
            const uint32_t w[4] = {f.x, f.y, f.z, f.w};
#pragma unroll
            for (int j = 0; j < MM_PER_THREAD; ++j)
                if ((w[j >> 2] >> (8 * (j & 3))) & 0xffu) fmask |= 1u << j;
        }

        // ---- the recurrence inside the thread ----
        V run = v[0];
#pragma unroll
        for (int j = 1; j < MM_PER_THREAD; ++j) {
            run = ((fmask >> j) & 1u) ? v[j] : Op::op(run, v[j]);
            v[j] = run;
        }
        // ---- segmented warp scan of (has a start, value of the open tail) ----
        V val = run;
        uint32_t flg = fmask ? 1u : 0u;
        const unsigned starts = __ballot_sync(0xffffffffu, fmask != 0u);
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t tv = __shfl_up_sync(0xffffffffu, Op::bits(val), o);
            const uint32_t tf = __shfl_up_sync(0xffffffffu, flg, o);
            if (lane >= o) {
                if (!flg) val = Op::op(Op::from_bits(tv), val);
                flg |= tf;
            }
        }
        uint32_t ev_bits = __shfl_up_sync(0xffffffffu, Op::bits(val), 1);          // open value of the lanes in front of mine
        uint32_t ef = __shfl_up_sync(0xffffffffu, flg, 1);
        if (lane == 0) {
            ev_bits = Op::bits(Op::identity());
            ef = 0u;
        }
        // position of the warp's first segment start inside the tile
        const int lead = starts ? __ffs(starts) - 1 : 0;
        const uint32_t lead_mask = __shfl_sync(0xffffffffu, fmask, lead);
        if (lane == 31) {
            warp_val[warp] = Op::bits(val);
            warp_flg[warp] = flg;
            warp_first[warp] = starts ? warp * 32 * MM_PER_THREAD + lead * MM_PER_THREAD + __ffs(lead_mask) - 1 : MM_TILE;
        }
        if (tid == 0) s_tile[b ^ 1] = static_cast<long long>(atomicAdd(&prm.hdr->tile_counter, 1u));
        __syncthreads();
        const long long next = s_tile[b ^ 1];

        // ---- across the warps of the tile ----
        V pre = Op::identity();                            // open value of the warps in front of mine
        uint32_t pre_flg = 0u;
        V tile_val = Op::identity();
        uint32_t tile_flg = 0u;
        int tile_first = MM_TILE;                          // first segment start of the tile (MM_TILE: none)
#pragma unroll
        for (int q = 0; q < kWarps; ++q) {
            if (q == warp) {
                pre = tile_val;
                pre_flg = tile_flg;
            }
            const V wv = Op::from_bits(warp_val[q]);
            tile_val = warp_flg[q] ? wv : Op::op(tile_val, wv);
            tile_flg |= warp_flg[q];
            tile_first = min(tile_first, warp_first[q]);
        }
        const bool first = tile == 0;
        if (tid == 0)
            st_relaxed_gpu_u64(prm.status + tile, pack_status((tile_flg || first) ? ST_PREFIX : ST_AGG, Op::bits(tile_val)));
        stage(next, b ^ 1);                                // the next tile comes in behind the look-back and the stores

        // ---- finish inside the tile, park the results ----
        const V ex = ef ? Op::from_bits(ev_bits) : Op::op(pre, Op::from_bits(ev_bits));
        const int first_flag = fmask ? __ffs(fmask) - 1 : MM_PER_THREAD;
#pragma unroll
        for (int q = 0; q < MM_PER_THREAD / 4; ++q) {
            uint32_t o[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int j = 4 * q + i;
                o[i] = Op::bits(j < first_flag ? Op::op(ex, v[j]) : v[j]);
            }
            const int c = tid * 4 + q;
            outb[c ^ ((c >> 3) & 7)] = make_uint4(o[0], o[1], o[2], o[3]);
        }

        // ---- the first warp looks back for the carry ----
        if (warp == 0) {
            V carry = Op::identity();
            bool ok = true;
            if (!first) {
                long long idx = tile - 1;
                const uint64_t tstart = global_timer_ns();
                uint32_t polls = 0;
                while (true) {
                    const long long my = idx - lane;
                    const uint64_t w = my >= 0 ? ld_relaxed_gpu_u64(prm.status + my) : pack_status(ST_PREFIX, Op::bits(Op::identity()));
                    const uint32_t st = static_cast<uint32_t>(w >> 32);
                    const unsigned term = __ballot_sync(0xffffffffu, st == ST_PREFIX || st == ST_ABORT);
                    const int L = term ? __ffs(term) - 1 : 32;               // nearest lane with a final word
                    const bool needed = lane <= L;
                    if (__all_sync(0xffffffffu, !needed || st != ST_NONE)) {
                        if (__any_sync(0xffffffffu, needed && st == ST_ABORT)) { ok = false; break; }
                        // combine the needed words (the operator is commutative and associative: any order)
                        V part = needed ? Op::from_bits(static_cast<uint32_t>(w)) : Op::identity();
#pragma unroll
                        for (int o = 16; o >= 1; o >>= 1) part = Op::op(part, Op::from_bits(__shfl_xor_sync(0xffffffffu, Op::bits(part), o)));
                        carry = Op::op(carry, part);
                        if (L < 32) break;
                        idx -= 32;
                    } else {
                        if ((++polls & 7u) == 0u && global_timer_ns() - tstart > prm.budget_ns) { ok = false; break; }
                        __nanosleep(20);
                    }
                }
            }
            if (lane == 0) {
                if (!ok) {
                    st_relaxed_gpu_u64(prm.status + tile, pack_status(ST_ABORT, 0u));
                    report_error(prm.hdr, 5u);
                    s_failed = 1;
                } else if (!tile_flg && !first) {
                    st_relaxed_gpu_u64(prm.status + tile, pack_status(ST_PREFIX, Op::bits(Op::op(carry, tile_val))));
                }
                s_carry = Op::bits(carry);
            }
        }
        __syncthreads();
        if (s_failed) break;

        // ---- out: coalesced, the carry goes to the elements before the tile's first start ----
        const V carry = Op::from_bits(s_carry);
        const bool whole = t0 + MM_TILE <= prm.n;
#pragma unroll
        for (int k = 0; k < MM_TILE / 4 / MM_THREADS; ++k) {
            const int c = k * MM_THREADS + tid;
            uint4 r = outb[c ^ ((c >> 3) & 7)];
            const int e = 4 * c;
            if (e < tile_first) {
                r.x = Op::bits(Op::op(carry, Op::from_bits(r.x)));
                if (e + 1 < tile_first) r.y = Op::bits(Op::op(carry, Op::from_bits(r.y)));
                if (e + 2 < tile_first) r.z = Op::bits(Op::op(carry, Op::from_bits(r.z)));
                if (e + 3 < tile_first) r.w = Op::bits(Op::op(carry, Op::from_bits(r.w)));
            }
            if (whole) {
                *reinterpret_cast<uint4*>(outp + t0 + e) = r;
            } else {
                const uint32_t rr[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
                for (int i = 0; i < 4; ++i)
                    if (t0 + e + i < prm.n) outp[t0 + e + i] = rr[i];
            }
        }
        tile = next;
        b ^= 1;
    }
    cp_async_wait_all();
}

}  // namespace mmv
