// Segmented running maximum / minimum: Eq. (1) with max or min in place of the addition.
// These operators have no inverse, and the matrix-product method of the paper reverts its
// speculation by subtracting (Section 2: the operator has to form a group), so this scan is the
// plain recurrence on the CUDA cores -- no tensor-core product, nothing to revert.  No arithmetic
// is involved, so results are exact; the kernel is bound by instruction issue and by memory, and
// is laid out to spend few instructions per element:
//
//  * a CTA of 256 threads takes a run of 8192 consecutive elements (runs are handed out by an
//    atomic counter, so a run's predecessors have always started) as two halves of 4096; a thread
//    scans 16 consecutive elements, a segmented warp scan (starts known from one ballot) and the
//    same scan over the eight warp aggregates give the prefix inside the run.  Four CTAs share an
//    SM: with 512 threads and 16384-element runs, two per SM, the CTA-wide barriers cost 10 %;
//  * everything per element is done in the values' own 16-bit format (fp16 or bfloat16): the maximum
//    of such values is one of them; int8 values are fp16 values too.  So a thread's 16 elements live
//    in eight packed registers and the results are parked in shared memory in place of the inputs;
//  * runs are chained with a single-pass decoupled look-back over one status word per run.  Only
//    the elements in front of the run's first segment start need the carry, so all other results
//    leave (fp32 / int32, coalesced 16-byte stores) while the first warp is still looking back;
//  * inputs arrive by 16-byte asynchronous copies into one of two shared-memory buffers; the next
//    run is requested as soon as its number is known.
//
// NaN inputs and the sign of a zero result are unspecified (max(+0, -0) may be either).
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <type_traits>
#include <cuda_runtime.h>
#include <stdint.h>
#include "common.cuh"
#include "ptx.cuh"

namespace mmv {

#ifndef MMV_MM_THREADS
#define MMV_MM_THREADS 256
#endif
constexpr int MM_THREADS = MMV_MM_THREADS;
constexpr int MM_WARPS = MM_THREADS / 32;
constexpr int MM_PER_THREAD = 16;
constexpr int MM_SUB = MM_THREADS * MM_PER_THREAD;       // 4096 elements: one pass of the CTA
constexpr int MM_SUBS = 2;
constexpr int MM_TILE = MM_SUB * MM_SUBS;                // 8192 elements: one run, one status word
static_assert(MM_WARPS <= 32 && 1024 % MM_THREADS == 0, "the warp aggregates are scanned by one warp");
constexpr int MM_CTAS_PER_SM = 1024 / MM_THREADS;
constexpr int MM_X_BYTES = MM_TILE * 2;                  // values (and, later, results) as fp16
constexpr int MM_STAGE_BYTES = MM_X_BYTES + MM_TILE;     // ... and the flag bytes behind them
constexpr int MM_SMEM_BYTES = 2 * MM_STAGE_BYTES;
#ifndef MMV_MM_STRIDE
#define MMV_MM_STRIDE 4
#endif
#ifndef MMV_MM_LOOK
#define MMV_MM_LOOK 1
#endif
// The status words of consecutive runs lie MM_STATUS_STRIDE words apart: the few hundred words that the runs in
// flight poll then spread over the L2 slices instead of queueing at the one or two that a dense array maps to.
constexpr int MM_STATUS_STRIDE = MMV_MM_STRIDE;
#ifndef MMV_MM_EARLY
#define MMV_MM_EARLY 1
#endif
constexpr bool MM_EARLY = MMV_MM_EARLY != 0;           // publish the next run's aggregate ahead of time (see the kernel)
constexpr int MM_LOOK = MMV_MM_LOOK;                               // status words per lane and poll of the look-back

struct MinMaxParams {
    const void* x;              // n values (fp16 or int8)
    const uint8_t* flags;       // n start flags, or null: one segment
    void* out;                  // n results (fp32 or int32)
    long long n;
    long long num_tiles;        // runs of MM_TILE elements
    WorkspaceHeader* hdr;       // tile_counter and error, cleared by the caller
    uint64_t* status;           // one word per run, cleared by the caller; payload: the value as fp32 bits
    unsigned long long budget_ns;
    long long debug_skip_run;   // test hook: this run never publishes a status word (-1: none)
};

template <bool MIN>
struct MinMaxOp {
    __device__ static __forceinline__ float f(float a, float b) { return MIN ? fminf(a, b) : fmaxf(a, b); }
    __device__ static __forceinline__ __half h(__half a, __half b) { return MIN ? __hmin(a, b) : __hmax(a, b); }
    __device__ static __forceinline__ __half2 h2(__half2 a, __half2 b) { return MIN ? __hmin2(a, b) : __hmax2(a, b); }
    __device__ static __forceinline__ __nv_bfloat16 h(__nv_bfloat16 a, __nv_bfloat16 b) { return MIN ? __hmin(a, b) : __hmax(a, b); }
    __device__ static __forceinline__ __nv_bfloat162 h2(__nv_bfloat162 a, __nv_bfloat162 b) { return MIN ? __hmin2(a, b) : __hmax2(a, b); }
    __device__ static __forceinline__ float identity() { return __int_as_float(MIN ? 0x7f800000 : 0xff800000); }
};

// The two 16-bit formats behind one set of names.
__device__ __forceinline__ __half mm_lo(__half2 p) { return __low2half(p); }
__device__ __forceinline__ __half mm_hi(__half2 p) { return __high2half(p); }
__device__ __forceinline__ __nv_bfloat16 mm_lo(__nv_bfloat162 p) { return __low2bfloat16(p); }
__device__ __forceinline__ __nv_bfloat16 mm_hi(__nv_bfloat162 p) { return __high2bfloat16(p); }
__device__ __forceinline__ float mm_tof(__half v) { return __half2float(v); }
__device__ __forceinline__ float mm_tof(__nv_bfloat16 v) { return __bfloat162float(v); }
__device__ __forceinline__ float2 mm_tof2(__half2 p) { return __half22float2(p); }
__device__ __forceinline__ float2 mm_tof2(__nv_bfloat162 p) { return __bfloat1622float2(p); }
__device__ __forceinline__ __half2 mm_dup(__half v) { return __half2half2(v); }
__device__ __forceinline__ __nv_bfloat162 mm_dup(__nv_bfloat16 v) { return __bfloat162bfloat162(v); }
__device__ __forceinline__ __half2 mm_pack(__half a, __half b) { return __halves2half2(a, b); }
__device__ __forceinline__ __nv_bfloat162 mm_pack(__nv_bfloat16 a, __nv_bfloat16 b) { return __halves2bfloat162(a, b); }
template <typename H> __device__ __forceinline__ H mm_fromf(float v);
template <> __device__ __forceinline__ __half mm_fromf<__half>(float v) { return __float2half_rn(v); }
template <> __device__ __forceinline__ __nv_bfloat16 mm_fromf<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

// Bit i of the result: byte i of w is not zero.
__device__ __forceinline__ uint32_t nonzero_byte_bits(uint32_t w) {
    const uint32_t t = (((w & 0x7f7f7f7fu) + 0x7f7f7f7fu) | w) >> 7;
    return ((t & 0x01010101u) * 0x01020408u) >> 24 & 0xfu;
}

// FMT 0: fp16 values, fp32 results; 1: int8 values (handled as fp16), int32 results; 2: bfloat16 values, fp32
// results.  MIN selects the operator.
template <int FMT, bool MIN>
__global__ void __launch_bounds__(MM_THREADS, MM_CTAS_PER_SM)
seg_scan_minmax_kernel(const MinMaxParams prm) {
    using Op = MinMaxOp<MIN>;
    constexpr bool INT8 = FMT == 1;
    using H = typename std::conditional<FMT == 2, __nv_bfloat16, __half>::type;
    using H2 = typename std::conditional<FMT == 2, __nv_bfloat162, __half2>::type;
    constexpr unsigned short kNeutralBits = FMT == 2 ? (MIN ? 0x7f80u : 0xff80u) : (MIN ? 0x7c00u : 0xfc00u);   // +inf / -inf
    constexpr int kElem = INT8 ? 1 : 2;                    // bytes per input value
    // int8 values land in the upper half of the value area: their fp16 results then never overwrite
    // a value that has not been read (the first half's results fill the lower half of the area, the
    // second half's are written after the barrier that follows the reading of its values)
    constexpr int kRawOff = INT8 ? MM_TILE : 0;
    extern __shared__ __align__(128) uint8_t smem[];
    __shared__ float warp_val[MM_SUBS][MM_WARPS];
    __shared__ int warp_first[MM_SUBS][MM_WARPS];
    __shared__ float early_val[MM_WARPS];
    __shared__ long long s_tile[2];
    __shared__ float s_carry;
    __shared__ int s_failed;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t lanes_below = (1u << lane) - 1u;

    // Requests run t into buffer b (nothing for a run past the end).
    auto stage = [&](long long t, int b) {
        if (t >= prm.num_tiles) return;
        uint8_t* xs = smem + b * MM_STAGE_BYTES;
        uint8_t* fs = xs + MM_X_BYTES;
        const long long t0 = t * MM_TILE;
        if (t0 + MM_TILE <= prm.n) {
            const uint8_t* gx = static_cast<const uint8_t*>(prm.x) + t0 * kElem;
#pragma unroll
            for (int c = 0; c < MM_TILE * kElem / 16 / MM_THREADS; ++c)
                cp_async_16(xs + kRawOff + (c * MM_THREADS + tid) * 16, gx + (c * MM_THREADS + tid) * 16);
            if (prm.flags) {
#pragma unroll
                for (int c = 0; c < MM_TILE / 16 / MM_THREADS; ++c)
                    cp_async_16(fs + (c * MM_THREADS + tid) * 16, prm.flags + t0 + (c * MM_THREADS + tid) * 16);
            }
        } else {
            // the ragged end of the input: element by element; what lies past n is neutral and starts nothing
            for (int e = tid; e < MM_TILE; e += MM_THREADS) {
                const bool in = t0 + e < prm.n;
                if constexpr (INT8)
                    xs[kRawOff + e] = in ? static_cast<const uint8_t*>(prm.x)[t0 + e] : static_cast<uint8_t>(MIN ? 0x7fu : 0x80u);
                else
                    reinterpret_cast<unsigned short*>(xs)[e] =
                        in ? static_cast<const unsigned short*>(prm.x)[t0 + e] : kNeutralBits;
                fs[e] = (in && prm.flags) ? prm.flags[t0 + e] : uint8_t(0);
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
    bool published = false;                                // this run's aggregate went out ahead of time (below)
    stage(tile, 0);

    while (tile < prm.num_tiles) {
        cp_async_wait_all();
        __syncthreads();                                   // this run's inputs are in; the previous run has left its buffer
        uint8_t* xs = smem + b * MM_STAGE_BYTES;
        const uint8_t* fs = xs + MM_X_BYTES;
        const long long t0 = tile * MM_TILE;
        long long next = 0;
        // what is known of the run so far: value of its open tail, whether a segment started, where the first one did
        float run_val = Op::identity();
        bool run_flg = false;
        int run_first = MM_TILE;

#pragma unroll
        for (int s = 0; s < MM_SUBS; ++s) {
            const int base = s * MM_SUB + tid * MM_PER_THREAD;          // my first element inside the run
            // ---- my 16 values as fp16 pairs, my 16 flags as bits ----
            H h[MM_PER_THREAD];
            if constexpr (INT8) {
                const uint4 a = *reinterpret_cast<const uint4*>(xs + kRawOff + base);
                const uint32_t w[4] = {a.x, a.y, a.z, a.w};
#pragma unroll
                for (int j = 0; j < MM_PER_THREAD; ++j)
                    h[j] = __short2half_rn(static_cast<short>(static_cast<int8_t>((w[j >> 2] >> (8 * (j & 3))) & 0xffu)));
            } else {
                const uint4 a = *reinterpret_cast<const uint4*>(xs + base * 2);
                const uint4 c = *reinterpret_cast<const uint4*>(xs + base * 2 + 16);
                const uint32_t w[8] = {a.x, a.y, a.z, a.w, c.x, c.y, c.z, c.w};
#pragma unroll
                for (int k = 0; k < MM_PER_THREAD / 2; ++k) {
                    const H2 p = *reinterpret_cast<const H2*>(&w[k]);
                    h[2 * k] = mm_lo(p);
                    h[2 * k + 1] = mm_hi(p);
                }
            }
            uint32_t fmask = 0u;                                        // bit j: element j starts a segment
            if (prm.flags) {
                const uint4 f = *reinterpret_cast<const uint4*>(fs + base);
                if (f.x | f.y | f.z | f.w)
                    fmask = nonzero_byte_bits(f.x) | nonzero_byte_bits(f.y) << 4 | nonzero_byte_bits(f.z) << 8 | nonzero_byte_bits(f.w) << 12;
            }
            // ---- the recurrence inside the thread ----
            H run = h[0];
            if (fmask == 0u) {
#pragma unroll
                for (int j = 1; j < MM_PER_THREAD; ++j) {
                    run = Op::h(run, h[j]);
                    h[j] = run;
                }
            } else {
#pragma unroll
                for (int j = 1; j < MM_PER_THREAD; ++j) {
                    run = ((fmask >> j) & 1u) ? h[j] : Op::h(run, h[j]);
                    h[j] = run;
                }
            }
            // ---- segmented warp scan of the threads' open tails; the starts are known from one ballot ----
            const unsigned starts = __ballot_sync(0xffffffffu, fmask != 0u);
            const int seg_lane = 31 - __clz((starts & (lanes_below | (1u << lane))) | 1u);   // nearest lane at or below mine with a start (else 0)
            float val = mm_tof(run);
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const float tv = __shfl_up_sync(0xffffffffu, val, o);
                if (lane - o >= seg_lane) val = Op::f(tv, val);
            }
            float ev = __shfl_up_sync(0xffffffffu, val, 1);               // open value of the lanes in front of mine
            if (lane == 0) ev = Op::identity();
            const bool ef = (starts & lanes_below) != 0u;
            const int lead = starts ? __ffs(starts) - 1 : 0;
            const uint32_t lead_mask = __shfl_sync(0xffffffffu, fmask, lead);
            if (lane == 31) {
                warp_val[s][warp] = val;
                warp_first[s][warp] = starts ? (warp * 32 + lead) * MM_PER_THREAD + __ffs(lead_mask) - 1 : MM_SUB;
            }
            if (s == 0 && tid == 0) s_tile[b ^ 1] = static_cast<long long>(atomicAdd(&prm.hdr->tile_counter, 1u));
            __syncthreads();
            if (s == 0) {
                next = s_tile[b ^ 1];
                stage(next, b ^ 1);                                     // the next run comes in behind everything below
            }
            // ---- across the warps: the same scan over one value per lane ----
            const float wv = lane < MM_WARPS ? warp_val[s][lane] : Op::identity();
            const int wf = lane < MM_WARPS ? warp_first[s][lane] : MM_SUB;
            const unsigned wstarts = __ballot_sync(0xffffffffu, wf < MM_SUB);
            const int wseg = 31 - __clz((wstarts & (lanes_below | (1u << lane))) | 1u);
            float wval = wv;
#pragma unroll
            for (int o = 1; o < MM_WARPS; o <<= 1) {
                const float tv = __shfl_up_sync(0xffffffffu, wval, o);
                if (lane - o >= wseg) wval = Op::f(tv, wval);
            }
            const float sub_val = __shfl_sync(0xffffffffu, wval, MM_WARPS - 1);
            const bool sub_flg = wstarts != 0u;
            const int sub_first = static_cast<int>(__reduce_min_sync(0xffffffffu, static_cast<unsigned>(wf)));
            float pre = __shfl_sync(0xffffffffu, wval, (warp + 31) & 31);  // open value of the warps in front of mine
            if (warp == 0) pre = Op::identity();
            const bool pre_flg = (wstarts & ((1u << warp) - 1u)) != 0u;

            // ---- what is open in front of my elements inside the run; finish my elements up to my first start ----
            float ex = ef ? ev : Op::f(pre, ev);
            if (!(ef || pre_flg)) ex = Op::f(run_val, ex);
            const H exh = mm_fromf<H>(ex);                              // exact: one of the values, or the identity
            H2 w2[MM_PER_THREAD / 2];
            if (fmask == 0u) {
                const H2 ex2 = mm_dup(exh);
#pragma unroll
                for (int k = 0; k < MM_PER_THREAD / 2; ++k) w2[k] = Op::h2(ex2, mm_pack(h[2 * k], h[2 * k + 1]));
            } else {
                const int first_flag = __ffs(fmask) - 1;
#pragma unroll
                for (int k = 0; k < MM_PER_THREAD / 2; ++k)
                    w2[k] = mm_pack(2 * k < first_flag ? Op::h(exh, h[2 * k]) : h[2 * k],
                                           2 * k + 1 < first_flag ? Op::h(exh, h[2 * k + 1]) : h[2 * k + 1]);
            }
            uint4* park = reinterpret_cast<uint4*>(xs + base * 2);
            const uint32_t* wb = reinterpret_cast<const uint32_t*>(w2);
            park[0] = make_uint4(wb[0], wb[1], wb[2], wb[3]);
            park[1] = make_uint4(wb[4], wb[5], wb[6], wb[7]);
            // ---- the run so far ----
            if (!run_flg && sub_flg) run_first = s * MM_SUB + sub_first;
            run_val = sub_flg ? sub_val : Op::f(run_val, sub_val);
            run_flg = run_flg || sub_flg;
        }
        const bool first = tile == 0;
        const bool silent = tile == prm.debug_skip_run;
        if (tid == 0 && !published && !silent)
            st_relaxed_gpu_u64(prm.status + tile * MM_STATUS_STRIDE, pack_status((run_flg || first) ? ST_PREFIX : ST_AGG, __float_as_uint(run_val)));
        __syncthreads();                                   // every result of the run is parked

        // ---- where segment starts are rare: the NEXT run's aggregate, ahead of time ----
        // This CTA took the next run's number long ago, and the runs behind it wait for that run's word.  Left to
        // the next iteration, the word would come only after this run's look-back: one slow look-back would then
        // hold up the look-backs of the runs behind, and theirs the ones behind them.  So when this run saw no
        // start, the next run (already in shared memory, or nearly) is reduced here, before the look-back, and
        // its aggregate published if it holds no start either; the scan proper recomputes it later.
        published = false;
        if (MM_EARLY && !run_flg && next < prm.num_tiles) {
            cp_async_wait_all();
            __syncthreads();
            const uint8_t* nx = smem + (b ^ 1) * MM_STAGE_BYTES;
            int any = 0;
            if (prm.flags) {
                const uint4* nf = reinterpret_cast<const uint4*>(nx + MM_X_BYTES + tid * 32);
                const uint4 f0 = nf[0], f1 = nf[1];
                any = (f0.x | f0.y | f0.z | f0.w | f1.x | f1.y | f1.z | f1.w) != 0u;
            }
            if (!__syncthreads_or(any)) {
                float m;
                if constexpr (INT8) {
                    const uint4* p4 = reinterpret_cast<const uint4*>(nx + kRawOff + tid * 32);
                    const uint4 a = p4[0], c = p4[1];
                    const uint32_t w[8] = {a.x, a.y, a.z, a.w, c.x, c.y, c.z, c.w};
                    int mi = MIN ? 127 : -128;
#pragma unroll
                    for (int k = 0; k < 8; ++k)
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const int e = static_cast<int8_t>((w[k] >> (8 * i)) & 0xffu);
                            mi = MIN ? min(mi, e) : max(mi, e);
                        }
                    m = static_cast<float>(mi);
                } else {
                    const uint4* p4 = reinterpret_cast<const uint4*>(nx + tid * 64);
                    H2 m2 = *reinterpret_cast<const H2*>(&p4[0].x);
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        const uint4 a = p4[k];
                        m2 = Op::h2(m2, *reinterpret_cast<const H2*>(&a.x));
                        m2 = Op::h2(m2, *reinterpret_cast<const H2*>(&a.y));
                        m2 = Op::h2(m2, *reinterpret_cast<const H2*>(&a.z));
                        m2 = Op::h2(m2, *reinterpret_cast<const H2*>(&a.w));
                    }
                    m = mm_tof(Op::h(mm_lo(m2), mm_hi(m2)));
                }
#pragma unroll
                for (int o = 16; o >= 1; o >>= 1) m = Op::f(m, __shfl_xor_sync(0xffffffffu, m, o));
                if (lane == 0) early_val[warp] = m;
                __syncthreads();
                if (tid == 0 && next != prm.debug_skip_run) {
                    float r = early_val[0];
#pragma unroll
                    for (int q = 1; q < MM_WARPS; ++q) r = Op::f(r, early_val[q]);
                    st_relaxed_gpu_u64(prm.status + next * MM_STATUS_STRIDE, pack_status(ST_AGG, __float_as_uint(r)));
                }
                published = true;
            }
        }

        // Results leave as fp32 / int32, 16 bytes per thread and store.  late = false: the elements that need no
        // carry (all but those in front of the run's first start); late = true: the rest, and the first warp's share.
        const bool whole = t0 + MM_TILE <= prm.n;
        auto copy_out = [&](bool late, float carry) {
#pragma unroll
            for (int k = 0; k < MM_TILE / 4 / MM_THREADS; ++k) {
                const int c = k * MM_THREADS + tid;
                const int e = 4 * c;
                const bool needs = e < run_first;
                if (warp == 0 ? !late : needs != late) continue;
                const uint2 r = *reinterpret_cast<const uint2*>(xs + c * 8);
                const float2 lo = mm_tof2(*reinterpret_cast<const H2*>(&r.x));
                const float2 hi = mm_tof2(*reinterpret_cast<const H2*>(&r.y));
                float v[4] = {lo.x, lo.y, hi.x, hi.y};
                if (needs) {
#pragma unroll
                    for (int i = 0; i < 4; ++i)
                        if (e + i < run_first) v[i] = Op::f(carry, v[i]);
                }
                uint32_t o[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) o[i] = INT8 ? static_cast<uint32_t>(__float2int_rn(v[i])) : __float_as_uint(v[i]);
                uint32_t* dst = static_cast<uint32_t*>(prm.out) + t0 + e;
                if (whole) {
                    *reinterpret_cast<uint4*>(dst) = make_uint4(o[0], o[1], o[2], o[3]);
                } else {
#pragma unroll
                    for (int i = 0; i < 4; ++i)
                        if (t0 + e + i < prm.n) dst[i] = o[i];
                }
            }
        };

        if (warp == 0) {
            // ---- the first warp looks back for the carry ----
            float carry = Op::identity();
            bool ok = true;
            if (!first) {
                long long idx = tile - 1;
                const uint64_t tstart = global_timer_ns();
                uint32_t polls = 0;
                while (true) {
                    // a window of 32 * MM_LOOK runs, MM_LOOK per lane, nearest first
                    uint64_t w[MM_LOOK];
#pragma unroll
                    for (int q = 0; q < MM_LOOK; ++q) {
                        const long long my = idx - MM_LOOK * lane - q;
                        w[q] = my >= 0 ? ld_relaxed_gpu_u64(prm.status + my * MM_STATUS_STRIDE)
                                       : pack_status(ST_PREFIX, __float_as_uint(Op::identity()));
                    }
                    // my words up to and including my first final one
                    bool mine_final = false, mine_none = false, mine_abort = false;
                    float mine = Op::identity();
#pragma unroll
                    for (int q = 0; q < MM_LOOK; ++q) {
                        const uint32_t st = static_cast<uint32_t>(w[q] >> 32);
                        if (!mine_final) {
                            mine_none = mine_none || st == ST_NONE;
                            mine_abort = mine_abort || st == ST_ABORT;
                            mine = Op::f(mine, __uint_as_float(static_cast<uint32_t>(w[q])));
                            mine_final = st == ST_PREFIX || st == ST_ABORT;
                        }
                    }
                    const unsigned term = __ballot_sync(0xffffffffu, mine_final);
                    const int L = term ? __ffs(term) - 1 : 32;               // nearest lane with a final word
                    const bool needed = lane <= L;
                    if (__all_sync(0xffffffffu, !needed || !mine_none)) {
                        if (__any_sync(0xffffffffu, needed && mine_abort)) { ok = false; break; }
                        // combine the needed words (the operator is commutative and associative: any order)
                        float part = needed ? mine : Op::identity();
#pragma unroll
                        for (int o = 16; o >= 1; o >>= 1) part = Op::f(part, __shfl_xor_sync(0xffffffffu, part, o));
                        carry = Op::f(carry, part);
                        if (L < 32) break;
                        idx -= 32 * MM_LOOK;
                    } else {
                        if ((++polls & 7u) == 0u && global_timer_ns() - tstart > prm.budget_ns) { ok = false; break; }
                    }
                }
            }
            if (lane == 0) {
                if (!ok) {
                    st_relaxed_gpu_u64(prm.status + tile * MM_STATUS_STRIDE, pack_status(ST_ABORT, 0u));
                    report_error(prm.hdr, 5u);
                    s_failed = 1;
                } else if (!run_flg && !first && !silent) {
                    st_relaxed_gpu_u64(prm.status + tile * MM_STATUS_STRIDE, pack_status(ST_PREFIX, __float_as_uint(Op::f(carry, run_val))));
                }
                s_carry = carry;
            }
        } else {
            copy_out(false, 0.0f);
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
