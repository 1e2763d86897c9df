// COMPRESS of the segment-start flags (Section 2; the compaction step of Algorithm 4.2):
// the positions of the start flags, in order, are exactly the CSR offsets of the segments,
//     off[r] = position of the r-th start,   off[K] = n,   K = 1 + #{i >= 1 : f(i) != 0},
// so the flag-encoded segmented sum is this compaction followed by the offset-encoded kernel.
// Three small streaming kernels: per-chunk counts, one-block exclusive scan of the counts,
// in-order scatter of the positions.  Element 0 always starts a segment, whatever f(0) holds.
// The count pass is the only one that reads the flag bytes: it leaves one bit per flag (a 64-bit
// mask per thread, n / 8 bytes in the workspace) and the scatter pass reads those instead, an
// eighth of the bytes.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace mmv {

constexpr int CMP_THREADS = 256;
constexpr int CMP_PER_THREAD = 64;                              // flag bytes per thread: four 16-byte vectors
constexpr int CMP_CHUNK = CMP_THREADS * CMP_PER_THREAD;         // 16384 flags per block iteration

// The 64 flag bytes of thread t of chunk c as 16 words (zero past n; with first_is_start byte 0 of the
// vector is forced to 1: element 0 opens a segment whatever its flag says).
__device__ __forceinline__ void load_thread_flags(const uint8_t* __restrict__ f, long long n, long long base, uint32_t (&w)[16],
                                                  bool first_is_start = true) {
#pragma unroll
    for (int v = 0; v < 4; ++v) {
        const long long p = base + 16 * v;
        uint4 q = make_uint4(0u, 0u, 0u, 0u);
        if (p + 16 <= n) {
            q = *reinterpret_cast<const uint4*>(f + p);
        } else if (p < n) {
            uint32_t t[4] = {0u, 0u, 0u, 0u};
            for (int b = 0; b < 16 && p + b < n; ++b) t[b >> 2] |= static_cast<uint32_t>(f[p + b]) << (8 * (b & 3));
            q = make_uint4(t[0], t[1], t[2], t[3]);
        }
        w[4 * v] = q.x;
        w[4 * v + 1] = q.y;
        w[4 * v + 2] = q.z;
        w[4 * v + 3] = q.w;
    }
    if (base == 0 && first_is_start) w[0] |= 1u;          // element 0 starts the first segment
}

// Exclusive scan of one int per thread over the block; returns this thread's offset, *total = block sum.
__device__ __forceinline__ int block_exclusive_scan(int v, int* total, int* warp_sums /* >= 32 ints of shared memory */) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = (blockDim.x + 31) >> 5;
    int inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += t;
    }
    if (lane == 31) warp_sums[warp] = inc;
    __syncthreads();
    if (warp == 0) {
        int s = lane < nwarps ? warp_sums[lane] : 0;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int t = __shfl_up_sync(0xffffffffu, s, o);
            if (lane >= o) s += t;
        }
        warp_sums[lane] = s;            // inclusive over warps
    }
    __syncthreads();
    const int before = warp ? warp_sums[warp - 1] : 0;
    *total = warp_sums[nwarps - 1];
    __syncthreads();                    // warp_sums may be reused by the caller's next round
    return before + inc - v;
}

// bit b of the result = byte b of the 64 flag bytes in w is non-zero
__device__ __forceinline__ unsigned long long flag_words_to_mask(const uint32_t (&w)[16]) {
    uint32_t lo = 0u, hi = 0u;
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        const uint32_t t = (((w[i] & 0x7F7F7F7Fu) + 0x7F7F7F7Fu) | w[i]) & 0x80808080u;      // bit 8b+7 set: byte b non-zero
        const uint32_t four = (t * 0x00204081u) >> 28;                                        // those four bits, packed
        if (i < 8) lo |= four << (4 * i);
        else hi |= four << (4 * (i - 8));
    }
    return (static_cast<unsigned long long>(hi) << 32) | lo;
}

// chunk_count[c] = number of segment starts among the flags of chunk c; masks[c * CMP_THREADS + t] = the 64
// flags of thread t as bits.
// warp_off[c * CMP_WARPS + w] = number of set flags of chunk c in front of warp w's 2048 flags: with it the
// scatter passes need no block-wide barrier, a warp scan of its own 32 counts is enough.
constexpr int CMP_WARPS = CMP_THREADS / 32;
constexpr int CMP_BATCH = 4;               // chunks a block of a scatter pass requests together
__global__ void __launch_bounds__(CMP_THREADS)
flag_count_kernel(const uint8_t* __restrict__ f, long long n, long long nchunks, int32_t* __restrict__ chunk_count,
                  unsigned long long* __restrict__ masks, int32_t* __restrict__ warp_off, bool first_is_start = true) {
    __shared__ int warp_sums[32];
    for (long long c = blockIdx.x; c < nchunks; c += gridDim.x) {
        uint32_t w[16];
        load_thread_flags(f, n, c * CMP_CHUNK + static_cast<long long>(threadIdx.x) * CMP_PER_THREAD, w, first_is_start);
        const unsigned long long m = flag_words_to_mask(w);
        masks[c * CMP_THREADS + threadIdx.x] = m;
        const int cnt = __popcll(m);
        int total;
        const int before = block_exclusive_scan(cnt, &total, warp_sums);
        if ((threadIdx.x & 31) == 0) warp_off[c * CMP_WARPS + (threadIdx.x >> 5)] = before;
        if (threadIdx.x == 0) chunk_count[c] = total;
    }
}

// exclusive scan of one int per lane over the warp
__device__ __forceinline__ int warp_exclusive_scan(int v) {
    const int lane = threadIdx.x & 31;
    int inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += t;
    }
    return inc - v;
}

// ---------------------------------------------------------------------------
// Warps with many set flags.  The scatter passes let every lane walk its own 64-bit mask, which is right for the
// segment-start flags they were built for (one flag in a thousand): a round costs a few instructions and touches
// one element per lane.  With dense flags that loop runs as long as the fullest mask and every access is a sector
// of its own (2^30 flags, half of them set: COMPRESS took 4.7 ms).  A warp whose 2048 flags hold CMP_DENSE_MIN or
// more set ones therefore takes the routes below, after the sparse loop (which stays as small and as fast as it was):
// the warp notes the rounds in which it met such flags and comes back to exactly those.
// ---------------------------------------------------------------------------
constexpr int CMP_WARP_ELEMS = 32 * CMP_PER_THREAD;            // 2048 elements per warp and chunk
constexpr int CMP_DENSE_MIN = 224;          // (about a ninth of the flags: below that the sparse loop measured faster)
// A warp remembers which of its rounds (chunk = block + round * grid) were dense: one bit per round.
constexpr int CMP_DENSE_ROUNDS = 128;       // rounds it can remember (more than any grid here needs); later ones take the sparse loop

// Positions: the warp takes the masks one after the other, lane l the flags l and l + 32 of the mask at hand, so
// that one store instruction writes consecutive offsets.
// m: my mask; slot: output index of my first set flag; wbase: position of the warp's first element.
__device__ __forceinline__ void warp_scatter_positions_dense(unsigned long long m, int slot, long long wbase, int32_t* __restrict__ off) {
    const int lane = threadIdx.x & 31;
    const uint32_t below = (1u << lane) - 1u;
#pragma unroll 4
    for (int j = 0; j < 32; ++j) {
        const unsigned long long mj = __shfl_sync(0xffffffffu, m, j);
        const int sj = __shfl_sync(0xffffffffu, slot, j);
        const uint32_t lo = static_cast<uint32_t>(mj), hi = static_cast<uint32_t>(mj >> 32);
        const int32_t pos = static_cast<int32_t>(wbase + j * CMP_PER_THREAD + lane);
        if ((lo >> lane) & 1u) off[sj + __popc(lo & below)] = pos;
        if ((hi >> lane) & 1u) off[sj + __popc(lo) + __popc(hi & below)] = pos + 32;
    }
}

// Values: the warp reads its 2048 elements as 16-byte vectors, packs the kept ones into shared memory at the
// phase the output has inside a 16-byte vector, and writes them out as 16-byte vectors (elements only at the two
// ragged ends) -- in two halves of 1024 elements, so that eight blocks of the kernel still fit an SM.
// stage: CMP_STAGE_ELEMS elements of this warp, 16-byte aligned.
// slotrel: number of kept elements of the warp in front of my mask; out_start: output index of the warp's first.
constexpr int CMP_STAGE_ELEMS = CMP_WARP_ELEMS / 2 + 16;
template <typename T>
__device__ __forceinline__ void warp_compress_values_dense(const T* __restrict__ x, long long n, long long wbase, unsigned long long m,
                                                        int slotrel, int warp_total, long long out_start, T* __restrict__ out,
                                                        T* __restrict__ stage) {
    constexpr int EPV = 16 / static_cast<int>(sizeof(T));          // elements per vector: 8 or 16
    constexpr int ROUNDS = CMP_WARP_ELEMS / (32 * EPV);
    static_assert(CMP_PER_THREAD % EPV == 0, "a vector lies inside one mask");
    static_assert(ROUNDS % 2 == 0, "two halves");
    const int lane = threadIdx.x & 31;
    const int first_half = __shfl_sync(0xffffffffu, slotrel, 16);      // kept elements among the first 1024
#pragma unroll 1
    for (int half = 0; half < 2; ++half) {
    const long long ostart = out_start + (half ? first_half : 0);
    const int htotal = half ? warp_total - first_half : first_half;
    const int a = static_cast<int>((reinterpret_cast<uintptr_t>(out + ostart) & 15u) / sizeof(T));
#pragma unroll 2
    for (int r = half * (ROUNDS / 2); r < (half + 1) * (ROUNDS / 2); ++r) {
        const int e0 = (r * 32 + lane) * EPV;                      // first element of my vector inside the warp's 2048
        const int j = e0 / CMP_PER_THREAD, b0 = e0 % CMP_PER_THREAD;
        const unsigned long long mj = __shfl_sync(0xffffffffu, m, j);
        const int sj = __shfl_sync(0xffffffffu, slotrel, j);
        uint32_t bits = static_cast<uint32_t>(mj >> b0) & ((1u << EPV) - 1u);
        if (bits == 0u) continue;
        __align__(16) T e[EPV];
        if (wbase + e0 + EPV <= n) {
            *reinterpret_cast<uint4*>(e) = *reinterpret_cast<const uint4*>(x + wbase + e0);
        } else {
#pragma unroll
            for (int t = 0; t < EPV; ++t) e[t] = (wbase + e0 + t < n) ? x[wbase + e0 + t] : T(0);
        }
        int r0 = a + sj - (half ? first_half : 0) + __popcll(mj & ((1ull << b0) - 1ull));
#pragma unroll
        for (int t = 0; t < EPV; ++t) {
            if ((bits >> t) & 1u) stage[r0++] = e[t];
        }
    }
    __syncwarp();
    const int total = a + htotal;
    T* obase = out + (ostart - a);                                  // 16-byte aligned
    for (int i0 = lane * EPV; i0 < total; i0 += 32 * EPV) {
        if (i0 >= a && i0 + EPV <= total) {
            *reinterpret_cast<uint4*>(obase + i0) = *reinterpret_cast<const uint4*>(stage + i0);
        } else {
            for (int t = 0; t < EPV; ++t)
                if (i0 + t >= a && i0 + t < total) obase[i0 + t] = stage[i0 + t];
        }
    }
    __syncwarp();
    }
}

// chunk_base = exclusive scan of chunk_count; K = total is written to nseg_dev and, when given, to the caller's
// d_num_segments; off[K] = n closes the last segment.  A few blocks share the work: block b first adds up the
// counts in front of its part (all its threads, 16-byte loads; the counts are a few hundred KB and stay in the
// L2), then scans its part.  One block alone took 21 us for the 65,536 chunks of 2^30 flags.
constexpr int CMP_SCAN_BLOCKS = 32;
__global__ void __launch_bounds__(1024)
chunk_scan_kernel(const int32_t* __restrict__ chunk_count, long long nchunks, int32_t* __restrict__ chunk_base,
                  long long* __restrict__ nseg_dev, long long* __restrict__ d_num_segments, int32_t* __restrict__ off,
                  long long n) {
    __shared__ int warp_sums[32];
    __shared__ int s_front;
    // parts are multiples of 4 * blockDim.x counts so that every thread reads and writes 16-byte vectors
    const long long unit = 4ll * blockDim.x;
    const long long part = ((nchunks + gridDim.x - 1) / gridDim.x + unit - 1) / unit * unit;
    const long long p0 = static_cast<long long>(blockIdx.x) * part;
    const long long p1 = p0 + part < nchunks ? p0 + part : nchunks;
    // (1) the counts in front of my part
    int front = 0;
    for (long long c = 4ll * threadIdx.x; c < p0; c += unit) {          // p0 is a multiple of 4
        const int4 v = __ldg(reinterpret_cast<const int4*>(chunk_count + c));
        front += v.x + v.y + v.z + v.w;
    }
    int total;
    block_exclusive_scan(front, &total, warp_sums);
    if (threadIdx.x == 0) s_front = total;
    __syncthreads();
    int run_base = s_front;
    // (2) my part: each thread takes `per` consecutive counts, a multiple of four
    const long long per = part / blockDim.x;
    const long long lo = p0 + static_cast<long long>(threadIdx.x) * per;
    const long long hi = lo + per < p1 ? lo + per : p1;
    int local = 0;
    for (long long c = lo; c < hi; c += 4) {
        if (c + 4 <= hi) {
            const int4 v = __ldg(reinterpret_cast<const int4*>(chunk_count + c));
            local += v.x + v.y + v.z + v.w;
        } else {
            for (long long d = c; d < hi; ++d) local += __ldg(chunk_count + d);
        }
    }
    int run = run_base + block_exclusive_scan(local, &total, warp_sums);
    for (long long c = lo; c < hi; c += 4) {
        if (c + 4 <= hi) {
            const int4 v = __ldg(reinterpret_cast<const int4*>(chunk_count + c));
            *reinterpret_cast<int4*>(chunk_base + c) = make_int4(run, run + v.x, run + v.x + v.y, run + v.x + v.y + v.z);
            run += v.x + v.y + v.z + v.w;
        } else {
            for (long long d = c; d < hi; ++d) {
                chunk_base[d] = run;
                run += __ldg(chunk_count + d);
            }
        }
    }
    // the block that holds the last chunk knows the grand total
    if (threadIdx.x == 0 && p0 < nchunks && p1 == nchunks) {
        const int grand = run_base + total;
        *nseg_dev = grand;
        if (d_num_segments) *d_num_segments = grand;
        if (off) off[grand] = static_cast<int32_t>(n);
    }
}

// off[chunk_base[c] + j] = position of the j-th start flag of chunk c (in order).  A chunk is four
// 4096-element spans of the segmented-sum kernel, and the number of starts in front of a span is
// exactly that kernel's span_q entry (the first offset index at or after the span's start), so
// the span partition comes for free here: span_q[s] = #starts before s * 4096, K when the span
// starts at n, K + 1 ("none") beyond.
__global__ void __launch_bounds__(CMP_THREADS, 6)
flag_scatter_kernel(const unsigned long long* __restrict__ masks, long long n, long long nchunks, const int32_t* __restrict__ chunk_base,
                    const int32_t* __restrict__ warp_off, int32_t* __restrict__ off, int32_t* __restrict__ span_q,
                    const long long* __restrict__ nseg_dev) {
    constexpr int kThreadsPerSpan = 4096 / CMP_PER_THREAD;
    const long long K = *nseg_dev;
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        const long long end = nchunks * CMP_CHUNK;
        span_q[nchunks * (CMP_CHUNK / 4096)] = static_cast<int32_t>(end == n ? K : K + 1);
    }
    // (four chunks per round, their loads requested together: the pass is bound by the latency of its loads)
    unsigned long long dense_rounds[CMP_DENSE_ROUNDS / 64] = {0ull, 0ull};
    int round0 = 0;
    for (long long c0 = blockIdx.x; c0 < nchunks; c0 += static_cast<long long>(CMP_BATCH) * gridDim.x, round0 += CMP_BATCH) {
        unsigned long long mk[CMP_BATCH];
        int start[CMP_BATCH];
#pragma unroll
        for (int k = 0; k < CMP_BATCH; ++k) {
            const long long c = c0 + static_cast<long long>(k) * gridDim.x;
            mk[k] = 0ull;
            start[k] = 0;
            if (c < nchunks) {
                mk[k] = masks[c * CMP_THREADS + threadIdx.x];
                start[k] = chunk_base[c] + warp_off[c * CMP_WARPS + (threadIdx.x >> 5)];
            }
        }
#pragma unroll
        for (int k = 0; k < CMP_BATCH; ++k) {
            const long long c = c0 + static_cast<long long>(k) * gridDim.x;
            if (c >= nchunks) break;
            const long long base = c * CMP_CHUNK + static_cast<long long>(threadIdx.x) * CMP_PER_THREAD;
            unsigned long long m = mk[k];
            const int cnt = __popcll(m);
            int slot = start[k] + warp_exclusive_scan(cnt);
            if (threadIdx.x % kThreadsPerSpan == 0)
                span_q[c * (CMP_CHUNK / 4096) + threadIdx.x / kThreadsPerSpan] =
                    static_cast<int32_t>(base < n ? slot : (base == n ? K : K + 1));
            if (__shfl_sync(0xffffffffu, slot + cnt, 31) - start[k] >= CMP_DENSE_MIN && round0 + k < CMP_DENSE_ROUNDS) {
                if (round0 + k < 64) dense_rounds[0] |= 1ull << (round0 + k);
                else dense_rounds[1] |= 1ull << (round0 + k - 64);
                continue;
            }
            while (m) {
                off[slot++] = static_cast<int32_t>(base + (__ffsll(static_cast<long long>(m)) - 1));
                m &= m - 1;
            }
        }
    }
    // the rounds in which this warp met many set flags
#pragma unroll 1
    for (int h = 0; h < CMP_DENSE_ROUNDS / 64; ++h) {
        unsigned long long todo = dense_rounds[h];
        while (todo) {
            const long long c = blockIdx.x + static_cast<long long>(64 * h + __ffsll(static_cast<long long>(todo)) - 1) * gridDim.x;
            todo &= todo - 1;
            const unsigned long long m = masks[c * CMP_THREADS + threadIdx.x];
            const int st = chunk_base[c] + warp_off[c * CMP_WARPS + (threadIdx.x >> 5)];
            const int slot = st + warp_exclusive_scan(__popcll(m));
            warp_scatter_positions_dense(m, slot, c * CMP_CHUNK + static_cast<long long>(threadIdx.x & ~31) * CMP_PER_THREAD, off);
        }
    }
}

// COMPRESS of the values themselves (Section 2): out[chunk_base[c] + j] = the value at the j-th non-zero flag
// of chunk c.  T is the element as stored (2 bytes for fp16 / bf16, 1 byte for int8); nothing is converted.
template <typename T>
__global__ void __launch_bounds__(CMP_THREADS, 8)
compress_values_kernel(const T* __restrict__ x, const unsigned long long* __restrict__ masks, long long n, long long nchunks,
                       const int32_t* __restrict__ chunk_base, const int32_t* __restrict__ warp_off, T* __restrict__ out) {
    __shared__ __align__(16) T stage_all[CMP_WARPS][CMP_STAGE_ELEMS];
    T* stage = stage_all[threadIdx.x >> 5];
    unsigned long long dense_rounds[CMP_DENSE_ROUNDS / 64] = {0ull, 0ull};
    int round0 = 0;
    for (long long c0 = blockIdx.x; c0 < nchunks; c0 += static_cast<long long>(CMP_BATCH) * gridDim.x, round0 += CMP_BATCH) {
        unsigned long long mk[CMP_BATCH];
        int start[CMP_BATCH];
#pragma unroll
        for (int k = 0; k < CMP_BATCH; ++k) {
            const long long c = c0 + static_cast<long long>(k) * gridDim.x;
            mk[k] = 0ull;
            start[k] = 0;
            if (c < nchunks) {
                mk[k] = masks[c * CMP_THREADS + threadIdx.x];
                start[k] = chunk_base[c] + warp_off[c * CMP_WARPS + (threadIdx.x >> 5)];
            }
        }
#pragma unroll
        for (int k = 0; k < CMP_BATCH; ++k) {
            const long long c = c0 + static_cast<long long>(k) * gridDim.x;
            if (c >= nchunks) break;
            const long long base = c * CMP_CHUNK + static_cast<long long>(threadIdx.x) * CMP_PER_THREAD;
            unsigned long long m = mk[k];
            const int cnt = __popcll(m);
            const int rel = warp_exclusive_scan(cnt);
            const int warp_total = __shfl_sync(0xffffffffu, rel + cnt, 31);
            if (warp_total >= CMP_DENSE_MIN && round0 + k < CMP_DENSE_ROUNDS) {
                if (round0 + k < 64) dense_rounds[0] |= 1ull << (round0 + k);
                else dense_rounds[1] |= 1ull << (round0 + k - 64);
                continue;
            }
            long long slot = start[k] + rel;
            while (m) {
                out[slot++] = x[base + (__ffsll(static_cast<long long>(m)) - 1)];
                m &= m - 1;
            }
        }
    }
    // the rounds in which this warp met many kept elements
#pragma unroll 1
    for (int h = 0; h < CMP_DENSE_ROUNDS / 64; ++h) {
        unsigned long long todo = dense_rounds[h];
        while (todo) {
            const long long c = blockIdx.x + static_cast<long long>(64 * h + __ffsll(static_cast<long long>(todo)) - 1) * gridDim.x;
            todo &= todo - 1;
            const unsigned long long m = masks[c * CMP_THREADS + threadIdx.x];
            const int st = chunk_base[c] + warp_off[c * CMP_WARPS + (threadIdx.x >> 5)];
            const int cnt = __popcll(m);
            const int rel = warp_exclusive_scan(cnt);
            warp_compress_values_dense<T>(x, n, c * CMP_CHUNK + static_cast<long long>(threadIdx.x & ~31) * CMP_PER_THREAD, m, rel,
                                          __shfl_sync(0xffffffffu, rel + cnt, 31), st, out, stage);
        }
    }
}

}  // namespace mmv
