// Shared constants and small helpers of the segmented-operation kernels.
#pragma once
#include <cstdint>
#include <cuda_fp16.h>
#include "ptx.cuh"

namespace mmv {

// Geometry.  The value vector is viewed as rows of CHUNK consecutive elements
// (the paper's ceil(n/s) x s matrix view of MATMUL(x, U_s), with s = CHUNK).  A
// warp owns a SPAN of NCOL consecutive rows: its 32 lanes are the 32 positions
// of a row and the rows are the columns of its TMEM accumulator.  A TILE is the
// four spans handled by the four warps of one epilogue warpgroup and is the
// unit of one tensor-core product.
constexpr int CHUNK = 32;
constexpr int NCOL = 128;
constexpr int SPAN = CHUNK * NCOL;       // 4096 elements
constexpr int SPANS_PER_TILE = 4;
constexpr int TILE = SPANS_PER_TILE * SPAN;   // 16384 elements
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
    static constexpr int kRowBytes = CHUNK * 2;            // 64-byte rows -> 64-byte swizzle
    static constexpr int kSlabBytes = NCOL * kRowBytes;    // one K-slab of an operand: 8 KB
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
};
struct I8Path {
    using Acc = uint32_t;                                  // wrap-around arithmetic on unsigned
    static constexpr int kElemBytes = 1;
    static constexpr bool kIsFloat = false;
    static constexpr int kRowBytes = CHUNK;                // 32-byte rows -> 32-byte swizzle
    static constexpr int kSlabBytes = NCOL * kRowBytes;    // 4 KB
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

// Shared-memory matrix descriptor of a K-major swizzled slab (see ptx.cuh for the fields).
__device__ __forceinline__ uint64_t make_desc(uint32_t addr, uint32_t sbo_bytes, uint32_t layout_type) {
    uint64_t d = 0;
    d |= static_cast<uint64_t>((addr & 0x3FFFFu) >> 4);
    d |= static_cast<uint64_t>(1) << 16;
    d |= static_cast<uint64_t>(sbo_bytes >> 4) << 32;
    d |= static_cast<uint64_t>(1) << 46;
    d |= static_cast<uint64_t>(layout_type) << 61;
    return d;
}

__device__ __forceinline__ void report_error(WorkspaceHeader* hdr, unsigned int code) {
    atomicCAS(&hdr->error, 0u, code);
}

}  // namespace mmv
