// Range arithmetic of A2SGD_DEBUG_CHECKS, shared by the device accessors and by a host-compiled
// unit test (this header is plain C++: no CUDA types).
//
// A range describes one caller buffer as `rows` rows of `row_bytes` live bytes, row r starting at
// base + r * stride_bytes (stride_bytes == 0: a single row).  An access of `bytes` bytes at `addr`
// is inside the range when it lies entirely within the live part of one row — not in the padding
// between rows, not past the last row, not straddling a row end.
#pragma once

#include <stdint.h>

#if defined(__CUDACC__)
#define A2SGD_HD __host__ __device__ __forceinline__
#else
#define A2SGD_HD inline
#endif

namespace a2sgd_check {

struct DebugRange {
    uint64_t base;         // address of row 0
    uint64_t stride_bytes; // distance between rows (0: one row)
    uint64_t row_bytes;    // live bytes per row
    uint64_t rows;
};

A2SGD_HD bool debug_range_contains(const DebugRange &r, uint64_t addr, uint64_t bytes)
{
    if (r.rows == 0 || addr < r.base) return false;
    const uint64_t off = addr - r.base;
    uint64_t row = 0, col = off;
    if (r.stride_bytes != 0) {
        row = off / r.stride_bytes;
        col = off - row * r.stride_bytes;
    }
    if (row >= r.rows) return false;
    return col + bytes <= r.row_bytes && col + bytes >= col; // second clause: no wrap-around
}

constexpr int kDebugMaxRanges = 8;

A2SGD_HD bool debug_any_range_contains(const DebugRange *ranges, int count, uint64_t addr, uint64_t bytes)
{
    for (int k = 0; k < count && k < kDebugMaxRanges; ++k)
        if (debug_range_contains(ranges[k], addr, bytes)) return true;
    return false;
}

// Index form, for buffers that are not described by a range (the tensors of a segment list):
// `count` elements starting at element `first` of a tensor of `numel` elements.
A2SGD_HD bool debug_span_inside(uint64_t first, uint64_t count, uint64_t numel)
{
    return first + count <= numel && first + count >= first;
}

} // namespace a2sgd_check
