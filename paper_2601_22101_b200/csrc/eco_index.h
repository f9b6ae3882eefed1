// Index arithmetic shared by the kernels and their launchers, for every shape the boundary admits
// (rows * cols < 2^34, cols < 2^32).  Plain functions, usable on the host and on the device, so that a
// host-side test can walk them at the admitted maxima (tests/index_arithmetic_check.cpp): nothing here
// may wrap a 32-bit value, because a wrapped loop bound is an endless loop on a GPU.
#pragma once

#include <stdint.h>

#if defined(__CUDACC__)
#define ECO_HD __host__ __device__ __forceinline__
#else
#define ECO_HD inline
#endif

namespace eco {

// ceil(a / b) without forming a + b - 1 (which wraps for a near 2^32).
ECO_HD uint32_t div_ceil_u32(uint32_t a, uint32_t b) { return a / b + (a % b != 0u ? 1u : 0u); }

// Number of valid elements (0..4) of the 4-element tile starting at column c of a row of `cols` columns.
ECO_HD int tile_valid(uint32_t cols, uint64_t c) {
    if (c >= cols) return 0;
    const uint64_t rem = static_cast<uint64_t>(cols) - c;
    return rem > 4 ? 4 : static_cast<int>(rem);
}

// Whether the 32-element scale block g (0..3) of the 128-column chunk j of a row lies inside the row.
ECO_HD bool block32_inside(uint32_t cols, uint32_t j, uint32_t g) {
    return static_cast<uint64_t>(j) * 128u + 32u * g < cols;
}

// eco_dequantize, vector form: work units of `ept` consecutive elements (cols % 16 == 0, so ept | cols).
ECO_HD uint64_t dequant_units(uint64_t rows, uint32_t cols, uint32_t ept) { return rows * (cols / ept); }

// Row and first column of unit u of that form.
ECO_HD void dequant_unit_position(uint64_t u, uint32_t units_per_row, uint32_t ept, uint64_t& row, uint32_t& c0) {
    row = u / units_per_row;
    c0 = static_cast<uint32_t>(u - row * units_per_row) * ept;      // < cols
}

// Index of the scale that unit u of that form reads.  gran: 0 per tensor, 1 per matrix row, 2 per block of `block`
// elements of a row.  shift >= 0 says that every row is made of whole blocks of 2^shift elements, so the blocks of the
// tensor are numbered like its elements divided by the block length and no division is needed.  Otherwise the row
// comes from ONE 32-bit division: u < n_units <= 2^32 - 4 for every admitted shape.
ECO_HD uint64_t dequant_scale_index(uint64_t u, uint32_t units_per_row, uint32_t ept, int gran, uint32_t block,
                                    uint32_t scales_per_row, int shift) {
    if (gran == 0) return 0;
    if (gran == 2 && shift >= 0) return (u * ept) >> shift;
    const uint32_t u32 = static_cast<uint32_t>(u);
    const uint32_t row = u32 / units_per_row;
    if (gran == 1) return row;
    const uint32_t c0 = (u32 - row * units_per_row) * ept;           // < cols
    return static_cast<uint64_t>(row) * scales_per_row + c0 / block;
}

// Tickets of a persistent launch over n_units work units walked as W regions: W * ceil(n_units / W).  The
// unit tables hold at most 2^31 - 1 units, so this (and the few tickets every CTA draws past the end) fits 32 bits.
ECO_HD uint32_t ticket_count(uint32_t n_units, uint32_t W) { return div_ceil_u32(n_units, W) * W; }

}  // namespace eco
