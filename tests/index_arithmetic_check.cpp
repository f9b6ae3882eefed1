// Host-side walk of the kernels' index arithmetic (paper_2601_22101_b200/csrc/eco_index.h) at the largest shapes
// the boundary admits (rows * cols < 2^34, cols < 2^32).  Built with g++ and run by
// tests/test_index_arithmetic_cpu.py; exits 0 and prints "ok" when every check holds.  No GPU involved:
// a loop bound that wraps would be an endless loop on the device, so it is walked here instead.
#include <cstdint>
#include <cstdio>
#include <cstdlib>
#include <initializer_list>

#include "../paper_2601_22101_b200/csrc/eco_index.h"

#define CHECK(cond)                                                          \
    do {                                                                     \
        if (!(cond)) {                                                       \
            std::printf("FAILED line %d: %s\n", __LINE__, #cond);            \
            return 1;                                                        \
        }                                                                    \
    } while (0)

int main() {
    using namespace eco;
    // ---- ceilings at cols = 2^32 - 1, where cols + d - 1 wraps to a small number ----
    const uint32_t big = 0xFFFFFFFFu;
    CHECK(div_ceil_u32(big, 128u) == (1u << 25));
    CHECK(div_ceil_u32(big, 32u) == (1u << 27));
    CHECK(div_ceil_u32(big, 4u) == (1u << 30));
    CHECK((big + 127u) / 128u == 0u);                     // the form that must not be used
    CHECK(div_ceil_u32(10944u, 128u) == 86u && div_ceil_u32(128u, 128u) == 1u && div_ceil_u32(1u, 4u) == 1u);

    // ---- one CTA per row: thread t walks columns 4t, 4t + 1024, ... (256 threads) ----
    for (uint32_t cols : {big, big - 1023u, big - 1024u, 0xFFFFFC00u, 4097u, 1u}) {
        for (uint32_t t : {0u, 1u, 255u}) {
            uint64_t iters = 0, valid = 0;
            for (uint64_t c = 4u * t; c < cols; c += 1024u) {
                CHECK(++iters <= (1ull << 23));           // ends: at most 2^32 / 1024 trips
                valid += static_cast<uint64_t>(tile_valid(cols, c));
                CHECK(c + 3 < cols || tile_valid(cols, c) == static_cast<int>(cols - c));
            }
            // what a 32-bit counter would do on the last trip for thread 0 of the longest rows: wrap and go on
            if (t == 0 && cols > 0xFFFFFC00u) {
                const uint32_t last = (cols - 1u) / 1024u * 1024u;
                CHECK(static_cast<uint32_t>(last + 1024u) < cols);
            }
            (void)valid;
        }
    }
    CHECK(tile_valid(10u, 8) == 2 && tile_valid(10u, 12) == 0 && tile_valid(big, 0xFFFFFFFCull) == 3);
    {   // every column of a long row is covered exactly once
        const uint32_t cols = 0xFFFFFFFBu;
        uint64_t covered = 0;
        for (uint64_t c = 0; c < cols; c += 4) covered += static_cast<uint64_t>(tile_valid(cols, c));
        CHECK(covered == cols);
    }

    // ---- eco_dequantize, vector form, largest tensor: 2^34 - 16 elements, 4 per unit ----
    {
        const uint64_t rows = (1ull << 30) - 1;
        const uint32_t cols = 16u, ept = 4u;
        const uint64_t n_units = dequant_units(rows, cols, ept);
        CHECK(n_units == (1ull << 32) - 4);
        const uint64_t stride = 148ull * 16 * 256;
        uint64_t wrapped_32 = 0;
        for (uint64_t first : {uint64_t(0), uint64_t(1), stride / 2, stride - 1}) {
            uint64_t iters = 0, u = first, last = first;
            for (; u < n_units; u += stride) {
                CHECK(++iters <= 8192);
                last = u;
            }
            CHECK(u >= n_units && u - stride == last);
            // the 32-bit counter this replaces: does last + stride wrap to below n_units?
            if (static_cast<uint32_t>(static_cast<uint32_t>(last) + static_cast<uint32_t>(stride)) < n_units &&
                last + stride >= (1ull << 32))
                ++wrapped_32;
        }
        CHECK(wrapped_32 > 0);                            // it did, for some threads: the reason for 64 bits
        uint64_t row;
        uint32_t c0;
        dequant_unit_position(n_units - 1, cols / ept, ept, row, c0);
        CHECK(row == rows - 1 && c0 == cols - ept);
        dequant_unit_position(0, cols / ept, ept, row, c0);
        CHECK(row == 0 && c0 == 0);
        // a wide matrix: 3 rows of 2^32 - 16 columns, 8 elements per unit
        const uint32_t wide = 0xFFFFFFF0u;
        CHECK(dequant_units(3, wide, 8u) == 3ull * (wide / 8u));
        dequant_unit_position(3ull * (wide / 8u) - 1, wide / 8u, 8u, row, c0);
        CHECK(row == 2 && c0 == wide - 8u);
    }

    // ---- scale index of a unit of that form, against the definition (row * scales per row + column / block) ----
    {
        struct Shape { uint64_t rows; uint32_t cols, ept, block; };
        const Shape shapes[] = {{(1ull << 30) - 1, 16u, 4u, 128u}, {3, 0xFFFFFFF0u, 8u, 128u}, {1ull << 20, 16384u - 128u, 8u, 128u},
                                {5, 208u, 4u, 128u}, {7, 4096u, 8u, 32u}, {9, 48u, 8u, 32u}, {(1ull << 27), 96u, 4u, 32u}};
        for (const Shape& sh : shapes) {
            const uint32_t upr = sh.cols / sh.ept, spr = div_ceil_u32(sh.cols, sh.block);
            const uint64_t n_units = dequant_units(sh.rows, sh.cols, sh.ept);
            CHECK(n_units <= (1ull << 32) - 4);
            const int shift = sh.cols % sh.block == 0u ? (sh.block == 128u ? 7 : 5) : -1;
            const uint64_t probes[] = {0, 1, upr - 1ull, upr, n_units / 2, n_units / 3 + 5, n_units - 2, n_units - 1};
            for (uint64_t u : probes) {
                if (u >= n_units) continue;
                uint64_t row;
                uint32_t c0;
                dequant_unit_position(u, upr, sh.ept, row, c0);
                CHECK(dequant_scale_index(u, upr, sh.ept, 0, sh.block, spr, -1) == 0);
                CHECK(dequant_scale_index(u, upr, sh.ept, 1, sh.block, spr, -1) == row);
                CHECK(dequant_scale_index(u, upr, sh.ept, 2, sh.block, spr, -1) == row * spr + c0 / sh.block);
                if (shift >= 0) CHECK(dequant_scale_index(u, upr, sh.ept, 2, sh.block, spr, shift) == row * spr + c0 / sh.block);
            }
        }
    }

    // ---- 1x32 blocks inside ragged rows ----
    CHECK(block32_inside(200u, 1u, 2u) && !block32_inside(200u, 1u, 3u) && block32_inside(193u, 1u, 2u));
    CHECK(block32_inside(big, (1u << 25) - 1u, 3u) && !block32_inside(0xFFFFFF9Cu, (1u << 25) - 1u, 1u));

    // ---- ticket counts of the persistent launches: unit tables hold at most 2^31 - 1 units ----
    CHECK(ticket_count(0x7FFFFFFFu, 8u) == 0x80000000u);
    CHECK(ticket_count(1u, 8u) == 8u && ticket_count(16u, 8u) == 16u && ticket_count(17u, 1u) == 17u);
    std::printf("ok\n");
    return 0;
}
