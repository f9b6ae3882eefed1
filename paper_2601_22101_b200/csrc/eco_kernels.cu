// Kernels of the ECO step (Algorithm 1-3) for sm_100a and their launchers.
//
// Work decomposition.  A tensor is cut into rows of 128 consecutive elements;
// a warp owns 4 such rows at a time and lane l owns elements 4l..4l+3 of each,
// so that every global access of the warp is one contiguous span (16 B per
// lane for m and v, 8 B for the bf16 gradient, 4 B / 2 B for FP8 / INT4
// codes).  A CTA of 8 warps owns one "unit" of 32 rows (4096 elements).  A
// launch covers the units of many tensors: unit -> tensor through a table
// built at eco_create.
//
//   1x128 block scales : one pass.  The 128-element row IS the scale block; its
//                        amax is a warp reduction, no memory traffic beyond
//                        the algorithmic bytes.
//   per-tensor scale   : two kernels.  Pass 1 recomputes theta~ and reduces
//                        max|theta~| into a per-tensor slot (atomicMax on the
//                        bit pattern of a non-negative float: exact and
//                        order-free); pass 2 recomputes theta~ and finishes.
//   per-row scale      : one CTA per row, two loops over the row (the second
//                        loop re-reads the row from L1/L2).
#include <algorithm>

#include "eco_device.cuh"
#include "eco_index.h"
#include "eco_launch.h"

namespace eco {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kRowsPerWarp = 4;
constexpr int kRowsPerUnit = kWarps * kRowsPerWarp;   // 32 rows of 128 = 4096 elements

// Reduce 4 per-lane maxima (one per row) over the warp.  Afterwards every lane
// of lane-group g = lane / 8 holds the maximum of row g.  6 shuffles instead of 20.
__device__ __forceinline__ float reduce_rows4(const float a[4], int lane) {
    const bool b4 = lane & 16, b3 = lane & 8;
    const float send_x = b4 ? a[0] : a[2], send_y = b4 ? a[1] : a[3];
    const float keep_x = b4 ? a[2] : a[0], keep_y = b4 ? a[3] : a[1];
    const float x = fmaxf(keep_x, __shfl_xor_sync(0xFFFFFFFFu, send_x, 16));
    const float y = fmaxf(keep_y, __shfl_xor_sync(0xFFFFFFFFu, send_y, 16));
    const float send = b3 ? x : y, keep = b3 ? y : x;
    float z = fmaxf(keep, __shfl_xor_sync(0xFFFFFFFFu, send, 8));
    z = fmaxf(z, __shfl_xor_sync(0xFFFFFFFFu, z, 4));
    z = fmaxf(z, __shfl_xor_sync(0xFFFFFFFFu, z, 2));
    z = fmaxf(z, __shfl_xor_sync(0xFFFFFFFFu, z, 1));
    return z;
}

__device__ __forceinline__ float warp_max(float z) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) z = fmaxf(z, __shfl_xor_sync(0xFFFFFFFFu, z, o));
    return z;
}

// Element range of row `blk` for the lane.
template <bool GENERIC>
__device__ __forceinline__ void row_extent(const TensorDesc& T, uint64_t blk, int lane, uint64_t& i0, int& nvalid, bool& vec) {
    if (!GENERIC) {
        i0 = blk * 128 + 4 * lane;
        nvalid = blk < T.n_blocks ? 4 : 0;
        vec = true;
        return;
    }
    if (blk >= T.n_blocks) { i0 = 0; nvalid = 0; vec = false; return; }
    const uint64_t row = blk / T.blocks_per_row;
    const uint32_t j = static_cast<uint32_t>(blk - row * T.blocks_per_row);
    const uint32_t c0 = j * 128u;
    const uint32_t len = min(128u, T.cols - c0);
    const uint64_t start = row * T.cols + c0;
    i0 = start + 4 * lane;
    const int rem = static_cast<int>(len) - 4 * lane;
    nvalid = rem < 0 ? 0 : (rem > 4 ? 4 : rem);
    vec = (start & 3) == 0;
}

// Maximum over each group of 8 lanes (one 32-element scale block); every lane of the group gets it.
__device__ __forceinline__ float group8_max(float z) {
    z = fmaxf(z, __shfl_xor_sync(0xFFFFFFFFu, z, 4));
    z = fmaxf(z, __shfl_xor_sync(0xFFFFFFFFu, z, 2));
    z = fmaxf(z, __shfl_xor_sync(0xFFFFFFFFu, z, 1));
    return z;
}

// Index of the scale of 32-element block g (0..3) of 128-element chunk `blk`; the chunk's blocks that lie
// inside the row are those with 128 j + 32 g < cols.
template <bool GENERIC>
__device__ __forceinline__ bool scale32_index(const TensorDesc& T, uint64_t blk, int g, uint64_t& k) {
    if (blk >= T.n_blocks) return false;
    if (!GENERIC) { k = blk * 4 + g; return true; }
    const uint64_t row = blk / T.blocks_per_row;
    const uint32_t j = static_cast<uint32_t>(blk - row * T.blocks_per_row);
    k = row * T.scales_per_row + j * 4u + g;
    return block32_inside(T.cols, j, static_cast<uint32_t>(g));
}

// ---------------------------------------------------------------------------
// Block scales along the row: the whole step in one pass.  A warp handles chunks of 128 consecutive elements
// of a row; SUB = 1: the chunk is one scale block (1x128), SUB = 4: four blocks of 32 (8 lanes each).
// GENERIC = false: cols is a multiple of 128, so chunk k is elements
// 128k..128k+127 of the flat tensor.  GENERIC = true: any cols; the last chunk
// of a row may be short and rows need not start on a 4-element boundary.
// ---------------------------------------------------------------------------
template <int FMT, int OPT, int RND, bool GENERIC, int SUB>
__global__ void __launch_bounds__(kThreads)
eco_block128_kernel(const TensorDesc* __restrict__ descs, const uint32_t* __restrict__ unit_tensor,
                    const StepParams P, const int scale_kind) {
    const uint32_t unit = blockIdx.x;
    const TensorDesc T = descs[unit_tensor[unit]];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint64_t blk0 = static_cast<uint64_t>(unit - T.first_unit) * kRowsPerUnit + warp * kRowsPerWarp;
    if (blk0 >= T.n_blocks) return;

    Lane4<OPT> L[kRowsPerWarp];
    uint64_t i0[kRowsPerWarp];
    int nvalid[kRowsPerWarp];
    bool vec[kRowsPerWarp];
    float amax[kRowsPerWarp];
    const int g = lane >> 3;
    if constexpr (SUB == 4) {
#pragma unroll
        for (int k = 0; k < kRowsPerWarp; ++k) {
            row_extent<GENERIC>(T, blk0 + k, lane, i0[k], nvalid[k], vec[k]);
            uint64_t sk;
            const bool present = scale32_index<GENERIC>(T, blk0 + k, g, sk);
            const float s_old = present ? load_scale(T.scale, sk, scale_kind) : 1.0f;
            amax[k] = lane_front<FMT, OPT>(T, P, i0[k], nvalid[k], vec[k], s_old, L[k], true);
        }
#pragma unroll
        for (int k = 0; k < kRowsPerWarp; ++k) {
            float s, inv;
            uint32_t bits;
            make_scale<FMT>(group8_max(amax[k]), scale_kind, s, inv, bits);
            uint64_t sk;
            if (scale32_index<GENERIC>(T, blk0 + k, g, sk) && (lane & 7) == 0) store_scale(T.scale, sk, scale_kind, s, bits);
            lane_back<FMT, OPT, RND>(T, P, i0[k], nvalid[k], vec[k], s, inv, L[k]);
        }
    } else {
#pragma unroll
        for (int k = 0; k < kRowsPerWarp; ++k) {
            row_extent<GENERIC>(T, blk0 + k, lane, i0[k], nvalid[k], vec[k]);
            const float s_old = (blk0 + k < T.n_blocks) ? load_scale(T.scale, blk0 + k, scale_kind) : 1.0f;
            amax[k] = lane_front<FMT, OPT>(T, P, i0[k], nvalid[k], vec[k], s_old, L[k], true);
        }
        const float my_amax = reduce_rows4(amax, lane);   // row (lane / 8)
        float s_mine, inv_mine;
        uint32_t bits_mine;
        make_scale<FMT>(my_amax, scale_kind, s_mine, inv_mine, bits_mine);
        if ((lane & 7) == 0 && blk0 + g < T.n_blocks) store_scale(T.scale, blk0 + g, scale_kind, s_mine, bits_mine);
#pragma unroll
        for (int k = 0; k < kRowsPerWarp; ++k) {
            const float s = __shfl_sync(0xFFFFFFFFu, s_mine, 8 * k);
            const float inv = __shfl_sync(0xFFFFFFFFu, inv_mine, 8 * k);
            lane_back<FMT, OPT, RND>(T, P, i0[k], nvalid[k], vec[k], s, inv, L[k]);
        }
    }
}

// ---------------------------------------------------------------------------
// Per-tensor scale, pass 1: max |theta~| over the tensor.
// scratch_amax[slot] accumulates the bit pattern; unit 0 also saves the old scale.
// ---------------------------------------------------------------------------
template <int FMT, int OPT>
__global__ void __launch_bounds__(kThreads)
eco_tensor_amax_kernel(const TensorDesc* __restrict__ descs, const uint32_t* __restrict__ unit_tensor,
                       const StepParams P, const int scale_kind,
                       uint32_t* __restrict__ scratch_amax, float* __restrict__ scratch_s_old) {
    __shared__ float smax[kWarps];
    const uint32_t unit = blockIdx.x;
    const TensorDesc T = descs[unit_tensor[unit]];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t local = unit - T.first_unit;
    const uint64_t blk0 = static_cast<uint64_t>(local) * kRowsPerUnit + warp * kRowsPerWarp;
    const float s_old = load_scale(T.scale, 0, scale_kind);
    if (local == 0 && threadIdx.x == 0) scratch_s_old[T.slot] = s_old;
    float amax = 0.0f;
#pragma unroll
    for (int k = 0; k < kRowsPerWarp; ++k) {
        const uint64_t i0 = (blk0 + k) * 128 + 4 * lane;
        const int64_t rem = static_cast<int64_t>(T.numel) - static_cast<int64_t>(i0);
        const int nvalid = rem < 0 ? 0 : (rem > 4 ? 4 : static_cast<int>(rem));
        Lane4<OPT> L;
        amax = fmaxf(amax, lane_front<FMT, OPT>(T, P, i0, nvalid, true, s_old, L, false));
    }
    amax = warp_max(amax);
    if (lane == 0) smax[warp] = amax;
    __syncthreads();
    if (threadIdx.x == 0) {
        float a = smax[0];
#pragma unroll
        for (int i = 1; i < kWarps; ++i) a = fmaxf(a, smax[i]);
        atomicMax(scratch_amax + T.slot, __float_as_uint(a));
    }
}

// Per-tensor scale, pass 2: recompute theta~, quantize with the tensor's scale, inject, store.
// Also clears the amax slot of the NEXT step (the two slots alternate by step parity).
template <int FMT, int OPT, int RND>
__global__ void __launch_bounds__(kThreads)
eco_tensor_apply_kernel(const TensorDesc* __restrict__ descs, const uint32_t* __restrict__ unit_tensor,
                        const StepParams P, const int scale_kind,
                        const uint32_t* __restrict__ scratch_amax, uint32_t* __restrict__ scratch_amax_next,
                        const float* __restrict__ scratch_s_old, const int reverse, const uint32_t n_units) {
    const uint32_t unit = reverse ? (n_units - 1 - blockIdx.x) : blockIdx.x;
    const TensorDesc T = descs[unit_tensor[unit]];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t local = unit - T.first_unit;
    const uint64_t blk0 = static_cast<uint64_t>(local) * kRowsPerUnit + warp * kRowsPerWarp;
    const float s_old = scratch_s_old[T.slot];
    float s, inv;
    uint32_t s_bits;
    make_scale<FMT>(__uint_as_float(scratch_amax[T.slot]), scale_kind, s, inv, s_bits);
    if (local == 0 && threadIdx.x == 0) {
        store_scale(T.scale, 0, scale_kind, s, s_bits);
        scratch_amax_next[T.slot] = 0u;
    }
#pragma unroll
    for (int k = 0; k < kRowsPerWarp; ++k) {
        const uint64_t i0 = (blk0 + k) * 128 + 4 * lane;
        const int64_t rem = static_cast<int64_t>(T.numel) - static_cast<int64_t>(i0);
        const int nvalid = rem < 0 ? 0 : (rem > 4 ? 4 : static_cast<int>(rem));
        if (nvalid == 0) continue;
        Lane4<OPT> L;
        lane_front<FMT, OPT>(T, P, i0, nvalid, true, s_old, L, true);
        lane_back<FMT, OPT, RND>(T, P, i0, nvalid, true, s, inv, L);
    }
}

// ---------------------------------------------------------------------------
// Per-row scale: one CTA per row, two loops over the row.
// ---------------------------------------------------------------------------
template <int FMT, int OPT, int RND>
__global__ void __launch_bounds__(kThreads)
eco_row_kernel(const TensorDesc* __restrict__ descs, const uint32_t* __restrict__ unit_tensor,
               const StepParams P, const int scale_kind) {
    __shared__ float smax[kWarps];
    __shared__ float s_sh, inv_sh;
    const uint32_t unit = blockIdx.x;
    const TensorDesc T = descs[unit_tensor[unit]];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint64_t row = unit - T.first_unit;
    const uint64_t start = row * T.cols;
    const bool vec = (start & 3) == 0;
    const float s_old = load_scale(T.scale, row, scale_kind);
    float amax = 0.0f;
    // 64-bit column counter: cols may be anything below 2^32, and c + 1024 must not wrap
    for (uint64_t c = 4 * threadIdx.x; c < T.cols; c += 4 * kThreads) {
        Lane4<OPT> L;
        amax = fmaxf(amax, lane_front<FMT, OPT>(T, P, start + c, tile_valid(T.cols, c), vec, s_old, L, false));
    }
    amax = warp_max(amax);
    if (lane == 0) smax[warp] = amax;
    __syncthreads();
    if (threadIdx.x == 0) {
        float a = smax[0];
#pragma unroll
        for (int i = 1; i < kWarps; ++i) a = fmaxf(a, smax[i]);
        float s, inv;
        uint32_t s_bits;
        make_scale<FMT>(a, scale_kind, s, inv, s_bits);
        store_scale(T.scale, row, scale_kind, s, s_bits);
        s_sh = s;
        inv_sh = inv;
    }
    __syncthreads();
    const float s = s_sh, inv = inv_sh;
    for (uint64_t c = 4 * threadIdx.x; c < T.cols; c += 4 * kThreads) {
        const int nvalid = tile_valid(T.cols, c);
        Lane4<OPT> L;
        lane_front<FMT, OPT>(T, P, start + c, nvalid, vec, s_old, L, true);
        lane_back<FMT, OPT, RND>(T, P, start + c, nvalid, vec, s, inv, L);
    }
}

// ---------------------------------------------------------------------------
// q(x) for the initial state: theta~ = x (f32 input), same scale and rounding rules.
// mode 0: per-tensor pass 1 (amax only); 1: per-tensor pass 2; 2: per-row; 3: 1x128 blocks.
// One warp per 128-element row of work (blocks), one CTA per row (rows),
// grid-stride over 1024-element tiles (tensor).
// ---------------------------------------------------------------------------
template <int FMT, int RND>
__device__ __forceinline__ void quantize_lane(const float* x, uint8_t* w, uint64_t i0, int nvalid, bool vec,
                                              float s_inv, const StepParams& P, uint32_t tensor_id) {
    float xv[4];
    load_f32x4(x, i0, nvalid, vec, xv);
    uint32_t word[4] = {0u, 0u, 0u, 0u};
    if (RND == RND_SR) random_words4(P, tensor_id, i0, vec, word);
    float y[4], q[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) y[e] = __fmul_rn(xv[e], s_inv);
    round4<FMT, RND>(y, word, q);
    store_codes4<FMT>(w, i0, nvalid, vec, pack4<FMT>(q));
}

__device__ __forceinline__ float amax_lane(const float* x, uint64_t i0, int nvalid, bool vec) {
    float xv[4];
    load_f32x4(x, i0, nvalid, vec, xv);
    float a = 0.0f;
#pragma unroll
    for (int e = 0; e < 4; ++e)
        if (e < nvalid) a = fmaxf(a, fabsf(xv[e]));
    return a;
}

template <int FMT, int RND>
__global__ void __launch_bounds__(kThreads)
eco_quantize_kernel(const float* __restrict__ x, uint8_t* __restrict__ w, void* __restrict__ scale,
                    const uint64_t rows, const uint32_t cols, const int mode, const int scale_kind,
                    const StepParams P, const uint32_t tensor_id, uint32_t* __restrict__ scratch_amax) {
    __shared__ float smax[kWarps];
    __shared__ float s_sh, inv_sh;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint64_t numel = rows * cols;
    if (mode == 0 || mode == 1) {
        float s = 0.f, inv = 0.f;
        uint32_t s_bits;
        if (mode == 1) {
            make_scale<FMT>(__uint_as_float(*scratch_amax), scale_kind, s, inv, s_bits);
            if (blockIdx.x == 0 && threadIdx.x == 0) store_scale(scale, 0, scale_kind, s, s_bits);
        }
        float amax = 0.0f;
        for (uint64_t i0 = (static_cast<uint64_t>(blockIdx.x) * kThreads + threadIdx.x) * 4; i0 < numel;
             i0 += static_cast<uint64_t>(gridDim.x) * kThreads * 4) {
            const uint64_t rem = numel - i0;
            const int nvalid = rem > 4 ? 4 : static_cast<int>(rem);
            if (mode == 0) amax = fmaxf(amax, amax_lane(x, i0, nvalid, true));
            else quantize_lane<FMT, RND>(x, w, i0, nvalid, true, inv, P, tensor_id);
        }
        if (mode == 0) {
            amax = warp_max(amax);
            if (lane == 0) atomicMax(scratch_amax, __float_as_uint(amax));
        }
        return;
    }
    if (mode == 2) {
        for (uint64_t row = blockIdx.x; row < rows; row += gridDim.x) {
            const uint64_t start = row * cols;
            const bool vec = (start & 3) == 0;
            float amax = 0.0f;
            for (uint64_t c = 4 * threadIdx.x; c < cols; c += 4 * kThreads)
                amax = fmaxf(amax, amax_lane(x, start + c, tile_valid(cols, c), vec));
            amax = warp_max(amax);
            if (lane == 0) smax[warp] = amax;
            __syncthreads();
            if (threadIdx.x == 0) {
                float a = smax[0];
                for (int i = 1; i < kWarps; ++i) a = fmaxf(a, smax[i]);
                float s, inv;
                uint32_t s_bits;
                make_scale<FMT>(a, scale_kind, s, inv, s_bits);
                store_scale(scale, row, scale_kind, s, s_bits);
                s_sh = s;
                inv_sh = inv;
            }
            __syncthreads();
            const float inv = inv_sh;
            for (uint64_t c = 4 * threadIdx.x; c < cols; c += 4 * kThreads)
                quantize_lane<FMT, RND>(x, w, start + c, tile_valid(cols, c), vec, inv, P, tensor_id);
            __syncthreads();
        }
        return;
    }
    // mode 3 / 4: one warp per chunk of 128 elements of a row = one scale block (mode 3) or four of 32 (mode 4)
    const uint32_t bpr = div_ceil_u32(cols, 128u);
    const uint64_t n_blocks = rows * bpr;
    for (uint64_t blk = static_cast<uint64_t>(blockIdx.x) * kWarps + warp; blk < n_blocks;
         blk += static_cast<uint64_t>(gridDim.x) * kWarps) {
        const uint64_t row = blk / bpr;
        const uint32_t c0 = static_cast<uint32_t>(blk - row * bpr) * 128u;
        const uint32_t len = min(128u, cols - c0);
        const uint64_t start = row * cols + c0;
        const bool vec = (start & 3) == 0;
        const int rem = static_cast<int>(len) - 4 * lane;
        const int nvalid = rem < 0 ? 0 : (rem > 4 ? 4 : rem);
        const float mine = amax_lane(x, start + 4 * lane, nvalid, vec);
        float s, inv;
        uint32_t s_bits;
        if (mode == 4) {
            make_scale<FMT>(group8_max(mine), scale_kind, s, inv, s_bits);
            const uint32_t g = static_cast<uint32_t>(lane) >> 3;
            if ((lane & 7) == 0 && block32_inside(cols, c0 / 128u, g))
                store_scale(scale, row * div_ceil_u32(cols, 32u) + c0 / 32u + g, scale_kind, s, s_bits);
        } else {
            make_scale<FMT>(warp_max(mine), scale_kind, s, inv, s_bits);
            if (lane == 0) store_scale(scale, blk, scale_kind, s, s_bits);
        }
        quantize_lane<FMT, RND>(x, w, start + 4 * lane, nvalid, vec, inv, P, tensor_id);
    }
}

// ---------------------------------------------------------------------------
// Launchers: runtime configuration -> template instance.
// ---------------------------------------------------------------------------
#define ECO_DISPATCH_FMT(fmt, ...)                                   \
    if ((fmt) == FMT_FP8) { constexpr int F = FMT_FP8; __VA_ARGS__ } \
    else if ((fmt) == FMT_E5M2) { constexpr int F = FMT_E5M2; __VA_ARGS__ } \
    else { constexpr int F = FMT_INT4; __VA_ARGS__ }
#define ECO_DISPATCH_OPT(opt, ...)                                    \
    if ((opt) == OPT_SGDM) { constexpr int O = OPT_SGDM; __VA_ARGS__ } \
    else { constexpr int O = OPT_ADAM; __VA_ARGS__ }
#define ECO_DISPATCH_RND(rnd, ...)                                  \
    if ((rnd) == RND_RTN) { constexpr int R = RND_RTN; __VA_ARGS__ } \
    else { constexpr int R = RND_SR; __VA_ARGS__ }

cudaError_t launch_block128(const LaunchConfig& c, const TensorDesc* descs, const uint32_t* unit_tensor,
                            uint32_t n_units, bool generic, const StepParams& P, cudaStream_t stream) {
    if (n_units == 0) return cudaSuccess;
    ECO_DISPATCH_FMT(c.format, ECO_DISPATCH_OPT(c.optimizer, ECO_DISPATCH_RND(c.rounding, {
        if (c.sub == 4) {
            if (generic) eco_block128_kernel<F, O, R, true, 4><<<n_units, kThreads, 0, stream>>>(descs, unit_tensor, P, c.scale_kind);
            else eco_block128_kernel<F, O, R, false, 4><<<n_units, kThreads, 0, stream>>>(descs, unit_tensor, P, c.scale_kind);
        } else {
            if (generic) eco_block128_kernel<F, O, R, true, 1><<<n_units, kThreads, 0, stream>>>(descs, unit_tensor, P, c.scale_kind);
            else eco_block128_kernel<F, O, R, false, 1><<<n_units, kThreads, 0, stream>>>(descs, unit_tensor, P, c.scale_kind);
        }
    })))
    return cudaGetLastError();
}

cudaError_t launch_tensor_amax(const LaunchConfig& c, const TensorDesc* descs, const uint32_t* unit_tensor,
                               uint32_t n_units, const StepParams& P, uint32_t* scratch_amax, float* scratch_s_old,
                               cudaStream_t stream) {
    if (n_units == 0) return cudaSuccess;
    ECO_DISPATCH_FMT(c.format, ECO_DISPATCH_OPT(c.optimizer, {
        eco_tensor_amax_kernel<F, O><<<n_units, kThreads, 0, stream>>>(descs, unit_tensor, P, c.scale_kind,
                                                                     scratch_amax, scratch_s_old);
    }))
    return cudaGetLastError();
}

cudaError_t launch_tensor_apply(const LaunchConfig& c, const TensorDesc* descs, const uint32_t* unit_tensor,
                                uint32_t n_units, const StepParams& P, const uint32_t* scratch_amax,
                                uint32_t* scratch_amax_next, const float* scratch_s_old, bool reverse,
                                cudaStream_t stream) {
    if (n_units == 0) return cudaSuccess;
    ECO_DISPATCH_FMT(c.format, ECO_DISPATCH_OPT(c.optimizer, ECO_DISPATCH_RND(c.rounding, {
        eco_tensor_apply_kernel<F, O, R><<<n_units, kThreads, 0, stream>>>(
            descs, unit_tensor, P, c.scale_kind, scratch_amax, scratch_amax_next, scratch_s_old, reverse ? 1 : 0, n_units);
    })))
    return cudaGetLastError();
}

cudaError_t launch_row(const LaunchConfig& c, const TensorDesc* descs, const uint32_t* unit_tensor,
                       uint32_t n_units, const StepParams& P, cudaStream_t stream) {
    if (n_units == 0) return cudaSuccess;
    ECO_DISPATCH_FMT(c.format, ECO_DISPATCH_OPT(c.optimizer, ECO_DISPATCH_RND(c.rounding, {
        eco_row_kernel<F, O, R><<<n_units, kThreads, 0, stream>>>(descs, unit_tensor, P, c.scale_kind);
    })))
    return cudaGetLastError();
}

cudaError_t launch_quantize(const LaunchConfig& c, const float* x, uint8_t* w, void* scale, uint64_t rows,
                            uint32_t cols, int mode, const StepParams& P, uint32_t tensor_id,
                            uint32_t* scratch_amax, uint32_t grid, cudaStream_t stream) {
    ECO_DISPATCH_FMT(c.format, ECO_DISPATCH_RND(c.rounding, {
        eco_quantize_kernel<F, R><<<grid, kThreads, 0, stream>>>(x, w, scale, rows, cols, mode, c.scale_kind, P,
                                                                tensor_id, scratch_amax);
    }))
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------
// x^ = value(code) * scale (Sec. 3.1) for a whole tensor: what the forward pass of quantized training reads.
// One thread per 4 consecutive elements of a row (cols is even for INT4, so a thread never splits a byte);
// gran: 0 per-tensor, 1 per-row, 2 blocks of `block` (128 or 32) elements along the row.  OUT_BF16: round the product to bf16 (nearest even).
// ---------------------------------------------------------------------------
template <int FMT, bool OUT_BF16>
__global__ void __launch_bounds__(kThreads)
eco_dequantize_kernel(const uint8_t* __restrict__ w, const void* __restrict__ scale, void* __restrict__ out,
                      const uint64_t rows, const uint32_t cols, const int gran, const uint32_t block, const int scale_kind) {
    const uint32_t quads_per_row = div_ceil_u32(cols, 4u);
    const uint32_t scales_per_row = div_ceil_u32(cols, block);
    const uint64_t n_quads = rows * quads_per_row;
    for (uint64_t qd = static_cast<uint64_t>(blockIdx.x) * kThreads + threadIdx.x; qd < n_quads;
         qd += static_cast<uint64_t>(gridDim.x) * kThreads) {
        const uint64_t row = qd / quads_per_row;
        const uint32_t c0 = static_cast<uint32_t>(qd - row * quads_per_row) * 4u;
        const int nvalid = static_cast<int>(min(4u, cols - c0));
        const uint64_t i0 = row * cols + c0;
        const bool vec = (i0 & 3) == 0;
        const uint32_t codes = load_codes4<FMT>(w, i0, nvalid, vec);
        float val[4];
        unpack4<FMT>(codes, val);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            if (e >= nvalid) break;
            const uint64_t k = gran == 0 ? 0 : (gran == 1 ? row : row * scales_per_row + (c0 + e) / block);
            const float x = __fmul_rn(val[e], load_scale(scale, k, scale_kind));
            if (OUT_BF16) static_cast<uint16_t*>(out)[i0 + e] = static_cast<uint16_t>(f32_to_bf16_bits_rne(x));
            else static_cast<float*>(out)[i0 + e] = x;
        }
    }
}

// The same for rows whose length is a multiple of 16 and 16-byte aligned buffers: one thread per EPT consecutive
// elements (they share a scale: 4, 8 and 16 divide both block lengths).  EPT is chosen so that a lane stores exactly
// 16 bytes, contiguous with its neighbours': 8 elements for bf16 output, 4 for f32.
// Two binary32 values to two bf16 in one register (first value in the low half), each rounded to nearest even: one
// instruction of the arithmetic pipes instead of two conversions, a shift and an OR.
__device__ __forceinline__ uint32_t f32x2_to_bf16x2_rne(float lo, float hi) {
    uint32_t d;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
    return d;
}

template <int FMT, bool OUT_BF16, int EPT>
__global__ void __launch_bounds__(kThreads)
eco_dequantize_vec_kernel(const uint8_t* __restrict__ w, const void* __restrict__ scale, void* __restrict__ out,
                          const uint64_t n_units, const uint32_t units_per_row, const int gran, const uint32_t block,
                          const uint32_t scales_per_row, const int scale_kind, const int shift) {
    static_assert(EPT == 4 || EPT == 8, "4 or 8 elements per thread");
    constexpr int Q = EPT / 4;
    constexpr int U = 4;                     // units per thread and trip: all loads are issued before any is used
    // 64-bit unit counter and stride: n_units reaches 2^32 - 4 for the largest admitted tensor, and u + stride
    // must not wrap below it
    const uint64_t stride = static_cast<uint64_t>(gridDim.x) * kThreads;
    for (uint64_t u0 = static_cast<uint64_t>(blockIdx.x) * (U * kThreads) + threadIdx.x; u0 < n_units; u0 += U * stride) {
        uint32_t codes[U][Q];
        float s[U];
#pragma unroll
        for (int j = 0; j < U; ++j) {
            const uint64_t u = u0 + j * kThreads;            // the CTA's units of a trip are neighbours
            if (u >= n_units) continue;
            const uint64_t i0 = u * EPT;
            if (FMT != FMT_INT4) {
                if constexpr (EPT == 8) {
                    const uint2 r = __ldg(reinterpret_cast<const uint2*>(w + i0));
                    codes[j][0] = r.x; codes[j][1] = r.y;
                } else {
                    codes[j][0] = __ldg(reinterpret_cast<const uint32_t*>(w + i0));
                }
            } else {
                if constexpr (EPT == 8) {
                    const uint32_t r = __ldg(reinterpret_cast<const uint32_t*>(w + (i0 >> 1)));
                    codes[j][0] = r & 0xFFFFu; codes[j][1] = r >> 16;
                } else {
                    codes[j][0] = __ldg(reinterpret_cast<const uint16_t*>(w + (i0 >> 1)));
                }
            }
            s[j] = load_scale(scale, dequant_scale_index(u, units_per_row, EPT, gran, block, scales_per_row, shift), scale_kind);
        }
#pragma unroll
        for (int j = 0; j < U; ++j) {
            const uint64_t u = u0 + j * kThreads;            // the CTA's units of a trip are neighbours
            if (u >= n_units) continue;
            const uint64_t i0 = u * EPT;
            float x[EPT];
#pragma unroll
            for (int q = 0; q < Q; ++q) {
                float val[4];
                unpack4<FMT>(codes[j][q], val);
#pragma unroll
                for (int e = 0; e < 4; e += 2) {
                    const float2 t = mul2(make_float2(val[e], val[e + 1]), dup2(s[j]));
                    x[4 * q + e] = t.x; x[4 * q + e + 1] = t.y;
                }
            }
            if (OUT_BF16) {
                uint32_t p[EPT / 2];
#pragma unroll
                for (int t = 0; t < EPT / 2; ++t)
                    p[t] = f32x2_to_bf16x2_rne(x[2 * t], x[2 * t + 1]);
                uint4* o = reinterpret_cast<uint4*>(static_cast<uint16_t*>(out) + i0);
#pragma unroll
                for (int t = 0; t < (EPT + 7) / 8; ++t) o[t] = make_uint4(p[4 * t], p[4 * t + 1], p[4 * t + 2], p[4 * t + 3]);
            } else {
                float4* o = reinterpret_cast<float4*>(static_cast<float*>(out) + i0);
#pragma unroll
                for (int t = 0; t < Q; ++t) o[t] = make_float4(x[4 * t], x[4 * t + 1], x[4 * t + 2], x[4 * t + 3]);
            }
        }
    }
}

cudaError_t launch_dequantize(const LaunchConfig& c, const uint8_t* w, const void* scale, void* out, uint64_t rows,
                              uint32_t cols, int gran, bool out_bf16, uint32_t grid, cudaStream_t stream) {
    const uint32_t block = static_cast<uint32_t>(128 / c.sub);
    const bool aligned = ((reinterpret_cast<uintptr_t>(w) | reinterpret_cast<uintptr_t>(out)) & 15u) == 0;
    if (cols % 16 == 0 && aligned) {
        const uint32_t ept = out_bf16 ? 8u : 4u;
        const uint64_t n_units = dequant_units(rows, cols, ept);
        const uint64_t cap = static_cast<uint64_t>((c.sm_count > 0 ? c.sm_count : 148) * 16);
        const uint32_t g = static_cast<uint32_t>(std::max<uint64_t>(1, std::min(cap, (n_units + kThreads - 1) / kThreads)));
        const uint32_t spr = div_ceil_u32(cols, block);
        // rows made of whole blocks of 128 or 32 elements: scale blocks are numbered like elements / block
        const int shift = (gran == 2 && cols % block == 0u) ? (block == 128u ? 7 : (block == 32u ? 5 : -1)) : -1;
        ECO_DISPATCH_FMT(c.format, {
            if (out_bf16) eco_dequantize_vec_kernel<F, true, 8><<<g, kThreads, 0, stream>>>(w, scale, out, n_units, cols / 8, gran, block, spr, c.scale_kind, shift);
            else eco_dequantize_vec_kernel<F, false, 4><<<g, kThreads, 0, stream>>>(w, scale, out, n_units, cols / 4, gran, block, spr, c.scale_kind, shift);
        })
        return cudaGetLastError();
    }
    ECO_DISPATCH_FMT(c.format, {
        if (out_bf16) eco_dequantize_kernel<F, true><<<grid, kThreads, 0, stream>>>(w, scale, out, rows, cols, gran, static_cast<uint32_t>(128 / c.sub), c.scale_kind);
        else eco_dequantize_kernel<F, false><<<grid, kThreads, 0, stream>>>(w, scale, out, rows, cols, gran, static_cast<uint32_t>(128 / c.sub), c.scale_kind);
    })
    return cudaGetLastError();
}

int rows_per_unit() { return kRowsPerUnit; }

}  // namespace eco
