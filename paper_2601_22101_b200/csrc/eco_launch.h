// Host-side interface between the C-ABI layer (eco_api.cu) and the kernel
// launchers (eco_kernels.cu).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "eco_device.cuh"

namespace eco {

struct LaunchConfig {
    int format;      // FMT_*
    int optimizer;   // OPT_*
    int rounding;    // RND_*
    int scale_kind;  // SCALE_KIND_*: f32, bf16 or power-of-two (one exponent byte) scales
    int sm_count;    // SMs of the device (sizes the persistent grids)
    int sub;         // block scales: scale blocks per 128 elements of a row (1: 1x128 blocks, 4: 1x32 blocks)
};

// Rows of 128 elements that one CTA (work unit) covers.
int rows_per_unit();
int stream_unit_rows();

// Modes of the TMA-fed streaming kernel (eco_stream_kernels.cu).
enum : int { STREAM_BLOCK = 0, STREAM_TENSOR_AMAX = 1, STREAM_TENSOR_APPLY = 2, STREAM_ROW = 3, STREAM_BLOCK32 = 4 };
enum : int { MODE_BLOCK = STREAM_BLOCK, MODE_TENSOR_AMAX = STREAM_TENSOR_AMAX, MODE_TENSOR_APPLY = STREAM_TENSOR_APPLY,
             MODE_ROW = STREAM_ROW, MODE_BLOCK32 = STREAM_BLOCK32 };

// Persistent launch over n_units work units; grid = min(n_units, grid_cap), where grid_cap = 0 stands for the kernel's
// own number of resident CTAs per SM (3 for momentum SGD, 2 for Adam) times LaunchConfig::sm_count.  `tickets` are two device
// words, zero before the first launch, that the kernel uses to hand out units and rewinds before it ends
// (launches sharing them must be ordered on the device).  `status` is a device word that receives a
// non-zero code if a bounded wait inside the kernel expires.  with_errors selects the instantiation that also
// reads / writes the tensors' error buffers (TensorDesc::e must then be set for every tensor of the launch).
cudaError_t launch_stream(const LaunchConfig& c, int mode, const TensorDesc* descs, const uint32_t* unit_tensor,
                          uint32_t n_units, const StepParams& P, uint32_t* amax, uint32_t* amax_next, float* s_old,
                          bool reverse, uint32_t* tickets, uint32_t* status, int grid_cap, cudaStream_t stream,
                          bool with_errors = false, int cluster = 1);
// cluster > 1 (STREAM_ROW only): the units are single matrix rows of up to 32 * cluster segments of 128 columns; the
// launch runs thread-block clusters of that many CTAs, each CTA streaming its slice of the row, the row maximum
// exchanged through distributed shared memory (TensorDesc::n_blocks = rows * segments, one unit per matrix row).
int stream_max_cluster();

// A wave of the single-launch per-tensor step: the units [first_unit, first_unit + n_units) of the launch's unit table,
// made of whole tensors.
struct WaveDesc {
    uint32_t first_unit, n_units;
};

// Per-tensor scales in one cooperative launch (see eco_wave_kernel): both passes of every wave, a grid barrier in
// between.  `grid_counter`: two device words, zero before the first launch, rewound by the kernel itself.
// `wave_tickets`: NULL = every CTA owns a fixed share of each wave (what it streamed in pass 1 is still in its
// shared memory for pass 2: the form for a single wave); else 2 * n_waves device words, zero before the first launch
// and rewound by the kernel, from which the units of each pass are handed out.  The grid is the number of CTAs the
// device can hold at once (or grid_cap, if that is smaller).
cudaError_t launch_wave(const LaunchConfig& c, const TensorDesc* descs, const uint32_t* unit_tensor, const WaveDesc* waves,
                        uint32_t n_waves, const StepParams& P, uint32_t* amax, uint32_t* amax_next, float* s_old,
                        uint32_t* grid_counter, uint32_t* wave_tickets, uint32_t* status, int grid_cap, cudaStream_t stream,
                        bool with_errors);

// One warp waits, for at most limit_cycles, on a barrier nothing arrives on; then writes code 7 to *status.
cudaError_t launch_wait_selftest(uint32_t* status, long long limit_cycles, cudaStream_t stream);
// Two CTAs wait, for at most limit_cycles, at a grid barrier that expects a third; then code 6 is written to *status.
// `counter`: a device word, zero before the launch (left non-zero).
cudaError_t launch_grid_wait_selftest(uint32_t* counter, uint32_t* status, long long limit_cycles, cudaStream_t stream);

cudaError_t launch_block128(const LaunchConfig& c, const TensorDesc* descs, const uint32_t* unit_tensor,
                            uint32_t n_units, bool generic, const StepParams& P, cudaStream_t stream);
cudaError_t launch_tensor_amax(const LaunchConfig& c, const TensorDesc* descs, const uint32_t* unit_tensor,
                               uint32_t n_units, const StepParams& P, uint32_t* scratch_amax, float* scratch_s_old,
                               cudaStream_t stream);
cudaError_t launch_tensor_apply(const LaunchConfig& c, const TensorDesc* descs, const uint32_t* unit_tensor,
                                uint32_t n_units, const StepParams& P, const uint32_t* scratch_amax,
                                uint32_t* scratch_amax_next, const float* scratch_s_old, bool reverse,
                                cudaStream_t stream);
cudaError_t launch_row(const LaunchConfig& c, const TensorDesc* descs, const uint32_t* unit_tensor,
                       uint32_t n_units, const StepParams& P, cudaStream_t stream);
cudaError_t launch_quantize(const LaunchConfig& c, const float* x, uint8_t* w, void* scale, uint64_t rows,
                            uint32_t cols, int mode, const StepParams& P, uint32_t tensor_id,
                            uint32_t* scratch_amax, uint32_t grid, cudaStream_t stream);

cudaError_t launch_dequantize(const LaunchConfig& c, const uint8_t* w, const void* scale, void* out, uint64_t rows,
                              uint32_t cols, int gran, bool out_bf16, uint32_t grid, cudaStream_t stream);

}  // namespace eco
