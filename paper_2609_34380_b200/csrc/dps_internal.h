// Host-side declarations shared by the translation units of libdps (not part of the ABI).
#pragma once
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include <mutex>

#include "../../include/dps.h"

namespace dps {

// One-time set-up that must happen once PER DEVICE (function attributes, occupancy queries): keyed by
// the current device's ordinal, safe against concurrent first calls.  The error of a failed set-up is
// kept and returned to every later caller on that device.
constexpr int kMaxDevices = 64;
struct PerDeviceOnce {
    std::once_flag once[kMaxDevices];
    cudaError_t err[kMaxDevices] = {};
    // Runs f() the first time the current device is seen; returns its (cached) result.  *device, if
    // given, receives the ordinal.
    template <typename F>
    cudaError_t run(F f, int* device = nullptr) {
        int dev = 0;
        cudaError_t e = cudaGetDevice(&dev);
        if (e != cudaSuccess) return e;
        if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
        if (device) *device = dev;
        std::call_once(once[dev], [&] { err[dev] = f(); });
        return err[dev];
    }
};

// Every launcher enqueues on `stream`, never synchronises and returns the CUDA error of the
// launch.  `status` is the address of the current device's status word.

// max over the tensor of (word & 0x7FFF), written with atomicMax into *stat (caller zeroes it).
cudaError_t launch_magnitude_stat(const uint16_t* w, int64_t n, unsigned* stat, cudaStream_t stream);
cudaError_t launch_split(const uint16_t* w, uint8_t* p, uint8_t* r, int64_t n, int enc, cudaStream_t stream);
cudaError_t launch_reconstruct(const uint8_t* p, const uint8_t* r, uint16_t* w, int64_t n, int enc,
                               cudaStream_t stream);

// Dense linear, CUDA-core path (any M; efficient for M <= 4).
cudaError_t launch_gemv(int mode, int enc, const void* x, const uint8_t* p, const uint8_t* r, void* y,
                        int64_t M, int64_t N, int64_t K, cudaStream_t stream);

// Dense linear for M <= 16: register-streaming kernel with warp-level MMAs.
cudaError_t launch_decode_mma(int mode, int enc, const void* x, const uint8_t* p, const uint8_t* r, void* y,
                              int64_t M, int64_t N, int64_t K, cudaStream_t stream);

// Dense linear, tensor-core path (tcgen05 + TMEM).  `status` receives DPS_ERR_CUDA if a bounded
// wait inside the kernel ever gives up.
cudaError_t launch_umma_linear(int mode, int enc, const void* x, const uint8_t* p, const uint8_t* r, void* y,
                               int64_t M, int64_t N, int64_t K, int* status, cudaStream_t stream);

// Grouped linear on the tensor-core path.  e5m2_mask: 64 words, bit e of the first 32 set for an E5M2
// expert, of the last 32 for a rounded nest.  x_sorted: [A][K] activations grouped by expert;
// tiles / num_tiles / sorted_rows: device tables built by the routing pre-pass; tn: token-tile
// width the tile list was built for (grouped_tile_tokens); max_tiles: upper bound on num_tiles.
int grouped_tile_tokens(int64_t A, int32_t E);
cudaError_t launch_umma_grouped(int mode, const uint32_t* e5m2_mask, const void* x_sorted, const uint8_t* p,
                                const uint8_t* r, void* y, int64_t A, int64_t N, int64_t K, int32_t E, int tn,
                                const void* tiles, const int32_t* num_tiles, const int32_t* sorted_rows,
                                int max_tiles, int* status, cudaStream_t stream);

// Fast mode with FP8 activations: per-token E4M3 quantisation, then an FP8 x FP8 tensor-core linear
// that reads the persistent plane as it is.
cudaError_t launch_quantize_activations(const void* x, uint8_t* q, float* scale, int64_t M, int64_t K, int* status,
                                        cudaStream_t stream);
cudaError_t launch_linear_fp8act(int enc, const uint8_t* q, const float* scale, const uint8_t* p, void* y, int64_t M,
                                 int64_t N, int64_t K, int* status, cudaStream_t stream);

// Grouped linear.
size_t moe_workspace_bytes(int64_t A, int32_t E, int64_t K);
cudaError_t launch_moe(int mode, const int32_t* enc_host, const void* x, const int32_t* token_of_row,
                       const int32_t* expert_of_row, const uint8_t* p, const uint8_t* r, void* y, int64_t A,
                       int64_t T, int64_t N, int64_t K, int32_t E, void* workspace, int* status,
                       cudaStream_t stream);

// Host-side checks shared by dps_moe_linear and dps_moe_linear_static (everything but the workspace).
// *empty is set when there is nothing to do (A == 0) and the pointers were therefore not looked at.
dps_status check_moe_args(int32_t mode, const int32_t* enc_per_expert, const void* x, const int32_t* token_of_row,
                          const int32_t* expert_of_row, const uint8_t* w_persist, const uint8_t* w_resid, const void* y,
                          int64_t A, int64_t T, int64_t N, int64_t K, int32_t E, bool* empty);

// Checks that the current device can run the kernels and returns the address of its status word.
dps_status device_status_word(int** status);

void count_launch(int n = 1);
int sm_count();

}  // namespace dps
