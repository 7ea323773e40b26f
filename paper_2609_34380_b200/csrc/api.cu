// The C ABI of libdps: argument validation, the per-device status word, and dispatch of each
// call to a kernel family.  Nothing here allocates or frees device memory.
#include <atomic>
#include <cstdlib>
#include <cstring>
#include <mutex>

#include "sm100.cuh"

#include "bits.cuh"
#include "dps_internal.h"

namespace dps {

namespace {

// Per-device words that kernels write: the status word (data-dependent errors) and the
// scratch word of the load-time magnitude statistic.
__device__ int g_status_word;
__device__ unsigned g_stat_word;

// Self-test of the bounded device-side waits: ONE warp initialises an mbarrier that nobody will ever
// arrive on and waits for it with the given limit -- the same wait (and the same reaction: set the
// status word, give up, return) as every pipeline wait in the tensor-core kernels.  No copy is in
// flight, no tensor memory is held, no other CTA is involved.
__global__ void wait_timeout_selftest_kernel(unsigned long long limit_ns, int* status) {
    __shared__ __align__(8) uint64_t bar;
    if (threadIdx.x == 0) {
        sm100::mbar_init(sm100::smem_u32(&bar), 1);
        sm100::fence_barrier_init();
    }
    __syncwarp();
    if (!sm100::mbar_wait_limit(sm100::smem_u32(&bar), 0, limit_ns) && threadIdx.x == 0)
        atomicExch(status, (int)DPS_ERR_CUDA);
}

std::atomic<int64_t> g_launches{0};
std::mutex g_stat_mutex;  // the statistic word is shared by all AUTO / checked-E4M3 splits

struct DeviceInfo {
    std::once_flag once;
    cudaError_t err = cudaSuccess;
    int* status = nullptr;
    unsigned* stat = nullptr;
    int sms = 0;
    int cc_major = 0;
};
DeviceInfo g_dev[kMaxDevices];

DeviceInfo* device_info() {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
    DeviceInfo& d = g_dev[dev];
    std::call_once(d.once, [&] {
        d.err = cudaGetSymbolAddress((void**)&d.status, g_status_word);
        if (d.err == cudaSuccess) d.err = cudaGetSymbolAddress((void**)&d.stat, g_stat_word);
        if (d.err == cudaSuccess) d.err = cudaDeviceGetAttribute(&d.sms, cudaDevAttrMultiProcessorCount, dev);
        if (d.err == cudaSuccess) d.err = cudaDeviceGetAttribute(&d.cc_major, cudaDevAttrComputeCapabilityMajor, dev);
    });
    return &d;
}

// Tuning / debugging knob: DPS_FORCE_PATH=gemv, =umma or =stream pins the dense kernel family.
int forced_path() {
    static const int path = [] {
        const char* v = getenv("DPS_FORCE_PATH");
        if (!v) return 0;
        if (!strcmp(v, "gemv")) return 1;
        if (!strcmp(v, "umma")) return 2;
        if (!strcmp(v, "stream")) return 3;
        return 0;
    }();
    return path;
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

dps_status check_device(DeviceInfo*& d) {
    d = device_info();
    if (d == nullptr || d->err != cudaSuccess) return DPS_ERR_CUDA;
    if (d->cc_major != 10) return DPS_ERR_UNSUPPORTED;  // the kernels are built for sm_100a only
    return DPS_OK;
}

}  // namespace

void count_launch(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }

dps_status check_moe_args(int32_t mode, const int32_t* enc_per_expert, const void* x, const int32_t* token_of_row,
                          const int32_t* expert_of_row, const uint8_t* w_persist, const uint8_t* w_resid, const void* y,
                          int64_t A, int64_t T, int64_t N, int64_t K, int32_t E, bool* empty) {
    *empty = false;
    if (mode != DPS_MODE_FAST && mode != DPS_MODE_FULL) return DPS_ERR_MODE;
    if (A < 0 || T < 0 || N <= 0 || K <= 0 || E <= 0 || (K % 16) != 0 || (N % 8) != 0) return DPS_ERR_SHAPE;
    if (A > ((int64_t)1 << 30) || T > ((int64_t)1 << 30) || N >= ((int64_t)1 << 31) || K >= ((int64_t)1 << 31))
        return DPS_ERR_SHAPE;
    // the kernels address plane rows of all experts with 32-bit coordinates
    if ((int64_t)E * N >= ((int64_t)1 << 31)) return DPS_ERR_SHAPE;
    if (!enc_per_expert) return DPS_ERR_NULL;
    if (moe_workspace_bytes(A, E, K) == 0) return DPS_ERR_SHAPE;
    for (int32_t e = 0; e < E; ++e) {
        const int32_t enc = enc_per_expert[e];
        if (enc != DPS_ENC_E4M3 && enc != DPS_ENC_E5M2 && enc != DPS_ENC_E4M3_RN && enc != DPS_ENC_E5M2_RN)
            return DPS_ERR_ENCODING;
    }
    if (A == 0) {
        *empty = true;
        return DPS_OK;
    }
    if (!x || !expert_of_row || !w_persist || !y) return DPS_ERR_NULL;
    if (mode == DPS_MODE_FULL && !w_resid) return DPS_ERR_NULL;
    if (!aligned16(x) || !aligned16(w_persist) || !aligned16(y)) return DPS_ERR_ALIGN;
    if (mode == DPS_MODE_FULL && !aligned16(w_resid)) return DPS_ERR_ALIGN;
    if ((reinterpret_cast<uintptr_t>(expert_of_row) & 3u) || (reinterpret_cast<uintptr_t>(token_of_row) & 3u))
        return DPS_ERR_ALIGN;
    return DPS_OK;
}

dps_status device_status_word(int** status) {
    DeviceInfo* d = nullptr;
    const dps_status st = check_device(d);
    *status = (st == DPS_OK) ? d->status : nullptr;
    return st;
}

int sm_count() {
    DeviceInfo* d = device_info();
    return (d && d->sms > 0) ? d->sms : 148;
}

}  // namespace dps

using namespace dps;

namespace {
bool known_encoding(int32_t enc) {
    return enc == DPS_ENC_E4M3 || enc == DPS_ENC_E5M2 || enc == DPS_ENC_E4M3_RN || enc == DPS_ENC_E5M2_RN;
}
}  // namespace

extern "C" {

dps_status dps_split_weights(const void* w_fp16, uint8_t* w_persist, uint8_t* w_resid, int64_t rows, int64_t cols,
                             int32_t* enc_inout, void* cuda_stream) {
    if (enc_inout == nullptr) return DPS_ERR_NULL;
    const int32_t req = *enc_inout;
    if (req != DPS_ENC_AUTO && req != DPS_ENC_AUTO_RN && !known_encoding(req)) return DPS_ERR_ENCODING;
    if (rows < 0 || cols < 0 || (cols % 16) != 0) return DPS_ERR_SHAPE;
    if (rows > 0 && cols > 0 && rows > INT64_MAX / cols) return DPS_ERR_SHAPE;
    const int64_t n = rows * cols;
    if (n == 0) {
        if (req == DPS_ENC_AUTO) *enc_inout = DPS_ENC_E4M3;
        if (req == DPS_ENC_AUTO_RN) *enc_inout = DPS_ENC_E4M3_RN;
        return DPS_OK;
    }
    if (!w_fp16 || !w_persist || !w_resid) return DPS_ERR_NULL;
    if (!aligned16(w_fp16) || !aligned16(w_persist) || !aligned16(w_resid)) return DPS_ERR_ALIGN;
    DeviceInfo* d;
    dps_status st = check_device(d);
    if (st != DPS_OK) return st;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    int enc = req;
    if (req != DPS_ENC_E5M2) {
        // Load-time statistics: max over the tensor of (word & 0x7FFF).  A word with the exponent
        // MSB set is >= 0x4000, so one maximum answers both questions:
        //   AUTO  -> E4M3 iff max <= 0x3F00 (|w| <= 1.75), else E5M2
        //   E4M3  -> legal iff max <  0x3F80 (exponent MSB clear and the byte is not 0x7F/0xFF)
        //   rounded nests: the same limits must hold after half a unit of the last kept bit is added
        //     E4M3_RN -> legal iff max + 0x40 < 0x3F80;  E5M2_RN -> legal iff max + 0x80 < 0x7C00 (no Inf code)
        std::lock_guard<std::mutex> lock(g_stat_mutex);
        unsigned maxmag = 0;
        if (cudaMemsetAsync(d->stat, 0, sizeof(unsigned), stream) != cudaSuccess) return DPS_ERR_CUDA;
        if (launch_magnitude_stat(static_cast<const uint16_t*>(w_fp16), n, d->stat, stream) != cudaSuccess)
            return DPS_ERR_CUDA;
        if (cudaMemcpyAsync(&maxmag, d->stat, sizeof(unsigned), cudaMemcpyDeviceToHost, stream) != cudaSuccess)
            return DPS_ERR_CUDA;
        if (cudaStreamSynchronize(stream) != cudaSuccess) return DPS_ERR_CUDA;
        if (req == DPS_ENC_AUTO) enc = (maxmag <= 0x3F00u) ? DPS_ENC_E4M3 : DPS_ENC_E5M2;
        else if (req == DPS_ENC_AUTO_RN) {
            enc = (maxmag <= 0x3F00u) ? DPS_ENC_E4M3_RN : DPS_ENC_E5M2_RN;
            if (enc == DPS_ENC_E5M2_RN && maxmag + 0x80u >= 0x7C00u) return DPS_ERR_DATA;
        }
        else if (req == DPS_ENC_E4M3 && maxmag >= 0x3F80u) return DPS_ERR_DATA;
        else if (req == DPS_ENC_E4M3_RN && maxmag + 0x40u >= 0x3F80u) return DPS_ERR_DATA;
        else if (req == DPS_ENC_E5M2_RN && maxmag + 0x80u >= 0x7C00u) return DPS_ERR_DATA;
    }
    if (launch_split(static_cast<const uint16_t*>(w_fp16), w_persist, w_resid, n, enc, stream) != cudaSuccess)
        return DPS_ERR_CUDA;
    *enc_inout = enc;
    return DPS_OK;
}

dps_status dps_reconstruct(const uint8_t* w_persist, const uint8_t* w_resid, void* w_fp16_out, int64_t rows,
                           int64_t cols, int32_t enc, void* cuda_stream) {
    if (!known_encoding(enc)) return DPS_ERR_ENCODING;
    if (rows < 0 || cols < 0 || (cols % 16) != 0) return DPS_ERR_SHAPE;
    if (rows > 0 && cols > 0 && rows > INT64_MAX / cols) return DPS_ERR_SHAPE;
    const int64_t n = rows * cols;
    if (n == 0) return DPS_OK;
    if (!w_persist || !w_fp16_out) return DPS_ERR_NULL;
    if (!aligned16(w_persist) || !aligned16(w_resid) || !aligned16(w_fp16_out)) return DPS_ERR_ALIGN;
    DeviceInfo* d;
    dps_status st = check_device(d);
    if (st != DPS_OK) return st;
    if (launch_reconstruct(w_persist, w_resid, static_cast<uint16_t*>(w_fp16_out), n, enc,
                           static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess)
        return DPS_ERR_CUDA;
    return DPS_OK;
}

dps_status dps_linear(int32_t mode, int32_t enc, const void* x, const uint8_t* w_persist, const uint8_t* w_resid,
                      void* y, int64_t M, int64_t N, int64_t K, void* cuda_stream) {
    if (mode != DPS_MODE_FAST && mode != DPS_MODE_FULL) return DPS_ERR_MODE;
    if (!known_encoding(enc)) return DPS_ERR_ENCODING;
    if (M < 0 || N <= 0 || K <= 0 || (K % 16) != 0 || (N % 8) != 0) return DPS_ERR_SHAPE;
    if (N >= ((int64_t)1 << 31) || K >= ((int64_t)1 << 31) || M >= ((int64_t)1 << 31)) return DPS_ERR_SHAPE;
    if (M == 0) return DPS_OK;
    if (!x || !w_persist || !y) return DPS_ERR_NULL;
    if (mode == DPS_MODE_FULL && !w_resid) return DPS_ERR_NULL;
    if (!aligned16(x) || !aligned16(w_persist) || !aligned16(y)) return DPS_ERR_ALIGN;
    if (mode == DPS_MODE_FULL && !aligned16(w_resid)) return DPS_ERR_ALIGN;
    DeviceInfo* d;
    dps_status st = check_device(d);
    if (st != DPS_OK) return st;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const uint8_t* r = (mode == DPS_MODE_FULL) ? w_resid : nullptr;  // fast mode never sees the pointer
    // A handful of tokens makes the layer a pure weight stream: up to 8 tokens (one MMA column group)
    // the register-streaming kernel serves it.  For 9-16 tokens the choice was measured on Llama-7B
    // and hidden-8192 shapes, in both modes: the tensor-core kernel's set-up and cluster reduction
    // cost a few microseconds per launch, its TMA stream is faster once running; it wins from 2^25
    // weights on (by 0-20 %), the streaming kernel below (4096 x 4096: by 15-30 %).  Beyond 16
    // tokens the tcgen05 tiles take over.  (The CUDA-core GEMV is kept as a cross-check.)
    const bool stream_mid = N * K < ((int64_t)1 << 25);
    const int path = forced_path();
    cudaError_t err;
    if (path == 1) err = launch_gemv(mode, enc, x, w_persist, r, y, M, N, K, stream);
    else if (path == 2) err = launch_umma_linear(mode, enc, x, w_persist, r, y, M, N, K, d->status, stream);
    else if (path == 3 || M <= 8 || (M <= 16 && stream_mid)) {
        if (M > 16) return DPS_ERR_UNSUPPORTED;      // (only reachable with DPS_FORCE_PATH=stream)
        err = launch_decode_mma(mode, enc, x, w_persist, r, y, M, N, K, stream);
    } else err = launch_umma_linear(mode, enc, x, w_persist, r, y, M, N, K, d->status, stream);
    return err == cudaSuccess ? DPS_OK : DPS_ERR_CUDA;
}

size_t dps_moe_workspace_bytes(int64_t A, int32_t E, int64_t K) { return moe_workspace_bytes(A, E, K); }

dps_status dps_moe_linear(int32_t mode, const int32_t* enc_per_expert, const void* x, const int32_t* token_of_row,
                          const int32_t* expert_of_row, const uint8_t* w_persist, const uint8_t* w_resid, void* y,
                          int64_t A, int64_t T, int64_t N, int64_t K, int32_t E, void* workspace,
                          size_t workspace_bytes, void* cuda_stream) {
    bool empty = false;
    const dps_status ok = check_moe_args(mode, enc_per_expert, x, token_of_row, expert_of_row, w_persist, w_resid, y, A, T,
                                         N, K, E, &empty);
    if (ok != DPS_OK || empty) return ok;
    const size_t need = moe_workspace_bytes(A, E, K);
    if (!workspace || !aligned16(workspace) || workspace_bytes < need) return DPS_ERR_WORKSPACE;
    DeviceInfo* d;
    dps_status st = check_device(d);
    if (st != DPS_OK) return st;
    const uint8_t* r = (mode == DPS_MODE_FULL) ? w_resid : nullptr;
    if (launch_moe(mode, enc_per_expert, x, token_of_row, expert_of_row, w_persist, r, y, A, T, N, K, E, workspace,
                   d->status, static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess)
        return DPS_ERR_CUDA;
    return DPS_OK;
}

dps_status dps_stream_status(void* cuda_stream) {
    DeviceInfo* d;
    dps_status st = check_device(d);
    if (st != DPS_OK) return st;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    int word = 0;
    if (cudaMemcpyAsync(&word, d->status, sizeof(int), cudaMemcpyDeviceToHost, stream) != cudaSuccess)
        return DPS_ERR_CUDA;
    if (cudaMemsetAsync(d->status, 0, sizeof(int), stream) != cudaSuccess) return DPS_ERR_CUDA;
    if (cudaStreamSynchronize(stream) != cudaSuccess) return DPS_ERR_CUDA;
    return word == 0 ? DPS_OK : (word == (int)DPS_ERR_DATA ? DPS_ERR_DATA : DPS_ERR_CUDA);
}

dps_status dps_quantize_activations(const void* x, uint8_t* x_fp8, float* scale, int64_t M, int64_t K,
                                    void* cuda_stream) {
    if (M < 0 || K <= 0 || (K % 16) != 0 || M >= ((int64_t)1 << 31) || K >= ((int64_t)1 << 31)) return DPS_ERR_SHAPE;
    if (M == 0) return DPS_OK;
    if (!x || !x_fp8 || !scale) return DPS_ERR_NULL;
    if (!aligned16(x) || !aligned16(x_fp8)) return DPS_ERR_ALIGN;
    DeviceInfo* d;
    dps_status st = check_device(d);
    if (st != DPS_OK) return st;
    return launch_quantize_activations(x, x_fp8, scale, M, K, d->status, static_cast<cudaStream_t>(cuda_stream)) ==
                   cudaSuccess
               ? DPS_OK
               : DPS_ERR_CUDA;
}

dps_status dps_linear_fp8act(int32_t enc, const uint8_t* x_fp8, const float* scale, const uint8_t* w_persist, void* y,
                             int64_t M, int64_t N, int64_t K, void* cuda_stream) {
    if (!known_encoding(enc)) return DPS_ERR_ENCODING;
    enc = base_enc(enc);   // the persistent byte of a rounded nest is an FP8 value like any other
    if (M < 0 || N <= 0 || K <= 0 || (K % 16) != 0 || (N % 8) != 0) return DPS_ERR_SHAPE;
    if (N >= ((int64_t)1 << 31) || K >= ((int64_t)1 << 31) || M >= ((int64_t)1 << 31)) return DPS_ERR_SHAPE;
    if (M == 0) return DPS_OK;
    if (!x_fp8 || !scale || !w_persist || !y) return DPS_ERR_NULL;
    if (!aligned16(x_fp8) || !aligned16(w_persist) || !aligned16(y)) return DPS_ERR_ALIGN;
    DeviceInfo* d;
    dps_status st = check_device(d);
    if (st != DPS_OK) return st;
    return launch_linear_fp8act(enc, x_fp8, scale, w_persist, y, M, N, K, d->status,
                                static_cast<cudaStream_t>(cuda_stream)) == cudaSuccess
               ? DPS_OK
               : DPS_ERR_CUDA;
}

namespace {
dps_status chunked_copy(void* dst, const void* src, size_t bytes, size_t chunk, cudaMemcpyKind kind, void* cuda_stream) {
    if (bytes == 0) return DPS_OK;
    if (!dst || !src) return DPS_ERR_NULL;
    if (chunk == 0) chunk = (size_t)4 << 20;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    for (size_t off = 0; off < bytes; off += chunk) {
        const size_t n = bytes - off < chunk ? bytes - off : chunk;
        if (cudaMemcpyAsync(static_cast<char*>(dst) + off, static_cast<const char*>(src) + off, n, kind, stream) !=
            cudaSuccess)
            return DPS_ERR_CUDA;
    }
    return DPS_OK;
}
}  // namespace

dps_status dps_backup_residual(const uint8_t* w_resid, uint8_t* backup_host, size_t bytes, size_t chunk_bytes,
                               void* cuda_stream) {
    return chunked_copy(backup_host, w_resid, bytes, chunk_bytes, cudaMemcpyDeviceToHost, cuda_stream);
}

dps_status dps_restore_residual(uint8_t* w_resid, const uint8_t* backup_host, size_t bytes, size_t chunk_bytes,
                                void* cuda_stream) {
    return chunked_copy(w_resid, backup_host, bytes, chunk_bytes, cudaMemcpyHostToDevice, cuda_stream);
}

dps_status dps_debug_wait_timeout(uint64_t limit_ns, void* cuda_stream) {
    if (limit_ns == 0 || limit_ns > 1000000000ull) return DPS_ERR_SHAPE;   // at most one second
    DeviceInfo* d;
    dps_status st = check_device(d);
    if (st != DPS_OK) return st;
    wait_timeout_selftest_kernel<<<1, 32, 0, static_cast<cudaStream_t>(cuda_stream)>>>(limit_ns, d->status);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? DPS_OK : DPS_ERR_CUDA;
}

int64_t dps_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

const char* dps_status_string(dps_status status) {
    switch (status) {
        case DPS_OK: return "ok";
        case DPS_ERR_NULL: return "null pointer";
        case DPS_ERR_SHAPE: return "bad shape";
        case DPS_ERR_MODE: return "bad mode";
        case DPS_ERR_ENCODING: return "bad encoding";
        case DPS_ERR_ALIGN: return "misaligned pointer";
        case DPS_ERR_UNSUPPORTED: return "unsupported device or request";
        case DPS_ERR_CUDA: return "CUDA error";
        case DPS_ERR_DATA: return "data-dependent error";
        case DPS_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    }
    return "unknown status";
}

int dps_version(void) { return 1; }

}  // extern "C"
