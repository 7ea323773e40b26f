// Grouped (MoE) linear layer: device-side routing pre-pass, activation gather, grouped kernel.
// Paper: "Scheduler: Dual-Precision Execution", paragraph "Dual-mode serving (DPS) with
// asymmetric switching" -- GroupedGEMM kernels with nested reconstruction serve MoE models.
//
// Steps, all enqueued on the caller's stream without synchronising:
//   1. route   (one CTA): validate rows, count rows per expert, group row ids by expert in
//               ascending row order (stable, no atomics), and cut every group into token tiles.
//   2. gather  : x_sorted[i][:] = x[token(sorted_rows[i])][:], so that each expert's activations
//               are one contiguous matrix a TMA tile load can address.
//   3. grouped tensor-core kernel over (weight-row tile, token tile): every expert's planes are
//               streamed once per token tile; results are scattered to the caller's row order.
//
// Workspace layout (E4 = E rounded up to 4, A4 = A rounded up to 4, all parts 16-byte aligned):
//   int32 counts[E4] | int32 offsets[E4 + 4] | int32 sorted_rows[A4] | int32 num_tiles[4]
//   | int4 tiles[A4 / 16 + E + 4] | fp16 x_sorted[A][K]
#include <mutex>

#include "dps_internal.h"
#include "gemv.cuh"
#include "sm100.cuh"

namespace dps {

namespace {

constexpr int kRouteThreads = 1024;
constexpr int kMaxExperts = 1024;

inline int64_t round4(int64_t v) { return (v + 3) / 4 * 4; }

struct Workspace {
    int32_t* counts;
    int32_t* offsets;
    int32_t* sorted_rows;
    int32_t* num_tiles;
    int4* tiles;
    __half* x_sorted;
    int64_t max_tiles;
    size_t bytes;
};

Workspace carve(void* base, int64_t A, int32_t E, int64_t K) {
    Workspace w;
    const int64_t e4 = round4(E), a4 = round4(A);
    int32_t* p = static_cast<int32_t*>(base);
    w.counts = p;
    w.offsets = w.counts + e4;
    w.sorted_rows = w.offsets + e4 + 4;
    w.num_tiles = w.sorted_rows + a4;
    w.max_tiles = a4 / 16 + E + 4;
    w.tiles = reinterpret_cast<int4*>(w.num_tiles + 4);
    w.x_sorted = reinterpret_cast<__half*>(w.tiles + w.max_tiles);
    const size_t head = (size_t)(e4 + e4 + 4 + a4 + 4) * 4 + (size_t)w.max_tiles * 16;
    w.bytes = (head + (size_t)A * (size_t)K * 2 + 255) / 256 * 256;
    return w;
}

__device__ __forceinline__ bool row_valid(const int32_t* token_of_row, const int32_t* expert_of_row, int a,
                                          int T, int E) {
    const int e = expert_of_row[a];
    const int t = token_of_row ? token_of_row[a] : a;
    return e >= 0 && e < E && t >= 0 && t < T;
}

// One CTA.  Warp w owns experts w, w+32, ...; for each it walks all rows in order, so the
// grouping is stable without any atomics.  Invalid rows belong to no group and raise the
// status word.
__global__ void __launch_bounds__(kRouteThreads)
moe_route_kernel(const int32_t* __restrict__ token_of_row, const int32_t* __restrict__ expert_of_row, int A, int T,
                 int E, int tile_tokens, int32_t* counts, int32_t* offsets, int32_t* sorted_rows,
                 int32_t* num_tiles, int4* tiles, int* status) {
    __shared__ int s_cnt[kMaxExperts];
    __shared__ int s_off[kMaxExperts];
    // the gather and the grouped kernel may be made resident now; both wait for their predecessor
    // (griddepcontrol.wait) before they read anything this kernel writes
    sm100::grid_launch_dependents();
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    int bad = 0;
    for (int a = tid; a < A; a += kRouteThreads) bad |= !row_valid(token_of_row, expert_of_row, a, T, E);
    if (__syncthreads_or(bad) && tid == 0) atomicExch(status, (int)DPS_ERR_DATA);
    for (int e = warp; e < E; e += kRouteThreads / 32) {
        int c = 0;
        for (int base = 0; base < A; base += 32) {
            const int a = base + lane;
            const bool hit = a < A && expert_of_row[a] == e && row_valid(token_of_row, expert_of_row, a, T, E);
            c += __popc(__ballot_sync(0xFFFFFFFFu, hit));
        }
        if (lane == 0) s_cnt[e] = c;
    }
    __syncthreads();
    if (tid == 0) {
        int run = 0, nt = 0;
        for (int e = 0; e < E; ++e) {
            s_off[e] = run;
            offsets[e] = run;
            counts[e] = s_cnt[e];
            for (int first = 0; first < s_cnt[e]; first += tile_tokens) {
                const int rows = s_cnt[e] - first < tile_tokens ? s_cnt[e] - first : tile_tokens;
                tiles[nt++] = make_int4(e, run + first, rows, 0);
            }
            run += s_cnt[e];
        }
        offsets[E] = run;
        num_tiles[0] = nt;
        num_tiles[1] = run;  // number of valid rows
    }
    __syncthreads();
    for (int e = warp; e < E; e += kRouteThreads / 32) {
        int pos = s_off[e];
        for (int base = 0; base < A; base += 32) {
            const int a = base + lane;
            const bool hit = a < A && expert_of_row[a] == e && row_valid(token_of_row, expert_of_row, a, T, E);
            const unsigned b = __ballot_sync(0xFFFFFFFFu, hit);
            if (hit) sorted_rows[pos + __popc(b & ((1u << lane) - 1u))] = a;
            pos += __popc(b);
        }
    }
}

// x_sorted[i][:] = x[token(sorted_rows[i])][:] for the valid rows; 16 bytes per thread.
__global__ void __launch_bounds__(256)
moe_gather_kernel(const uint4* __restrict__ x, const int32_t* __restrict__ token_of_row,
                  const int32_t* __restrict__ sorted_rows, const int32_t* __restrict__ num_tiles,
                  uint4* __restrict__ x_sorted, int64_t k16) {
    sm100::grid_launch_dependents();
    sm100::grid_dependency_wait();   // sorted_rows and num_tiles come from the routing kernel
    const int valid = num_tiles[1];
    for (int i = blockIdx.x; i < valid; i += gridDim.x) {
        const int a = sorted_rows[i];
        const int64_t tok = token_of_row ? token_of_row[a] : a;
        const uint4* src = x + tok * k16;
        uint4* dst = x_sorted + (int64_t)i * k16;
        for (int64_t c = threadIdx.x; c < k16; c += blockDim.x) dst[c] = src[c];
    }
}

}  // namespace

size_t moe_workspace_bytes(int64_t A, int32_t E, int64_t K) {
    if (A < 0 || E <= 0 || E > kMaxExperts || A > (int64_t)1 << 30 || K <= 0 || K > (int64_t)1 << 31) return 0;
    return carve(nullptr, A, E, K).bytes;
}

cudaError_t launch_moe(int mode, const int32_t* enc_host, const void* x, const int32_t* token_of_row,
                       const int32_t* expert_of_row, const uint8_t* p, const uint8_t* r, void* y, int64_t A,
                       int64_t T, int64_t N, int64_t K, int32_t E, void* workspace, int* status,
                       cudaStream_t stream) {
    const Workspace w = carve(workspace, A, E, K);
    const int tn = grouped_tile_tokens(A, E);
    moe_route_kernel<<<1, kRouteThreads, 0, stream>>>(token_of_row, expert_of_row, (int)A, (int)T, E, tn, w.counts,
                                                      w.offsets, w.sorted_rows, w.num_tiles, w.tiles, status);
    count_launch();
    cudaError_t err = cudaGetLastError();
    if (err != cudaSuccess) return err;
    const int gather_grid = (int)(A < 4096 ? A : 4096);
    {   // programmatic dependent launch: resident while the routing kernel runs, waits before its first read
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)gather_grid, 1, 1);
        cfg.blockDim = dim3(256, 1, 1);
        cfg.stream = stream;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        err = cudaLaunchKernelEx(&cfg, moe_gather_kernel, static_cast<const uint4*>(x), token_of_row,
                                 (const int32_t*)w.sorted_rows, (const int32_t*)w.num_tiles,
                                 reinterpret_cast<uint4*>(w.x_sorted), (int64_t)(K / 8));
        count_launch();
        if (err != cudaSuccess) return err;
    }

    // 32 words of E5M2 bits, then 32 words of rounded-nest bits
    static_assert(kMaxExperts == 1024, "the grouped kernels take two 32-word masks");
    uint32_t mask[64];
    for (int i = 0; i < 64; ++i) mask[i] = 0;
    for (int e = 0; e < E; ++e) {
        if (enc_host[e] == DPS_ENC_E5M2 || enc_host[e] == DPS_ENC_E5M2_RN) mask[e >> 5] |= 1u << (e & 31);
        if (enc_host[e] == DPS_ENC_E4M3_RN || enc_host[e] == DPS_ENC_E5M2_RN) mask[32 + (e >> 5)] |= 1u << (e & 31);
    }
    // an upper bound on the number of token tiles that needs no device round trip
    const int max_tiles = (int)((A + tn - 1) / tn + E);
    return launch_umma_grouped(mode, mask, w.x_sorted, p, r, y, A, N, K, E, tn, w.tiles, w.num_tiles, w.sorted_rows,
                               max_tiles < w.max_tiles ? max_tiles : (int)w.max_tiles, status, stream);
}

}  // namespace dps

// ---- allocation-free variant ---------------------------------------------------------------------
// Scratch for dps_moe_linear_static: one fixed array per GPU that loads the library, held until the
// process exits.  In host code the array's name is only a stand-in; the device address is looked up
// once per device (with that device current) and handed to the kernels as an ordinary pointer.
namespace dps {
namespace {

constexpr size_t kStaticScratchBytes = (size_t)DPS_MOE_STATIC_SCRATCH_BYTES;
static __device__ __align__(256) unsigned char g_moe_static_scratch[kStaticScratchBytes];

// Device address of the array, per device.  Only a successful look-up is kept: a failed one (made
// inside a stream capture, say) is tried again by the next call.
std::mutex g_static_scratch_mutex;
unsigned char* g_static_scratch_ptr[kMaxDevices] = {};

cudaError_t static_scratch_address(unsigned char** out) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_static_scratch_mutex);
    if (g_static_scratch_ptr[dev] == nullptr) {
        unsigned char* ptr = nullptr;
        e = cudaGetSymbolAddress((void**)&ptr, g_moe_static_scratch);
        if (e != cudaSuccess) {
            (void)cudaGetLastError();   // leave no sticky error behind: the next call tries again
            return e;
        }
        g_static_scratch_ptr[dev] = ptr;
    }
    *out = g_static_scratch_ptr[dev];
    return cudaSuccess;
}

}  // namespace
}  // namespace dps

extern "C" DPS_API dps_status dps_moe_linear_static(int32_t mode, const int32_t* enc_per_expert, const void* x,
                                                    const int32_t* token_of_row, const int32_t* expert_of_row,
                                                    const uint8_t* w_persist, const uint8_t* w_resid, void* y,
                                                    int64_t A, int64_t T, int64_t N, int64_t K, int32_t E,
                                                    void* cuda_stream) {
    using namespace dps;
    bool empty = false;
    const dps_status ok = check_moe_args(mode, enc_per_expert, x, token_of_row, expert_of_row, w_persist, w_resid, y, A, T,
                                         N, K, E, &empty);
    if (ok != DPS_OK) return ok;
    if (moe_workspace_bytes(A, E, K) > kStaticScratchBytes) return DPS_ERR_WORKSPACE;  // use dps_moe_linear instead
    if (empty) return DPS_OK;
    int* status = nullptr;
    const dps_status st = device_status_word(&status);
    if (st != DPS_OK) return st;
    unsigned char* scratch = nullptr;
    if (static_scratch_address(&scratch) != cudaSuccess || scratch == nullptr) return DPS_ERR_CUDA;
    const uint8_t* r = (mode == DPS_MODE_FULL) ? w_resid : nullptr;
    if (launch_moe(mode, enc_per_expert, x, token_of_row, expert_of_row, w_persist, r, y, A, T, N, K, E, scratch,
                   status, static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess)
        return DPS_ERR_CUDA;
    return DPS_OK;
}
