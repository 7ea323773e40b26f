// Grouped (MoE) linear layer: device-side routing pre-pass + grouped kernels.
// Paper: "Scheduler: Dual-Precision Execution", paragraph "Dual-mode serving (DPS) with
// asymmetric switching" -- GroupedGEMM kernels with nested reconstruction serve MoE models.
//
// Workspace layout (int32 words, E4 = E rounded up to 4, A4 = A rounded up to 4):
//   counts[E4] | offsets[E4 + 4] | sorted_rows[A4] | reserved
// sorted_rows lists the valid row ids grouped by expert, in ascending row order inside each
// group (a stable grouping, so the layout is reproducible).
#include "dps_internal.h"
#include "gemv.cuh"

namespace dps {

namespace {

constexpr int kRouteThreads = 1024;
constexpr int kMaxExperts = 1024;

struct EncMask {
    uint32_t e5m2[kMaxExperts / 32];  // bit e set: expert e uses E5M2, else E4M3
};

inline int64_t round4(int64_t v) { return (v + 3) / 4 * 4; }

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
                 int E, int32_t* counts, int32_t* offsets, int32_t* sorted_rows, int* status) {
    __shared__ int s_cnt[kMaxExperts];
    __shared__ int s_off[kMaxExperts];
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
        int run = 0;
        for (int e = 0; e < E; ++e) {
            s_off[e] = run;
            offsets[e] = run;
            counts[e] = s_cnt[e];
            run += s_cnt[e];
        }
        offsets[E] = run;
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

// Interim grouped kernel on the CUDA-core GEMV body: blockIdx.y = expert, blockIdx.x = row
// range of that expert's matrix; tokens of the group are taken four at a time.
template <bool FULL>
__global__ void __launch_bounds__(kGemvThreads, 2)
moe_gemv_kernel(const __half* __restrict__ x, const int32_t* __restrict__ token_of_row,
                const int32_t* __restrict__ sorted_rows, const int32_t* __restrict__ counts,
                const int32_t* __restrict__ offsets, const uint8_t* __restrict__ P,
                const uint8_t* __restrict__ Rp, __half* __restrict__ y, int64_t N, int64_t K, EncMask enc,
                int rows_per_cta, int red_stride) {
    extern __shared__ float red[];
    const int e = blockIdx.y;
    const int cnt = counts[e];
    if (cnt == 0) return;
    const int off = offsets[e];
    const int64_t row_begin = (int64_t)blockIdx.x * rows_per_cta;
    const int64_t row_end = (row_begin + rows_per_cta < N) ? row_begin + rows_per_cta : N;
    if (row_begin >= row_end) return;
    const uint8_t* Pe = P + (int64_t)e * N * K;
    const uint8_t* Re = FULL ? Rp + (int64_t)e * N * K : nullptr;
    const bool e5m2 = (enc.e5m2[e >> 5] >> (e & 31)) & 1u;
    for (int g = 0; g < cnt; g += 4) {
        const __half* xrow[4];
        __half* yrow[4];
#pragma unroll
        for (int t = 0; t < 4; ++t) {
            xrow[t] = nullptr;
            yrow[t] = nullptr;
            if (g + t < cnt) {
                const int a = sorted_rows[off + g + t];
                const int tok = token_of_row ? token_of_row[a] : a;
                xrow[t] = x + (int64_t)tok * K;
                yrow[t] = y + (int64_t)a * N;
            }
        }
        if (e5m2) gemv_rows<kEncE5M2, FULL, 4>(xrow, yrow, Pe, Re, K, row_begin, row_end, red, red_stride);
        else gemv_rows<kEncE4M3, FULL, 4>(xrow, yrow, Pe, Re, K, row_begin, row_end, red, red_stride);
    }
}

}  // namespace

size_t moe_workspace_bytes(int64_t A, int32_t E) {
    if (A < 0 || E <= 0 || E > kMaxExperts || A > (int64_t)1 << 30) return 0;
    const int64_t words = round4(E) + (round4(E) + 4) + round4(A);
    const int64_t reserved = 16 * (A / 16 + E + 16);
    return (size_t)((words * 4 + reserved + 255) / 256 * 256);
}

cudaError_t launch_moe(int mode, const int32_t* enc_host, const void* x, const int32_t* token_of_row,
                       const int32_t* expert_of_row, const uint8_t* p, const uint8_t* r, void* y, int64_t A,
                       int64_t T, int64_t N, int64_t K, int32_t E, void* workspace, int* status,
                       cudaStream_t stream) {
    int32_t* counts = static_cast<int32_t*>(workspace);
    int32_t* offsets = counts + round4(E);
    int32_t* sorted_rows = offsets + round4(E) + 4;
    moe_route_kernel<<<1, kRouteThreads, 0, stream>>>(token_of_row, expert_of_row, (int)A, (int)T, E, counts, offsets,
                                                      sorted_rows, status);
    count_launch();
    cudaError_t err = cudaGetLastError();
    if (err != cudaSuccess) return err;

    EncMask enc;
    for (int i = 0; i < kMaxExperts / 32; ++i) enc.e5m2[i] = 0;
    for (int e = 0; e < E; ++e)
        if (enc_host[e] == DPS_ENC_E5M2) enc.e5m2[e >> 5] |= 1u << (e & 31);

    constexpr int MT = 4;
    const int64_t max_rows = (32 * 1024) / (kGemvWarps * MT * 4) / kGemvRows * kGemvRows;
    int64_t per_expert = ((int64_t)sm_count() * 2 + E - 1) / E;
    int64_t rows = (N + per_expert - 1) / per_expert;
    if (rows < 1) rows = 1;
    if (rows > max_rows) rows = max_rows;
    const int64_t gx = (N + rows - 1) / rows;
    const int red_stride = (int)((rows + kGemvRows - 1) / kGemvRows) * kGemvRows * MT;
    const size_t smem = (size_t)kGemvWarps * red_stride * sizeof(float);
    dim3 grid((unsigned)gx, (unsigned)E);
    const __half* xh = static_cast<const __half*>(x);
    __half* yh = static_cast<__half*>(y);
    if (mode == DPS_MODE_FULL)
        moe_gemv_kernel<true><<<grid, kGemvThreads, smem, stream>>>(xh, token_of_row, sorted_rows, counts, offsets, p,
                                                                    r, yh, N, K, enc, (int)rows, red_stride);
    else
        moe_gemv_kernel<false><<<grid, kGemvThreads, smem, stream>>>(xh, token_of_row, sorted_rows, counts, offsets,
                                                                     p, r, yh, N, K, enc, (int)rows, red_stride);
    count_launch();
    return cudaGetLastError();
}

}  // namespace dps
