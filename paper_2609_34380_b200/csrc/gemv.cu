// Dense linear layer on the CUDA-core GEMV path (see gemv.cuh for the design).
#include "dps_internal.h"
#include "gemv.cuh"
#include "sm100.cuh"

namespace dps {

namespace {

template <int ENC, bool FULL, int MT>
__global__ void __launch_bounds__(kGemvThreads, 2)
gemv_dense_kernel(const __half* __restrict__ x, const uint8_t* __restrict__ P, const uint8_t* __restrict__ Rp,
                  __half* __restrict__ y, int m_count, int64_t N, int64_t K, int rows_per_cta, int red_stride) {
    extern __shared__ float red[];
    sm100::grid_launch_dependents();  // let the next kernel's CTAs take the slots this grid frees
    sm100::grid_dependency_wait();    // activations (and possibly planes) come from the preceding kernel
    const int64_t row_begin = (int64_t)blockIdx.x * rows_per_cta;
    const int64_t row_end = (row_begin + rows_per_cta < N) ? row_begin + rows_per_cta : N;
    if (row_begin >= row_end) return;
    const __half* xrow[MT];
    __half* yrow[MT];
#pragma unroll
    for (int t = 0; t < MT; ++t) {
        xrow[t] = (t < m_count) ? x + (int64_t)t * K : nullptr;
        yrow[t] = (t < m_count) ? y + (int64_t)t * N : nullptr;
    }
    gemv_rows<ENC, FULL, MT>(xrow, yrow, P, Rp, K, row_begin, row_end, red, red_stride);
}

template <int ENC, bool FULL, int MT>
cudaError_t launch_one(const __half* x, const uint8_t* p, const uint8_t* r, __half* y, int m_count, int64_t N,
                       int64_t K, cudaStream_t stream) {
    // Two CTAs per SM; shrink the row range if the per-warp partial-sum table would outgrow 32 KB.
    const int64_t max_rows = (32 * 1024) / (kGemvWarps * MT * 4) / kGemvRows * kGemvRows;
    int64_t target = (int64_t)sm_count() * 2;
    int64_t rows = (N + target - 1) / target;
    if (rows < 1) rows = 1;
    if (rows > max_rows) rows = max_rows;
    const int64_t grid = (N + rows - 1) / rows;
    const int red_stride = (int)((rows + kGemvRows - 1) / kGemvRows) * kGemvRows * MT;
    const size_t smem = (size_t)kGemvWarps * red_stride * sizeof(float);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid, 1, 1);
    cfg.blockDim = dim3(kGemvThreads, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, gemv_dense_kernel<ENC, FULL, MT>, x, p, r, y, m_count, N, K, (int)rows,
                                       red_stride);
    count_launch();
    return e;
}

template <int ENC, bool FULL>
cudaError_t launch_tokens(const __half* x, const uint8_t* p, const uint8_t* r, __half* y, int m_count, int64_t N,
                          int64_t K, cudaStream_t stream) {
    if (m_count == 1) return launch_one<ENC, FULL, 1>(x, p, r, y, m_count, N, K, stream);
    if (m_count == 2) return launch_one<ENC, FULL, 2>(x, p, r, y, m_count, N, K, stream);
    return launch_one<ENC, FULL, 4>(x, p, r, y, m_count, N, K, stream);
}

}  // namespace

cudaError_t launch_gemv(int mode, int enc, const void* x, const uint8_t* p, const uint8_t* r, void* y, int64_t M,
                        int64_t N, int64_t K, cudaStream_t stream) {
    const __half* xh = static_cast<const __half*>(x);
    __half* yh = static_cast<__half*>(y);
    const bool full = mode == DPS_MODE_FULL;
    for (int64_t m0 = 0; m0 < M; m0 += 4) {
        const int mc = (int)((M - m0) < 4 ? (M - m0) : 4);
        const __half* xs = xh + m0 * K;
        __half* ys = yh + m0 * N;
        cudaError_t e;
        const int enc_here = full ? enc : base_enc(enc);
        if (enc_here == kEncE4M3R) e = launch_tokens<kEncE4M3R, true>(xs, p, r, ys, mc, N, K, stream);
        else if (enc_here == kEncE5M2R) e = launch_tokens<kEncE5M2R, true>(xs, p, r, ys, mc, N, K, stream);
        else if (enc_here == kEncE4M3)
            e = full ? launch_tokens<kEncE4M3, true>(xs, p, r, ys, mc, N, K, stream)
                     : launch_tokens<kEncE4M3, false>(xs, p, r, ys, mc, N, K, stream);
        else
            e = full ? launch_tokens<kEncE5M2, true>(xs, p, r, ys, mc, N, K, stream)
                     : launch_tokens<kEncE5M2, false>(xs, p, r, ys, mc, N, K, stream);
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

}  // namespace dps
