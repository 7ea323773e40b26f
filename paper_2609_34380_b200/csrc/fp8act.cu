// Fast mode with FP8 activations: the persistent plane is consumed by the FP8 tensor cores AS IT IS.
//
// Paper: "Mapper: Semi-Unified Memory Abstraction", "Persistent Region" paragraph -- FP8 execution
// can halve memory accesses "or double peak tensor-core throughput with hardware support".  The
// persistent byte of the nested format is a valid FP8 number (E5M2: the fast-mode weight itself;
// E4M3: 2^8 times it), so with activations quantised to E4M3 the layer is a plain FP8 x FP8
// contraction: no rebuilding of weights, both operands straight from shared memory
// (tcgen05.mma kind::f8f6f4, SS form), FP32 accumulation in tensor memory.
//
// Activation quantisation (the paper gives no recipe; per-token dynamic scaling is the reading
// taken): scale[m] = max_k |x[m][k]| / 448 (1 for an all-zero token), q = E4M3(x / scale), round to
// nearest even, saturating; y[m][n] = scale[m] * sum_k q[m][k] * W_fast[n][k].
//
// Kernel: tiles of 128 weight rows x 256 tokens, K in blocks of 128 bytes, one persistent CTA per
// SM.  Warp 0 TMA producer (P tile 128 x 128 B, activation tile 256 x 128 B, 128-byte swizzle), warp 1
// MMA issuer (two accumulators in tensor memory), warps 2-5 epilogue (TMEM -> scale -> FP16 ->
// shared-memory buffer -> 16-byte stores), overlapped with the next tile's MMAs.
#include <cuda.h>
#include <cuda_fp16.h>
#include <cuda_fp8.h>

#include "dps_internal.h"
#include "sm100.cuh"

namespace dps {

bool make_byte_map_sw128(CUtensorMap* map, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows);

namespace {

using namespace sm100;

// ---- activation quantisation ------------------------------------------------------------------
constexpr int kQuantThreads = 256;

// One CTA per token: maximum magnitude, scale, then the E4M3 codes.  Rows of up to 8192 elements stay
// in registers between the two passes (four 16-byte pieces per thread); longer rows are read again.
constexpr int kQuantKeep = 4;

__device__ __forceinline__ uint2 quantize8(const uint4& v, float sc) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
    uint32_t out[2] = {0u, 0u};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&w[j]));
        const float2 d = make_float2(__fdiv_rn(f.x, sc), __fdiv_rn(f.y, sc));
        const uint32_t pair = (uint32_t)__nv_cvt_float2_to_fp8x2(d, __NV_SATFINITE, __NV_E4M3);   // .x in the low byte
        out[j >> 1] |= pair << ((j & 1) * 16);
    }
    return make_uint2(out[0], out[1]);
}

__global__ void __launch_bounds__(kQuantThreads)
quantize_activations_kernel(const uint4* __restrict__ x, uint2* __restrict__ q, float* __restrict__ scale, int64_t k8,
                            int* status) {
    __shared__ float s_max[kQuantThreads / 32];
    __shared__ float s_scale;
    grid_launch_dependents();
    grid_dependency_wait();   // the activations are the preceding kernel's output
    const int64_t m = blockIdx.x;
    const uint4* row = x + m * k8;
    const bool keep = k8 <= (int64_t)kQuantKeep * kQuantThreads;
    uint4 held[kQuantKeep];
    float amax = 0.f;
    bool bad = false;
    auto scan = [&](const uint4& v) {
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&w[j]));
            const float a = fabsf(f.x), b = fabsf(f.y);
            bad |= !(a <= 65504.f) || !(b <= 65504.f);   // Inf or NaN
            amax = fmaxf(amax, fmaxf(a, b));
        }
    };
    if (keep) {
#pragma unroll
        for (int u = 0; u < kQuantKeep; ++u) {
            const int64_t i = (int64_t)u * kQuantThreads + threadIdx.x;
            held[u] = make_uint4(0u, 0u, 0u, 0u);
            if (i < k8) held[u] = row[i];
            scan(held[u]);
        }
    } else {
        for (int64_t i = threadIdx.x; i < k8; i += kQuantThreads) scan(row[i]);
    }
    for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, o));
    if (__syncthreads_or(bad) && threadIdx.x == 0) atomicExch(status, (int)DPS_ERR_DATA);
    if ((threadIdx.x & 31) == 0) s_max[threadIdx.x >> 5] = amax;
    __syncthreads();
    if (threadIdx.x == 0) {
        float a = 0.f;
        for (int w = 0; w < kQuantThreads / 32; ++w) a = fmaxf(a, s_max[w]);
        const float sc = a > 0.f ? __fdiv_rn(a, 448.0f) : 1.0f;
        s_scale = sc;
        scale[m] = sc;
    }
    __syncthreads();
    const float sc = s_scale;
    uint2* qrow = q + m * k8;
    if (keep) {
#pragma unroll
        for (int u = 0; u < kQuantKeep; ++u) {
            const int64_t i = (int64_t)u * kQuantThreads + threadIdx.x;
            if (i < k8) qrow[i] = quantize8(held[u], sc);
        }
    } else {
        for (int64_t i = threadIdx.x; i < k8; i += kQuantThreads) qrow[i] = quantize8(row[i], sc);
    }
}

// ---- FP8 x FP8 linear ---------------------------------------------------------------------------
constexpr int kRows = 128;      // weight rows per tile (UMMA M)
constexpr int kBlockBytes = 128;                                  // K per stage (one swizzle atom of bytes)
constexpr int kThreads = 192;
// Tokens per tile (UMMA N): 256, or 128 when 256-token tiles would leave SMs without one.
__host__ __device__ constexpr int stage_bytes_fp8(int tokens) { return (kRows + tokens) * kBlockBytes; }   // 48 / 32 KB
__host__ __device__ constexpr int stages_fp8(int tokens) { return tokens == 256 ? 4 : 6; }

// Instruction descriptor for kind::f8f6f4: FP32 accumulator, K-major operands; formats 0 = E4M3, 1 = E5M2.
__host__ __device__ constexpr uint32_t idesc_f8(int m, int n, int a_format, int b_format) {
    return (1u << 4) | ((uint32_t)a_format << 7) | ((uint32_t)b_format << 10) | ((uint32_t)(n >> 3) << 17) |
           ((uint32_t)(m >> 4) << 24);
}

// D[tmem] (+)= A[smem] * B[smem], FP8 operands; issued by ONE thread.
__device__ __forceinline__ void umma_f8_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                           uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(0u)
        : "memory");
}

struct Fp8Params {
    __half* y;
    const float* scale;
    int M, N, K;
    int e5m2;      // the persistent plane is E5M2 (else E4M3, whose bytes read as FP8 are 2^8 times the weights)
    int* status;
};

constexpr int kEpiCols = 32;                                      // token columns per epilogue chunk
constexpr int kEpiBytes = kEpiCols * kRows * 2;                   // 8 KB buffer behind the ring

// Persistent: one CTA per SM walks the tiles (groups of 8 row tiles x all token tiles).  Two
// accumulators of 256 columns fill tensor memory, so the MMA warp starts the next tile while the
// four epilogue warps drain the previous one -- at FP8 rates the epilogue of a 128 x 256 tile is a
// fifth of the tile's MMA time.  The epilogue goes through a small buffer, 32 token columns at a
// time: the stage ring never idles.
template <int kTokens>
__global__ void __launch_bounds__(kThreads, 1)
fp8act_linear_kernel(const __grid_constant__ CUtensorMap map_p, const __grid_constant__ CUtensorMap map_x,
                     const Fp8Params prm) {
    constexpr int kStageBytes = stage_bytes_fp8(kTokens);
    constexpr int kStages = stages_fp8(kTokens);
    constexpr uint32_t kTmemCols = 2 * kTokens;   // two accumulators
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bar_full[kStages];
    __shared__ __align__(8) uint64_t bar_empty[kStages];
    __shared__ __align__(8) uint64_t bar_d_full[2];
    __shared__ __align__(8) uint64_t bar_d_empty[2];
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;    // set by an epilogue warp whose wait timed out; the four leave together

    grid_launch_dependents();
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t epi_base = smem_base + (uint32_t)(kStages * kStageBytes);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int row_tiles = (prm.N + kRows - 1) / kRows, tok_tiles = (prm.M + kTokens - 1) / kTokens;
    const int total = row_tiles * tok_tiles;
    const int num_kb = (prm.K + kBlockBytes - 1) / kBlockBytes;
    auto tile_origin = [&](int lin, int& n0, int& m0) {
        int row_tile = lin, tok_tile = 0;
        if (tok_tiles > 1) {
            constexpr int kRowGroup = 8;
            const int per_group = kRowGroup * tok_tiles;
            const int group = lin / per_group, within = lin % per_group;
            const int rows_here = min(kRowGroup, row_tiles - group * kRowGroup);
            row_tile = group * kRowGroup + within % rows_here;
            tok_tile = within / rows_here;
        }
        n0 = row_tile * kRows;
        m0 = tok_tile * kTokens;
    };

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(smem_u32(&bar_full[s]), 1);
            mbar_init(smem_u32(&bar_empty[s]), 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(smem_u32(&bar_d_full[a]), 1);
            mbar_init(smem_u32(&bar_d_empty[a]), 4);   // one arrival per epilogue warp
        }
        abort_flag = 0;
        fence_barrier_init();
        prefetch_tensormap(&map_p);
        prefetch_tensormap(&map_x);
    }
    if (warp == 1) tmem_alloc(smem_u32(&tmem_base_slot), kTmemCols);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = tmem_base_slot;

    bool ok = true;
    if (warp == 0) {
        // ---------------- TMA producer ----------------
        grid_dependency_wait();   // the activation codes come from the quantisation kernel
        int s = 0;
        uint32_t ph = 0;
        for (int lin = blockIdx.x; lin < total && ok; lin += gridDim.x) {
            int n0, m0;
            tile_origin(lin, n0, m0);
            for (int i = 0; i < num_kb && ok; ++i, s = (s + 1 == kStages) ? 0 : s + 1, ph ^= (s == 0)) {
                ok = mbar_wait(smem_u32(&bar_empty[s]), ph ^ 1u);
                ok = __all_sync(0xFFFFFFFFu, ok);
                if (!ok) break;
                if (elect_one()) {
                    const uint32_t full = smem_u32(&bar_full[s]);
                    const uint32_t dst = smem_base + (uint32_t)s * kStageBytes;
                    mbar_arrive_expect_tx(full, (uint32_t)kStageBytes);
                    tma_load_2d(dst, &map_p, full, i * kBlockBytes, n0);
                    tma_load_2d(dst + kRows * kBlockBytes, &map_x, full, i * kBlockBytes, m0);
                }
                __syncwarp();
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        const uint32_t idesc = idesc_f8(kRows, kTokens, prm.e5m2 ? 1 : 0, 0);
        int s = 0, it = 0;
        uint32_t ph = 0;
        for (int lin = blockIdx.x; lin < total && ok; lin += gridDim.x, ++it) {
            const int acc = it & 1;
            if (it >= 2) {   // the tile before last used this accumulator: its epilogue must have read it out
                ok = mbar_wait(smem_u32(&bar_d_empty[acc]), (uint32_t)((it >> 1) - 1) & 1u);
                ok = __all_sync(0xFFFFFFFFu, ok);
                if (!ok) break;
                tc_fence_after_sync();
            }
            const uint32_t tmem_d = tmem_base + (uint32_t)(acc * kTokens);
            for (int i = 0; i < num_kb && ok; ++i, s = (s + 1 == kStages) ? 0 : s + 1, ph ^= (s == 0)) {
                ok = mbar_wait(smem_u32(&bar_full[s]), ph);
                ok = __all_sync(0xFFFFFFFFu, ok);
                if (!ok) break;
                tc_fence_after_sync();
                if (elect_one()) {
                    const uint32_t abase = smem_base + (uint32_t)s * kStageBytes;
                    const uint64_t adesc = umma_desc_k_sw128(abase), bdesc = umma_desc_k_sw128(abase + kRows * kBlockBytes);
#pragma unroll
                    for (int j = 0; j < kBlockBytes / 32; ++j)   // 32 K elements = 32 bytes per instruction
                        umma_f8_ss(tmem_d, adesc + (uint64_t)(j * 2), bdesc + (uint64_t)(j * 2), idesc,
                                   (i > 0 || j > 0) ? 1u : 0u);
                    umma_commit(smem_u32(&bar_empty[s]));
                    if (i == num_kb - 1) umma_commit(smem_u32(&bar_d_full[acc]));
                }
                __syncwarp();
            }
        }
    } else {
        // ---------------- epilogue: D[row][token] * scale[token] -> FP16 -> y[token][n0 + row] ----------------
        const int q = warp & 3;                          // TMEM lane quarter this warp may touch
        const int row = q * 32 + lane;
        const uint32_t lane_base = (uint32_t)(q * 32) << 16;
        const float wscale = prm.e5m2 ? 1.0f : 0.00390625f;   // E4M3 bytes read as FP8 are 2^8 times the weights
        const int et = (int)threadIdx.x - 64;            // index among the 128 epilogue threads
        int it = 0;
        for (int lin = blockIdx.x; lin < total; lin += gridDim.x, ++it) {
            int n0, m0;
            tile_origin(lin, n0, m0);
            const int acc = it & 1;
            const uint32_t tmem_d = tmem_base + (uint32_t)(acc * kTokens);
            const int ncols = min(kTokens, prm.M - m0);
            if (ok) ok = mbar_wait(smem_u32(&bar_d_full[acc]), (uint32_t)(it >> 1) & 1u);
            ok = __all_sync(0xFFFFFFFFu, ok);
            if (ok) tc_fence_after_sync();
            else abort_flag = 1;
            // same trip count in all four warps (it depends on the tile only): the barriers always match
            for (int c0 = 0; c0 < ncols; c0 += kEpiCols) {
                if (ok) {
#pragma unroll
                    for (int h = 0; h < kEpiCols / 16; ++h) {
                        const int cb = c0 + 16 * h;
                        if (cb >= ncols) break;
                        uint32_t v[16];
                        tmem_ld_32x32b_x16(tmem_d + lane_base + (uint32_t)cb, v);
                        tmem_wait_ld();
#pragma unroll
                        for (int j = 0; j < 16; ++j) {
                            const int c = cb + j;
                            const float sc = c < ncols ? prm.scale[m0 + c] * wscale : 0.f;
                            const __half hv = __float2half_rn(__uint_as_float(v[j]) * sc);
                            const uint32_t addr = epi_base + (uint32_t)(((c - c0) * kRows + row) * 2);
                            asm volatile("st.shared.u16 [%0], %1;" ::"r"(addr), "h"(__half_as_ushort(hv)) : "memory");
                        }
                    }
                }
                if (c0 + kEpiCols >= ncols) {            // last chunk read: the accumulator is free again
                    tc_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&bar_d_empty[acc]));
                }
                named_barrier_sync(1, 128);
                if (ok) {
                    constexpr int kChunks = kRows / 8;   // 16-byte pieces of one token's rows
                    const int cols_here = min(kEpiCols, ncols - c0);
                    for (int item = et; item < cols_here * kChunks; item += 128) {
                        const int c = item / kChunks, qq = item % kChunks;
                        const int n = n0 + qq * 8;
                        if (n >= prm.N) continue;        // N is a multiple of 8
                        uint4 val;
                        asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];"
                                     : "=r"(val.x), "=r"(val.y), "=r"(val.z), "=r"(val.w)
                                     : "r"(epi_base + (uint32_t)((c * kRows + qq * 8) * 2)));
                        *reinterpret_cast<uint4*>(prm.y + (int64_t)(m0 + c0 + c) * prm.N + n) = val;
                    }
                }
                named_barrier_sync(1, 128);              // the buffer is free for the next chunk
            }
            if (*reinterpret_cast<volatile int*>(&abort_flag)) {   // read after the tile's last barrier: the same in all four warps
                ok = false;
                break;
            }
        }
    }
    if (!ok) atomicExch(prm.status, (int)DPS_ERR_CUDA);
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

}  // namespace

cudaError_t launch_quantize_activations(const void* x, uint8_t* q, float* scale, int64_t M, int64_t K, int* status,
                                        cudaStream_t stream) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)M, 1, 1);
    cfg.blockDim = dim3(kQuantThreads, 1, 1);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, quantize_activations_kernel, static_cast<const uint4*>(x),
                                       reinterpret_cast<uint2*>(q), scale, (int64_t)(K / 8), status);
    count_launch();
    return e;
}

namespace {
template <int kTokens>
cudaError_t launch_fp8_tokens(int enc, const uint8_t* q, const float* scale, const uint8_t* p, void* y, int64_t M, int64_t N,
                              int64_t K, int* status, cudaStream_t stream) {
    static PerDeviceOnce setup;     // per instantiation and per device
    const size_t smem = (size_t)stages_fp8(kTokens) * stage_bytes_fp8(kTokens) + kEpiBytes + 1024;
    auto kernel = fp8act_linear_kernel<kTokens>;
    {
        const cudaError_t e = setup.run(
            [&] { return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem); });
        if (e != cudaSuccess) return e;
    }
    CUtensorMap mp, mx;
    if (!make_byte_map_sw128(&mp, p, (uint64_t)N, (uint64_t)K, kRows) ||
        !make_byte_map_sw128(&mx, q, (uint64_t)M, (uint64_t)K, kTokens))
        return cudaErrorInvalidValue;
    Fp8Params prm;
    prm.y = static_cast<__half*>(y);
    prm.scale = scale;
    prm.M = (int)M;
    prm.N = (int)N;
    prm.K = (int)K;
    prm.e5m2 = enc == DPS_ENC_E5M2;
    prm.status = status;
    const int64_t tiles = ((N + kRows - 1) / kRows) * ((M + kTokens - 1) / kTokens);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(tiles < sm_count() ? tiles : sm_count()), 1, 1);   // one CTA per SM walks the tiles
    cfg.blockDim = dim3(kThreads, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, kernel, mp, mx, prm);
    count_launch();
    return e;
}
}  // namespace

cudaError_t launch_linear_fp8act(int enc, const uint8_t* q, const float* scale, const uint8_t* p, void* y, int64_t M,
                                 int64_t N, int64_t K, int* status, cudaStream_t stream) {
    // 256-token tiles unless they would leave SMs without a tile (few weight rows, few tokens)
    const int64_t tiles256 = ((N + kRows - 1) / kRows) * ((M + 255) / 256);
    if (tiles256 < sm_count() && M > 128) return launch_fp8_tokens<128>(enc, q, scale, p, y, M, N, K, status, stream);
    return launch_fp8_tokens<256>(enc, q, scale, p, y, M, N, K, status, stream);
}

}  // namespace dps
