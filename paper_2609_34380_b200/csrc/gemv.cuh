// CUDA-core GEMV body for very small token counts (decode with 1-4 tokens), shared by the
// dense and the grouped (MoE) launchers.
//
// Paper: "Scheduler: Dual-Precision Execution" -- fast mode streams the persistent plane only,
// full mode streams both planes and rebuilds the FP16 weights on chip.  Decode is a
// memory-bound GEMV, so the design goal is bytes in flight, not arithmetic:
//   * a CTA owns a contiguous range of weight rows; its 256 threads split K, each thread
//     keeping 16 consecutive activations per token in registers for a whole pass over the rows;
//   * weights arrive as 128-bit streaming loads of P (and R), eight rows in flight per thread;
//   * the planes are zipped to FP16 with byte permutes, products are exact in FP32;
//   * partial sums are folded across the warp with a transposing shuffle butterfly (V-1
//     shuffles for V values instead of 5V), parked per warp in shared memory and summed across
//     warps in a fixed order at the end -- no atomics, so results are bit-stable.
#pragma once
#include "bits.cuh"

namespace dps {

constexpr int kGemvThreads = 256;
constexpr int kGemvWarps = kGemvThreads / 32;
constexpr int kGemvRows = 8;                      // weight rows reduced together (one butterfly)
constexpr int kGemvBatch = 2;                     // row groups whose loads are issued together when only
                                                  // one plane is read, so both modes keep 256 B per thread in flight
constexpr int kGemvKPass = kGemvThreads * 16;     // K covered by one pass of the CTA

__device__ __forceinline__ uint4 ldg_stream16(const void* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

// Sum V values per lane across the 32 lanes.  Returns the total of value index
// (lane >> (5 - log2 V)); every lane of that group holds the same total.
template <int V>
__device__ __forceinline__ float butterfly_sum(float (&v)[V], int lane) {
    static_assert(V == 1 || V == 2 || V == 4 || V == 8 || V == 16 || V == 32, "V must be a power of two <= 32");
    int off = 16;
#pragma unroll
    for (int n = V; n > 1; n >>= 1) {
        const int half = n >> 1;
        const bool upper = (lane & off) != 0;
#pragma unroll
        for (int j = 0; j < half; ++j) {
            float keep = upper ? v[j + half] : v[j];
            float send = upper ? v[j] : v[j + half];
            v[j] = keep + __shfl_xor_sync(0xFFFFFFFFu, send, off);
        }
        off >>= 1;
    }
    float s = v[0];
    for (; off > 0; off >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, off);
    return s;
}

// One CTA computes y[t][row] for rows [row_begin, row_end) of one weight matrix and up to MT
// tokens.  xrow[t] / yrow[t] point at the token's activation row and output row (NULL = no
// token in that slot).  red is shared memory for kGemvWarps * red_stride floats with
// red_stride >= ceil(rows / kGemvRows) * kGemvRows * MT.
template <int ENC, bool FULL, int MT>
__device__ __forceinline__ void gemv_rows(const __half* const (&xrow)[MT], __half* const (&yrow)[MT],
                                          const uint8_t* __restrict__ P, const uint8_t* __restrict__ Rp,
                                          int64_t K, int64_t row_begin, int64_t row_end, float* red,
                                          int red_stride) {
    constexpr int V = kGemvRows * MT;
    constexpr int kGroup = 32 / V;  // lanes that end up holding the same total
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int nrows = (int)(row_end - row_begin);
    const int nblocks = (nrows + kGemvRows - 1) / kGemvRows;

    for (int64_t k0 = 0; k0 < K; k0 += kGemvKPass) {
        const int64_t k = k0 + (int64_t)tid * 16;
        const bool active = k < K;
        float xf[MT][16];
#pragma unroll
        for (int t = 0; t < MT; ++t) {
            uint4 a = make_uint4(0, 0, 0, 0), b = a;
            if (active && xrow[t] != nullptr) {
                a = *reinterpret_cast<const uint4*>(xrow[t] + k);
                b = *reinterpret_cast<const uint4*>(xrow[t] + k + 8);
            }
            const uint32_t h[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                float2 f = h2f2(h[j]);
                xf[t][2 * j] = f.x;
                xf[t][2 * j + 1] = f.y;
            }
        }
        constexpr int kBatch = FULL ? 1 : kGemvBatch;
        for (int b0 = 0; b0 < nblocks; b0 += kBatch) {
            uint4 pw[kBatch][kGemvRows], rw[kBatch][kGemvRows];
#pragma unroll
            for (int u = 0; u < kBatch; ++u) {
#pragma unroll
                for (int i = 0; i < kGemvRows; ++i) {
                    const int64_t row = row_begin + (int64_t)(b0 + u) * kGemvRows + i;
                    pw[u][i] = make_uint4(0, 0, 0, 0);
                    rw[u][i] = make_uint4(0, 0, 0, 0);
                    if (active && row < row_end) {
                        pw[u][i] = ldg_stream16(P + row * K + k);
                        if (FULL) rw[u][i] = ldg_stream16(Rp + row * K + k);
                    }
                }
            }
#pragma unroll
            for (int u = 0; u < kBatch; ++u) {
                const int b = b0 + u;
                if (b >= nblocks) break;
                float acc[V];
#pragma unroll
                for (int v = 0; v < V; ++v) acc[v] = 0.f;
#pragma unroll
                for (int i = 0; i < kGemvRows; ++i) {
                    uint32_t h[8];
                    join16<ENC, FULL>(pw[u][i], rw[u][i], h);
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const float2 w = h2f2(h[j]);
#pragma unroll
                        for (int t = 0; t < MT; ++t) {
                            acc[i * MT + t] = fmaf(w.x, xf[t][2 * j], acc[i * MT + t]);
                            acc[i * MT + t] = fmaf(w.y, xf[t][2 * j + 1], acc[i * MT + t]);
                        }
                    }
                }
                const float s = butterfly_sum<V>(acc, lane);
                if ((lane & (kGroup - 1)) == 0) {
                    float* slot = red + warp * red_stride + b * V + (lane / kGroup);
                    *slot = (k0 == 0) ? s : (*slot + s);
                }
            }
        }
    }
    __syncthreads();
    for (int o = tid; o < nblocks * V; o += kGemvThreads) {
        const int b = o / V, rem = o % V, i = rem / MT, t = rem % MT;
        const int row = b * kGemvRows + i;
        if (row < nrows && yrow[t] != nullptr) {
            float s = 0.f;
#pragma unroll
            for (int w = 0; w < kGemvWarps; ++w) s += red[w * red_stride + o];
            yrow[t][row_begin + row] = __float2half_rn(s);
        }
    }
    __syncthreads();  // red is reused by the caller's next group of tokens
}

}  // namespace dps
