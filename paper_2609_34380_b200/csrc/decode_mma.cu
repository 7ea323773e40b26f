// Decode linear layer for a handful of tokens (up to 16): a register-streaming kernel.
//
// Paper: "Scheduler: Dual-Precision Execution" -- fast mode streams the FP8 tensor only, full mode
// streams the FP8 and the residual tensor and rebuilds the FP16 weights during computation.  With
// a handful of tokens the layer is a weight stream bound by HBM, so the kernel is built around the
// stream, not around the arithmetic:
//   * every warp owns the same 16 weight rows as its CTA and every 8th 64-byte slice of K; each lane
//     issues 128-bit loads of P (and R) for two rows, several K rounds ahead, so that a CTA keeps
//     32-64 KB in flight and its eight warps together read 512 contiguous bytes of each row;
//   * the plane bytes become packed FP16 pairs in registers -- E4M3 fast mode with the hardware
//     FP8->FP16 conversion (exact, it yields 2^8 times the weight; the factor is taken out at the
//     store), the other variants with byte permutes -- and those registers ARE the A fragments of
//     a warp-level m16n8k16 MMA.  The activations are already FP16 pairs, i.e. B fragments.  No
//     conversion to FP32, no FMA per weight: about one integer instruction per weight;
//   * the K order inside an MMA is free as long as both operands agree, which is what lets each
//     lane feed 16 consecutive bytes of one row (four MMAs' worth) without any shuffle;
//   * partial sums of the eight warps are added in a fixed order through shared memory, so the
//     result is bit-stable.  One CTA per 16-row block: the hardware scheduler balances the SMs;
//   * the first batch of weight loads is issued before the kernel waits for its predecessor in
//     the stream (programmatic dependent launch): the planes are model state, only the
//     activations can be that predecessor's output.
// Tensor memory and TMA buy nothing here (no reuse, nothing to stage); the wide tcgen05 tiles take
// over once the token count makes the layer a real contraction.
#include <cuda_fp16.h>
#include <cuda_fp8.h>

#include <cstdlib>

#include "bits.cuh"
#include "dps_internal.h"
#include "sm100.cuh"

namespace dps {

namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kRowsPerBlock = 16;
constexpr int kRoundK = kWarps * 64;  // K covered by the CTA per round: each warp 64 bytes per row

__device__ __forceinline__ uint4 ldg_stream(const void* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

// Optional timeline (compile with -DDPS_TRACE): time stamps of the CTAs of the last eight launches, read
// back with dps_debug_decode_times().
#ifdef DPS_TRACE
constexpr int kTraceCtas = 1536, kTraceEvents = 8, kTraceLaunches = 8;
__device__ unsigned long long g_decode_times[kTraceLaunches * kTraceCtas * kTraceEvents];
#define DPS_DSTAMP(ev)                                                                                          \
    do {                                                                                                        \
        if (threadIdx.x == 0 && blockIdx.x < kTraceCtas)                                                        \
            g_decode_times[((trace_slot % kTraceLaunches) * kTraceCtas + blockIdx.x) * kTraceEvents + (ev)] =  \
                sm100::global_timer_ns();                                                                       \
    } while (0)
#else
#define DPS_DSTAMP(ev) do { } while (0)
#endif

// D (16x8, FP32) += A (16x16 FP16, row) * B (16x8 FP16, col)
__device__ __forceinline__ void mma_16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                          uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// 16 plane bytes (+ residual bytes) of one row -> 8 packed FP16 pairs, element order preserved.
// E4M3 fast mode returns 2^8 times the weights; the kernel's kScale undoes it at the store.
template <int ENC, bool FULL>
__device__ __forceinline__ void to_half_pairs(const uint4& p, const uint4& r, uint32_t (&h)[8]) {
    if (!FULL) fast16<ENC>(p, h);
    else join16<ENC, FULL>(p, r, h);
}

// HALF: the CTA owns 8 weight rows instead of 16 (the upper half of every MMA tile is zero).  It
// doubles the number of CTAs for matrices with few rows; the MMA work wasted is irrelevant here.
// Three CTAs per SM for the variant that fits them (full mode, 8 tokens, two rounds in flight:
// 80 registers); one register more and the allocation granularity drops it to two CTAs, which
// was measured 10 % slower on the wide Llama-7B layers.
template <int ENC, bool FULL, int NT, int U, bool HALF>
__global__ void __launch_bounds__(kThreads, (FULL && NT == 1 && U == 2) ? 3 : 2)
decode_mma_kernel(const __half* __restrict__ x, const uint8_t* __restrict__ P, const uint8_t* __restrict__ Rp,
                  __half* __restrict__ y, int M, int64_t N, int64_t K, int prefetch_steps,
                  int prefetch_ctas, int trace_slot) {
    constexpr float kScale = (ENC == kEncE4M3 && !FULL) ? 0.00390625f : 1.0f;  // 2^-8, exact
    __shared__ float red[kWarps][kRowsPerBlock][NT * 8 + 1];
    sm100::grid_launch_dependents();
    DPS_DSTAMP(0);
    // A CTA that becomes resident while the preceding kernel drains has no activations yet (they are
    // that kernel's output), but its weights are model state: the first batch of weight loads is
    // issued BEFORE the dependency wait (below), and the first wave of CTAs asks L2 for the stretch
    // of its rows behind that batch, so that the DRAM pipe keeps working through the other
    // kernel's tail.  Thread i takes row i / 16 and every 16th 128-byte line of it.
    if (prefetch_steps > 0 && (int)blockIdx.x < prefetch_ctas) {
        const int64_t prow = (int64_t)blockIdx.x * (HALF ? 8 : kRowsPerBlock) + (threadIdx.x >> 4);
        if (prow < N && (!HALF || (threadIdx.x >> 4) < 8)) {
            const int64_t first = (int64_t)U * kRoundK;   // bytes of a row the first batch loads itself
            const int64_t pbase = prow * K + first + (threadIdx.x & 15) * 128;
            for (int j = 0; j < prefetch_steps; ++j) {
                const int64_t off = first + (int64_t)j * 2048 + (threadIdx.x & 15) * 128;
                if (off < K) {
                    sm100::prefetch_l2(P + pbase + (int64_t)j * 2048);
                    if (FULL) sm100::prefetch_l2(Rp + pbase + (int64_t)j * 2048);
                }
            }
        }
    }
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int g = lane >> 2, t = lane & 3;
    constexpr int kRows = HALF ? 8 : kRowsPerBlock;
    const int full_rounds = (int)(K / kRoundK);           // rounds in which every lane is inside K
    const bool has_tail = (K % kRoundK) != 0;
    const int kl = warp * 64 + t * 16;                    // this lane's byte offset inside a round

    // activation rows this lane feeds as B fragments (token 8 * n + g of every token group);
    // lanes without a token read row 0 and have their product discarded at the store
    const __half* xrow[NT];
#pragma unroll
    for (int n = 0; n < NT; ++n) xrow[n] = x + (int64_t)((n * 8 + g < M) ? n * 8 + g : 0) * K + kl;

    {   // one row block per CTA: the hardware block scheduler balances the SMs
        const int64_t rb = blockIdx.x;
        // rows past N are clamped for the loads and dropped at the store
        const int64_t row_lo = rb * kRows + g, row_hi = row_lo + 8;
        const uint8_t* p_lo = P + (row_lo < N ? row_lo : N - 1) * K + kl;
        const uint8_t* p_hi = P + (row_hi < N ? row_hi : N - 1) * K + kl;
        const uint8_t* r_lo = FULL ? Rp + (row_lo < N ? row_lo : N - 1) * K + kl : nullptr;
        const uint8_t* r_hi = FULL ? Rp + (row_hi < N ? row_hi : N - 1) * K + kl : nullptr;
        float acc[NT][4];
#pragma unroll
        for (int n = 0; n < NT; ++n)
#pragma unroll
            for (int c = 0; c < 4; ++c) acc[n][c] = 0.f;

        auto load_x = [&](uint4 (&xb)[NT][2], int koff, bool in) {
#pragma unroll
            for (int n = 0; n < NT; ++n) {
                xb[n][0] = xb[n][1] = make_uint4(0, 0, 0, 0);
                if (in) {
                    xb[n][0] = *reinterpret_cast<const uint4*>(xrow[n] + koff);
                    xb[n][1] = *reinterpret_cast<const uint4*>(xrow[n] + koff + 8);
                }
            }
        };
        auto multiply = [&](const uint4& wp_lo, const uint4& wp_hi, const uint4& wr_lo, const uint4& wr_hi,
                            const uint4 (&xb)[NT][2]) {
            uint32_t a_lo[8], a_hi[8];
            to_half_pairs<ENC, FULL>(wp_lo, wr_lo, a_lo);
            if (HALF) {
#pragma unroll
                for (int i = 0; i < 8; ++i) a_hi[i] = 0u;
            } else {
                to_half_pairs<ENC, FULL>(wp_hi, wr_hi, a_hi);
            }
#pragma unroll
            for (int n = 0; n < NT; ++n) {
                const uint4 b0 = xb[n][0], b1 = xb[n][1];
                const uint32_t bb[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
                // MMA j takes bytes 4j..4j+3 of the lane's 16: K slots (2t, 2t+1) <- pair 2j and
                // K slots (2t+8, 2t+9) <- pair 2j+1, for the weights and the activations alike.
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    mma_16816(acc[n], a_lo[2 * j], a_hi[2 * j], a_lo[2 * j + 1], a_hi[2 * j + 1], bb[2 * j],
                              bb[2 * j + 1]);
            }
        };

        int r0 = 0;
        for (; r0 + U <= full_rounds; r0 += U) {          // U rounds in flight, immediate offsets
            const int base = r0 * kRoundK;
            uint4 wp_lo[U], wp_hi[U], wr_lo[U], wr_hi[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                wp_hi[u] = wr_lo[u] = wr_hi[u] = make_uint4(0, 0, 0, 0);
                wp_lo[u] = ldg_stream(p_lo + base + u * kRoundK);
                if (!HALF) wp_hi[u] = ldg_stream(p_hi + base + u * kRoundK);
                if (FULL) {
                    wr_lo[u] = ldg_stream(r_lo + base + u * kRoundK);
                    if (!HALF) wr_hi[u] = ldg_stream(r_hi + base + u * kRoundK);
                }
            }
            // Everything but the planes may come from the preceding kernel: wait for it here, with the
            // first batch of weight loads already in flight.
            if (r0 == 0) {
                DPS_DSTAMP(1);
                sm100::grid_dependency_wait();
                DPS_DSTAMP(2);
            }
            // the activation fragments of the batch are fetched together with the weights, so that
            // their (L1 / L2) latency hides behind the DRAM latency of the weight loads
            uint4 xb[U][NT][2];
#pragma unroll
            for (int u = 0; u < U; ++u) load_x(xb[u], base + u * kRoundK, true);
#pragma unroll
            for (int u = 0; u < U; ++u) multiply(wp_lo[u], wp_hi[u], wr_lo[u], wr_hi[u], xb[u]);
        }
        const int total_rounds = full_rounds + (has_tail ? 1 : 0);
        // Leftover rounds and the ragged end of K: predicated batches (of at most 128 bytes per lane, which
        // keeps the predicated copy of the loop body free of register spills), never one round at
        // a time -- a lone round costs a full DRAM latency.
        constexpr int UT = FULL ? 2 : (U > 4 ? 4 : U);
        if (r0 == 0) sm100::grid_dependency_wait();   // K shorter than one full batch: nothing was loaded ahead
        for (; r0 < total_rounds; r0 += UT) {
            uint4 wp_lo[UT], wp_hi[UT], wr_lo[UT], wr_hi[UT];
            uint4 xb[UT][NT][2];
#pragma unroll
            for (int u = 0; u < UT; ++u) {
                const int base = (r0 + u) * kRoundK;
                const bool in = r0 + u < total_rounds && (int64_t)base + kl < K;
                wp_lo[u] = wp_hi[u] = wr_lo[u] = wr_hi[u] = make_uint4(0, 0, 0, 0);
                if (in) {
                    wp_lo[u] = ldg_stream(p_lo + base);
                    if (!HALF) wp_hi[u] = ldg_stream(p_hi + base);
                    if (FULL) {
                        wr_lo[u] = ldg_stream(r_lo + base);
                        if (!HALF) wr_hi[u] = ldg_stream(r_hi + base);
                    }
                }
                load_x(xb[u], base, in);
            }
#pragma unroll
            for (int u = 0; u < UT; ++u) {
                // warp-uniform skip (the MMA needs the whole warp); lanes past K multiply zeros
                const bool warp_in = r0 + u < total_rounds && (int64_t)(r0 + u) * kRoundK + warp * 64 < K;
                if (warp_in) multiply(wp_lo[u], wp_hi[u], wr_lo[u], wr_hi[u], xb[u]);
            }
        }
        // accumulator fragment: c0,c1 = (row g, tokens 2t, 2t+1), c2,c3 = (row g+8, same tokens)
#ifdef DPS_TRACE
        asm volatile("" ::"f"(acc[0][0] + acc[0][3]));
        DPS_DSTAMP(3);
#endif
#pragma unroll
        for (int n = 0; n < NT; ++n) {
            red[warp][g][n * 8 + 2 * t] = acc[n][0];
            red[warp][g][n * 8 + 2 * t + 1] = acc[n][1];
            if (!HALF) {
                red[warp][g + 8][n * 8 + 2 * t] = acc[n][2];
                red[warp][g + 8][n * 8 + 2 * t + 1] = acc[n][3];
            }
        }
        __syncthreads();
        for (int o = threadIdx.x; o < kRows * NT * 8; o += kThreads) {
            const int tok = o / kRows, row = o % kRows;
            const int64_t n_out = rb * kRows + row;
            if (tok < M && n_out < N) {
                float s = 0.f;
#pragma unroll
                for (int w = 0; w < kWarps; ++w) s += red[w][row][tok];
                y[(int64_t)tok * N + n_out] = __float2half_rn(s * kScale);
            }
        }
        __syncthreads();
        DPS_DSTAMP(4);
    }
}

template <int ENC, bool FULL, int NT, int U, bool HALF>
cudaError_t launch_one(const __half* x, const uint8_t* p, const uint8_t* r, __half* y, int M, int64_t N, int64_t K,
                       cudaStream_t stream) {
    constexpr int kRows = HALF ? 8 : kRowsPerBlock;
    const int64_t grid = (N + kRows - 1) / kRows;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid, 1, 1);
    cfg.blockDim = dim3(kThreads, 1, 1);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    // DPS_STREAM_PREFETCH=<steps> overrides how many 2 KB column steps of its row block a CTA asks
    // L2 for before it waits for the preceding kernel (0 = none), DPS_STREAM_PREFETCH_CTAS how many
    // CTAs of the grid do so.  Measured on Llama-7B shapes, every launch timed in a loop of its own: one step
    // by the first wave of CTAs gains 1-10 %; whole row blocks, or every CTA of a grid of several waves, lose.
    // Inside a decoder's chain of launches (graphs of 128 launches, the four Llama-7B linears in turn) the
    // picture differs by mode: fast mode keeps 2 % of that gain at 8 tokens, full mode LOSES 4-6 % to it (1 and
    // 8 tokens: 0.85 / 0.83 of the copy bandwidth with the prefetch, 0.90 / 0.87 without -- the requests compete
    // with the tail of the launch in front, which in full mode streams twice as long).  So: fast mode only.
    static const int prefetch_forced = [] {
        const char* e = getenv("DPS_STREAM_PREFETCH");
        return e ? atoi(e) : -1;
    }();
    const int prefetch_steps = prefetch_forced >= 0 ? prefetch_forced : (FULL ? 0 : 1);
    static const int prefetch_ctas = [] {
        const char* e = getenv("DPS_STREAM_PREFETCH_CTAS");
        return e ? atoi(e) : 2 * sm_count();
    }();
    int trace_slot = 0;
#ifdef DPS_TRACE
    static int trace_launches = 0;
    trace_slot = trace_launches++;
#endif
    cudaError_t e = cudaLaunchKernelEx(&cfg, decode_mma_kernel<ENC, FULL, NT, U, HALF>, x, p, r, y, M, N, K,
                                       prefetch_steps, prefetch_ctas, trace_slot);
    count_launch();
    return e;
}

template <int ENC, bool FULL>
cudaError_t launch_enc(const __half* x, const uint8_t* p, const uint8_t* r, __half* y, int M, int64_t N, int64_t K,
                       cudaStream_t stream) {
    // Rounds in flight per lane: 256 bytes (fast mode: 8 rounds of one plane; full mode: 4 rounds of
    // two), two CTAs per SM.  Half as much with three CTAs per SM in full mode was the default until the
    // first batch of weight loads moved in front of the dependency wait; since then the deeper
    // batches measure 2-26 % faster on every Llama-7B and hidden-8192 shape but one (QKV, full mode,
    // 8 tokens: -3 %).  DPS_STREAM_U2=0 selects the shallower batches (tuning knob).
    // Half-height blocks were measured slower for every Llama-7B shape (the kernel is bound by
    // instruction issue, and they double the MMA and activation-load instructions per weight), so
    // they stay off.
    static const int u_forced = [] {
        const char* e = getenv("DPS_STREAM_U2");
        return e ? atoi(e) : -1;
    }();
    constexpr int U = FULL ? 2 : 4;
    const bool wide_batches = u_forced >= 0 ? u_forced != 0 : true;
    if (wide_batches) {
        if (M <= 8) return launch_one<ENC, FULL, 1, 2 * U, false>(x, p, r, y, M, N, K, stream);
        if (M <= 16) return launch_one<ENC, FULL, 2, 2 * U, false>(x, p, r, y, M, N, K, stream);
    }
    if (M <= 8) return launch_one<ENC, FULL, 1, U, false>(x, p, r, y, M, N, K, stream);
    return launch_one<ENC, FULL, 2, U, false>(x, p, r, y, M, N, K, stream);   // (callers never pass more than 16 tokens)
}

}  // namespace

cudaError_t launch_decode_mma(int mode, int enc, const void* x, const uint8_t* p, const uint8_t* r, void* y,
                              int64_t M, int64_t N, int64_t K, cudaStream_t stream) {
    const __half* xh = static_cast<const __half*>(x);
    __half* yh = static_cast<__half*>(y);
    const bool full = mode == DPS_MODE_FULL;
    if (!full) enc = base_enc(enc);   // fast mode: the persistent byte of a rounded nest is an FP8 value like any other
    if (enc == kEncE4M3R) return launch_enc<kEncE4M3R, true>(xh, p, r, yh, (int)M, N, K, stream);
    if (enc == kEncE5M2R) return launch_enc<kEncE5M2R, true>(xh, p, r, yh, (int)M, N, K, stream);
    if (enc == kEncE4M3)
        return full ? launch_enc<kEncE4M3, true>(xh, p, r, yh, (int)M, N, K, stream)
                    : launch_enc<kEncE4M3, false>(xh, p, r, yh, (int)M, N, K, stream);
    return full ? launch_enc<kEncE5M2, true>(xh, p, r, yh, (int)M, N, K, stream)
                : launch_enc<kEncE5M2, false>(xh, p, r, yh, (int)M, N, K, stream);
}

#ifdef DPS_TRACE
extern "C" __attribute__((visibility("default"))) int dps_debug_decode_times(unsigned long long* out) {
    return (int)cudaMemcpyFromSymbol(out, g_decode_times, sizeof(g_decode_times));
}
#endif

}  // namespace dps
