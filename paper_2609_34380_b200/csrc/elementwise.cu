// Load-time kernels: tensor statistics for the encoding choice, nested split, reconstruction.
// Paper: "Mapper: Semi-Unified Memory Abstraction" ("Persistent Region" paragraph) for the
// split; "Scheduler: Dual-Precision Execution" for the reconstruction and the per-layer
// encoding choice.  All three are pure streams: 16 elements per thread per step, 128-bit
// loads and stores, grid sized to the SM count.
#include "bits.cuh"
#include "dps_internal.h"

namespace dps {

namespace {

constexpr int kThreads = 256;

__device__ __forceinline__ uint4 ldg_stream(const void* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

__device__ __forceinline__ uint32_t max_mag2(uint32_t a, uint32_t m) {
    // per-half max of (word & 0x7FFF)
    a &= 0x7FFF7FFFu;
    return __vmaxu2(a, m);
}

__global__ void __launch_bounds__(kThreads) magnitude_stat_kernel(const uint4* __restrict__ w, int64_t n8,
                                                                   unsigned* stat) {
    uint32_t m = 0;
    for (int64_t i = blockIdx.x * (int64_t)kThreads + threadIdx.x; i < n8; i += (int64_t)gridDim.x * kThreads) {
        uint4 v = ldg_stream(w + i);
        m = max_mag2(v.x, m);
        m = max_mag2(v.y, m);
        m = max_mag2(v.z, m);
        m = max_mag2(v.w, m);
    }
    unsigned best = max(m & 0xFFFFu, m >> 16);
    for (int o = 16; o > 0; o >>= 1) best = max(best, __shfl_xor_sync(0xFFFFFFFFu, best, o));
    if ((threadIdx.x & 31) == 0 && best) atomicMax(stat, best);
}

template <int ENC>
__global__ void __launch_bounds__(kThreads) split_kernel(const uint4* __restrict__ w, uint4* __restrict__ p,
                                                         uint4* __restrict__ r, int64_t n16) {
    for (int64_t i = blockIdx.x * (int64_t)kThreads + threadIdx.x; i < n16; i += (int64_t)gridDim.x * kThreads) {
        uint4 a = ldg_stream(w + 2 * i);
        uint4 b = ldg_stream(w + 2 * i + 1);
        uint4 pp, rr;
        split4<ENC>(a.x, a.y, pp.x, rr.x);
        split4<ENC>(a.z, a.w, pp.y, rr.y);
        split4<ENC>(b.x, b.y, pp.z, rr.z);
        split4<ENC>(b.z, b.w, pp.w, rr.w);
        p[i] = pp;
        r[i] = rr;
    }
}

template <int ENC, bool FULL>
__global__ void __launch_bounds__(kThreads) reconstruct_kernel(const uint4* __restrict__ p,
                                                               const uint4* __restrict__ r, uint4* __restrict__ w,
                                                               int64_t n16) {
    for (int64_t i = blockIdx.x * (int64_t)kThreads + threadIdx.x; i < n16; i += (int64_t)gridDim.x * kThreads) {
        uint4 pp = ldg_stream(p + i);
        uint4 rr = make_uint4(0, 0, 0, 0);
        if (FULL) rr = ldg_stream(r + i);
        uint32_t h[8];
        join16<ENC, FULL>(pp, rr, h);
        w[2 * i] = make_uint4(h[0], h[1], h[2], h[3]);
        w[2 * i + 1] = make_uint4(h[4], h[5], h[6], h[7]);
    }
}

int stream_grid(int64_t items) {
    int64_t blocks = (items + kThreads - 1) / kThreads;
    int64_t cap = (int64_t)sm_count() * 8;
    return (int)(blocks < cap ? (blocks > 0 ? blocks : 1) : cap);
}

// Empty kernel launched (as an ordinary, fully ordered launch) after the planes have been written.
// A linear kernel that follows on the stream may start early and fetch planes before it waits for
// its predecessor; with this launch in between, that predecessor is the fence, and the fence did
// not start before the split kernel had finished and its writes were visible.
__global__ void plane_fence_kernel() {}

}  // namespace

cudaError_t launch_magnitude_stat(const uint16_t* w, int64_t n, unsigned* stat, cudaStream_t stream) {
    int64_t n8 = n / 8;
    magnitude_stat_kernel<<<stream_grid(n8), kThreads, 0, stream>>>(reinterpret_cast<const uint4*>(w), n8, stat);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_split(const uint16_t* w, uint8_t* p, uint8_t* r, int64_t n, int enc, cudaStream_t stream) {
    int64_t n16 = n / 16;
    int grid = stream_grid(n16);
    if (enc == kEncE4M3)
        split_kernel<kEncE4M3><<<grid, kThreads, 0, stream>>>(reinterpret_cast<const uint4*>(w),
                                                               reinterpret_cast<uint4*>(p),
                                                               reinterpret_cast<uint4*>(r), n16);
    else
        split_kernel<kEncE5M2><<<grid, kThreads, 0, stream>>>(reinterpret_cast<const uint4*>(w),
                                                               reinterpret_cast<uint4*>(p),
                                                               reinterpret_cast<uint4*>(r), n16);
    count_launch();
    plane_fence_kernel<<<1, 32, 0, stream>>>();
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_reconstruct(const uint8_t* p, const uint8_t* r, uint16_t* w, int64_t n, int enc,
                               cudaStream_t stream) {
    int64_t n16 = n / 16;
    int grid = stream_grid(n16);
    const uint4* pp = reinterpret_cast<const uint4*>(p);
    const uint4* rr = reinterpret_cast<const uint4*>(r);
    uint4* ww = reinterpret_cast<uint4*>(w);
    if (enc == kEncE4M3) {
        if (r) reconstruct_kernel<kEncE4M3, true><<<grid, kThreads, 0, stream>>>(pp, rr, ww, n16);
        else reconstruct_kernel<kEncE4M3, false><<<grid, kThreads, 0, stream>>>(pp, rr, ww, n16);
    } else {
        if (r) reconstruct_kernel<kEncE5M2, true><<<grid, kThreads, 0, stream>>>(pp, rr, ww, n16);
        else reconstruct_kernel<kEncE5M2, false><<<grid, kThreads, 0, stream>>>(pp, rr, ww, n16);
    }
    count_launch();
    return cudaGetLastError();
}

}  // namespace dps
