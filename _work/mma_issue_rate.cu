// Microbenchmark: cycles per tcgen05.mma (M=128, N=16, A in tensor memory) for different ways of writing the
// issue loop: a lone diverged lane versus the elected lane of a converged warp.
// Build: python -m paper_2609_34380_b200.build --microbench ; run: paper_2609_34380_b200/microbench/mma_issue_rate
#include <cuda.h>
#include <cuda_runtime.h>
#include <cstdio>
#include <cstdint>
#include "../csrc/sm100.cuh"
using namespace dps::sm100;

// accumulate always: no setp needed
__device__ __forceinline__ void umma_ts_acc(uint32_t d, uint32_t a, uint64_t b, uint32_t idesc) {
    asm volatile("{\n\t.reg .pred p;\n\tsetp.eq.u32 p, 1, 1;\n\t"
                 "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}" ::"r"(d), "r"(a), "l"(b), "r"(idesc) : "memory");
}

template <int VARIANT>
__global__ void __launch_bounds__(128, 1) rate_kernel(int iters, int per_commit, long long* out) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bar;
    __shared__ uint32_t slot;
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    if (threadIdx.x == 0) { mbar_init(smem_u32(&bar), 1); fence_barrier_init(); }
    if (threadIdx.x < 32) tmem_alloc(smem_u32(&slot), 256);
    tc_fence_before_sync(); __syncthreads(); tc_fence_after_sync();
    const uint32_t tm = slot;
    const uint32_t idesc = umma_idesc_f16(128, 16);
    const uint64_t bdesc = umma_desc_k_sw128(base);
    if (VARIANT == 0) {          // single diverged lane, current wrapper
        if (threadIdx.x == 0) {
            long long t0 = clock64(); uint32_t ph = 0;
            for (int i = 0; i < iters; ++i) {
                for (int j = 0; j < per_commit; ++j) umma_f16_ts(tm, tm + 128 + (j & 7) * 8, bdesc + (uint64_t)((j & 3) * 2), idesc, 1u);
                umma_commit(smem_u32(&bar));
                if (!mbar_wait(smem_u32(&bar), ph)) break; ph ^= 1;
            }
            out[blockIdx.x] = clock64() - t0;
        }
    } else if (VARIANT == 1) {   // single lane, no disable mask / constant predicate
        if (threadIdx.x == 0) {
            long long t0 = clock64(); uint32_t ph = 0;
            for (int i = 0; i < iters; ++i) {
                for (int j = 0; j < per_commit; ++j) umma_ts_acc(tm, tm + 128 + (j & 7) * 8, bdesc + (uint64_t)((j & 3) * 2), idesc);
                umma_commit(smem_u32(&bar));
                if (!mbar_wait(smem_u32(&bar), ph)) break; ph ^= 1;
            }
            out[blockIdx.x] = clock64() - t0;
        }
    } else if (VARIANT == 2) {   // converged warp, elected lane issues
        if (threadIdx.x < 32) {
            long long t0 = clock64(); uint32_t ph = 0;
            for (int i = 0; i < iters; ++i) {
                if (elect_one()) {
#pragma unroll 8
                    for (int j = 0; j < per_commit; ++j) umma_ts_acc(tm, tm + 128 + (j & 7) * 8, bdesc + (uint64_t)((j & 3) * 2), idesc);
                    umma_commit(smem_u32(&bar));
                }
                __syncwarp();
                if (!mbar_wait(smem_u32(&bar), ph)) break; ph ^= 1;
            }
            if (threadIdx.x == 0) out[blockIdx.x] = clock64() - t0;
        }
    } else if (VARIANT == 3) {   // single lane, fully unrolled by 8 with immediate offsets
        if (threadIdx.x == 0) {
            long long t0 = clock64(); uint32_t ph = 0;
            for (int i = 0; i < iters; ++i) {
                for (int j0 = 0; j0 < per_commit; j0 += 8) {
#pragma unroll
                    for (int j = 0; j < 8; ++j) umma_ts_acc(tm, tm + 128 + j * 8, bdesc + (uint64_t)((j & 3) * 2), idesc);
                }
                umma_commit(smem_u32(&bar));
                if (!mbar_wait(smem_u32(&bar), ph)) break; ph ^= 1;
            }
            out[blockIdx.x] = clock64() - t0;
        }
    }
    tc_fence_before_sync(); __syncthreads();
    if (threadIdx.x < 32) { tc_fence_after_sync(); tmem_dealloc(tm, 256); }
}

template <int V> void run(const char* name, int per_commit) {
    long long* out; cudaMalloc(&out, 8 * 1024);
    cudaFuncSetAttribute(rate_kernel<V>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    const int iters = 100, ctas = 148;
    rate_kernel<V><<<ctas, 128, 100 * 1024>>>(iters, per_commit, out);
    cudaDeviceSynchronize();
    long long h[1024]; cudaMemcpy(h, out, 8 * ctas, cudaMemcpyDeviceToHost);
    double avg = 0; for (int i = 0; i < ctas; ++i) avg += h[i]; avg /= ctas;
    printf("%-44s mma/commit=%3d: %.1f cycles per MMA  %s\n", name, per_commit, avg / (iters * per_commit), cudaGetErrorString(cudaGetLastError()));
    cudaFree(out);
}
int main() {
    for (int pc : {16, 128}) {
        run<0>("single lane, masks + setp", pc);
        run<1>("single lane, no mask, const pred", pc);
        run<2>("converged warp + elect", pc);
        run<3>("single lane unrolled x8", pc);
    }
}
