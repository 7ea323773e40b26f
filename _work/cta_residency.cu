// Microbenchmark: how many CTAs of a 320-thread kernel become co-resident, depending on dynamic shared
// memory, cluster size, the shared-memory carve-out preference and tensor-memory allocation.
// Build: python -m paper_2609_34380_b200.build --microbench ; run: paper_2609_34380_b200/microbench/cta_residency
#include <cuda_runtime.h>
#include <cstdio>
#include <cstdint>
#include <vector>
#include <algorithm>
#include "../csrc/sm100.cuh"
using namespace dps::sm100;
__global__ void __launch_bounds__(320, 1) k(unsigned long long* t, unsigned* sm, int use_tmem, int tmem_cols) {
    extern __shared__ uint8_t s[];
    __shared__ uint32_t slot;
    const int cta = blockIdx.x + gridDim.x * blockIdx.z;
    if (threadIdx.x == 0) { t[cta] = global_timer_ns(); unsigned id; asm volatile("mov.u32 %0, %%smid;" : "=r"(id)); sm[cta] = id; s[0] = 1; }
    if (use_tmem && threadIdx.x < 32) tmem_alloc(smem_u32(&slot), tmem_cols);
    __syncthreads();
    unsigned long long t0 = global_timer_ns();
    while (global_timer_ns() - t0 < 30000) { }
    __syncthreads();
    if (use_tmem && threadIdx.x < 32) tmem_dealloc(slot, tmem_cols);
}
void run(const char* name, int smem_kb, int cluster, int carve, int use_tmem, int cols) {
    const int ctas = 296 / cluster * cluster;
    unsigned long long* t; unsigned* sm; cudaMalloc(&t, 8 * 1024); cudaMalloc(&sm, 4 * 1024);
    cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, 224 * 1024);
    cudaFuncSetAttribute(k, cudaFuncAttributePreferredSharedMemoryCarveout, carve ? (int)cudaSharedmemCarveoutMaxShared : (int)cudaSharedmemCarveoutDefault);
    cudaLaunchConfig_t cfg = {}; cfg.gridDim = dim3(ctas / cluster, 1, cluster); cfg.blockDim = dim3(320); cfg.dynamicSmemBytes = smem_kb * 1024;
    cudaLaunchAttribute a[1]; a[0].id = cudaLaunchAttributeClusterDimension; a[0].val.clusterDim.x = 1; a[0].val.clusterDim.y = 1; a[0].val.clusterDim.z = cluster;
    cfg.attrs = a; cfg.numAttrs = cluster > 0 ? 1 : 0;
    for (int rep = 0; rep < 2; ++rep) { cudaLaunchKernelEx(&cfg, k, t, sm, use_tmem, cols); cudaDeviceSynchronize(); }
    std::vector<unsigned long long> h(ctas); std::vector<unsigned> hs(ctas);
    cudaMemcpy(h.data(), t, 8 * ctas, cudaMemcpyDeviceToHost); cudaMemcpy(hs.data(), sm, 4 * ctas, cudaMemcpyDeviceToHost);
    unsigned long long t0 = *std::min_element(h.begin(), h.end());
    int first = 0; int per_sm[256] = {0}; int mx = 0;
    for (int i = 0; i < ctas; ++i) if (h[i] - t0 < 10000) { ++first; mx = std::max(mx, ++per_sm[hs[i]]); }
    printf("%-50s first-wave CTAs=%3d of %d, max per SM=%d  %s\n", name, first, ctas, mx, cudaGetErrorString(cudaGetLastError()));
}
int main() {
    run("smem 82KB no-cluster default-carve", 82, 1, 0, 0, 0);
    run("smem 82KB no-cluster max-carve", 82, 1, 1, 0, 0);
    run("smem 82KB cluster3 max-carve", 82, 3, 1, 0, 0);
    run("smem 82KB cluster8 max-carve", 82, 8, 1, 0, 0);
    run("smem 82KB no-cluster max-carve tmem256", 82, 1, 1, 1, 256);
    run("smem 82KB cluster3 max-carve tmem256", 82, 3, 1, 1, 256);
    run("smem 104KB cluster3 max-carve tmem256", 104, 3, 1, 1, 256);
    run("smem 40KB cluster3 max-carve tmem128", 40, 3, 1, 1, 128);
    run("smem 40KB cluster3 default-carve tmem128", 40, 3, 0, 1, 128);
}
