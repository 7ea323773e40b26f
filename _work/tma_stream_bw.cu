// Microbenchmark: bandwidth of streaming a row-major [N][K] byte matrix through TMA tile loads, for
// different box shapes (row width, swizzle, K-adjacent boxes issued together, 3-D boxes).  The result
// picked the stage shape of the tensor-core linear kernel.
// Build: python -m paper_2609_34380_b200.build --microbench ; run: paper_2609_34380_b200/microbench/tma_stream_bw
#include <cuda.h>
#include <cuda_runtime.h>
#include <cstdio>
#include <cstdlib>
#include <cstdint>
#include <vector>
#include "../csrc/sm100.cuh"
using namespace dps::sm100;

struct P { int num_kb; int stages; int stage_bytes; int box_w; int box_h; int kb_per_cta; int rows_per_tile; int boxes_per_stage; int kdir; int three_d; int chunks; };

__global__ void __launch_bounds__(64, 1) stream_kernel(const __grid_constant__ CUtensorMap map, P p, unsigned long long* sink) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t full[16], empty[16];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    if (threadIdx.x == 0) { for (int s = 0; s < p.stages; ++s) { mbar_init(smem_u32(&full[s]), 1); mbar_init(smem_u32(&empty[s]), 1);} fence_barrier_init(); }
    __syncthreads();
    const int row0 = blockIdx.x * p.rows_per_tile;
    const int kb0 = blockIdx.y * p.kb_per_cta;
    int nkb = p.num_kb - kb0; if (nkb > p.kb_per_cta) nkb = p.kb_per_cta;
    if (threadIdx.x == 0) {
        for (int i = 0; i < nkb; ++i) {
            int s = i % p.stages; uint32_t ph = (i / p.stages) & 1;
            if (!mbar_wait(smem_u32(&empty[s]), ph ^ 1)) break;
            mbar_arrive_expect_tx(smem_u32(&full[s]), p.stage_bytes);
            for (int b = 0; b < p.boxes_per_stage; ++b) {
                uint32_t dst = base + s * p.stage_bytes + b * (p.stage_bytes / p.boxes_per_stage);
                if (p.three_d) tma_load_3d(dst, &map, smem_u32(&full[s]), 0, (kb0 + i) * p.chunks, row0);
                else if (p.kdir) tma_load_2d(dst, &map, smem_u32(&full[s]), ((kb0 + i) * p.boxes_per_stage + b) * p.box_w, row0);
                else tma_load_2d(dst, &map, smem_u32(&full[s]), (kb0 + i) * p.box_w, row0 + b * p.box_h);
            }
        }
    } else if (threadIdx.x == 32) {
        unsigned long long acc = 0;
        for (int i = 0; i < nkb; ++i) {
            int s = i % p.stages; uint32_t ph = (i / p.stages) & 1;
            if (!mbar_wait(smem_u32(&full[s]), ph)) break;
            acc += *reinterpret_cast<volatile unsigned*>(smem_raw + (base - smem_u32(smem_raw)) + s * p.stage_bytes);
            mbar_arrive(smem_u32(&empty[s]));
        }
        if (acc == 0x123456789ull) *sink = acc;
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

int main(int argc, char** argv) {
    const int64_t N = 49152, K = 4096;
    uint8_t* buf; cudaMalloc(&buf, N * K); cudaMemset(buf, 1, N * K);
    unsigned long long* sink; cudaMalloc(&sink, 8);
    void* fp; cudaDriverEntryPointQueryResult q;
    cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fp, cudaEnableDefault, &q);
    EncodeTiledFn enc = (EncodeTiledFn)fp;
    cudaFuncSetAttribute(stream_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 224 * 1024);
    struct Cfg { int w, h, boxes, swz, elem; int split; int smem_kb; const char* name; int kdir; int chunks; };
    // w in bytes; elem = bytes per element of the tensor-map type
    std::vector<Cfg> cfgs = {
        {64, 128, 1, 2, 1, 1, 100, "64x128 sw64 split1 2cta"},
        {128, 128, 1, 3, 1, 1, 100, "128x128 sw128 split1 2cta"},
        {128, 128, 1, 3, 1, 4, 100, "128x128 sw128 split4 2cta"},
        {128, 128, 1, 3, 1, 1, 200, "128x128 sw128 split1 1cta"},
        {128, 128, 1, 3, 1, 1, 50, "128x128 sw128 split1 4cta"},
        {128, 128, 1, 3, 1, 4, 50, "128x128 sw128 split4 4cta"},
        {256, 64, 2, 0, 1, 1, 100, "256x(2x64) none split1 2cta"},
        {256, 64, 2, 0, 1, 4, 100, "256x(2x64) none split4 2cta"},
        {256, 128, 1, 0, 1, 1, 100, "256x128 none split1 2cta"},
        {256, 128, 1, 0, 1, 4, 100, "256x128 none split4 2cta"},
        {512, 32, 4, 0, 4, 1, 100, "512x(4x32) u32 none split1 2cta"},
        {1024, 16, 8, 0, 4, 1, 100, "1024x(8x16) u32 none split1 2cta"},
        {1024, 16, 8, 0, 4, 2, 100, "1024x(8x16) u32 none split2 2cta"},
        {1024, 32, 4, 0, 4, 1, 200, "1024x(4x32) u32 none split1 1cta"},
        {128, 128, 2, 3, 1, 1, 100, "2x(128x128) sw128 kdir 2cta", 1, 0},
        {128, 128, 4, 3, 1, 1, 200, "4x(128x128) sw128 kdir 1cta", 1, 0},
        {128, 128, 1, 3, 1, 1, 100, "3D {128,2,128} sw128 2cta", 0, 2},
        {128, 128, 1, 3, 1, 1, 200, "3D {128,4,128} sw128 1cta", 0, 4},
        {128, 64, 1, 3, 1, 1, 100, "3D {128,4,64} sw128 2cta", 0, 4},
        {4096, 8, 16, 0, 16, 1, 100, "NA", },
    };
    for (auto& c : cfgs) {
        if (c.elem == 16) continue;
        CUtensorMap map;
        cuuint64_t dims[2] = {(cuuint64_t)(K / c.elem), (cuuint64_t)N};
        cuuint64_t strides[1] = {(cuuint64_t)K};
        cuuint32_t box[2] = {(cuuint32_t)(c.w / c.elem), (cuuint32_t)c.h};
        cuuint32_t es[2] = {1, 1};
        CUtensorMapDataType dt = c.elem == 1 ? CU_TENSOR_MAP_DATA_TYPE_UINT8 : CU_TENSOR_MAP_DATA_TYPE_UINT32;
        CUtensorMapSwizzle sw = c.swz == 3 ? CU_TENSOR_MAP_SWIZZLE_128B : c.swz == 2 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_NONE;
        CUresult r;
        if (c.chunks) {
            cuuint64_t d3[3] = {128, (cuuint64_t)(K / 128), (cuuint64_t)N};
            cuuint64_t s3[2] = {128, (cuuint64_t)K};
            cuuint32_t b3[3] = {128, (cuuint32_t)c.chunks, (cuuint32_t)c.h};
            cuuint32_t e3[3] = {1, 1, 1};
            r = enc(&map, dt, 3, buf, d3, s3, b3, e3, CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        } else
        r = enc(&map, dt, 2, buf, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) { printf("%s: encode failed %d\n", c.name, (int)r); continue; }
        P p; p.box_w = c.w / c.elem; p.box_h = c.h; p.boxes_per_stage = c.boxes; p.stage_bytes = c.w * c.h * c.boxes;
        p.kdir = c.kdir; p.three_d = c.chunks > 0; p.chunks = c.chunks;
        if (c.chunks) p.stage_bytes = 128 * c.chunks * c.h;
        p.rows_per_tile = c.kdir || c.chunks ? c.h : c.h * c.boxes;
        p.num_kb = c.chunks ? K / (128 * c.chunks) : c.kdir ? K / (c.w * c.boxes) : K / c.w; p.kb_per_cta = (p.num_kb + c.split - 1) / c.split;
        p.stages = (c.smem_kb * 1024) / p.stage_bytes; if (p.stages > 16) p.stages = 16; if (p.stages < 1) p.stages = 1;
        size_t smem = (size_t)p.stages * p.stage_bytes + 1024;
        dim3 grid(N / p.rows_per_tile, c.split);
        cudaEvent_t e0, e1; cudaEventCreate(&e0); cudaEventCreate(&e1);
        for (int it = 0; it < 2; ++it) stream_kernel<<<grid, 64, smem>>>(map, p, sink);
        cudaEventRecord(e0);
        for (int it = 0; it < 5; ++it) stream_kernel<<<grid, 64, smem>>>(map, p, sink);
        cudaEventRecord(e1); cudaEventSynchronize(e1);
        float ms; cudaEventElapsedTime(&ms, e0, e1);
        cudaError_t err = cudaGetLastError();
        printf("%-36s stages=%2d stage=%6dB grid=%5dx%d  %.1f us  %.0f GB/s  %s\n", c.name, p.stages, p.stage_bytes, grid.x, grid.y, ms * 200, N * K / (ms / 5 * 1e-3) / 1e9, err == cudaSuccess ? "" : cudaGetErrorString(err));
    }
    return 0;
}
