// Tensor-core path of the dense linear layer: tcgen05.mma with the reconstructed weights as the
// A operand in tensor memory and the activations as the B operand in shared memory.
//
// Paper: "Scheduler: Dual-Precision Execution" -- full mode combines the FP8 tensor with the
// residual tensor into the original FP16 values *during computation*; fast mode uses the FP8
// tensor alone.  Here that combination happens on the way from shared memory to tensor memory.
//
// Tile: 128 weight rows (UMMA M) x TN tokens (UMMA N), K walked in blocks of 64.  The problem
// is "swapped": D[row][token] = sum_k W[row][k] * x[token][k], so that even a handful of decode
// tokens fills the 128-lane datapath with weight rows and every weight byte is fetched once.
//
// Roles (6 warps):
//   warp 0     TMA producer: P tile (128 x 64 bytes), R tile (full mode), x tile (TN x 64 halves)
//              into a ring of shared-memory stages, completion counted on mbarriers.
//   warp 1     allocates tensor memory; one lane issues tcgen05.mma (A from TMEM, B from smem)
//              and commits stage-release barriers.
//   warps 2-5  "zip" warps: each owns 32 TMEM lanes = 32 weight rows.  Per K block a thread
//              reads its row's 64 plane bytes (swizzled, conflict-free), rebuilds 64 FP16 words
//              in registers with byte permutes and writes them to the A ring in TMEM with one
//              tcgen05.st.  After the K loop the same warps drain the accumulator
//              (tcgen05.ld), round to FP16 and store y.
// Shared memory never holds FP16 weights, so its bandwidth is spent on 1-2 bytes per weight
// instead of 5-6, and the tensor core reads only the small activation tile from it.
#include <cuda_fp16.h>

#include <cstdlib>

#include "bits.cuh"
#include "dps_internal.h"
#include "sm100.cuh"

namespace dps {

namespace {

using namespace sm100;

constexpr int kTileRows = 128;   // weight rows per CTA (UMMA M)
constexpr int kBlockK = 64;      // K elements per pipeline stage
constexpr int kAStages = 4;      // A ring in tensor memory (32 columns each)
constexpr int kZipGroups = 2;    // groups of 4 zip warps; group g takes K blocks g, g + G, ...
constexpr int kThreads = 64 + kZipGroups * 128;
constexpr int kPlaneStageBytes = kTileRows * kBlockK;  // 8 KB per plane per stage
constexpr int kMaxStages = 12;
constexpr int kMaxSplit = 8;     // portable cluster size
static_assert(kAStages % kZipGroups == 0, "each A stage must belong to one zip group");

__host__ __device__ constexpr int stage_bytes(bool full, int tn) {
    return kPlaneStageBytes * (full ? 2 : 1) + tn * kBlockK * 2;
}
__host__ __device__ constexpr int tmem_cols(int tn) {
    int need = tn + kAStages * 32;
    int c = 32;
    while (c < need) c <<= 1;
    return c;
}

struct UmmaParams {
    __half* y;
    int M, N, K;
    int num_stages;
    int split;       // K split = cluster size along z; partial tiles are summed through DSMEM
    int* status;
};

template <int ENC, bool FULL, int TN>
__global__ void __launch_bounds__(kThreads, 1)
umma_linear_kernel(const __grid_constant__ CUtensorMap map_p, const __grid_constant__ CUtensorMap map_r,
                   const __grid_constant__ CUtensorMap map_x, const UmmaParams prm) {
    constexpr int kStage = stage_bytes(FULL, TN);
    constexpr int kXOffset = kPlaneStageBytes * (FULL ? 2 : 1);
    constexpr uint32_t kCols = tmem_cols(TN);
    constexpr uint32_t kIdesc = umma_idesc_f16(kTileRows, TN);

    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bar_full[kMaxStages];
    __shared__ __align__(8) uint64_t bar_empty[kMaxStages];
    __shared__ __align__(8) uint64_t bar_a_full[kAStages];
    __shared__ __align__(8) uint64_t bar_a_empty[kAStages];
    __shared__ __align__(8) uint64_t bar_d_full;
    __shared__ uint32_t tmem_base_slot;

    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int num_stages = prm.num_stages;
    const int n0 = blockIdx.x * kTileRows;
    const int m0 = blockIdx.y * TN;
    const int total_kb = (prm.K + kBlockK - 1) / kBlockK;
    const int split = prm.split;
    const int rank = (split > 1) ? (int)cluster_ctarank() : 0;   // == blockIdx.z
    const int kb_begin = (int)((int64_t)total_kb * rank / split);
    const int kb_end = (int)((int64_t)total_kb * (rank + 1) / split);
    const int num_kb = kb_end - kb_begin;

    if (threadIdx.x == 0) {
        for (int s = 0; s < num_stages; ++s) {
            mbar_init(smem_u32(&bar_full[s]), 1);
            mbar_init(smem_u32(&bar_empty[s]), 5);  // 4 zip warps + 1 tcgen05.commit
        }
        for (int a = 0; a < kAStages; ++a) {
            mbar_init(smem_u32(&bar_a_full[a]), 4);
            mbar_init(smem_u32(&bar_a_empty[a]), 1);
        }
        mbar_init(smem_u32(&bar_d_full), 1);
        fence_barrier_init();
        prefetch_tensormap(&map_p);
        if (FULL) prefetch_tensormap(&map_r);
        prefetch_tensormap(&map_x);
    }
    if (warp == 1) tmem_alloc(smem_u32(&tmem_base_slot), kCols);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = tmem_base_slot;
    const uint32_t tmem_d = tmem_base;           // TN accumulator columns
    const uint32_t tmem_a = tmem_base + TN;      // kAStages x 32 columns of packed FP16 pairs

    // Partial tile for the split-K sum, token-major: red[token][row].  It overlays the stage ring,
    // which is idle once the accumulator is complete.
    float* red = reinterpret_cast<float*>(smem_raw + (smem_base - smem_u32(smem_raw)));

    bool ok = true;
    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (lane == 0) {
            for (int i = 0; i < num_kb && ok; ++i) {
                const int s = i % num_stages;
                const uint32_t ph = (uint32_t)(i / num_stages) & 1u;
                ok = mbar_wait(smem_u32(&bar_empty[s]), ph ^ 1u);
                if (!ok) break;
                const uint32_t full = smem_u32(&bar_full[s]);
                const uint32_t dst = smem_base + (uint32_t)s * kStage;
                const int k = (kb_begin + i) * kBlockK;
                mbar_arrive_expect_tx(full, (uint32_t)kStage);
                tma_load_2d(dst, &map_p, full, k, n0);
                if (FULL) tma_load_2d(dst + kPlaneStageBytes, &map_r, full, k, n0);
                tma_load_2d(dst + kXOffset, &map_x, full, k, m0);
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (lane == 0) {
            for (int i = 0; i < num_kb && ok; ++i) {
                const int s = i % num_stages, a = i % kAStages;
                ok = mbar_wait(smem_u32(&bar_full[s]), (uint32_t)(i / num_stages) & 1u);
                if (ok) ok = mbar_wait(smem_u32(&bar_a_full[a]), (uint32_t)(i / kAStages) & 1u);
                if (!ok) break;
                tc_fence_after_sync();
                const uint64_t bdesc = umma_desc_k_sw128(smem_base + (uint32_t)s * kStage + kXOffset);
#pragma unroll
                for (int j = 0; j < kBlockK / 16; ++j)
                    umma_f16_ts(tmem_d, tmem_a + (uint32_t)(a * 32 + j * 8), bdesc + (uint64_t)(j * 2), kIdesc,
                                (i > 0 || j > 0) ? 1u : 0u);
                umma_commit(smem_u32(&bar_empty[s]));
                umma_commit(smem_u32(&bar_a_empty[a]));
            }
            if (ok) umma_commit(smem_u32(&bar_d_full));
        }
    } else {
        // ---------------- zip warps: planes -> FP16 -> tensor memory; then epilogue ----------------
        const int group = (warp - 2) >> 2;
        const int q = warp & 3;                  // TMEM lane quarter this warp may touch
        const int row = q * 32 + lane;           // weight row inside the tile
        const uint32_t lane_base = (uint32_t)(q * 32) << 16;
        const uint32_t sw = (uint32_t)((row >> 1) & 3);  // 64-byte swizzle: chunk ^= (row / 2) % 4
        for (int i = group; i < num_kb && ok; i += kZipGroups) {
            const int s = i % num_stages, a = i % kAStages;
            ok = mbar_wait(smem_u32(&bar_full[s]), (uint32_t)(i / num_stages) & 1u);
            if (ok) ok = mbar_wait(smem_u32(&bar_a_empty[a]), ((uint32_t)(i / kAStages) & 1u) ^ 1u);
            ok = __all_sync(0xFFFFFFFFu, ok);
            if (!ok) break;
            tc_fence_after_sync();
            const uint32_t prow = smem_base + (uint32_t)s * kStage + (uint32_t)row * kBlockK;
            uint32_t h[32];
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const uint32_t off = ((uint32_t)c ^ sw) * 16u;
                uint4 pv, rv = make_uint4(0, 0, 0, 0);
                asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];"
                             : "=r"(pv.x), "=r"(pv.y), "=r"(pv.z), "=r"(pv.w)
                             : "r"(prow + off));
                if (FULL)
                    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];"
                                 : "=r"(rv.x), "=r"(rv.y), "=r"(rv.z), "=r"(rv.w)
                                 : "r"(prow + kPlaneStageBytes + off));
                uint32_t h8[8];
                join16<ENC, FULL>(pv, rv, h8);
#pragma unroll
                for (int j = 0; j < 8; ++j) h[c * 8 + j] = h8[j];
            }
            tmem_st_32x32b_x32(tmem_a + lane_base + (uint32_t)(a * 32), h);
            tmem_wait_st();
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(smem_u32(&bar_a_full[a]));
                mbar_arrive(smem_u32(&bar_empty[s]));
            }
        }
        // epilogue (first zip group): D[row][token] -> y[token][n0 + row], or -> red for split K
        if (group == 0) {
            if (ok) ok = mbar_wait(smem_u32(&bar_d_full), 0u);
            ok = __all_sync(0xFFFFFFFFu, ok);
            if (ok) {
                tc_fence_after_sync();
                const int n = n0 + row;
#pragma unroll
                for (int c0 = 0; c0 < TN; c0 += 16) {
                    uint32_t v[16];
                    tmem_ld_32x32b_x16(tmem_d + lane_base + (uint32_t)c0, v);
                    tmem_wait_ld();
                    if (split > 1) {
#pragma unroll
                        for (int j = 0; j < 16; ++j) red[(c0 + j) * kTileRows + row] = __uint_as_float(v[j]);
                    } else if (n < prm.N) {
#pragma unroll
                        for (int j = 0; j < 16; ++j) {
                            const int m = m0 + c0 + j;
                            if (m < prm.M) prm.y[(int64_t)m * prm.N + n] = __float2half_rn(__uint_as_float(v[j]));
                        }
                    }
                }
            }
        }
    }
    if (!ok) atomicExch(prm.status, (int)DPS_ERR_CUDA);

    if (split > 1) {
        // Split-K: every CTA of the cluster holds a partial tile in its shared memory.  CTA `rank`
        // sums tokens rank, rank + split, ... over all partials in rank order (fixed order, so the
        // result is deterministic) straight out of its peers' shared memory.
        __syncthreads();
        cluster_sync_all();
        const uint32_t red_addr = smem_base;
        for (int e = threadIdx.x; e < (TN / 1) * kTileRows; e += kThreads) {
            const int c = e / kTileRows, r = e % kTileRows;
            if ((c % split) != rank) continue;
            const int m = m0 + c, n = n0 + r;
            if (m >= prm.M || n >= prm.N) continue;
            float acc = 0.f;
            for (int j = 0; j < split; ++j)
                acc += ld_cluster_f32(map_to_cta(red_addr + (uint32_t)(c * kTileRows + r) * 4u, (uint32_t)j));
            prm.y[(int64_t)m * prm.N + n] = __float2half_rn(acc);
        }
        cluster_sync_all();
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, kCols);
    }
}

// ---- host side ---------------------------------------------------------------------------------

using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                   const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// Tuning / debugging knob: DPS_FORCE_SPLIT=<1..8> pins the K split.
int forced_split() {
    static const int v = [] {
        const char* e = getenv("DPS_FORCE_SPLIT");
        return e ? atoi(e) : 0;
    }();
    return v;
}

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            p = nullptr;
        return reinterpret_cast<EncodeTiledFn>(p);
    }();
    return fn;
}

// 2-D row-major tensor [rows][cols] of `elem_bytes`-sized elements, tiles of box_rows x box_cols.
bool make_map_2d(CUtensorMap* map, const void* base, CUtensorMapDataType dt, int elem_bytes, uint64_t rows,
                 uint64_t cols, uint32_t box_rows, uint32_t box_cols, CUtensorMapSwizzle swizzle) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {cols * (uint64_t)elem_bytes};
    const cuuint32_t box[2] = {box_cols, box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return fn(map, dt, 2, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle,
              CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// K split for a launch of `tiles` output tiles: the factor (<= 8, a portable cluster) that fills
// the machine's CTA slots most evenly, keeping at least 6 K blocks per CTA; ties go to the
// smaller factor (less reduction traffic).
int choose_split(int64_t tiles, int total_kb, int slots) {
    int best = 1;
    double best_eff = 0.0;
    for (int s = 1; s <= kMaxSplit; ++s) {
        if (s > 1 && total_kb / s < 6) break;
        const int64_t units = tiles * s;
        const int64_t waves = (units + slots - 1) / slots;
        const double eff = (double)units / (double)(waves * slots);
        if (eff > best_eff + 0.02) {
            best_eff = eff;
            best = s;
        }
    }
    return best;
}

template <int ENC, bool FULL, int TN>
cudaError_t launch_tn(const void* x, const uint8_t* p, const uint8_t* r, void* y, int64_t M, int64_t N, int64_t K,
                      int* status, cudaStream_t stream) {
    constexpr int kStage = stage_bytes(FULL, TN);
    constexpr int kCtasPerSm = tmem_cols(TN) <= 256 ? 2 : 1;
    constexpr int kSmemBudget = kCtasPerSm == 2 ? 100 * 1024 : 200 * 1024;
    int stages = kSmemBudget / kStage;
    if (stages > 8) stages = 8;
    if (stages < 3) stages = 3;
    const size_t smem = (size_t)stages * kStage + 1024;
    static bool configured = false;  // per instantiation
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(umma_linear_kernel<ENC, FULL, TN>,
                                             cudaFuncAttributeMaxDynamicSharedMemorySize, 220 * 1024);
        if (e != cudaSuccess) return e;
        configured = true;
    }
    CUtensorMap mp, mr, mx;
    if (!make_map_2d(&mp, p, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, (uint64_t)N, (uint64_t)K, kTileRows, kBlockK,
                     CU_TENSOR_MAP_SWIZZLE_64B))
        return cudaErrorInvalidValue;
    if (FULL) {
        if (!make_map_2d(&mr, r, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, (uint64_t)N, (uint64_t)K, kTileRows, kBlockK,
                         CU_TENSOR_MAP_SWIZZLE_64B))
            return cudaErrorInvalidValue;
    } else {
        mr = mp;
    }
    if (!make_map_2d(&mx, x, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, (uint64_t)M, (uint64_t)K, TN, kBlockK,
                     CU_TENSOR_MAP_SWIZZLE_128B))
        return cudaErrorInvalidValue;
    const int64_t row_tiles = (N + kTileRows - 1) / kTileRows, tok_tiles = (M + TN - 1) / TN;
    const int total_kb = (int)((K + kBlockK - 1) / kBlockK);
    int split = forced_split();
    if (split <= 0) split = choose_split(row_tiles * tok_tiles, total_kb, sm_count() * kCtasPerSm);
    if (split > total_kb) split = total_kb;
    if (split > kMaxSplit) split = kMaxSplit;
    if ((size_t)stages * kStage < (size_t)TN * kTileRows * 4) split = 1;  // partial tile overlays the stage ring
    UmmaParams prm;
    prm.y = static_cast<__half*>(y);
    prm.M = (int)M;
    prm.N = (int)N;
    prm.K = (int)K;
    prm.num_stages = stages;
    prm.split = split;
    prm.status = status;

    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)row_tiles, (unsigned)tok_tiles, (unsigned)split);
    cfg.blockDim = dim3(kThreads, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 1;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = (unsigned)split;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, umma_linear_kernel<ENC, FULL, TN>, mp, mr, mx, prm);
    count_launch();
    return e;
}

template <int ENC, bool FULL>
cudaError_t launch_enc(const void* x, const uint8_t* p, const uint8_t* r, void* y, int64_t M, int64_t N, int64_t K,
                       int* status, cudaStream_t stream) {
    if (M <= 16) return launch_tn<ENC, FULL, 16>(x, p, r, y, M, N, K, status, stream);
    if (M <= 32) return launch_tn<ENC, FULL, 32>(x, p, r, y, M, N, K, status, stream);
    if (M <= 64) return launch_tn<ENC, FULL, 64>(x, p, r, y, M, N, K, status, stream);
    if (M <= 128 || M > 256) return launch_tn<ENC, FULL, 128>(x, p, r, y, M, N, K, status, stream);
    return launch_tn<ENC, FULL, 256>(x, p, r, y, M, N, K, status, stream);
}

}  // namespace

cudaError_t launch_umma_linear(int mode, int enc, const void* x, const uint8_t* p, const uint8_t* r, void* y,
                               int64_t M, int64_t N, int64_t K, int* status, cudaStream_t stream) {
    const bool full = mode == DPS_MODE_FULL;
    if (enc == kEncE4M3)
        return full ? launch_enc<kEncE4M3, true>(x, p, r, y, M, N, K, status, stream)
                    : launch_enc<kEncE4M3, false>(x, p, r, y, M, N, K, status, stream);
    return full ? launch_enc<kEncE5M2, true>(x, p, r, y, M, N, K, status, stream)
                : launch_enc<kEncE5M2, false>(x, p, r, y, M, N, K, status, stream);
}

}  // namespace dps
