// Tensor-core path of the dense linear layer: tcgen05.mma with the reconstructed weights as the
// A operand in tensor memory and the activations as the B operand in shared memory.
//
// Paper: "Scheduler: Dual-Precision Execution" -- full mode combines the FP8 tensor with the
// residual tensor into the original FP16 values *during computation*; fast mode uses the FP8
// tensor alone.  Here that combination happens on the way from shared memory to tensor memory.
//
// Tile: 128 weight rows (UMMA M) x TN tokens (UMMA N), K walked in blocks of 128 or 64.  The problem
// is "swapped": D[row][token] = sum_k W[row][k] * x[token][k], so that even a handful of decode
// tokens fills the 128-lane datapath with weight rows and every weight byte is fetched once.
//
// Roles (10 warps; 11 in persistent tiles of two row blocks):
//   warp 0     TMA producer: P tile (128 rows x 128 or 64 bytes), R tile (full mode), x tile (TN rows
//              of 64-element swizzle atoms) into a ring of shared-memory stages, completion
//              counted on mbarriers.  Decode tiles with a K split and grouped persistent tiles keep x
//              in slots of their own, a second stream with its own barriers (see x_slots below).
//   warp 1     allocates tensor memory; one elected lane issues tcgen05.mma (A from TMEM, B from
//              smem) and commits stage-release barriers.  Persistent tiles of two row blocks have a
//              second issuer (warp 10), one per row block.
//   warps 2-9  two groups of four "zip" warps; a warp owns 32 TMEM lanes = 32 weight rows.  Per K
//              block a thread reads its row's plane bytes (swizzled, conflict-free), rebuilds the
//              FP16 words in registers (byte permutes; hardware FP8 conversion for E4M3 fast mode)
//              and writes them to the A ring in TMEM with tcgen05.st.  The groups alternate K
//              blocks, or (RB = 2) serve one 128-row block each of a 256-row CTA tile.  After the
//              K loop the zip warps drain the accumulator (tcgen05.ld), round to FP16 and store y
//              through a shared-memory tile with 16-byte stores.
// Shared memory never holds FP16 weights, so its bandwidth is spent on 1-2 bytes per weight
// instead of 5-6, and the tensor core reads only the small activation tile from it.
//
// Two kernels share these roles: umma_linear_kernel (one tile per CTA; K split over a cluster with
// a DSMEM mailbox for decode-sized tiles) and umma_persistent_kernel (one CTA per SM walks many tiles;
// prefill and grouped launches), see below.
#include <cuda_fp16.h>

#include <cstdio>
#include <cstdlib>

#include "bits.cuh"
#include "dps_internal.h"
#include "sm100.cuh"
#include "tensor_map.h"

namespace dps {

namespace {

using namespace sm100;

constexpr int kTileRows = 128;   // weight rows per CTA (UMMA M)
// K elements per pipeline stage.  128 (128-byte plane rows, the widest swizzled TMA box) where it
// still leaves a ring of at least three or four stages: fast mode with tiles of up to 64 tokens.
// 64 where it does not: tiles of 96 tokens and more (the activation tile alone is 32-64 KB per
// 128 K elements) and full mode with small tiles (two planes per stage).  A ring of two stages
// cannot cover the 1600-2150 cycles a stage load takes; halving the stage doubles the ring depth.
// Measured: 64 everywhere costs fast-mode decode 10-20 % (64-byte plane rows stream worse), 128
// everywhere costs full mode and the grouped kernel about as much.
#ifndef DPS_BK64_FROM
#define DPS_BK64_FROM 96
#endif
#ifndef DPS_RB2_FAST_BK
#define DPS_RB2_FAST_BK 128
#endif
// Full-mode tiles of up to 64 tokens read 64 columns per K block (two planes: the stage is as large as a
// fast-mode one), except the 32-token decode tiles: their stages are handed back as soon as the zip warps have
// read them, so two stages of 128-byte rows do, and 128-byte rows stream better than 64-byte ones (measured at
// 32 tokens, full mode, Llama-7B QKV / gate-up / o / down: 22.3 / 36.3 / 11.0 / 19.7 us against 22.8 / 38.9 /
// 11.5 / 20.2).
#ifndef DPS_FULL_BK128_MAX_TN
#define DPS_FULL_BK128_MAX_TN 32
#endif
#ifndef DPS_FULL_BK128_MIN_TN
#define DPS_FULL_BK128_MIN_TN 16   // 16-token tiles alike: 21.3 / 36.1 / 18.8 us against 23.0 / 38.4 / 20.0 (no o: too small)
#endif
__host__ __device__ constexpr int block_k(bool full, int tn, int rb = 1) {
    if (rb == 2) return (full || tn > 128) ? 64 : DPS_RB2_FAST_BK;   // two accumulators of tn columns + four A slots in 512
    return (tn >= DPS_BK64_FROM || (full && tn <= 64 && !(tn >= DPS_FULL_BK128_MIN_TN && tn <= DPS_FULL_BK128_MAX_TN))) ? 64 : 128;
}
// Widest tile whose split-K partial sums are pushed into a mailbox of their own; wider tiles keep
// the shared memory for the ring and pull the partial tiles out of it afterwards.
#ifndef DPS_PUSH_MAX_TN
#define DPS_PUSH_MAX_TN 64
#endif
constexpr int kMaxAStages = 4;   // barrier array size for the A ring in tensor memory
// Groups of 4 zip warps; group g takes K blocks g, g + G, ...  Two groups everywhere: four were
// measured for 256-token full-mode tiles (one CTA per SM) and changed nothing -- once the stage
// ring is four deep the zip warps no longer hold the tensor pipe back there.
__host__ __device__ constexpr int zip_groups(bool /*full*/, int /*tn*/) { return 2; }
__host__ __device__ constexpr int cta_threads(bool full, int tn) { return 64 + zip_groups(full, tn) * 128; }
constexpr int kMaxStages = 12;
constexpr int kMaxSplit = 8;     // portable cluster size

__host__ __device__ constexpr int plane_stage_bytes(bool full, int tn, int rb = 1) {
    return rb * kTileRows * block_k(full, tn, rb);
}
__host__ __device__ constexpr int stage_bytes(bool full, int tn, int rb = 1) {
    return plane_stage_bytes(full, tn, rb) * (full ? 2 : 1) + tn * block_k(full, tn, rb) * 2;
}
// Columns to allocate: accumulator + A ring.  Tiles of up to 64 tokens leave room for three A
// slots inside 256 columns (two CTAs per SM); wider tiles keep two.
// A ring with an even stage ring: slots alternate between the zip groups (slot = block % slots).
__host__ __device__ constexpr int a_slots(bool full, int tn) { return block_k(full, tn) == 64 ? 4 : 2; }
__host__ __device__ constexpr int a_slots_max(bool full, int tn) {
    return (tn <= 64 && a_slots(full, tn) < 3) ? 3 : a_slots(full, tn);
}
// Two row blocks: two accumulators, and each zip group owns two A slots of its own.
__host__ __device__ constexpr int tmem_cols(bool full, int tn, int rb = 1) {
    int need = rb == 2 ? 2 * tn + 4 * (block_k(full, tn, rb) / 2)
                       : tn + a_slots_max(full, tn) * (block_k(full, tn) / 2);
    int c = 32;
    while (c < need) c <<= 1;
    return c;
}

// Activation slots kept apart from the plane ring.  Decode tiles (dense launches, 32 tokens): the plane
// stage and the activation tile of a K block have different consumers -- the zip warps take the planes into
// registers and hand the stage back at once, the MMAs read the activations several K blocks later -- and a
// tile fetched by the copy engine was measured to arrive 2000-2400 cycles after its request even out of L2.
// So the tiles get slots of their own, requested as soon as the MMAs that read a slot last are complete,
// five K blocks ahead in fast mode (three were 2-4 % slower on most Llama-7B shapes, six and eight leave
// too few plane stages in fast mode).  0 = the activation tile travels inside the stage.
// (16- and 64-token tiles: below.)
#ifndef DPS_XSLOT_MIN_TN
#define DPS_XSLOT_MIN_TN 32
#endif
#ifndef DPS_XSLOT_MAX_TN
#define DPS_XSLOT_MAX_TN 32
#endif
// Plane loading ahead of the dependency in decode tiles (see kPre in the kernel).  Measured inside the decode
// graphs at 32 tokens (fast / full, fraction of the copy bandwidth): nothing 0.55 / 0.60, the first ring pass
// 0.58 / 0.67, refills too 0.59 / 0.71, with the L2 prefetch of the second pass the same.
#ifndef DPS_PRE_DEP
#define DPS_PRE_DEP 3
#endif
#ifndef DPS_XSLOTS
#define DPS_XSLOTS 5        // fast mode
#endif
#ifndef DPS_XSLOTS_FULL
#define DPS_XSLOTS_FULL 3   // full mode: a stage is two planes of 16 KB, and three 8 KB slots leave room for two
#endif
constexpr int kMaxXSlots = 8;   // barrier array size
// 64-token tiles: the split-K mailbox takes 36 KB there, which leaves three plane stages and three slots in
// full mode and two of each in fast mode (one more slot each no longer fits two CTAs on an SM).  Measured
// at 64 tokens on the Llama-7B shapes against tiles that carry the activations in the stages: 0-14 % faster.
// 16-token tiles: slots in full mode only (fast mode with slots: gate-up 1-3 % faster, down 4 % slower).
#ifndef DPS_XSLOTS_FAST16
#define DPS_XSLOTS_FAST16 0
#endif
#ifndef DPS_XSLOTS_FULL64
#define DPS_XSLOTS_FULL64 3
#endif
#ifndef DPS_XSLOTS_FAST64
#define DPS_XSLOTS_FAST64 2
#endif
__host__ __device__ constexpr int x_slots(bool full, bool grouped, int tn, int rb) {
    if (grouped || rb != 1) return 0;
    if (tn == 64) return full ? DPS_XSLOTS_FULL64 : DPS_XSLOTS_FAST64;
    if (tn == 16) return full ? DPS_XSLOTS_FULL : DPS_XSLOTS_FAST16;
    return (tn >= DPS_XSLOT_MIN_TN && tn <= DPS_XSLOT_MAX_TN) ? (full ? DPS_XSLOTS_FULL : DPS_XSLOTS) : 0;
}
// Slots of a launch whose K is not split (no mailbox in shared memory): what the freed space holds best.
// 64-token tiles, fast mode: three slots and three stages instead of two and four (gate-up at 64 tokens:
// 22.3 us against 25.1); full mode: five slots beside the same number of stages.
__host__ __device__ constexpr int x_slots_alone(bool full, int tn) {
    if (x_slots(full, false, tn, 1) == 0) return 0;
    if (tn == 64) return full ? 5 : 3;
    return 5;
}
// The persistent kernel keeps the activations of GROUPED launches in slots as well: an MoE layer streams its
// planes once, three or four 56 KB stages of planes + activations per SM left the stream waiting for the ring
// (two stages instead of three: 25 % slower), and a plane stage is free again as soon as the zip warps have
// read it, while its activation tile has to stay until the MMAs are complete.  Dense persistent launches
// (prefill) are bound by the tensor pipe, not by the ring: their activations stay in the stages.
#ifndef DPS_PERSIST_XSLOTS
#define DPS_PERSIST_XSLOTS 4   // measured on Mixtral expert layers, 96-token tiles: 3 slots 3-5 % slower, 5 up to 13 %
#endif
__host__ __device__ constexpr int persist_x_slots(bool grouped) { return grouped ? DPS_PERSIST_XSLOTS : 0; }
// ... and tiles with two row blocks (grouped or dense) have two MMA-issuing warps, one per row block (the CTA's
// last warp is the second; dense fast-mode prefill on 256 x 192 tiles: +4 %, 1.30 -> 1.35 and 1.34 -> 1.39 PFLOP/s
// on Llama-7B QKV / gate-up at 2048 and 8192 tokens).  Probing the next K block's barriers before issuing the
// MMAs of the current one, so that a wait on a barrier that completed long ago costs nothing, was measured
// 3-5 % SLOWER on prefill in both modes and is not done.  Per-K-block stamps of a fast-mode Mixtral gate/up layer (96-token tiles, 16 MMAs of 48 cycles per
// K block): one warp spent 1240 cycles per block, 470 of them on its waits and commits with the tensor pipe
// running dry behind them; with two issuers one warp's waits hide behind the other's MMAs.
#ifndef DPS_PERSIST_TWO_MMA
#define DPS_PERSIST_TWO_MMA 2   // 0: never; 1: grouped launches only; 2: every tile with two row blocks
#endif
__host__ __device__ constexpr bool persist_two_mma(bool grouped, int rb) {
    return rb == 2 && (DPS_PERSIST_TWO_MMA == 2 || (DPS_PERSIST_TWO_MMA == 1 && persist_x_slots(grouped) > 0));
}
__host__ __device__ constexpr int persist_threads(bool full, int tn, bool grouped, int rb) {
    return cta_threads(full, tn) + (persist_two_mma(grouped, rb) ? 32 : 0);
}
__host__ __device__ constexpr int x_tile_bytes(bool full, int tn, int rb = 1) { return tn * block_k(full, tn, rb) * 2; }
// Bytes of one ring stage: planes and activations, or planes alone when the activations have slots.
__host__ __device__ constexpr int ring_stage_bytes(bool full, int tn, bool grouped, int rb = 1) {
    return stage_bytes(full, tn, rb) - (x_slots(full, grouped, tn, rb) ? x_tile_bytes(full, tn, rb) : 0);
}

// Optional timeline trace (compile with -DDPS_TRACE): lane 0 of each role of CTA (0,0,0) stamps
// the SM clock at pipeline events of every K block.  Read back with dps_debug_trace().
#ifdef DPS_TRACE
constexpr int kTraceBlocks = 64, kTraceEvents = 16;
__device__ long long g_trace[kTraceBlocks * kTraceEvents];
__device__ unsigned long long g_cta_times[2 * 2048 * 12];
#define DPS_CTA_STAMP(ev)                                                                          \
    do {                                                                                           \
        const int cta_ = blockIdx.x + gridDim.x * (blockIdx.y + gridDim.y * blockIdx.z);           \
        if (threadIdx.x == 64 && cta_ < 2048) g_cta_times[(prm.trace_slot * 2048 + cta_) * 12 + (ev)] = global_timer_ns(); \
    } while (0)
#define DPS_CTA_STAMP_T(ev, tid)                                                                   \
    do {                                                                                           \
        const int cta_ = blockIdx.x + gridDim.x * (blockIdx.y + gridDim.y * blockIdx.z);           \
        if (threadIdx.x == (tid) && cta_ < 2048)                                                   \
            g_cta_times[(prm.trace_slot * 2048 + cta_) * 12 + (ev)] = global_timer_ns();           \
    } while (0)
#ifdef DPS_TRACE_BLOCKS
#define DPS_STAMP(ev, i)                                                                          \
    do {                                                                                          \
        if (blockIdx.x == 0 && blockIdx.y == 0 && blockIdx.z == 0 && (threadIdx.x & 31) == 0 &&   \
            (i) < kTraceBlocks)                                                                   \
            g_trace[(i) * kTraceEvents + (ev)] = clock64();                                       \
    } while (0)
#else
#define DPS_STAMP(ev, i) do { } while (0)
#endif
#else
#define DPS_STAMP(ev, i) do { } while (0)
#define DPS_CTA_STAMP(ev) do { } while (0)
#define DPS_CTA_STAMP_T(ev, tid) do { } while (0)
#endif

// Grouped (MoE) launches: blockIdx.y indexes a list of token tiles built on the device by the
// routing pre-pass; each entry is (expert, first sorted row, rows in the tile, unused).
struct GroupedParams {
    const int4* tiles;
    const int32_t* num_tiles;
    const int32_t* sorted_rows;   // sorted position -> caller's row id
    uint32_t e5m2[32];            // bit e set: expert e is E5M2 (truncated or rounded)
    uint32_t rounded[32];         // bit e set: expert e is a rounded nest (full mode only; fast mode reads P alike)
};

struct UmmaParams {
    __half* y;
    int M, N, K;
    int num_stages;
    int split;       // K split = cluster size along z; partial tiles are summed through DSMEM
    int red_offset;  // byte offset (from the aligned base of dynamic smem) of the split-K mailbox
    int x_offset;    // byte offset of the activation slots (tiles whose activations do not ride in the stages)
    int x_slots;     // activation slots (tiles that keep the activations apart from the plane ring)
    int pair_min;    // ring depth from which stages are filled two at a time
    int tail_parts;  // persistent dense launches: the tiles of the last, partial round are cut into this many
                     // token ranges (1, 2 or 4), each a work item of its own
    int* status;
#ifdef DPS_TRACE
    int trace_slot;  // which half of the CTA time table this launch writes
#endif
};

// Two floats -> packed FP16 pair (first in the low half), round to nearest even.
__device__ __forceinline__ uint32_t pack_half2(float lo, float hi) {
    const __half2 h = __floats2half2_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&h);
}

// What a zip warp needs to know about its CTA's pipeline.
struct ZipCtx {
    int group, warp, lane, row, num_kb, num_stages, stage_bytes;
    uint32_t smem_base, tmem_a, lane_base, sw;
    uint64_t *bar_full, *bar_empty, *bar_a_full, *bar_a_empty;
};

// Ring position of a zip warp; carried from tile to tile by the persistent kernel.
struct ZipState {
    int s = 0;                // stage of the next K block
    uint32_t s_parity = 0;    // phase parity of that stage
    int cnt = 0;              // K blocks this warp's group has rebuilt so far
};

// Zip loop of one warp: for each of its K blocks, wait for the planes to land and for the A slot
// to be free, rebuild 128 FP16 weights of this thread's row from the plane bytes and store them
// into tensor memory.  Returns false if a wait timed out.
//
// RB == 2: the stage holds two row blocks (256 plane rows) that share one activation tile; zip
// group g rebuilds row block g of EVERY K block into its own two A slots (2g, 2g + 1).
// (Measured and dropped for single-row-block 256-token tiles: both groups rebuilding half of every K
// block -- half the time from a stage's arrival to its A slot being ready, same throughput -- was
// 4 % slower than alternating blocks.)
// EARLY: the stage holds planes only, so it is handed back as soon as this warp has it in registers.
template <int ENC, bool FULL, int TN, int RB, bool EARLY = false>
__device__ __forceinline__ bool zip_blocks(const ZipCtx& z, ZipState& st) {
    constexpr int kBlockK = block_k(FULL, TN, RB);
    constexpr int kACols = kBlockK / 2;
    constexpr int kPlaneStageBytes = plane_stage_bytes(FULL, TN, RB);
    bool ok = true;
    // Ring positions are advanced incrementally (no division in the loop).  Every stage and every A
    // slot always belongs to the same zip group, so that each waiter sees every phase of the barriers
    // it waits on: stage s belongs to group s % 2 (any ring depth; with an even ring that is simply
    // alternate K blocks), and group g owns the A slots g, g + 2, ... below the slot count, which
    // it uses in turn.
    constexpr int kTotalSlots = a_slots_max(FULL, TN);
    const int my_slots = RB == 2 ? 2 : (kTotalSlots - z.group + 1) / 2;   // 1 or 2
    int s = st.s;
    uint32_t s_parity = st.s_parity;   // phase parity of stage s
    int cnt = st.cnt;                  // K blocks this group has rebuilt so far
    int i = 0;
    for (; i < z.num_kb && ok; ++i, s = (s + 1 == z.num_stages) ? 0 : s + 1, s_parity ^= (s == 0)) {
        if (RB == 1 && (s & 1) != z.group) continue;
        const int turn = my_slots == 2 ? (cnt & 1) : 0;
        const int a = RB == 2 ? 2 * z.group + turn : z.group + 2 * turn;
        const uint32_t a_parity = (uint32_t)(my_slots == 2 ? (cnt >> 1) : cnt) & 1u;
        ++cnt;
        if (z.warp == 2 + 4 * z.group) DPS_STAMP(4, i);
        ok = mbar_wait(smem_u32(&z.bar_full[s]), s_parity);
        ok = __all_sync(0xFFFFFFFFu, ok);
        if (!ok) break;
        if (z.warp == 2 + 4 * z.group) DPS_STAMP(5, i);
        // Read and rebuild the weights FIRST, into registers: that needs the stage, not the A slot,
        // so it overlaps the MMAs that are still reading the slot's previous contents.
        const uint32_t prow = z.smem_base + (uint32_t)s * z.stage_bytes +
                              (uint32_t)((RB == 2 ? z.group * kTileRows : 0) + z.row) * kBlockK;
        uint32_t h[kACols];
#pragma unroll
        for (int c = 0; c < kBlockK / 16; ++c) {
            const uint32_t off = ((uint32_t)c ^ z.sw) * 16u;   // sw already reduced for the swizzle width
            uint4 pv, rv = make_uint4(0, 0, 0, 0);
            asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];"
                         : "=r"(pv.x), "=r"(pv.y), "=r"(pv.z), "=r"(pv.w)
                         : "r"(prow + off));
            if (FULL)
                asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];"
                             : "=r"(rv.x), "=r"(rv.y), "=r"(rv.z), "=r"(rv.w)
                             : "r"(prow + kPlaneStageBytes + off));
            uint32_t h8[8];
            if (FULL) join16<ENC, FULL>(pv, rv, h8);
            else fast16<ENC>(pv, h8);   // E4M3: 2^8 times the weights, undone in the epilogue
#pragma unroll
            for (int j = 0; j < 8; ++j) h[c * 8 + j] = h8[j];
        }
        if (EARLY) {
            __syncwarp();
            if (z.lane == 0) mbar_arrive(smem_u32(&z.bar_empty[s]));
        }
        ok = mbar_wait(smem_u32(&z.bar_a_empty[a]), a_parity ^ 1u);   // now the slot must be free
        ok = __all_sync(0xFFFFFFFFu, ok);
        if (!ok) break;
        if (z.warp == 2 + 4 * z.group) DPS_STAMP(6, i);
        tc_fence_after_sync();
#pragma unroll
        for (int t = 0; t < kACols / 32; ++t) {
            uint32_t part[32];
#pragma unroll
            for (int j = 0; j < 32; ++j) part[j] = h[t * 32 + j];
            tmem_st_32x32b_x32(z.tmem_a + z.lane_base + (uint32_t)(a * kACols + t * 32), part);
        }
        if (z.warp == 2 + 4 * z.group) DPS_STAMP(7, i);
        tmem_wait_st();
        tc_fence_before_sync();
        __syncwarp();
        if (z.lane == 0) {
            mbar_arrive(smem_u32(&z.bar_a_full[a]));
            if (!EARLY) mbar_arrive(smem_u32(&z.bar_empty[s]));
        }
        if (z.warp == 2 + 4 * z.group) DPS_STAMP(8, i);
    }
    st.s = s;
    st.s_parity = s_parity;
    st.cnt = cnt;
    return ok;
}

// ENC == 0 (grouped launches only): the encoding is a per-expert run-time value.
// RB = row blocks of 128 weight rows per CTA.  With RB == 2 one activation tile per stage feeds two
// accumulators, which halves the activation bytes an SM pulls out of L2 per weight byte -- the
// limit of the grouped (MoE) launches, whose token tiles are wide but whose planes are read once.
// RB == 2 supports neither a K split nor the odd ring; each zip group serves one row block.
template <int ENC, bool FULL, int TN, bool GROUPED, int RB = 1>
__global__ void __launch_bounds__(cta_threads(FULL, TN), (tmem_cols(FULL, TN, RB) <= 256 ? 2 : 1))
umma_linear_kernel(const __grid_constant__ CUtensorMap map_p, const __grid_constant__ CUtensorMap map_r,
                   const __grid_constant__ CUtensorMap map_x, const UmmaParams prm, const GroupedParams gp) {
    constexpr int kBlockK = block_k(FULL, TN, RB);
    constexpr int kXAtoms = kBlockK / 64;    // the x tile is stored as 64-element (128-byte) swizzle atoms
    constexpr int kACols = kBlockK / 2;      // TMEM columns of one A slot (two FP16 per column)
    constexpr int kPlaneStageBytes = plane_stage_bytes(FULL, TN, RB);
    constexpr int kStage = ring_stage_bytes(FULL, TN, GROUPED, RB);
    constexpr int kXOffset = kPlaneStageBytes * (FULL ? 2 : 1);
    constexpr bool kXS = x_slots(FULL, GROUPED, TN, RB) > 0;   // the activations have slots of their own ...
    const int xs_n = prm.x_slots;                               // ... this many (chosen per launch: what fits)
    constexpr int kXBytes = x_tile_bytes(FULL, TN, RB);
    constexpr uint32_t kCols = tmem_cols(FULL, TN, RB);
    static_assert(RB == 1 || RB == 2, "one or two row blocks per CTA");
    static_assert(RB == 1 || zip_groups(FULL, TN) == 2, "two row blocks need exactly two zip groups");

    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bar_full[kMaxStages];
    __shared__ __align__(8) uint64_t bar_empty[kMaxStages];
    __shared__ __align__(8) uint64_t bar_a_full[kMaxAStages];
    __shared__ __align__(8) uint64_t bar_a_empty[kMaxAStages];
    __shared__ __align__(8) uint64_t bar_d_full;
    __shared__ __align__(8) uint64_t bar_x_full[kMaxXSlots];
    __shared__ __align__(8) uint64_t bar_x_empty[kMaxXSlots];
    __shared__ __align__(8) uint64_t bar_dep;
    __shared__ uint32_t tmem_base_slot;
    __shared__ int s_rows[GROUPED ? TN : 1];   // grouped launches: row ids of the tile's tokens

    grid_launch_dependents();  // the next kernel's prologue may overlap this kernel's tail
    DPS_CTA_STAMP(0);
#ifdef DPS_TRACE
    {
        unsigned smid_;
        asm volatile("mov.u32 %0, %%smid;" : "=r"(smid_));
        const int cta_ = blockIdx.x + gridDim.x * (blockIdx.y + gridDim.y * blockIdx.z);
        if (threadIdx.x == 64 && cta_ < 2048) g_cta_times[(prm.trace_slot * 2048 + cta_) * 12 + 5] = smid_;
    }
#endif
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int num_stages = prm.num_stages;
    constexpr int kZipGroups = zip_groups(FULL, TN);
    constexpr int kThreads = cta_threads(FULL, TN);
    // Tile order (dense launches with several token tiles): CTAs are handed out x-fastest, so walk
    // groups of 8 row tiles x all token tiles.  The CTAs running at any moment then share 8 row
    // tiles of planes and a few dozen activation tiles, which stay in L2, instead of sweeping
    // the whole weight matrix once per token tile (measured: 1.04 GB of DRAM reads for a
    // 100 MB full-mode QKV layer at 2048 tokens before this, because P + R no longer fit in L2).
    int row_tile = blockIdx.x, tok_tile = blockIdx.y;
    if (!GROUPED && gridDim.y > 1) {
        constexpr int kRowGroup = 8;
        const int lin = blockIdx.x + gridDim.x * blockIdx.y;
        const int per_group = kRowGroup * gridDim.y;
        const int group = lin / per_group, within = lin % per_group;
        const int rows_here = min(kRowGroup, (int)gridDim.x - group * kRowGroup);
        row_tile = group * kRowGroup + within % rows_here;
        tok_tile = within / rows_here;
    }
    const int n0 = row_tile * kTileRows * RB;
    int m0 = tok_tile * TN;          // first token (dense) / first sorted row (grouped) of the tile
    int tile_tokens = TN;            // valid token columns of the tile (grouped)
    int plane_row0 = n0;             // first plane row of the tile in the [E * N][K] view
    bool e5m2 = (ENC == kEncE5M2);
    bool rounded = false;         // grouped launches: this tile's expert is a rounded nest (full mode)
    if (GROUPED) {
        grid_dependency_wait();      // the tile list comes from the routing pre-pass
        if ((int)blockIdx.y >= *gp.num_tiles) return;
        const int4 t = gp.tiles[blockIdx.y];
        m0 = t.y;
        tile_tokens = t.z;
        plane_row0 = t.x * prm.N + n0;
        e5m2 = (gp.e5m2[t.x >> 5] >> (t.x & 31)) & 1u;
        rounded = FULL && ((gp.rounded[t.x >> 5] >> (t.x & 31)) & 1u);
    }
    // UMMA N of this tile.  A grouped tile multiplies only the token columns it has (rounded up to
    // 16): at 64-96 tokens per expert a fast-mode MoE layer sits at the ridge between HBM and the
    // tensor pipe, and padded columns are tensor time.  The activation box still brings TN rows.
    const int mma_n = GROUPED ? min(TN, (tile_tokens + 15) & ~15) : TN;
    const uint32_t idesc = umma_idesc_f16(kTileRows, mma_n);
    const int total_kb = (prm.K + kBlockK - 1) / kBlockK;
    const int split = prm.split;
    const int rank = (split > 1) ? (int)cluster_ctarank() : 0;   // == blockIdx.z
    // K blocks are dealt round-robin to the CTAs of the cluster: at any moment the cluster reads
    // `split` adjacent 64-byte pieces of each weight row, which DRAM serves as one longer burst.
    const int num_kb = (total_kb - rank + split - 1) / split;

    if (threadIdx.x == 0) {
        for (int s = 0; s < num_stages; ++s) {
            mbar_init(smem_u32(&bar_full[s]), 1);
            // 4 zip warps per reader group + 1 tcgen05.commit; a stage that holds planes only (the activations
            // have slots) is read by the zip warps alone
            mbar_init(smem_u32(&bar_empty[s]), RB == 2 ? 9 : (kXS ? 4 : 5));
        }
        for (int a = 0; a < kMaxAStages; ++a) {
            mbar_init(smem_u32(&bar_a_full[a]), 4);
            mbar_init(smem_u32(&bar_a_empty[a]), 1);
        }
        mbar_init(smem_u32(&bar_d_full), 1);
        for (int a = 0; a < kMaxXSlots; ++a) {
            mbar_init(smem_u32(&bar_x_full[a]), 1);
            mbar_init(smem_u32(&bar_x_empty[a]), 1);   // the tcgen05.commit behind the MMAs that read the slot
        }
        mbar_init(smem_u32(&bar_dep), 1);
        fence_barrier_init();
        prefetch_tensormap(&map_p);
        if (FULL) prefetch_tensormap(&map_r);
        prefetch_tensormap(&map_x);
    }
    if (warp == 1) tmem_alloc(smem_u32(&tmem_base_slot), kCols);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    DPS_CTA_STAMP(1);
    const uint32_t tmem_base = tmem_base_slot;
    const uint32_t tmem_d = tmem_base;           // TN accumulator columns per row block
    const uint32_t tmem_a = tmem_base + RB * TN; // A ring: slots of kACols columns of packed FP16 pairs

    // Split-K sums.  TN <= 64 ("push"): every CTA owns the tokens c with c % split == rank and has a
    // mailbox mail[source rank][slot = c / split][row] in its own shared memory, outside the stage
    // ring; peers store their partial sums straight into it, one cluster barrier later the owner
    // adds them in rank order.  TN >= 128 ("pull"): the partial tile red[token][row] overlays the
    // idle stage ring and owners read it out of their peers' memory between two cluster barriers.
    constexpr bool kPush = TN <= DPS_PUSH_MAX_TN;
    float* red = reinterpret_cast<float*>(smem_raw + (smem_base - smem_u32(smem_raw)));
    const uint32_t mail_addr = smem_base + (uint32_t)prm.red_offset;
    const int slots = (TN + split - 1) / split;

    bool ok = true;
    if (warp == 0) {
        // ---------------- TMA producer (whole warp converged, one elected lane issues) ----------------
        // Optionally (tuning knob, off by default) stages are filled two at a time.
        const bool pair = (num_stages >= prm.pair_min) && (num_stages % 2 == 0);
        // First pass over the ring.  The planes are model state: (dense launches) their loads are
        // issued BEFORE the dependency wait, so that the ring fills while the preceding kernel
        // drains; only the activations -- that kernel's output in a decoder -- wait for it.  A
        // stage's barrier expects the bytes of both, so it completes when the later one lands.
        const int first = num_kb < num_stages ? num_kb : num_stages;
        auto load_planes = [&](int i, int s) {
            const uint32_t full = smem_u32(&bar_full[s]);
            const uint32_t dst = smem_base + (uint32_t)s * kStage;
            const int k = (rank + i * split) * kBlockK;
            mbar_arrive_expect_tx(full, (uint32_t)kStage);
            tma_load_2d(dst, &map_p, full, k, plane_row0);
            if (FULL) tma_load_2d(dst + kPlaneStageBytes, &map_r, full, k, plane_row0);
        };
        auto load_x = [&](int i, int s) {       // activation tile of K block i, riding in stage s
            const uint32_t full = smem_u32(&bar_full[s]);
            const uint32_t dst = smem_base + (uint32_t)s * kStage;
            const int k = (rank + i * split) * kBlockK;
#pragma unroll
            for (int t = 0; t < kXAtoms; ++t)
                tma_load_2d(dst + kXOffset + (uint32_t)(t * TN * 128), &map_x, full, k + t * 64, m0);
        };
        auto load_x_slot = [&](int j, int slot) {   // activation tile of K block j into its own slot
            const uint32_t full = smem_u32(&bar_x_full[slot]);
            const uint32_t dst = smem_base + (uint32_t)prm.x_offset + (uint32_t)(slot * kXBytes);
            const int k = (rank + j * split) * kBlockK;
            mbar_arrive_expect_tx(full, (uint32_t)kXBytes);
#pragma unroll
            for (int t = 0; t < kXAtoms; ++t)
                tma_load_2d(dst + (uint32_t)(t * TN * 128), &map_x, full, k + t * 64, m0);
        };
        // How much of that a tile with activation slots does ahead of the dependency (tuning knob): 0 nothing,
        // 1 the first ring pass, 2 also refills of stages the zip warps hand back, 3 also the L2 prefetch.
        constexpr int kPre = kXS ? DPS_PRE_DEP : 3;
        if (!GROUPED && elect_one()) {
            for (int i = 0; kPre >= 1 && i < first; ++i) load_planes(i, i);
            // ... and the plane tiles of the second pass are pulled into L2 meanwhile.
            // (A rolling L2 prefetch further ahead during the main loop was measured slower.)
            const int ahead = kPre >= 3 ? (num_kb < 2 * num_stages ? num_kb : 2 * num_stages) : 0;
            for (int i = first; i < ahead; ++i) {
                const int k = (rank + i * split) * kBlockK;
                tma_prefetch_l2_2d(&map_p, k, plane_row0);
                if (FULL) tma_prefetch_l2_2d(&map_r, k, plane_row0);
            }
        }
        __syncwarp();
        DPS_CTA_STAMP_T(8, 0);
        // grouped launches waited before reading the tile list; with activation slots the MMA warp waits and
        // reports on bar_dep, so that this warp can go on requesting planes meanwhile
        if (!GROUPED && !kXS) grid_dependency_wait();
        if (!kXS) DPS_CTA_STAMP_T(9, 0);
        if (!kXS && elect_one()) {
            for (int i = 0; i < first; ++i) {
                if (GROUPED) load_planes(i, i);
                load_x(i, i);
            }
        }
        __syncwarp();
        // Steady state without activation slots: wait for stage s to be free, refill it (planes and
        // activations of K block i).
        int s = first == num_stages ? 0 : first;
        uint32_t ph = first == num_stages ? 1u : 0u;
        for (int i = first; !kXS && i < num_kb && ok; ++i, s = (s + 1 == num_stages) ? 0 : s + 1, ph ^= (s == 0)) {
            if (!pair || (i & 1) == 0) {
                ok = mbar_wait(smem_u32(&bar_empty[s]), ph ^ 1u);
                if (ok && pair && (i & 1) == 0 && i + 1 < num_kb) {     // pairs never wrap: the ring depth is even
                    ok = mbar_wait(smem_u32(&bar_empty[s + 1]), ph ^ 1u);
                }
            }
            ok = __all_sync(0xFFFFFFFFu, ok);
            if (!ok) break;
            DPS_STAMP(0, i);
            if (elect_one()) {
                load_planes(i, s);
                load_x(i, s);
            }
            __syncwarp();
        }
        // Steady state with activation slots: two streams with different consumers.  A plane stage is free as
        // soon as its zip group holds it in registers; an activation slot is free when the MMAs that read it
        // are complete, several K blocks later.  One loop serves both by PROBING (test_wait never suspends)
        // whichever barrier comes next in each stream, so that neither stream waits for the other's consumer;
        // the clock is read once in a while to keep the wait bounded.
        if (kXS) {
            int ip = kPre >= 1 ? first : 0, ix = 0;                     // next K block of each stream
            int sp = ip == num_stages ? 0 : ip, sx = 0;                 // its stage / slot
            // parity of the "free" phase awaited there (a fresh barrier passes a wait for the phase before its first)
            uint32_t php = ip == num_stages ? 0u : 1u, phx = 0u;
            bool dep = false;                                           // the preceding kernel's output may be read
            uint32_t idle = 0;
            unsigned long long t0 = 0;
            while ((ip < num_kb || ix < num_kb) && ok) {
                bool progress = false;
                if (ip < num_kb && (kPre >= 2 || dep) &&
                    __any_sync(0xFFFFFFFFu, mbar_test_wait(smem_u32(&bar_empty[sp]), php))) {
                    DPS_STAMP(0, ip);
                    if (elect_one()) load_planes(ip, sp);
                    __syncwarp();
                    ++ip;
                    sp = (sp + 1 == num_stages) ? 0 : sp + 1;
                    php ^= (sp == 0);
                    progress = true;
                }
                if (!dep && __any_sync(0xFFFFFFFFu, mbar_test_wait(smem_u32(&bar_dep), 0u))) {
                    grid_dependency_wait();     // returns at once; orders this warp's loads behind the dependency
                    DPS_CTA_STAMP_T(9, 0);
                    dep = true;
                }
                if (dep && ix < num_kb &&
                    (ix < xs_n || __any_sync(0xFFFFFFFFu, mbar_test_wait(smem_u32(&bar_x_empty[sx]), phx)))) {
                    if (elect_one()) load_x_slot(ix, sx);
                    __syncwarp();
                    ++ix;
                    sx = (sx + 1 == xs_n) ? 0 : sx + 1;
                    if (sx == 0 && ix > xs_n) phx ^= 1u;
                    progress = true;
                }
                if (progress) {
                    idle = 0;
                } else if ((++idle & 1023u) == 0) {
                    const unsigned long long now = global_timer_ns();
                    if (idle == 1024u) t0 = now;
                    else if (now - t0 > kWaitLimitNs) ok = false;
                }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer (whole warp converged, one elected lane issues) ----------------
        constexpr int kTotalSlots = a_slots_max(FULL, TN);
        if (kXS) {
            // idle until the first activations arrive anyway: waits for the preceding kernel on the producer's behalf
            grid_dependency_wait();
            if (lane == 0) mbar_arrive(smem_u32(&bar_dep));
            __syncwarp();
        }
        if constexpr (RB == 2) {
            int s = 0;
            for (int i = 0; i < num_kb && ok; ++i, s = (s + 1 == num_stages) ? 0 : s + 1) {
                const uint32_t xbase = smem_base + (uint32_t)s * kStage + kXOffset;
                // row block g: A slot 2g + (i & 1) of zip group g, accumulator columns [g * TN, (g + 1) * TN)
#pragma unroll
                for (int g = 0; g < 2; ++g) {
                    const int a = 2 * g + (i & 1);
                    if (g == 0) DPS_STAMP(1, i);
                    ok = mbar_wait(smem_u32(&bar_a_full[a]), (uint32_t)(i >> 1) & 1u);
                    ok = __all_sync(0xFFFFFFFFu, ok);
                    if (!ok) break;
                    if (g == 0) DPS_STAMP(2, i);
                    tc_fence_after_sync();
                    if (elect_one()) {
#pragma unroll
                        for (int j = 0; j < kBlockK / 16; ++j) {
                            const uint64_t bdesc = umma_desc_k_sw128(xbase + (uint32_t)((j >> 2) * TN * 128)) +
                                                   (uint64_t)((j & 3) * 2);
                            umma_f16_ts(tmem_d + (uint32_t)(g * TN), tmem_a + (uint32_t)(a * kACols + j * 8), bdesc,
                                        idesc, (i > 0 || j > 0) ? 1u : 0u);
                        }
                        umma_commit(smem_u32(&bar_a_empty[a]));
                        if (g == 1) {
                            umma_commit(smem_u32(&bar_empty[s]));
                            if (i == num_kb - 1) umma_commit(smem_u32(&bar_d_full));
                        }
                    }
                    __syncwarp();
                }
                DPS_STAMP(3, i);
            }
        } else {
            // Stage s belongs to zip group s % 2, which rotates through its own A slots (see zip_blocks); the
            // activation tile rides in the stage or sits in a slot of its own (K block i: slot i % slots).  The zip warps waited for the stage's
            // TMA loads before they arrived on a_full, so a tile inside the stage is complete once a_full is;
            // a tile in a slot has a barrier of its own.
            int s = 0, xslot = 0;
            uint32_t xparity = 0, cnt0 = 0, cnt1 = 0;   // K blocks taken from each zip group so far
            for (int i = 0; i < num_kb && ok; ++i, s = (s + 1 == num_stages) ? 0 : s + 1) {
                constexpr int g0_slots = (kTotalSlots + 1) / 2, g1_slots = kTotalSlots / 2;   // 1 or 2 each
                int a;
                uint32_t a_parity;
                if ((s & 1) == 0) {
                    a = g0_slots == 2 ? 2 * (int)(cnt0 & 1u) : 0;
                    a_parity = (g0_slots == 2 ? cnt0 >> 1 : cnt0) & 1u;
                    ++cnt0;
                } else {
                    a = g1_slots == 2 ? 1 + 2 * (int)(cnt1 & 1u) : 1;
                    a_parity = (g1_slots == 2 ? cnt1 >> 1 : cnt1) & 1u;
                    ++cnt1;
                }
                const uint32_t xbase = kXS ? smem_base + (uint32_t)prm.x_offset + (uint32_t)(xslot * kXBytes)
                                           : smem_base + (uint32_t)s * kStage + kXOffset;
                DPS_STAMP(1, i);
                ok = mbar_wait(smem_u32(&bar_a_full[a]), a_parity);
                if (i == 0) DPS_CTA_STAMP_T(11, 32);
                DPS_STAMP(9, i);
                if (kXS && ok) ok = mbar_wait(smem_u32(&bar_x_full[xslot]), xparity);
                ok = __all_sync(0xFFFFFFFFu, ok);
                if (!ok) break;
                DPS_STAMP(2, i);
                if (i == 0) DPS_CTA_STAMP_T(10, 32);
                tc_fence_after_sync();
                if (elect_one()) {
#pragma unroll
                    for (int j = 0; j < kBlockK / 16; ++j) {
                        // 16 K elements = 32 bytes inside the 128-byte swizzle atom (j / 4)
                        const uint64_t bdesc = umma_desc_k_sw128(xbase + (uint32_t)((j >> 2) * TN * 128)) +
                                               (uint64_t)((j & 3) * 2);
                        umma_f16_ts(tmem_d, tmem_a + (uint32_t)(a * kACols + j * 8), bdesc, idesc,
                                    (i > 0 || j > 0) ? 1u : 0u);
                    }
                    DPS_STAMP(10, i);
                    if (kXS) umma_commit(smem_u32(&bar_x_empty[xslot]));   // the slot may be refilled ...
                    else umma_commit(smem_u32(&bar_empty[s]));             // ... or the stage that holds the tile
                    umma_commit(smem_u32(&bar_a_empty[a]));
                    if (i == num_kb - 1) umma_commit(smem_u32(&bar_d_full));
                }
                __syncwarp();
                DPS_STAMP(3, i);
                if (kXS) {
                    xslot = (xslot + 1 == xs_n) ? 0 : xslot + 1;
                    xparity ^= (xslot == 0);
                }
            }
        }
    } else {
        // ---------------- zip warps: planes -> FP16 -> tensor memory; then epilogue ----------------
        const int group = (warp - 2) >> 2;
        const int q = warp & 3;                  // TMEM lane quarter this warp may touch
        const int row = q * 32 + lane;           // weight row inside the tile
        const uint32_t lane_base = (uint32_t)(q * 32) << 16;
        ZipCtx zc;
        zc.group = group; zc.warp = warp; zc.lane = lane; zc.row = row;
        zc.num_kb = num_kb; zc.num_stages = num_stages; zc.stage_bytes = kStage;
        zc.smem_base = smem_base; zc.tmem_a = tmem_a; zc.lane_base = lane_base;
        // TMA swizzle of the plane tiles: 128-byte rows: 16-byte chunk index ^= row % 8;
        // 64-byte rows: chunk index ^= (row / 2) % 4
        zc.sw = kBlockK == 128 ? (uint32_t)(row & 7) : (uint32_t)((row >> 1) & 3);
        zc.bar_full = bar_full; zc.bar_empty = bar_empty; zc.bar_a_full = bar_a_full; zc.bar_a_empty = bar_a_empty;
        // grouped launches: the callers' row ids of the tile's tokens, fetched before the zip loop (which
        // hides the latency) rather than in front of every store of the epilogue
        if (GROUPED && (int)threadIdx.x - 64 < tile_tokens) s_rows[threadIdx.x - 64] = gp.sorted_rows[m0 + (int)threadIdx.x - 64];
        if (GROUPED && !(ENC == kEncE4M3 || ENC == kEncE5M2)) {
            // encoding known only at run time (one per expert): uniform branch per CTA
            ZipState zst;
            if (FULL && rounded)
                ok = e5m2 ? zip_blocks<kEncE5M2R, FULL, TN, RB>(zc, zst) : zip_blocks<kEncE4M3R, FULL, TN, RB>(zc, zst);
            else
                ok = e5m2 ? zip_blocks<kEncE5M2, FULL, TN, RB>(zc, zst) : zip_blocks<kEncE4M3, FULL, TN, RB>(zc, zst);
        } else {
            ZipState zst;
            ok = zip_blocks<ENC, FULL, TN, RB, kXS>(zc, zst);
        }
        // E4M3 fast mode multiplied with 2^8 times the weights (hardware FP8 conversion)
        const float out_scale = (!FULL && !e5m2) ? 0.00390625f : 1.0f;
        if (split == 1) {
            // ---- epilogue without a K split: D -> FP16 -> shared memory -> y, by all zip warps ----
            // The accumulator is drained into a [token][row] FP16 tile that overlays the idle stage
            // ring (every load has been consumed once the last MMA is complete), and then written
            // out with 16-byte stores: one warp instruction covers 512 contiguous bytes of a row
            // of y.  Storing straight from the accumulator registers (2 bytes per thread per
            // token, 64 bytes per warp instruction) took 5 us per 256 x 96 tile, with nothing
            // else running on the SM.
            constexpr int kRowsCta = kTileRows * RB;
            constexpr int kColsPerGroup = (RB == 2 || TN < 32) ? TN : TN / 2;   // RB == 1: the groups share the columns
            const int ncols = GROUPED ? tile_tokens : min(TN, prm.M - m0);     // token columns that exist
            if (ok) ok = mbar_wait(smem_u32(&bar_d_full), 0u);
            ok = __all_sync(0xFFFFFFFFu, ok);
            DPS_CTA_STAMP(2);
            const bool drains = RB == 2 || TN >= 32 || group == 0;
            if (ok && drains) {
                tc_fence_after_sync();
                const int rb = RB == 2 ? group : 0;
                const int cbeg = (RB == 1 && TN >= 32) ? group * kColsPerGroup : 0;
#pragma unroll
                for (int cc = 0; cc < kColsPerGroup; cc += 16) {
                    const int c0 = cbeg + cc;
                    if (c0 >= ncols) break;                       // warp-uniform
                    uint32_t v[16];
                    tmem_ld_32x32b_x16(tmem_d + lane_base + (uint32_t)(rb * TN + c0), v);
                    tmem_wait_ld();
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        const __half h = __float2half_rn(__uint_as_float(v[j]) * out_scale);
                        const uint32_t addr = smem_base + (uint32_t)(((c0 + j) * kRowsCta + rb * kTileRows + row) * 2);
                        asm volatile("st.shared.u16 [%0], %1;" ::"r"(addr), "h"(__half_as_ushort(h)) : "memory");
                    }
                }
            }
            named_barrier_sync(1, kZipGroups * 128);              // the zip warps only
            DPS_CTA_STAMP(3);
            if (ok) {
                constexpr int kChunks = kRowsCta / 8;             // 16-byte pieces of one token's rows
                const int zt = (int)threadIdx.x - 64;             // index among the zip threads
                for (int item = zt; item < ncols * kChunks; item += kZipGroups * 128) {
                    const int c = item / kChunks, q = item % kChunks;
                    const int n = n0 + q * 8;
                    if (n >= prm.N) continue;                     // N is a multiple of 8: a piece is in or out
                    const int m = GROUPED ? s_rows[c] : m0 + c;
                    uint4 val;
                    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];"
                                 : "=r"(val.x), "=r"(val.y), "=r"(val.z), "=r"(val.w)
                                 : "r"(smem_base + (uint32_t)((c * kRowsCta + q * 8) * 2)));
                    *reinterpret_cast<uint4*>(prm.y + (int64_t)m * prm.N + n) = val;
                }
            }
        } else if (group == 0 || TN >= 32) {
            // ---- epilogue with a K split: partial sums -> mailbox / red; the zip groups share the columns ----
            constexpr int kColsPerGroup = TN >= 32 ? TN / 2 : TN;
            const int cbeg = TN >= 32 ? group * kColsPerGroup : 0;
            if (ok) ok = mbar_wait(smem_u32(&bar_d_full), 0u);
            ok = __all_sync(0xFFFFFFFFu, ok);
            DPS_CTA_STAMP(2);
            // Both paths first put the partial tile into this CTA's own shared memory as red[token][row], over
            // the idle ring (every load has been consumed).  Push: the tile then goes out to the owners'
            // mailboxes four rows at a time -- sixteen scalar remote stores per thread straight out of the
            // accumulator registers took 0.75 us of every launch.
            if (ok) {
                tc_fence_after_sync();
#pragma unroll
                for (int cc = 0; cc < kColsPerGroup; cc += 16) {
                    const int c0 = cbeg + cc;
                    uint32_t v[16];
                    tmem_ld_32x32b_x16(tmem_d + lane_base + (uint32_t)c0, v);
                    tmem_wait_ld();
#pragma unroll
                    for (int j = 0; j < 16; ++j)
                        red[(c0 + j) * kTileRows + row] = __uint_as_float(v[j]) * out_scale;
                }
            }
            if (kPush) {
                constexpr int kPushers = TN >= 32 ? kZipGroups * 128 : 128;   // the threads in this branch
                asm volatile("bar.sync 2, %0;" ::"n"(kPushers) : "memory");
                if (ok) {
                    const int zt = (int)threadIdx.x - 64;
                    for (int e = zt; e < TN * (kTileRows / 4); e += kPushers) {
                        const int c = e / (kTileRows / 4), r4 = (e % (kTileRows / 4)) * 4;
                        const int owner = c % split, slot = c / split;
                        const float4 val = *reinterpret_cast<const float4*>(&red[c * kTileRows + r4]);
                        const uint32_t local = mail_addr + (uint32_t)(((rank * slots + slot) * kTileRows + r4) * 4);
                        st_cluster_v4_f32(map_to_cta(local, (uint32_t)owner), val);
                    }
                }
            }
        }
    }
    if (!ok) atomicExch(prm.status, (int)DPS_ERR_CUDA);
    if (split > 1) DPS_CTA_STAMP(3);

    if (split > 1 && kPush) {
        __syncthreads();
        cluster_sync_all();  // release/acquire: every peer's stores into this CTA's mailbox are visible
        DPS_CTA_STAMP(4);
        const float* mail = reinterpret_cast<const float*>(smem_raw + (smem_base - smem_u32(smem_raw)) + prm.red_offset);
        // one item = 8 consecutive rows of one owned token: 16 bytes of y
        for (int e = threadIdx.x; e < slots * (kTileRows / 8); e += kThreads) {
            const int slot = e / (kTileRows / 8), r = (e % (kTileRows / 8)) * 8;
            const int c = slot * split + rank;
            const int m = m0 + c, n = n0 + r;
            if (c >= TN || m >= prm.M || n >= prm.N) continue;   // N is a multiple of 8
            float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
            for (int j = 0; j < split; ++j) {
                const float4* src = reinterpret_cast<const float4*>(mail + (j * slots + slot) * kTileRows + r);
                const float4 a = src[0], b = src[1];
                acc[0] += a.x; acc[1] += a.y; acc[2] += a.z; acc[3] += a.w;
                acc[4] += b.x; acc[5] += b.y; acc[6] += b.z; acc[7] += b.w;
            }
            uint4 out;
            out.x = pack_half2(acc[0], acc[1]);
            out.y = pack_half2(acc[2], acc[3]);
            out.z = pack_half2(acc[4], acc[5]);
            out.w = pack_half2(acc[6], acc[7]);
            *reinterpret_cast<uint4*>(prm.y + (int64_t)m * prm.N + n) = out;
        }
    } else if (split > 1) {
        __syncthreads();
        cluster_sync_all();
        DPS_CTA_STAMP(4);
        const uint32_t red_addr = smem_base;
        for (int e = threadIdx.x; e < TN * kTileRows; e += kThreads) {
            const int c = e / kTileRows, r = e % kTileRows;
            if ((c % split) != rank) continue;
            const int m = m0 + c, n = n0 + r;
            if (m >= prm.M || n >= prm.N) continue;
            float acc = 0.f;
            for (int j = 0; j < split; ++j)
                acc += ld_cluster_f32(map_to_cta(red_addr + (uint32_t)(c * kTileRows + r) * 4u, (uint32_t)j));
            prm.y[(int64_t)m * prm.N + n] = __float2half_rn(acc);
        }
        cluster_sync_all();  // nobody leaves while a peer may still read its partial tile
    }
    DPS_CTA_STAMP(6);
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, kCols);
    }
    DPS_CTA_STAMP(7);
}

// ---- persistent variant ----------------------------------------------------------------------
//
// One CTA per SM walks a list of tiles.  The three roles run their loops over the same tile
// sequence without meeting between tiles, so the producer requests the next tile's first stages
// while the current tile is still being multiplied and drained: set-up, launch gap and the
// first-load latency are paid once per CTA instead of once per tile.  For the tile shapes that own
// an SM (256-token full-mode tiles, two-row-block tiles) nothing else would hide them.
// One accumulator: the MMA warp waits for the epilogue to have read the previous tile out of tensor
// memory (bar_d_empty) before it starts the next.  The epilogue goes through a small shared-memory
// buffer (32 token columns at a time), because the stage ring is busy with the next tile.
// No K split, no activation slots.
constexpr int kEpiChunkCols = 32;

struct TileCoords {
    int n0, m0, tile_tokens, plane_row0;
    int parts;   // 1, 2 or 4: this work item covers TN / parts token columns (activation box of that height)
    bool e5m2;
    bool rounded;   // grouped launches, full mode: the expert is a rounded nest
};

// Work item `step` of this CTA: whole tiles blockIdx.x + step * gridDim.x below `t_main`, then ONE
// more item from the last, partial round, in which otherwise a few CTAs would get a whole tile each
// and the rest nothing:
//   * `ksplit` (CTA pairs launched as clusters of two, at most half as many tiles left as CTAs): pair p
//     takes tile t_main + p and each CTA of it one half of K (khalf = its rank); the halves are summed
//     through the pair's shared memory at the very end;
//   * else `parts` > 1 (dense launches): the tiles are cut into `parts` token ranges (part), which
//     write disjoint parts of y.
// Returns false when the CTA is done.
__device__ __forceinline__ bool next_work(int step, int t_main, int total, int parts, bool ksplit, int& lin, int& part,
                                          int& khalf) {
    lin = (int)blockIdx.x + step * (int)gridDim.x;
    part = -1;    // a whole tile
    khalf = -1;   // all of K
    if (lin < t_main) return true;
    if (step != t_main / (int)gridDim.x) return false;
    if (ksplit) {
        const int pair = (int)blockIdx.x >> 1;
        if (pair >= total - t_main) return false;
        lin = t_main + pair;
        khalf = (int)blockIdx.x & 1;
        return true;
    }
    if (parts <= 1) return false;
    const int q = (int)blockIdx.x;
    if (q >= (total - t_main) * parts) return false;
    lin = t_main + q / parts;
    part = q % parts;
    return true;
}

template <int ENC, int TN, bool GROUPED, int RB>
__device__ __forceinline__ TileCoords tile_coords(int lin, int part, int parts, int row_tiles, int tok_tiles,
                                                  const UmmaParams& prm, const GroupedParams& gp) {
    TileCoords t;
    int row_tile, tok_tile;
    if (GROUPED) {
        row_tile = lin % row_tiles;
        tok_tile = lin / row_tiles;
    } else if (tok_tiles > 1) {
        // groups of 8 row tiles x all token tiles (keeps the planes of 8 row tiles and the activation
        // tiles in L2 while they are in use)
        constexpr int kRowGroup = 8;
        const int per_group = kRowGroup * tok_tiles;
        const int group = lin / per_group, within = lin % per_group;
        const int rows_here = min(kRowGroup, row_tiles - group * kRowGroup);
        row_tile = group * kRowGroup + within % rows_here;
        tok_tile = within / rows_here;
    } else {
        row_tile = lin;
        tok_tile = 0;
    }
    t.n0 = row_tile * kTileRows * RB;
    t.parts = part < 0 ? 1 : parts;
    t.m0 = tok_tile * TN + (part < 0 ? 0 : part * (TN / parts));
    t.tile_tokens = min(TN / t.parts, prm.M - t.m0);   // may be <= 0 for a piece past the last token: skipped
    t.plane_row0 = t.n0;
    t.e5m2 = (ENC == kEncE5M2);
    t.rounded = false;
    if (GROUPED) {
        const int4 g = gp.tiles[tok_tile];
        t.m0 = g.y;
        t.tile_tokens = g.z;
        t.plane_row0 = g.x * prm.N + t.n0;
        t.e5m2 = (gp.e5m2[g.x >> 5] >> (g.x & 31)) & 1u;
        t.rounded = (gp.rounded[g.x >> 5] >> (g.x & 31)) & 1u;
    }
    return t;
}

template <int ENC, bool FULL, int TN, bool GROUPED, int RB>
__global__ void __launch_bounds__(persist_threads(FULL, TN, GROUPED, RB), 1)
umma_persistent_kernel(const __grid_constant__ CUtensorMap map_p, const __grid_constant__ CUtensorMap map_r,
                       const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_x2,
                       const __grid_constant__ CUtensorMap map_x4, const UmmaParams prm, const GroupedParams gp) {
    // map_x2 / map_x4: the activation matrix again, with boxes of TN / 2 and TN / 4 rows (tail pieces)
    constexpr int kBlockK = block_k(FULL, TN, RB);
    constexpr int kXAtoms = kBlockK / 64;
    constexpr int kACols = kBlockK / 2;
    constexpr int kPlaneStageBytes = plane_stage_bytes(FULL, TN, RB);
    constexpr int kStage = stage_bytes(FULL, TN, RB);
    constexpr int kXOffset = kPlaneStageBytes * (FULL ? 2 : 1);
    constexpr uint32_t kCols = tmem_cols(FULL, TN, RB);
    constexpr int kRowsCta = kTileRows * RB;
    constexpr int kZipGroups = zip_groups(FULL, TN);
    constexpr int kZipThreads = kZipGroups * 128;
    constexpr int kTotalSlots = a_slots_max(FULL, TN);
    constexpr bool kXS = persist_x_slots(GROUPED) > 0;        // the activations have slots of their own ...
    constexpr int kRing = kXS ? kXOffset : kStage;            // ... and a ring stage holds planes only
    constexpr bool kTwoMma = persist_two_mma(GROUPED, RB);    // one MMA warp per row block
    constexpr int kMmaWarps = kTwoMma ? 2 : 1;
    constexpr int kZipEnd = 2 + 4 * zip_groups(FULL, TN);     // first warp behind the zip warps
    constexpr int kXBytes = x_tile_bytes(FULL, TN, RB);
    static_assert(TN % kEpiChunkCols == 0, "tiles are drained 32 token columns at a time");

    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bar_full[kMaxStages];
    __shared__ __align__(8) uint64_t bar_empty[kMaxStages];
    __shared__ __align__(8) uint64_t bar_a_full[kMaxAStages];
    __shared__ __align__(8) uint64_t bar_a_empty[kMaxAStages];
    __shared__ __align__(8) uint64_t bar_d_full;
    __shared__ __align__(8) uint64_t bar_d_empty;
    __shared__ __align__(8) uint64_t bar_x_full[kMaxXSlots];
    __shared__ __align__(8) uint64_t bar_x_empty[kMaxXSlots];
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;
    __shared__ int s_rows[GROUPED ? TN : 1];   // grouped launches: row ids of the current tile's tokens
    static_assert(!GROUPED || TN <= kZipThreads, "one zip thread per token fetches its row id");

    grid_launch_dependents();
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t epi_base = smem_base + (uint32_t)prm.red_offset;   // chunk buffer behind the ring
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int num_stages = prm.num_stages;
    const int num_kb = (prm.K + kBlockK - 1) / kBlockK;
    const int row_tiles = (prm.N + kRowsCta - 1) / kRowsCta;

    if (threadIdx.x == 0) {
        for (int s = 0; s < num_stages; ++s) {
            mbar_init(smem_u32(&bar_full[s]), 1);
            // the zip warps that read the stage, and the tcgen05.commit if the activations ride in it
            mbar_init(smem_u32(&bar_empty[s]), (RB == 2 ? 8 : 4) + (kXS ? 0 : kMmaWarps));
        }
        for (int a = 0; a < kMaxAStages; ++a) {
            mbar_init(smem_u32(&bar_a_full[a]), 4);
            mbar_init(smem_u32(&bar_a_empty[a]), 1);
        }
        for (int a = 0; a < kMaxXSlots; ++a) {
            mbar_init(smem_u32(&bar_x_full[a]), 1);
            mbar_init(smem_u32(&bar_x_empty[a]), kMmaWarps);   // one tcgen05.commit per MMA warp
        }
        mbar_init(smem_u32(&bar_d_full), kMmaWarps);
        mbar_init(smem_u32(&bar_d_empty), kZipGroups * 4);   // one arrival per zip warp
        abort_flag = 0;
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
    const uint32_t tmem_d = tmem_base;
    const uint32_t tmem_a = tmem_base + RB * TN;

    // Everything read from global memory may come from the preceding kernel (grouped launches: the
    // tile list does).  These launches run for tens of microseconds at least; fetching planes
    // ahead of the dependency, as the decode tiles do, would not be noticed.
    grid_dependency_wait();
    const int tok_tiles = GROUPED ? *gp.num_tiles : (prm.M + TN - 1) / TN;
    const int total = row_tiles * tok_tiles;
    // Last, partial round: halves of K for CTA pairs if the launch came as clusters of two and there
    // are at most half as many tiles left as CTAs; else token ranges (dense launches, if asked for).
    const int tail_tiles = total % (int)gridDim.x;
    const bool ksplit = prm.split == 2 && tail_tiles > 0 && 2 * tail_tiles <= (int)gridDim.x && num_kb >= 2;
    const int parts = (GROUPED || ksplit) ? 1 : prm.tail_parts;
    const int t_main = (ksplit || parts > 1) ? total - tail_tiles : total;
    const bool has_khalf = ksplit && ((int)blockIdx.x >> 1) < tail_tiles;   // same for both CTAs of a pair
    bool ok = true;
    int lin, part, khalf;
    int last_ncols = 0, last_n0 = 0, last_m0 = 0;   // the K-half item's tile, for the pair's reduction below
    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (kXS) {
            // Two streams over the same sequence of (work item, K block): planes into the ring, activation
            // tiles into their slots.  A stage is free when the zip warps have read it, a slot when the MMAs
            // that read it are complete; the loop probes (test_wait never suspends) whichever barrier is next
            // in each stream, so neither waits for the other's consumer.  The clock keeps the wait bounded.
            struct Cursor {
                int step = 0, i = 0, nkb = 0, kb0 = 0, row0 = 0, m0 = 0;
                bool live = false, done = false;
            };
            auto advance = [&](Cursor& c) {      // to the next K block of the stream, fetching work items as needed
                if (c.live && ++c.i < c.nkb) return;
                c.live = false;
                while (!c.done && !c.live) {
                    int l, pt, kh;
                    if (!next_work(c.step, t_main, total, parts, ksplit, l, pt, kh)) { c.done = true; break; }
                    ++c.step;
                    const TileCoords t = tile_coords<ENC, TN, GROUPED, RB>(l, pt, parts, row_tiles, tok_tiles, prm, gp);
                    if (t.tile_tokens <= 0) continue;
                    c.kb0 = kh == 1 ? num_kb / 2 : 0;
                    c.nkb = kh < 0 ? num_kb : (kh == 0 ? num_kb / 2 : num_kb - num_kb / 2);
                    c.row0 = t.plane_row0;
                    c.m0 = t.m0;
                    c.i = 0;
                    c.live = c.nkb > 0;
                }
            };
            Cursor cp, cx;
            advance(cp);
            advance(cx);
            int sp = 0, sx = 0;
            uint32_t php = 0, phx = 0;
            uint32_t idle = 0;
            unsigned long long t0 = 0;
            const int xs_n = prm.x_slots;
            while ((cp.live || cx.live) && ok) {
                bool progress = false;
                // (a fresh barrier passes a wait for the phase before its first at once)
                if (cp.live && __any_sync(0xFFFFFFFFu, mbar_test_wait(smem_u32(&bar_empty[sp]), php ^ 1u))) {
                    if (elect_one()) {
                        const uint32_t full = smem_u32(&bar_full[sp]);
                        const uint32_t dst = smem_base + (uint32_t)sp * kRing;
                        const int k = (cp.kb0 + cp.i) * kBlockK;
                        DPS_STAMP(0, cp.i);
                        mbar_arrive_expect_tx(full, (uint32_t)kRing);
                        tma_load_2d(dst, &map_p, full, k, cp.row0);
                        if (FULL) tma_load_2d(dst + kPlaneStageBytes, &map_r, full, k, cp.row0);
                    }
                    __syncwarp();
                    advance(cp);
                    sp = (sp + 1 == num_stages) ? 0 : sp + 1;
                    php ^= (sp == 0);
                    progress = true;
                }
                if (cx.live && __any_sync(0xFFFFFFFFu, mbar_test_wait(smem_u32(&bar_x_empty[sx]), phx ^ 1u))) {
                    if (elect_one()) {
                        const uint32_t full = smem_u32(&bar_x_full[sx]);
                        const uint32_t dst = smem_base + (uint32_t)prm.x_offset + (uint32_t)(sx * kXBytes);
                        const int k = (cx.kb0 + cx.i) * kBlockK;
                        mbar_arrive_expect_tx(full, (uint32_t)kXBytes);
#pragma unroll
                        for (int a = 0; a < kXAtoms; ++a)
                            tma_load_2d(dst + (uint32_t)(a * TN * 128), &map_x, full, k + a * 64, cx.m0);
                    }
                    __syncwarp();
                    advance(cx);
                    sx = (sx + 1 == xs_n) ? 0 : sx + 1;
                    phx ^= (sx == 0);
                    progress = true;
                }
                if (progress) {
                    idle = 0;
                } else if ((++idle & 1023u) == 0) {
                    const unsigned long long now = global_timer_ns();
                    if (idle == 1024u) t0 = now;
                    else if (now - t0 > kWaitLimitNs) ok = false;
                }
            }
        }
        int s = 0;
        uint32_t ph = 0;
        for (int step = 0; !kXS && ok && next_work(step, t_main, total, parts, ksplit, lin, part, khalf); ++step) {
            const TileCoords t = tile_coords<ENC, TN, GROUPED, RB>(lin, part, parts, row_tiles, tok_tiles, prm, gp);
            if (t.tile_tokens <= 0) continue;
            const CUtensorMap* xmap = t.parts == 4 ? &map_x4 : t.parts == 2 ? &map_x2 : &map_x;
            const uint32_t stage_tx = (uint32_t)(kStage - (TN - TN / t.parts) * kBlockK * 2);
            const int kb0 = khalf == 1 ? num_kb / 2 : 0;
            const int nkb = khalf < 0 ? num_kb : (khalf == 0 ? num_kb / 2 : num_kb - num_kb / 2);
            for (int i = 0; i < nkb && ok; ++i, s = (s + 1 == num_stages) ? 0 : s + 1, ph ^= (s == 0)) {
                ok = mbar_wait(smem_u32(&bar_empty[s]), ph ^ 1u);   // passes at once on the first ring pass
                ok = __all_sync(0xFFFFFFFFu, ok);
                if (!ok) break;
                if (elect_one()) {
                    const uint32_t full = smem_u32(&bar_full[s]);
                    const uint32_t dst = smem_base + (uint32_t)s * kStage;
                    const int k = (kb0 + i) * kBlockK;
                    mbar_arrive_expect_tx(full, stage_tx);
                    tma_load_2d(dst, &map_p, full, k, t.plane_row0);
                    if (FULL) tma_load_2d(dst + kPlaneStageBytes, &map_r, full, k, t.plane_row0);
#pragma unroll
                    for (int a = 0; a < kXAtoms; ++a)
                        tma_load_2d(dst + kXOffset + (uint32_t)(a * TN * 128), xmap, full, k + a * 64, t.m0);
                }
                __syncwarp();
            }
        }
    } else if (warp == 1 || (kTwoMma && warp == kZipEnd)) {
        // ---------------- MMA issuer (one, or one per row block) ----------------
        const int w = warp == 1 ? 0 : 1;
        int s = 0;
        int cnt0 = 0, cnt1 = 0;   // K blocks taken from each zip group (two scalars: an array indexed by the group lives in local memory)
        int it = 0;
        int xslot = 0;            // activation slot of the next K block (launches with activation slots)
        uint32_t xparity = 0;
        const int xs_n = prm.x_slots;
        for (int step = 0; ok && next_work(step, t_main, total, parts, ksplit, lin, part, khalf); ++step) {
            const TileCoords t = tile_coords<ENC, TN, GROUPED, RB>(lin, part, parts, row_tiles, tok_tiles, prm, gp);
            if (t.tile_tokens <= 0) continue;
            const int nkb = khalf < 0 ? num_kb : (khalf == 0 ? num_kb / 2 : num_kb - num_kb / 2);
            // UMMA N: only the token columns the item has, rounded up to 16
            const int mma_n = min(TN, (t.tile_tokens + 15) & ~15);
            const uint32_t idesc = umma_idesc_f16(kTileRows, mma_n);
            if (it > 0) {   // the previous tile must have been read out of the accumulator
                ok = mbar_wait(smem_u32(&bar_d_empty), (uint32_t)(it - 1) & 1u);
                ok = __all_sync(0xFFFFFFFFu, ok);
                if (!ok) break;
                tc_fence_after_sync();
            }
            for (int i = 0; i < nkb && ok; ++i, s = (s + 1 == num_stages) ? 0 : s + 1) {
                const uint32_t xbase = kXS ? smem_base + (uint32_t)prm.x_offset + (uint32_t)(xslot * kXBytes)
                                           : smem_base + (uint32_t)s * kStage + kXOffset;
                DPS_STAMP(1, i);
                if (kXS) {
                    ok = mbar_wait(smem_u32(&bar_x_full[xslot]), xparity);
                    ok = __all_sync(0xFFFFFFFFu, ok);
                    if (!ok) break;
                }
                DPS_STAMP(9, i);
#pragma unroll
                for (int rb = 0; rb < RB; ++rb) {
                    if (kTwoMma && rb != w) continue;
                    // RB == 2: zip group rb serves row block rb of every K block; RB == 1: group s % 2
                    const int g = RB == 2 ? rb : (s & 1);
                    const int g_slots = RB == 2 ? 2 : (kTotalSlots - g + 1) / 2;
                    const int cnt_g = g ? cnt1 : cnt0;
                    const int turn = g_slots == 2 ? (cnt_g & 1) : 0;
                    const int a = RB == 2 ? 2 * g + turn : g + 2 * turn;
                    const uint32_t a_parity = (uint32_t)(g_slots == 2 ? (cnt_g >> 1) : cnt_g) & 1u;
                    if (g) ++cnt1; else ++cnt0;
                    ok = mbar_wait(smem_u32(&bar_a_full[a]), a_parity);
                    ok = __all_sync(0xFFFFFFFFu, ok);
                    if (!ok) break;
                    if (rb == 0) DPS_STAMP(2, i); else DPS_STAMP(10, i);
                    tc_fence_after_sync();
                    if (elect_one()) {
#pragma unroll
                        for (int j = 0; j < kBlockK / 16; ++j) {
                            const uint64_t bdesc = umma_desc_k_sw128(xbase + (uint32_t)((j >> 2) * TN * 128)) +
                                                   (uint64_t)((j & 3) * 2);
                            umma_f16_ts(tmem_d + (uint32_t)(rb * TN), tmem_a + (uint32_t)(a * kACols + j * 8), bdesc,
                                        idesc, (i > 0 || j > 0) ? 1u : 0u);
                        }
                        umma_commit(smem_u32(&bar_a_empty[a]));
                        if (kTwoMma || rb == RB - 1) {
                            if (kXS) umma_commit(smem_u32(&bar_x_empty[xslot]));   // the slot may be refilled ...
                            else umma_commit(smem_u32(&bar_empty[s]));             // ... or the stage with the tile
                            if (i == nkb - 1) umma_commit(smem_u32(&bar_d_full));
                        }
                    }
                    __syncwarp();
                }
                DPS_STAMP(3, i);
                if (kXS) {
                    xslot = (xslot + 1 == xs_n) ? 0 : xslot + 1;
                    xparity ^= (xslot == 0);
                }
            }
            ++it;
        }
    } else if (warp < kZipEnd) {
        // ---------------- zip warps: planes -> FP16 -> tensor memory; then the tile's epilogue ----------------
        const int group = (warp - 2) >> 2;
        const int q = warp & 3;
        const int row = q * 32 + lane;
        const uint32_t lane_base = (uint32_t)(q * 32) << 16;
        const int zt = (int)threadIdx.x - 64;   // index among the zip threads
        ZipCtx zc;
        zc.group = group; zc.warp = warp; zc.lane = lane; zc.row = row;
        zc.num_kb = num_kb; zc.num_stages = num_stages; zc.stage_bytes = kRing;
        zc.smem_base = smem_base; zc.tmem_a = tmem_a; zc.lane_base = lane_base;
        zc.sw = kBlockK == 128 ? (uint32_t)(row & 7) : (uint32_t)((row >> 1) & 3);
        zc.bar_full = bar_full; zc.bar_empty = bar_empty; zc.bar_a_full = bar_a_full; zc.bar_a_empty = bar_a_empty;
        ZipState zst;
        int it = 0;
        for (int step = 0; next_work(step, t_main, total, parts, ksplit, lin, part, khalf); ++step) {
            const TileCoords t = tile_coords<ENC, TN, GROUPED, RB>(lin, part, parts, row_tiles, tok_tiles, prm, gp);
            if (t.tile_tokens <= 0) continue;
            zc.num_kb = khalf < 0 ? num_kb : (khalf == 0 ? num_kb / 2 : num_kb - num_kb / 2);
            // Grouped launches: the callers' row ids of this tile's tokens, fetched now (the zip loop hides
            // the latency) instead of one dependent global load in front of every store of the epilogue --
            // that gather cost 10 % of a fast-mode MoE layer.  The epilogue's barriers order the accesses.
            if (GROUPED && zt < t.tile_tokens) s_rows[zt] = gp.sorted_rows[t.m0 + zt];
            if (ok) {
                if (GROUPED && !(ENC == kEncE4M3 || ENC == kEncE5M2))
                    ok = (FULL && t.rounded)
                             ? (t.e5m2 ? zip_blocks<kEncE5M2R, FULL, TN, RB, kXS>(zc, zst)
                                       : zip_blocks<kEncE4M3R, FULL, TN, RB, kXS>(zc, zst))
                             : (t.e5m2 ? zip_blocks<kEncE5M2, FULL, TN, RB, kXS>(zc, zst)
                                       : zip_blocks<kEncE4M3, FULL, TN, RB, kXS>(zc, zst));
                else
                    ok = zip_blocks<ENC, FULL, TN, RB, kXS>(zc, zst);
            }
            const float out_scale = (!FULL && !t.e5m2) ? 0.00390625f : 1.0f;   // E4M3 fast mode carries 2^8
            if (ok) ok = mbar_wait(smem_u32(&bar_d_full), (uint32_t)it & 1u);
            ok = __all_sync(0xFFFFFFFFu, ok);
            if (ok) tc_fence_after_sync();
            if (!ok) abort_flag = 1;
            const int ncols = t.tile_tokens;
            if (khalf >= 0) {
                // Half of K (always this CTA's last item): the FP32 partial tile goes to shared memory,
                // red[token][row], over the ring -- nothing is in flight any more -- and the pair sums
                // the halves after the role loops.
                last_ncols = ncols; last_n0 = t.n0; last_m0 = t.m0;
                if (ok) {
                    const int rb = RB == 2 ? group : 0;
                    for (int cb = (RB == 2 ? 0 : 16 * group); cb < ncols; cb += (RB == 2 ? 16 : 32)) {
                        uint32_t v[16];
                        tmem_ld_32x32b_x16(tmem_d + lane_base + (uint32_t)(rb * TN + cb), v);
                        tmem_wait_ld();
#pragma unroll
                        for (int j = 0; j < 16; ++j) {
                            const uint32_t addr = smem_base + (uint32_t)(((cb + j) * kRowsCta + rb * kTileRows + row) * 4);
                            asm volatile("st.shared.f32 [%0], %1;" ::"r"(addr), "f"(__uint_as_float(v[j]) * out_scale)
                                         : "memory");
                        }
                    }
                }
                break;
            }
            // The chunk loop has the same trip count for every zip warp (it depends on the tile only),
            // so the barriers inside always match, also after a timeout somewhere.
            for (int c0 = 0; c0 < ncols; c0 += kEpiChunkCols) {
                // drain: RB == 2: this group's row block, all 32 columns; RB == 1: 16 columns per group
                if (ok) {
                    const int rb = RB == 2 ? group : 0;
#pragma unroll
                    for (int h = 0; h < (RB == 2 ? 2 : 1); ++h) {
                        const int cb = c0 + (RB == 2 ? 16 * h : 16 * group);
                        if (cb < ncols) {                     // warp-uniform
                            uint32_t v[16];
                            tmem_ld_32x32b_x16(tmem_d + lane_base + (uint32_t)(rb * TN + cb), v);
                            tmem_wait_ld();
#pragma unroll
                            for (int j = 0; j < 16; ++j) {
                                const __half hv = __float2half_rn(__uint_as_float(v[j]) * out_scale);
                                const uint32_t addr =
                                    epi_base + (uint32_t)(((cb - c0 + j) * kRowsCta + rb * kTileRows + row) * 2);
                                asm volatile("st.shared.u16 [%0], %1;" ::"r"(addr), "h"(__half_as_ushort(hv)) : "memory");
                            }
                        }
                    }
                }
                if (c0 + kEpiChunkCols >= ncols) {
                    // last chunk read: the accumulator may be overwritten by the next tile
                    tc_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&bar_d_empty));
                }
                named_barrier_sync(1, kZipThreads);
                if (ok) {
                    constexpr int kChunks = kRowsCta / 8;             // 16-byte pieces of one token's rows
                    const int cols_here = min(kEpiChunkCols, ncols - c0);
                    for (int item = zt; item < cols_here * kChunks; item += kZipThreads) {
                        const int c = item / kChunks, qq = item % kChunks;
                        const int n = t.n0 + qq * 8;
                        if (n >= prm.N) continue;                     // N is a multiple of 8
                        const int m = GROUPED ? s_rows[c0 + c] : t.m0 + c0 + c;
                        uint4 val;
                        asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];"
                                     : "=r"(val.x), "=r"(val.y), "=r"(val.z), "=r"(val.w)
                                     : "r"(epi_base + (uint32_t)((c * kRowsCta + qq * 8) * 2)));
                        *reinterpret_cast<uint4*>(prm.y + (int64_t)m * prm.N + n) = val;
                    }
                }
                named_barrier_sync(1, kZipThreads);   // the buffer is free for the next chunk
            }
            ++it;
            // after a timeout anywhere among the zip warps they all leave together
            if (*reinterpret_cast<volatile int*>(&abort_flag)) {
                ok = false;
                break;
            }
        }
    }
    if (!ok) atomicExch(prm.status, (int)DPS_ERR_CUDA);
    if (has_khalf) {
        // ---- the pair sums its two halves of K: every CTA takes the 8-row pieces of its parity, adds
        //      the peer's partial (read out of the peer's shared memory) to its own, writes FP16 ----
        __shared__ int s_tile[3];
        if (threadIdx.x == 64) { s_tile[0] = last_ncols; s_tile[1] = last_n0; s_tile[2] = last_m0; }   // a zip thread knows
        __syncthreads();
        cluster_sync_all();   // both partial tiles are complete and visible
        const int ncols = s_tile[0], n0 = s_tile[1], m0 = s_tile[2];
        const uint32_t rank = cluster_ctarank();
        // CTA `rank` takes the tokens of its parity; consecutive threads take consecutive 8-row pieces
        // of a token (32 contiguous bytes each, two 16-byte loads from each partial tile)
        constexpr int kPieces = kRowsCta / 8;
        const int my_cols = (ncols - (int)rank + 1) / 2;
        for (int idx = (int)threadIdx.x; idx < my_cols * kPieces; idx += (int)blockDim.x) {
            const int c = (int)rank + 2 * (idx / kPieces), qq = idx % kPieces;
            const int n = n0 + qq * 8;
            if (n >= prm.N) continue;
            const uint32_t local = smem_base + (uint32_t)((c * kRowsCta + qq * 8) * 4);
            const uint32_t remote = map_to_cta(local, rank ^ 1u);
            float4 a0, a1;
            asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];"
                         : "=f"(a0.x), "=f"(a0.y), "=f"(a0.z), "=f"(a0.w) : "r"(local));
            asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];"
                         : "=f"(a1.x), "=f"(a1.y), "=f"(a1.z), "=f"(a1.w) : "r"(local + 16u));
            const float4 b0 = ld_cluster_v4_f32(remote), b1 = ld_cluster_v4_f32(remote + 16u);
            const int m = GROUPED ? gp.sorted_rows[m0 + c] : m0 + c;
            uint4 out;
            out.x = pack_half2(a0.x + b0.x, a0.y + b0.y);
            out.y = pack_half2(a0.z + b0.z, a0.w + b0.w);
            out.z = pack_half2(a1.x + b1.x, a1.y + b1.y);
            out.w = pack_half2(a1.z + b1.z, a1.w + b1.w);
            *reinterpret_cast<uint4*>(prm.y + (int64_t)m * prm.N + n) = out;
        }
        cluster_sync_all();   // nobody leaves while its peer may still read its partial tile
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, kCols);
    }
}

// ---- host side ---------------------------------------------------------------------------------

// Tuning knob: DPS_PAIR_MIN=<depth> sets the (even) ring depth from which two stages are filled at a
// time, so that two boxes cover 256 adjacent bytes of every weight row.  Off by default: with rings
// of 5-7 stages it was measured equal or slower (up to 20 % on a 6-deep full-mode ring) than
// refilling every stage as soon as it is free.
int pair_min_depth() {
    static const int v = [] {
        const char* e = getenv("DPS_PAIR_MIN");
        return e ? atoi(e) : 1000;
    }();
    return v;
}

// Tuning / debugging knob: DPS_FORCE_SPLIT=<1..8> pins the K split.
int forced_split() {
    static const int v = [] {
        const char* e = getenv("DPS_FORCE_SPLIT");
        return e ? atoi(e) : 0;
    }();
    return v;
}

// K split for a launch of `tiles` output tiles.  capacity[s] = CTAs that can be resident at once
// when launched as clusters of s (clusters must fit inside one GPC, so this is not a multiple of
// the SM count).  Measured on B200: a second wave costs more than it buys, so take the largest
// factor (<= 8, a portable cluster) whose CTAs are all resident at once, keeping at least min_kb K
// blocks per CTA: 4 in fast mode, 5 in full mode (4096 x 4096 at 32-64 tokens in full mode: 6 CTAs per
// tile are 3-5 % faster than 8 with 4 blocks each, alone and inside the decode graphs; in fast mode they
// are as fast alone and 4 % slower inside the graphs).
int choose_split(int64_t tiles, int total_kb, const int* capacity, int min_kb) {
    int best = 1;
    for (int s = 2; s <= kMaxSplit; ++s) {
        if (total_kb / s < min_kb) break;
        if (tiles * s <= capacity[s]) best = s;
    }
    return best;
}

// Tuning knob: DPS_PERSIST=0 launches one CTA per tile even where the persistent kernel applies;
// DPS_PERSIST=2 uses the persistent kernel for such tile shapes even when there are fewer tiles than
// SMs (that is how the tests reach it with small shapes).
int persist_mode() {
    static const int v = [] {
        const char* e = getenv("DPS_PERSIST");
        return e ? atoi(e) : 1;
    }();
    return v;
}
// Dense launches of SM-owning tiles with at most half as many tiles as SMs: two CTAs per tile, each
// with one half of K, summed through the pair's shared memory (the persistent kernel's last-round
// path, with every tile in the "last round").  Chosen when the pairs fill at least three quarters of the SMs:
// measured +24-41 % on the Llama-7B O and down projections at 512 tokens and +18-30 % on the
// hidden-8192 ones at 256 (64 tiles -> 128 CTAs), against 128-token tiles with a cluster split or
// one CTA per 256-token tile; with 32 tiles (64 CTAs) it loses up to 15 %.
// DPS_PAIR_ALL=0 never, 2 whenever the tiles allow it (tuning knob).
bool pair_all_tiles(int64_t tiles) {
    static const int mode = [] {
        const char* e = getenv("DPS_PAIR_ALL");
        return e ? atoi(e) : 1;
    }();
    if (mode == 0 || tiles < 1 || 2 * tiles > sm_count()) return false;
    return mode == 2 || 8 * tiles >= 3 * (int64_t)sm_count();
}
bool use_persistent(int64_t tiles) { return persist_mode() == 2 || (persist_mode() == 1 && tiles > sm_count()); }

// Persistent launch: one CTA per SM (or fewer, if there are fewer tiles) walks `tiles` tiles.
// prm comes with y, M, N, K, status set; the ring is sized here.
// x / x_rows: the activation matrix (dense launches), needed for the half- and quarter-height
// boxes of the tail pieces.
template <int ENC, bool FULL, int TN, bool GROUPED, int RB>
cudaError_t launch_persistent(const CUtensorMap& mp, const CUtensorMap& mr, const CUtensorMap& mx, UmmaParams prm,
                              const GroupedParams& gp, int64_t tiles, const void* x, int64_t x_rows,
                              cudaStream_t stream) {
    constexpr int kXSlots = persist_x_slots(GROUPED);
    constexpr int kXTile = x_tile_bytes(FULL, TN, RB);
    // a ring stage: planes and activations, or planes only when the activations have slots
    constexpr int kStage = stage_bytes(FULL, TN, RB) - (kXSlots ? kXTile : 0);
    constexpr int kEpiBytes = kEpiChunkCols * kTileRows * RB * 2;
    constexpr int kThreads = persist_threads(FULL, TN, GROUPED, RB);
    int xs_n = kXSlots;     // one slot fewer where that buys the third plane stage (128-token tiles, fast mode)
    if (xs_n > 3 && (216 * 1024 - kEpiBytes - xs_n * kXTile) / kStage < 3) --xs_n;
    int stages = (216 * 1024 - kEpiBytes - xs_n * kXTile) / kStage;
    if (stages > 8) stages = 8;
    if (stages < 2) stages = 2;
    const size_t ring_bytes = (size_t)stages * kStage + (size_t)xs_n * kXTile;   // idle after a CTA's last item
    const size_t smem = ring_bytes + kEpiBytes + 1024;
    auto kernel = umma_persistent_kernel<ENC, FULL, TN, GROUPED, RB>;
    static PerDeviceOnce setup;     // per instantiation and per device
    {
        const cudaError_t e = setup.run([&] {
            cudaError_t a = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 224 * 1024);
            if (a != cudaSuccess) return a;
            return cudaFuncSetAttribute(kernel, cudaFuncAttributePreferredSharedMemoryCarveout,
                                        cudaSharedmemCarveoutMaxShared);
        });
        if (e != cudaSuccess) return e;
    }
    prm.num_stages = stages;
    prm.red_offset = (int)ring_bytes;   // the epilogue's chunk buffer
    prm.x_offset = stages * kStage;     // the activation slots, if any
    prm.x_slots = xs_n;
    prm.pair_min = pair_min_depth();
    int64_t grid = tiles < sm_count() ? tiles : sm_count();

    // CTA pairs (clusters of two) so that the tiles of a short last round can be shared out as halves
    // of K, summed through the pair's shared memory; the FP32 partial tile must fit over the ring.
    // DPS_TAIL_KSPLIT=0 launches single CTAs (tuning knob).
    static const int ksplit_mode = [] {   // 2: pairs launched, no split (isolates the cost of the cluster launch)
        const char* e = getenv("DPS_TAIL_KSPLIT");
        return e ? atoi(e) : 1;
    }();
    const bool ksplit_enabled = ksplit_mode != 0;
    // Dense launches with at most half as many tiles as SMs: two CTAs per tile, each with one half of K
    // (the kernel treats all of them as the "last round").
    if (!GROUPED && ksplit_mode == 1 && pair_all_tiles(tiles) && (size_t)TN * kTileRows * RB * 4 <= ring_bytes)
        grid = 2 * tiles;
    const bool pairs = ksplit_enabled && grid >= 2 && (size_t)TN * kTileRows * RB * 4 <= ring_bytes;
    if (pairs) grid &= ~(int64_t)1;
    prm.split = (pairs && ksplit_mode == 1) ? 2 : 1;
    // Last, partial round of a dense launch: cut its tiles into 2 or 4 token ranges if that gives
    // more CTAs something to do (each piece streams the tile's planes again, out of L2, but
    // multiplies and fetches only its share of the activations).  Measured gain: 0-4 % -- the
    // weight-side work (plane loads, rebuilding) of a piece is that of a whole tile.
    // DPS_TAIL_PARTS=1|2|4 overrides.
    static const int parts_forced = [] {
        const char* e = getenv("DPS_TAIL_PARTS");
        return e ? atoi(e) : 0;
    }();
    int parts = 1;
    CUtensorMap mx2 = mx, mx4 = mx;
    if (!GROUPED) {
        const int64_t tail = tiles % grid;
        if (!pairs && tail > 0 && tiles > grid) {   // with CTA pairs the short last round is split along K instead
            if (2 * tail <= grid) parts = 2;
            if (4 * tail <= grid) parts = 4;
        }
        if ((parts_forced == 1 || parts_forced == 2 || parts_forced == 4) && tail * parts_forced <= grid)
            parts = tiles > grid ? parts_forced : 1;   // every piece of the tail needs a CTA of its own
        if (parts > 1) {
            if (!make_map_2d(&mx2, x, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, (uint64_t)x_rows, (uint64_t)prm.K, TN / 2, 64,
                             CU_TENSOR_MAP_SWIZZLE_128B) ||
                !make_map_2d(&mx4, x, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, (uint64_t)x_rows, (uint64_t)prm.K, TN / 4, 64,
                             CU_TENSOR_MAP_SWIZZLE_128B))
                return cudaErrorInvalidValue;
        }
    }
    prm.tail_parts = parts;
    if (getenv("DPS_DEBUG"))
        fprintf(stderr, "[dps] persistent TN=%d full=%d RB=%d grouped=%d tiles<=%lld grid=%lld stages=%d tail_parts=%d pairs=%d\n",
                TN, (int)FULL, RB, (int)GROUPED, (long long)tiles, (long long)grid, stages, parts, (int)pairs);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid, 1, 1);
    cfg.blockDim = dim3(kThreads, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = 2;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pairs ? 2 : 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, kernel, mp, mr, mx, mx2, mx4, prm, gp);
    count_launch();
    return e;
}

template <int ENC, bool FULL, int TN>
cudaError_t launch_tn(const void* x, const uint8_t* p, const uint8_t* r, void* y, int64_t M, int64_t N, int64_t K,
                      int* status, cudaStream_t stream) {
    constexpr int kStage = ring_stage_bytes(FULL, TN, false);   // planes only when the activations have slots
    constexpr int kXSlots = x_slots(FULL, false, TN, 1);            // with a split-K mailbox in shared memory
    constexpr int kXSlotsAlone = x_slots_alone(FULL, TN);           // without one (K not split)
    constexpr int kXTile = x_tile_bytes(FULL, TN);
    constexpr int kZipGroups = zip_groups(FULL, TN);
    constexpr int kThreads = cta_threads(FULL, TN);
    constexpr int kCtasPerSm = tmem_cols(FULL, TN) <= 256 ? 2 : 1;
    constexpr int kSmemTotal = kCtasPerSm == 2 ? 111 * 1024 : 216 * 1024;
    constexpr int kMailMax = TN <= DPS_PUSH_MAX_TN ? (TN + kMaxSplit) * kTileRows * 4 : 0;  // push-mode mailbox, worst case
    // Ring depth for a given mailbox size: whatever fits (stage s is rebuilt by zip group s % 2, so
    // odd depths work; they just give the first group one stage more).
    static const int deep_forced = [] {
        const char* e = getenv("DPS_FORCE_DEEP");
        return e ? atoi(e) : -1;
    }();
    const int64_t tiles_total = ((N + kTileRows - 1) / kTileRows) * ((M + TN - 1) / TN);
    // One CTA per SM with a ring twice as deep when the tiles cannot fill two CTA slots per SM anyway.
    const bool deep = deep_forced >= 0 ? deep_forced != 0 : false;
    const int smem_total = (deep || kCtasPerSm == 1) ? 216 * 1024 : kSmemTotal;
    static const int max_stages = [] {   // DPS_MAX_STAGES=<n>: tuning knob, caps the ring depth
        const char* e = getenv("DPS_MAX_STAGES");
        return e ? atoi(e) : 8;
    }();
    auto ring_depth = [&](int mail_bytes) {
        const int x_ring = (mail_bytes > 0 ? kXSlots : kXSlotsAlone) * kXTile;
        int d = (smem_total - mail_bytes - x_ring) / kStage;
        if (d > max_stages) d = max_stages;
        if (d < 2) d = 2;
        return d;
    };
    const size_t smem_query = (size_t)ring_depth(kMailMax) * kStage + kXSlots * kXTile + kMailMax + 1024;
    auto kernel = umma_linear_kernel<ENC, FULL, TN, false>;
    // CTAs that can be resident at once for each cluster size: per instantiation and per device, filled by
    // the first call on that device and read only after that set-up has returned.
    static int capacity_of[kMaxDevices][kMaxSplit + 1] = {};
    static PerDeviceOnce setup;
    int dev = 0;
    {
        const cudaError_t e0 = setup.run([&] {
            int d = 0;
            cudaGetDevice(&d);
            int* capacity = capacity_of[d];
            cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 224 * 1024);
            if (e != cudaSuccess) return e;
            // Ask for the largest shared-memory carve-out, otherwise the driver may size it for ONE CTA
            // of this kernel and a second CTA never becomes resident on the SM.
            e = cudaFuncSetAttribute(kernel, cudaFuncAttributePreferredSharedMemoryCarveout,
                                     cudaSharedmemCarveoutMaxShared);
            if (e != cudaSuccess) return e;
            for (int s = 1; s <= kMaxSplit; ++s) {
                cudaLaunchConfig_t q = {};
                q.gridDim = dim3(1, 1, (unsigned)s);
                q.blockDim = dim3(kThreads, 1, 1);
                q.dynamicSmemBytes = smem_query;
                cudaLaunchAttribute qa[1];
                qa[0].id = cudaLaunchAttributeClusterDimension;
                qa[0].val.clusterDim.x = 1;
                qa[0].val.clusterDim.y = 1;
                qa[0].val.clusterDim.z = (unsigned)s;
                q.attrs = qa;
                q.numAttrs = 1;
                int clusters = 0;
                if (cudaOccupancyMaxActiveClusters(&clusters, kernel, &q) != cudaSuccess) clusters = 0;
                capacity[s] = clusters * s;
            }
            (void)cudaGetLastError();
            // The query can be more conservative about CTAs per SM than the hardware turns out to be
            // (it reported one where two were measured resident); keep its GPC packing ratios and
            // rescale to the CTAs per SM this kernel is sized for.
            const int slots = sm_count() * kCtasPerSm;
            if (capacity[1] <= 0) capacity[1] = slots;
            const int base = capacity[1];
            for (int s = 1; s <= kMaxSplit; ++s) capacity[s] = (int)((int64_t)capacity[s] * slots / base);
            // With two CTAs per SM a cluster of even size s needs only s / 2 SMs of a GPC, so it packs
            // like a cluster of s / 2 at one CTA per SM (32 row tiles split 8 ways, 256 CTAs, were
            // measured 5-11 % faster than split 6 ways, which the plain rescaling would have chosen).
            if (kCtasPerSm == 2)
                for (int s = kMaxSplit; s >= 2; s -= 2)
                    if (capacity[s / 2] > capacity[s]) capacity[s] = capacity[s / 2];
            return cudaSuccess;
        }, &dev);
        if (e0 != cudaSuccess) return e0;
    }
    const int* capacity = capacity_of[dev];
    CUtensorMap mp, mr, mx;
    constexpr int kBlockK = block_k(FULL, TN);
    constexpr CUtensorMapSwizzle kPlaneSwizzle = kBlockK == 128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B;
    if (!make_map_2d(&mp, p, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, (uint64_t)N, (uint64_t)K, kTileRows, kBlockK,
                     kPlaneSwizzle))
        return cudaErrorInvalidValue;
    if (FULL) {
        if (!make_map_2d(&mr, r, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, (uint64_t)N, (uint64_t)K, kTileRows, kBlockK,
                         kPlaneSwizzle))
            return cudaErrorInvalidValue;
    } else {
        mr = mp;
    }
    if (!make_map_2d(&mx, x, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, (uint64_t)M, (uint64_t)K, TN, 64,
                     CU_TENSOR_MAP_SWIZZLE_128B))
        return cudaErrorInvalidValue;
    const int64_t row_tiles = (N + kTileRows - 1) / kTileRows, tok_tiles = (M + TN - 1) / TN;
    const int total_kb = (int)((K + kBlockK - 1) / kBlockK);
    int split = forced_split();
    if (split <= 0) split = choose_split(row_tiles * tok_tiles, total_kb, capacity, FULL ? 5 : 4);
    if (deep) split = 1;
    (void)tiles_total;
    if (split > total_kb) split = total_kb;
    if (split > kMaxSplit) split = kMaxSplit;
    // the mailbox exists only when K is split, and then has its exact size
    const int slots = split > 1 ? (TN + split - 1) / split : 0;
    const int mail_bytes = (split > 1 && kMailMax > 0) ? split * slots * kTileRows * 4 : 0;
    const int stages = ring_depth(mail_bytes);
    const int xs_n = mail_bytes > 0 ? kXSlots : kXSlotsAlone;
    const int x_ring = xs_n * kXTile;
    const size_t smem = (size_t)stages * kStage + x_ring + mail_bytes + 1024;
    if (kMailMax == 0 && (size_t)stages * kStage < (size_t)TN * kTileRows * 4) split = 1;  // pull mode overlays the ring
    if (getenv("DPS_DEBUG"))
        fprintf(stderr, "[dps] umma TN=%d full=%d N=%lld K=%lld M=%lld stages=%d split=%d capacity=%d,%d,%d,%d,%d,%d,%d,%d\n",
                TN, (int)FULL, (long long)N, (long long)K, (long long)M, stages, split, capacity[1], capacity[2],
                capacity[3], capacity[4], capacity[5], capacity[6], capacity[7], capacity[8]);
    UmmaParams prm = {};
    prm.y = static_cast<__half*>(y);
    prm.M = (int)M;
    prm.N = (int)N;
    prm.K = (int)K;
    prm.status = status;
    if constexpr (kCtasPerSm == 1) {
        // a tile shape that owns its SM: with more tiles than SMs, let one CTA per SM walk them
        if ((split == 1 && use_persistent(row_tiles * tok_tiles)) || pair_all_tiles(row_tiles * tok_tiles))
            return launch_persistent<ENC, FULL, TN, false, 1>(mp, mr, mx, prm, GroupedParams{}, row_tiles * tok_tiles,
                                                             x, M, stream);
    }
    prm.num_stages = stages;
    prm.split = split;
    prm.x_offset = stages * kStage;
    prm.x_slots = xs_n;
    prm.red_offset = stages * kStage + x_ring;
    prm.status = status;
    prm.pair_min = pair_min_depth();
#ifdef DPS_TRACE
    static int trace_launches = 0;
    prm.trace_slot = (trace_launches++) & 1;
#endif

    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)row_tiles, (unsigned)tok_tiles, (unsigned)split);
    cfg.blockDim = dim3(kThreads, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 1;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = (unsigned)split;
    // Programmatic dependent launch: this kernel may start while the previous one drains; it
    // waits (griddepcontrol.wait) before its first global read.
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    GroupedParams gp = {};
    cudaError_t e = cudaLaunchKernelEx(&cfg, kernel, mp, mr, mx, prm, gp);
    count_launch();
    return e;
}

// Dense launch with two row blocks per CTA (256 weight rows share each activation tile): no K
// split, one CTA per SM unless the tile is narrow.
template <int ENC, bool FULL, int TN>
cudaError_t launch_tn_rb2(const void* x, const uint8_t* p, const uint8_t* r, void* y, int64_t M, int64_t N, int64_t K,
                          int* status, cudaStream_t stream) {
    constexpr int kRb = 2;
    constexpr int kStage = stage_bytes(FULL, TN, kRb);
    constexpr int kThreads = cta_threads(FULL, TN);
    constexpr int kCtasPerSm = tmem_cols(FULL, TN, kRb) <= 256 ? 2 : 1;
    constexpr int kSmemTotal = kCtasPerSm == 2 ? 111 * 1024 : 216 * 1024;
    constexpr int kBlockK = block_k(FULL, TN, kRb);
    constexpr CUtensorMapSwizzle kPlaneSwizzle = kBlockK == 128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B;
    int stages = kSmemTotal / kStage;
    if (stages > 8) stages = 8;
    if (stages < 2) stages = 2;
    const size_t smem = (size_t)stages * kStage + 1024;
    auto kernel = umma_linear_kernel<ENC, FULL, TN, false, kRb>;
    static PerDeviceOnce setup;     // per instantiation and per device
    {
        const cudaError_t e = setup.run([&] {
            cudaError_t a = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 224 * 1024);
            if (a != cudaSuccess) return a;
            return cudaFuncSetAttribute(kernel, cudaFuncAttributePreferredSharedMemoryCarveout,
                                        cudaSharedmemCarveoutMaxShared);
        });
        if (e != cudaSuccess) return e;
    }
    CUtensorMap mp, mr, mx;
    if (!make_map_2d(&mp, p, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, (uint64_t)N, (uint64_t)K, kTileRows * kRb, kBlockK,
                     kPlaneSwizzle))
        return cudaErrorInvalidValue;
    if (FULL) {
        if (!make_map_2d(&mr, r, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, (uint64_t)N, (uint64_t)K, kTileRows * kRb, kBlockK,
                         kPlaneSwizzle))
            return cudaErrorInvalidValue;
    } else {
        mr = mp;
    }
    if (!make_map_2d(&mx, x, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, (uint64_t)M, (uint64_t)K, TN, 64,
                     CU_TENSOR_MAP_SWIZZLE_128B))
        return cudaErrorInvalidValue;
    UmmaParams prm = {};
    prm.y = static_cast<__half*>(y);
    prm.M = (int)M;
    prm.N = (int)N;
    prm.K = (int)K;
    prm.status = status;
    if constexpr (kCtasPerSm == 1) {
        const int64_t tiles = ((N + kTileRows * kRb - 1) / (kTileRows * kRb)) * ((M + TN - 1) / TN);
        if (use_persistent(tiles))
            return launch_persistent<ENC, FULL, TN, false, kRb>(mp, mr, mx, prm, GroupedParams{}, tiles, x, M, stream);
    }
    prm.num_stages = stages;
    prm.split = 1;
    prm.red_offset = 0;
    prm.pair_min = pair_min_depth();
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)((N + kTileRows * kRb - 1) / (kTileRows * kRb)), (unsigned)((M + TN - 1) / TN), 1);
    cfg.blockDim = dim3(kThreads, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    GroupedParams gp = {};
    cudaError_t e = cudaLaunchKernelEx(&cfg, kernel, mp, mr, mx, prm, gp);
    count_launch();
    return e;
}

template <int ENC, bool FULL>
cudaError_t launch_enc(const void* x, const uint8_t* p, const uint8_t* r, void* y, int64_t M, int64_t N, int64_t K,
                       int* status, cudaStream_t stream) {
    if (M <= 16) return launch_tn<ENC, FULL, 16>(x, p, r, y, M, N, K, status, stream);
    if (M <= 32) return launch_tn<ENC, FULL, 32>(x, p, r, y, M, N, K, status, stream);
    if (M <= 64) return launch_tn<ENC, FULL, 64>(x, p, r, y, M, N, K, status, stream);
    // Prefill: in full mode the zip warps (two planes to read, more bit work) are the bottleneck,
    // and a 256-token tile halves their work per FLOP (one CTA per SM, each rebuilt weight block
    // feeds twice the columns); in fast mode two co-resident 128-token CTAs with deeper rings win.
    // DPS_FORCE_TN=64|128|256 overrides (tuning knob).
    static const int tn_forced = [] {
        const char* e = getenv("DPS_FORCE_TN");
        return e ? atoi(e) : 0;
    }();
    static const int rb_forced = [] {
        const char* e = getenv("DPS_DENSE_RB");
        return e ? atoi(e) : 0;
    }();
    // 65-128 tokens on matrices of moderate size: two 64-token tiles per 128 weight rows (the decode tiles with
    // their separate plane and activation streams) instead of one 128-token tile whose K is split over a
    // cluster and summed by remote loads.  Every weight is then streamed out of L2 and rebuilt twice, which
    // full mode and large matrices do not forgive.  Measured at 96 and 128 tokens: Llama-7B QKV / o / down in
    // fast mode 24.6 / 12.3-13.3 / 23.6 us against 31.7-33.8 / 19.5-20.5 / 25.6-26.6, o in full mode 17.4 against
    // 21.5-22.6; gate/up (90 M weights) 8 % slower in fast and 30 % in full mode, hidden-8192 layers 3-50 % slower
    // except o in fast mode (-8 %).  DPS_FORCE_TN=64|128 overrides.
    const bool two_by_64 = tn_forced ? tn_forced == 64 : N * K <= ((int64_t)1 << (FULL ? 25 : 26));
    if (M <= 128 && two_by_64) return launch_tn<ENC, FULL, 64>(x, p, r, y, M, N, K, status, stream);
    // Fast mode with more such tiles than SMs (the persistent kernel then walks them): 256 weight rows per CTA share
    // each 128-token activation tile, which halves the activation bytes pulled out of L2 per
    // FLOP (measured +2-8 % at 2048-8192 tokens; with fewer tiles the SMs run dry, and in full
    // mode the zip warps would rebuild twice the weights per MMA cycle: -20 %).
    // DPS_DENSE_RB=1|2 overrides (tuning knob).
    const int64_t tiles_rb2 = ((N + 2 * kTileRows - 1) / (2 * kTileRows)) * ((M + 127) / 128);
    const bool rb2 = rb_forced ? rb_forced == 2 : (!FULL && tiles_rb2 > (int64_t)sm_count());
    // ... and 192 tokens wide once there are at least two rounds of such tiles: 40 KB of planes and
    // activations per 256 x 192 x 64 block instead of 64 KB per 256 x 128 x 128, i.e. a sixth less out of L2 per
    // FLOP, which is what bounds the main loop (measured +5 % at 2048 tokens on the two wide Llama-7B layers,
    // +5-8 % at 8192 on all four; with fewer tiles the coarser last round costs more than that).  Two
    // accumulators of 192 columns and four A slots of 32 fill the tensor memory, hence 64-element K blocks.
    // DPS_RB2_TN=128|192 overrides (tuning knob).
    static const int rb2_tn = [] {
        const char* e = getenv("DPS_RB2_TN");
        return e ? atoi(e) : 0;
    }();
    if constexpr (!FULL) {
        const int64_t tiles192 = ((N + 2 * kTileRows - 1) / (2 * kTileRows)) * ((M + 191) / 192);
        // padded token columns are multiplied like real ones: at most 4 % more of them than with 128-token tiles
        const int64_t padded192 = ((M + 191) / 192) * 192, padded128 = ((M + 127) / 128) * 128;
        const bool wide192 = rb2_tn ? rb2_tn == 192
                                    : tiles192 >= 2 * (int64_t)sm_count() && 25 * padded192 <= 26 * padded128;
        if (rb2 && M > 128 && wide192) return launch_tn_rb2<ENC, FULL, 192>(x, p, r, y, M, N, K, status, stream);
    }
    if (rb2 && M > 64) return launch_tn_rb2<ENC, FULL, 128>(x, p, r, y, M, N, K, status, stream);
    // ... unless 256-token tiles would leave half the SMs without one (few weight rows, few tokens):
    // then 128-token tiles, two CTAs per SM, win by 10-40 % (measured at 256 tokens, N = 4096 / 8192).
    const int64_t tiles256 = ((N + kTileRows - 1) / kTileRows) * ((M + 255) / 256);
    // few 256-token tiles, but enough for CTA pairs (halves of K) to fill most SMs
    if (!tn_forced && M > 128 && pair_all_tiles(tiles256))
        return launch_tn<ENC, FULL, 256>(x, p, r, y, M, N, K, status, stream);
    const bool wide = tn_forced ? tn_forced == 256
                                : (FULL ? M > 128 : (M > 128 && M <= 256)) && 2 * tiles256 > (int64_t)sm_count();
    if (!wide) return launch_tn<ENC, FULL, 128>(x, p, r, y, M, N, K, status, stream);
    return launch_tn<ENC, FULL, 256>(x, p, r, y, M, N, K, status, stream);
}

}  // namespace

// Byte-matrix tensor map for the other translation units (row-major [rows][cols] bytes, boxes of
// box_rows x 128 bytes, 128-byte swizzle).
bool make_byte_map_sw128(CUtensorMap* map, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows) {
    return make_map_2d(map, base, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, rows, cols, box_rows, 128, CU_TENSOR_MAP_SWIZZLE_128B);
}

#ifdef DPS_TRACE
extern "C" __attribute__((visibility("default"))) int dps_debug_trace(long long* out, int max_words) {
    const int n = max_words < kTraceBlocks * kTraceEvents ? max_words : kTraceBlocks * kTraceEvents;
    return (int)cudaMemcpyFromSymbol(out, g_trace, sizeof(long long) * n);
}
extern "C" __attribute__((visibility("default"))) int dps_debug_cta_times(unsigned long long* out) {
    return (int)cudaMemcpyFromSymbol(out, g_cta_times, sizeof(unsigned long long) * 2 * 2048 * 12);
}
#endif

namespace {

template <bool FULL, int TN, int RB>
cudaError_t launch_grouped_tn(const uint32_t* e5m2_mask, const void* x_sorted, const uint8_t* p, const uint8_t* r,
                              void* y, int64_t A, int64_t N, int64_t K, int32_t E, const void* tiles,
                              const int32_t* num_tiles, const int32_t* sorted_rows, int max_tiles, int* status,
                              cudaStream_t stream) {
    constexpr int kStage = stage_bytes(FULL, TN, RB);
    constexpr int kZipGroups = zip_groups(FULL, TN);
    constexpr int kThreads = cta_threads(FULL, TN);
    constexpr int kCtasPerSm = tmem_cols(FULL, TN, RB) <= 256 ? 2 : 1;
    constexpr int kSmemTotal = kCtasPerSm == 2 ? 111 * 1024 : 216 * 1024;
    int stages = kSmemTotal / kStage;
    if (stages > 8) stages = 8;
    if (stages < 2) stages = 2;
    const size_t smem = (size_t)stages * kStage + 1024;
    auto kernel = umma_linear_kernel<0, FULL, TN, true, RB>;
    static PerDeviceOnce setup;     // per instantiation and per device
    {
        const cudaError_t e = setup.run([&] {
            cudaError_t a = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 224 * 1024);
            if (a != cudaSuccess) return a;
            return cudaFuncSetAttribute(kernel, cudaFuncAttributePreferredSharedMemoryCarveout,
                                        cudaSharedmemCarveoutMaxShared);
        });
        if (e != cudaSuccess) return e;
    }
    CUtensorMap mp, mr, mx;
    constexpr int kBlockK = block_k(FULL, TN, RB);
    constexpr CUtensorMapSwizzle kPlaneSwizzle = kBlockK == 128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B;
    if (!make_map_2d(&mp, p, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, (uint64_t)E * (uint64_t)N, (uint64_t)K, kTileRows * RB,
                     kBlockK, kPlaneSwizzle))
        return cudaErrorInvalidValue;
    if (FULL) {
        if (!make_map_2d(&mr, r, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, (uint64_t)E * (uint64_t)N, (uint64_t)K, kTileRows * RB,
                         kBlockK, kPlaneSwizzle))
            return cudaErrorInvalidValue;
    } else {
        mr = mp;
    }
    if (!make_map_2d(&mx, x_sorted, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, (uint64_t)A, (uint64_t)K, TN, 64,
                     CU_TENSOR_MAP_SWIZZLE_128B))
        return cudaErrorInvalidValue;
    UmmaParams prm = {};
    prm.y = static_cast<__half*>(y);
    prm.M = (int)A;
    prm.N = (int)N;
    prm.K = (int)K;
    prm.num_stages = stages;
    prm.split = 1;
    prm.red_offset = 0;
    prm.status = status;
    prm.pair_min = pair_min_depth();
    GroupedParams gp;
    gp.tiles = static_cast<const int4*>(tiles);
    gp.num_tiles = num_tiles;
    gp.sorted_rows = sorted_rows;
    for (int i = 0; i < 32; ++i) {   // the caller's array holds the E5M2 bits, then the rounded-nest bits
        gp.e5m2[i] = e5m2_mask[i];
        gp.rounded[i] = FULL ? e5m2_mask[32 + i] : 0u;
    }
    if constexpr (kCtasPerSm == 1 && TN % kEpiChunkCols == 0) {
        const int64_t upper = ((N + kTileRows * RB - 1) / (kTileRows * RB)) * max_tiles;
        if (use_persistent(upper))
            return launch_persistent<0, FULL, TN, true, RB>(mp, mr, mx, prm, gp, upper, x_sorted, A, stream);
    }

    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)((N + kTileRows * RB - 1) / (kTileRows * RB)), (unsigned)max_tiles, 1);
    cfg.blockDim = dim3(kThreads, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, kernel, mp, mr, mx, prm, gp);
    count_launch();
    return e;
}

}  // namespace

// Token-tile width of grouped launches: wide enough that an expert with 1.5 times the average
// number of rows still fits one tile (its planes are then streamed once), no wider than needed
// (every tile drags TN activation rows through L2 per weight block: at 128 tokens that is twice
// the plane bytes, and L2-to-SM bandwidth, not HBM, becomes the limit).
int grouped_tile_tokens(int64_t A, int32_t E) {
    const int64_t avg = (A + E - 1) / E;
    const int64_t target = avg + (avg + 1) / 2;
    return target <= 16 ? 16 : target <= 32 ? 32 : target <= 64 ? 64 : target <= 96 ? 96 : 128;
}

cudaError_t launch_umma_grouped(int mode, const uint32_t* e5m2_mask, const void* x_sorted, const uint8_t* p,
                                const uint8_t* r, void* y, int64_t A, int64_t N, int64_t K, int32_t E, int tn,
                                const void* tiles, const int32_t* num_tiles, const int32_t* sorted_rows,
                                int max_tiles, int* status, cudaStream_t stream) {
    // Two row blocks per CTA for wide token tiles, when that still leaves every SM a CTA: the
    // activation tile is then fetched from L2 once per 256 weight rows instead of once per 128.
    // DPS_GROUPED_RB=1|2 overrides (tuning knob).
    static const int rb_forced = [] {
        const char* e = getenv("DPS_GROUPED_RB");
        return e ? atoi(e) : 0;
    }();
    const bool two = rb_forced ? rb_forced == 2
                               : (tn >= 64 && ((N + 2 * kTileRows - 1) / (2 * kTileRows)) * max_tiles >= sm_count());
#define DPS_GROUPED_CALL(FULLV, TNV, RBV)                                                                         \
    launch_grouped_tn<FULLV, TNV, RBV>(e5m2_mask, x_sorted, p, r, y, A, N, K, E, tiles, num_tiles, sorted_rows,  \
                                       max_tiles, status, stream)
#define DPS_GROUPED_CASE(TNV)                                                                                     \
    if (tn == TNV)                                                                                                \
        return mode == DPS_MODE_FULL ? DPS_GROUPED_CALL(true, TNV, 1) : DPS_GROUPED_CALL(false, TNV, 1);
#define DPS_GROUPED_CASE2(TNV)                                                                                    \
    if (tn == TNV && two)                                                                                         \
        return mode == DPS_MODE_FULL ? DPS_GROUPED_CALL(true, TNV, 2) : DPS_GROUPED_CALL(false, TNV, 2);
    DPS_GROUPED_CASE2(64)
    DPS_GROUPED_CASE2(96)
    DPS_GROUPED_CASE2(128)
    DPS_GROUPED_CASE(16)
    DPS_GROUPED_CASE(32)
    DPS_GROUPED_CASE(64)
    DPS_GROUPED_CASE(96)
    DPS_GROUPED_CASE(128)
#undef DPS_GROUPED_CASE
#undef DPS_GROUPED_CASE2
#undef DPS_GROUPED_CALL
    return cudaErrorInvalidValue;
}

cudaError_t launch_umma_linear(int mode, int enc, const void* x, const uint8_t* p, const uint8_t* r, void* y,
                               int64_t M, int64_t N, int64_t K, int* status, cudaStream_t stream) {
    const bool full = mode == DPS_MODE_FULL;
    if (!full) enc = base_enc(enc);   // fast mode reads the persistent byte of a rounded nest like any other
    if (enc == kEncE4M3R) return launch_enc<kEncE4M3R, true>(x, p, r, y, M, N, K, status, stream);
    if (enc == kEncE5M2R) return launch_enc<kEncE5M2R, true>(x, p, r, y, M, N, K, status, stream);
    if (enc == kEncE4M3)
        return full ? launch_enc<kEncE4M3, true>(x, p, r, y, M, N, K, status, stream)
                    : launch_enc<kEncE4M3, false>(x, p, r, y, M, N, K, status, stream);
    return full ? launch_enc<kEncE5M2, true>(x, p, r, y, M, N, K, status, stream)
                : launch_enc<kEncE5M2, false>(x, p, r, y, M, N, K, status, stream);
}

}  // namespace dps
