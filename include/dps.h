/*
 * libdps -- dual-precision (fast / full mode) linear layers computed directly from
 * nested FP8 + residual weight planes, for NVIDIA B200 (sm_100a).
 *
 * The operations follow the DPS paper's statement of the problem:
 *   - an FP16 model is split into an FP8 model kept in the persistent region and a
 *     residual model kept in the shared region (section "Mapper: Semi-Unified Memory
 *     Abstraction", paragraph "Persistent Region");
 *   - in full mode the executor combines both tensors to reconstruct the original FP16
 *     values during computation; in fast mode only the FP8 tensor is used and the
 *     residual is not accessed, because its memory may be holding KV-cache data
 *     (section "Scheduler: Dual-Precision Execution", paragraph "Overall concept");
 *   - the encoding (E4M3 or E5M2) is chosen per layer at load time from weight
 *     statistics, and the kernels serve dense and MoE (grouped) layers (same section,
 *     paragraph "Dual-mode serving (DPS) with asymmetric switching");
 *   - every layer of one forward pass runs in the same mode and two CUDA graphs are
 *     captured per batch size (paragraph "Granularity of the precision switch").
 *
 * Conventions (all entry points):
 *   - W[N][K] is a linear layer's weight, N outputs by K inputs, row-major with K
 *     contiguous; y[M][N] = x[M][K] * W^T.  x and y are IEEE binary16, row-major.
 *   - The persistent plane P and the residual plane R are SEPARATE allocations of N*K
 *     bytes each, index-for-index identical to W.
 *   - The planes are MODEL STATE.  The linear kernels start fetching them while the
 *     kernel that precedes the call on the stream is still draining (programmatic
 *     dependent launch); only the activations wait for that kernel.  So a plane must not
 *     be written by the kernel launched immediately before dps_linear / dps_moe_linear
 *     on the same stream.  Planes written by dps_split_weights, by a copy
 *     (cudaMemcpyAsync) or by any kernel further back in the stream are safe:
 *     dps_split_weights ends with a fence launch for exactly this reason.
 *   - Pointers are DEVICE pointers unless a parameter says "host".  The caller owns
 *     every buffer; the library never allocates or frees device memory.
 *   - cuda_stream is a cudaStream_t passed as void* (NULL = the default stream).  Work
 *     is enqueued on it and, except where stated, the call returns without
 *     synchronising, so calls can be captured into CUDA graphs.
 *   - Every device base pointer must be 16-byte aligned; K must be a multiple of 16 and
 *     N a multiple of 8.  Violations return DPS_ERR_ALIGN / DPS_ERR_SHAPE.
 *   - The return value reports host-detectable errors only; on error nothing has been
 *     enqueued.  Data-dependent problems found on the device (an expert or token index
 *     out of range) set a per-device status word: the offending row is skipped, its
 *     output row is left untouched, and dps_stream_status() reports DPS_ERR_DATA.
 *   - No exception crosses this boundary.  Calls on distinct streams are thread-safe.
 */
#ifndef DPS_H_
#define DPS_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define DPS_API __attribute__((visibility("default")))
#else
#define DPS_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    DPS_OK = 0,
    DPS_ERR_NULL = 1,        /* a required pointer is NULL */
    DPS_ERR_SHAPE = 2,       /* negative or unsupported size */
    DPS_ERR_MODE = 3,        /* mode is neither FAST nor FULL */
    DPS_ERR_ENCODING = 4,    /* encoding value not valid for this call */
    DPS_ERR_ALIGN = 5,       /* pointer not 16-byte aligned */
    DPS_ERR_UNSUPPORTED = 6, /* valid request this build cannot serve (e.g. wrong GPU) */
    DPS_ERR_CUDA = 7,        /* a CUDA runtime call failed */
    DPS_ERR_DATA = 8,        /* data-dependent: E4M3 requested for an ineligible tensor, bad index */
    DPS_ERR_WORKSPACE = 9    /* workspace NULL, misaligned or too small */
} dps_status;

typedef enum { DPS_MODE_FAST = 0, DPS_MODE_FULL = 1 } dps_mode;
typedef enum {
    DPS_ENC_AUTO = 0,
    DPS_ENC_E4M3 = 1,
    DPS_ENC_E5M2 = 2,
    DPS_ENC_E4M3_RN = 3, /* rounded nests, see below */
    DPS_ENC_E5M2_RN = 4,
    DPS_ENC_AUTO_RN = 5  /* dps_split_weights only: AUTO's rule, answering with a rounded nest */
} dps_encoding;

/*
 * Nested split (paper: "Persistent Region" paragraph).  With b the FP16 word
 * (s = b[15], e = b[14:10], m = b[9:0]):
 *   E5M2: P = s e[4:0] m[9:8]          R = m[7:0]
 *   E4M3: P = s e[3:0] m[9:7]          R = 0 m[6:0]      (needs b[14] == 0 everywhere)
 * Bits are selected, never rounded, so (P, R) rebuilds W exactly.
 *
 * Rounded nests (an extension: the paper describes the bit selection only).  DPS_ENC_E5M2_RN and
 * DPS_ENC_E4M3_RN store the same fields of b' = b + 0x0080 (E5M2) or b + 0x0040 (E4M3), i.e. of
 * the word plus half a unit of the last bit P keeps.  P is then the FP8 value NEAREST to the
 * weight (ties away from zero) instead of the next one towards zero, which removes the
 * shrinking bias of fast mode, and join(P, R) - the same constant still rebuilds W exactly.
 * Legal iff no b' reaches an Inf / NaN code: max|b & 0x7FFF| + 0x80 < 0x7C00 (E5M2_RN),
 * + 0x40 < 0x3F80 (E4M3_RN).  Never chosen by AUTO; DPS_ENC_AUTO_RN chooses between them by
 * AUTO's rule (E4M3_RN iff max|w| <= 1.75, else E5M2_RN; DPS_ERR_DATA if that is not legal
 * either, i.e. |w| >= 61440 or Inf / NaN present).  Accepted wherever an encoding is.  In a legal
 * rounded pair a zero P byte never meets a zero R byte; the linear kernels read such a pair (their
 * own padding) as a zero weight.
 *
 * w_fp16: device, rows*cols FP16 words.  w_persist, w_resid: device, rows*cols bytes each.
 * enc_inout: HOST int32.  On entry DPS_ENC_AUTO, DPS_ENC_AUTO_RN or one of the four encodings; on return
 * the encoding that was used.
 *   AUTO  -> E4M3 iff every word has b[14] == 0 and max|w| <= 1.75, else E5M2.  The
 *            statistics pass needs its result on the host, so this variant SYNCHRONISES
 *            the stream (splitting is load-time work).
 *   E4M3  -> also synchronises: the tensor is checked first, and if any word has b[14] set
 *            or would produce the byte 0x7F/0xFF the call returns DPS_ERR_DATA with both
 *            planes untouched.
 *   E5M2  -> always legal, never synchronises.
 *   E4M3_RN, E5M2_RN -> checked like E4M3 (synchronise; DPS_ERR_DATA if not legal).
 * rows*cols == 0 returns DPS_OK (AUTO then reports E4M3, AUTO_RN E4M3_RN).  cols must be a
 * multiple of 16.
 */
DPS_API dps_status dps_split_weights(const void* w_fp16, uint8_t* w_persist, uint8_t* w_resid,
                             int64_t rows, int64_t cols, int32_t* enc_inout, void* cuda_stream);

/*
 * Reconstruction (paper: "Overall concept" paragraph, full mode): the inverse of the
 * split, W = join(P, R), bit-exact.  Bit 7 of an E4M3 residual byte is ignored.
 * w_resid == NULL rebuilds the fast-mode weights instead (residual taken as zero).
 * (for a rounded nest: the values of its persistent bytes, i.e. the rounded weights).
 * enc must be one of the four encodings, never AUTO.  Never synchronises.
 */
DPS_API dps_status dps_reconstruct(const uint8_t* w_persist, const uint8_t* w_resid, void* w_fp16_out,
                           int64_t rows, int64_t cols, int32_t enc, void* cuda_stream);

/*
 * Dense linear layer (paper: "Overall concept" paragraph).
 *   y[M][N] (FP16) = x[M][K] (FP16) * W_eff^T, FP32 accumulation, one FP16 rounding at the
 *   store.  FULL: W_eff = join(P, R), the original FP16 weights.  FAST: W_eff = join(P, 0);
 *   w_resid is never dereferenced and may be NULL or point at unrelated data.
 * enc must be one of the four encodings (the value dps_split_weights reported).  M == 0 returns DPS_OK
 * without a launch.  Never synchronises, never allocates.  Results are deterministic: the
 * same inputs give the same bits on every call.
 */
DPS_API dps_status dps_linear(int32_t mode, int32_t enc, const void* x, const uint8_t* w_persist,
                      const uint8_t* w_resid, void* y, int64_t M, int64_t N, int64_t K,
                      void* cuda_stream);

/*
 * Grouped (MoE) linear layer (paper: "Dual-mode serving" paragraph, GroupedGEMM kernels).
 * For each row a in [0, A):
 *   y[a][:] = x[token_of_row ? token_of_row[a] : a][:] * W_eff(expert_of_row[a])^T
 * x: [T][K] FP16.  y: [A][N] FP16.  w_persist / w_resid: [E][N][K] bytes (w_resid may be
 * NULL in FAST mode).  enc_per_expert: HOST array of E encodings (any of the four, never AUTO), read
 * before the call returns.  token_of_row (may be NULL) and expert_of_row: device int32[A].
 * workspace: device scratch of at least dps_moe_workspace_bytes(A, E, K) bytes, 16-byte
 * aligned, owned by the caller; its contents are overwritten (routing tables and the
 * activations regrouped by expert).  E may not exceed 1024.  A row whose expert is
 * outside [0, E) or whose token is outside [0, T) is skipped and flagged (see
 * dps_stream_status).  A == 0 returns DPS_OK without a launch.  Never synchronises.
 */
DPS_API dps_status dps_moe_linear(int32_t mode, const int32_t* enc_per_expert, const void* x,
                          const int32_t* token_of_row, const int32_t* expert_of_row,
                          const uint8_t* w_persist, const uint8_t* w_resid, void* y,
                          int64_t A, int64_t T, int64_t N, int64_t K, int32_t E,
                          void* workspace, size_t workspace_bytes, void* cuda_stream);

/* Bytes of scratch dps_moe_linear needs for A rows, E experts and K inputs (0 if an argument is
 * invalid). */
DPS_API size_t dps_moe_workspace_bytes(int64_t A, int32_t E, int64_t K);

/*
 * Grouped linear layer for callers that cannot allocate (the paper has no counterpart; this is a
 * convenience of this library).
 *
 * Some callers have no way to hand dps_moe_linear a workspace: a serving worker that gave all of
 * its free device memory to the weight planes and the KV cache at start-up and runs its steps under
 * a rule that nothing may call cudaMalloc afterwards (an allocation there synchronises the device,
 * can fail when memory is fully committed, and is forbidden outright in some runtimes), or a
 * plug-in that is only ever given its input and output buffers.  For them this variant computes
 * exactly what dps_moe_linear computes, with the same kernels, but keeps its scratch (routing tables
 * and the activations regrouped by expert) in a fixed array inside the library instead of a caller
 * buffer.  The call itself allocates nothing and frees nothing.
 *
 * Limits and rules:
 *   - The array is DPS_MOE_STATIC_SCRATCH_BYTES (16 MiB) per GPU and is held by every GPU that loads
 *     the library until the process exits.  A problem whose dps_moe_workspace_bytes(A, E, K) exceeds
 *     it is rejected with DPS_ERR_WORKSPACE and nothing is enqueued; use dps_moe_linear then.
 *   - The first call on each device looks up the array's device address (a one-time, host-side
 *     set-up step).  Make that first call outside any stream capture.  If the look-up fails the
 *     call returns DPS_ERR_CUDA and keeps nothing: a later call simply tries again.
 *   - All calls on a device share the one array and it keeps whatever the last call left in it.
 *     Nothing in it has to start at zero: every call rewrites all the tables it reads.  Two calls
 *     whose kernels can overlap on the GPU (different streams without an ordering between them)
 *     would overwrite each other's scratch: keep calls on one stream or order them with events.
 * Arguments, layouts, error codes and the status word are those of dps_moe_linear, minus the
 * workspace pair.  Never synchronises.
 */
#define DPS_MOE_STATIC_SCRATCH_BYTES (16u << 20)
DPS_API dps_status dps_moe_linear_static(int32_t mode, const int32_t* enc_per_expert, const void* x,
                                         const int32_t* token_of_row, const int32_t* expert_of_row,
                                         const uint8_t* w_persist, const uint8_t* w_resid, void* y,
                                         int64_t A, int64_t T, int64_t N, int64_t K, int32_t E,
                                         void* cuda_stream);

/*
 * Fast mode with FP8 activations (paper: "Persistent Region" paragraph, which notes that FP8
 * execution can raise the tensor-core peak where the hardware supports it).  The persistent plane is fed to the FP8
 * tensor cores as it is; the activations are quantised per token:
 *   scale[m] = max_k |x[m][k]| / 448 (1 for an all-zero token),
 *   x_fp8[m][k] = E4M3(x[m][k] / scale[m]), round to nearest even, saturating (both in binary32),
 *   y[m][n] = scale[m] * sum_k x_fp8[m][k] * W_fast[n][k], FP32 accumulation, one FP16 rounding.
 * This is a DIFFERENT result from dps_linear in fast mode (the activations lose precision: a few
 * per cent of the output scale on Gaussian data); it is meant for prefill-sized token counts.
 * dps_quantize_activations: x FP16 [M][K] -> x_fp8 uint8 [M][K] and scale float [M] (all device).
 * An Inf or NaN activation sets the device status word to DPS_ERR_DATA.
 * dps_linear_fp8act: enc as reported by dps_split_weights; the residual plane is not an argument.
 * Shapes, alignment and error rules as for dps_linear.  Neither call synchronises or allocates.
 */
DPS_API dps_status dps_quantize_activations(const void* x, uint8_t* x_fp8, float* scale, int64_t M, int64_t K,
                                            void* cuda_stream);
DPS_API dps_status dps_linear_fp8act(int32_t enc, const uint8_t* x_fp8, const float* scale,
                                     const uint8_t* w_persist, void* y, int64_t M, int64_t N, int64_t K,
                                     void* cuda_stream);

/*
 * Residual backup and restore (paper: "Scheduler: Dual-Precision Execution", the restore of the
 * lower byte before a switch back to full mode, done by a worker beside the running steps).
 * While a layer runs in fast mode the memory of its residual plane may be lent out; the bytes then
 * live in a host copy.  dps_backup_residual copies a residual plane to host memory,
 * dps_restore_residual copies it back, both as a sequence of plain asynchronous copies of
 * chunk_bytes each (0 = 4 MiB, the granularity at which a restore can yield to other copies) on
 * cuda_stream -- normally a stream of its own, so that fast-mode dps_linear calls on another stream
 * keep running meanwhile; they never read the residual plane.  backup_host should be page-locked
 * (pinned) host memory: with pageable memory the copies are staged and the call blocks.  Neither
 * call synchronises; the caller orders the switch to full mode after the restore (an event on
 * cuda_stream).  bytes == 0 returns DPS_OK without enqueuing anything.
 */
DPS_API dps_status dps_backup_residual(const uint8_t* w_resid, uint8_t* backup_host, size_t bytes,
                                       size_t chunk_bytes, void* cuda_stream);
DPS_API dps_status dps_restore_residual(uint8_t* w_resid, const uint8_t* backup_host, size_t bytes,
                                        size_t chunk_bytes, void* cuda_stream);

/*
 * Synchronises the stream, then returns and clears the current device's status word:
 * DPS_OK, DPS_ERR_DATA (a kernel skipped a row with a bad index) or DPS_ERR_CUDA.
 */
DPS_API dps_status dps_stream_status(void* cuda_stream);

/*
 * Diagnostic: exercises the bounded device-side wait that every pipeline of the tensor-core kernels
 * uses.  One warp waits, for at most limit_ns nanoseconds (1 .. 1e9), on a barrier that nothing
 * ever signals; when the limit passes it sets the status word and returns, exactly as a kernel does
 * whose copy never arrives.  Afterwards dps_stream_status() reports DPS_ERR_CUDA once, and the
 * device and the library remain fully usable.  Nothing faults, traps or spins without a limit.
 * (No counterpart in the paper: it tests this library's own failure handling.)
 */
DPS_API dps_status dps_debug_wait_timeout(uint64_t limit_ns, void* cuda_stream);

/* Number of kernel launches this process has enqueued through the library so far. */
DPS_API int64_t dps_launch_count(void);

DPS_API const char* dps_status_string(dps_status status);
DPS_API int dps_version(void);

#ifdef __cplusplus
}
#endif
#endif /* DPS_H_ */
