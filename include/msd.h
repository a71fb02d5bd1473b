/*
 * msd.h - C ABI of the B200 (sm_100a) hot path of Multi-Scale Dequant (MSD).
 *
 * MSD keeps quantized weights / KV in their low-precision format and instead splits each BF16
 * activation row (or query / softmax-probability tile) at run time into two low-precision components
 * with their own scales; both components are multiplied against the quantized operand on the tensor
 * cores and the partial products are combined with the scales in the epilogue.
 *
 * General rules for every call
 *  - All pointers are DEVICE pointers unless the argument name ends in `_host`.  The caller owns every
 *    buffer; the library allocates nothing on these paths and never synchronises the stream.
 *  - `stream` is a cudaStream_t (NULL = default stream).  Work is enqueued asynchronously.
 *  - BF16 tensors are raw 16-bit patterns; row-major, innermost dimension contiguous.
 *  - Host-detectable problems (null pointer, bad shape, misalignment, short workspace) return an error
 *    code BEFORE any launch.  A failed launch returns MSD_ERR_CUDA.  Device-side waits are bounded: a
 *    kernel that gives up records MSD_ERR_TIMEOUT in a device status word and exits without trapping;
 *    msd_last_device_status() reads and clears that word.
 *  - Non-finite activations give unspecified values but never a hang or a fault.
 *  - Workspaces: sizes come from the *_workspace_bytes functions; a workspace must be zero-filled once
 *    before its first use (msd_workspace_init) and is left in a reusable state by every successful call.
 *    Two calls that share a workspace must not overlap on the GPU.
 */
#ifndef MSD_H_
#define MSD_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  MSD_OK = 0,
  MSD_ERR_NULL_POINTER = 1,
  MSD_ERR_BAD_SHAPE = 2,
  MSD_ERR_BAD_ALIGNMENT = 3,
  MSD_ERR_UNSUPPORTED = 4,
  MSD_ERR_WORKSPACE_TOO_SMALL = 5,
  MSD_ERR_CUDA = 6,
  MSD_ERR_TIMEOUT = 7
} msd_status_t;

/* Scaling constants of the two INT8 passes: alpha = max|x| / c1, beta = alpha / c2.
 * DEFAULT: c1 = 127, c2 = 254 (Eq. alpha, Eq. beta).  FRACTIONAL: c1 = 127.49, c2 = 254.98 (Sec. 3.3, "fractional
 * scaling"): the extreme element keeps a residual of 0.49 alpha, the reconstruction bound tightens from max/64516 to
 * max/65015, still no clipping. */
typedef enum { MSD_SCALING_DEFAULT = 0, MSD_SCALING_FRACTIONAL = 1 } msd_scaling_t;

typedef enum { MSD_OUT_BF16 = 0, MSD_OUT_FP32 = 1 } msd_out_t;

const char* msd_status_string(msd_status_t s);

/* Reads and clears the device status word after synchronising `stream`.  Returns MSD_OK, MSD_ERR_TIMEOUT
 * (some kernel gave up on a bounded wait; its outputs are invalid and its workspace must be re-initialised),
 * MSD_ERR_BAD_SHAPE (a kernel found device-side input that contradicts the sizes the call was given) or
 * MSD_ERR_CUDA. */
msd_status_t msd_last_device_status(void* stream);

/* Self-test of the give-up path every device-side wait of this library has: launches a tiny kernel that waits, with
 * the given budget in SM cycles (clamped to [1e3, 2e8]), on a barrier nobody arrives on.  The kernel ends by itself,
 * and the next msd_last_device_status returns MSD_ERR_TIMEOUT; the context stays usable. */
msd_status_t msd_debug_timeout_selftest(int64_t budget_cycles, void* stream);

/* Testing and diagnostic switches.  Each is read from the environment variable of the same name once, when the first
 * call needs one; msd_debug_set_option overrides it afterwards (value -1 = unset), msd_debug_reset_options returns to
 * what the environment says.  Unknown names: MSD_ERR_UNSUPPORTED.  None of them changes results.
 *   MSD_NO_PDL (1: no programmatic dependent launches), MSD_GEMM_MODE / MSD_GEMM_CTAS (work split and CTA count of the
 *   W8A16 decode kernel: 0 stream-K, 1 row bands, 2 clusters), MSD_P8_PAIR / MSD_P8_KSPLIT (W8A16 many-row kernel: CTA
 *   pairs, K split), MSD_W4_PAIR / MSD_W4_TILEN / MSD_W4_KSPLIT (W4A16 kernels), MSD_ATTN_SPLITS / MSD_ATTN_CHUNK_TILES
 *   (context splits of the attention kernels; msd_attn_decode_schedule reports the schedule in force),
 *   MSD_ATTN_BALANCED (1: the balanced split schedule for every shape that has a kernel for it, 0: never; a forced
 *   split count or size switches it off as well). */
msd_status_t msd_debug_set_option(const char* name, int32_t value);
void msd_debug_reset_options(void);

/* Zero-fills a workspace (asynchronous memset on `stream`). */
msd_status_t msd_workspace_init(void* workspace, size_t workspace_bytes, void* stream);

/*
 * Two-pass INT8 decomposition of BF16 rows (Sec. 3.2, Eqs. alpha, x1, residual, beta, x2; Alg. 1 lines 1-5):
 *   alpha_i = max_k |x_ik| / 127,  q1 = clamp(rne(x/alpha), -128, 127),  r = x - alpha*q1 (one FMA, exact),
 *   beta_i = alpha_i / 254,        q2 = clamp(rne(r/beta), -128, 127);   a zero row gives zero scales and codes.
 * All scale arithmetic is IEEE FP32 with true division and round-half-to-even.
 *   x_bf16 [M, ldx] (ldx >= K elements, ldx % 8 == 0), q1/q2 [M, K] INT8, alpha/beta [M] FP32.
 * K % 16 == 0; x_bf16, q1, q2 16-byte aligned.  M = 0 is a no-op.
 */
msd_status_t msd_decompose_int8(const void* x_bf16, int64_t M, int64_t K, int64_t ldx, int8_t* q1, int8_t* q2,
                                float* alpha, float* beta, void* stream);
/* The same with the scaling constants chosen (msd_scaling_t above); anything else: MSD_ERR_UNSUPPORTED. */
msd_status_t msd_decompose_int8_ex(const void* x_bf16, int64_t M, int64_t K, int64_t ldx, int8_t* q1, int8_t* q2,
                                   float* alpha, float* beta, msd_scaling_t scaling, void* stream);

/*
 * Two-pass MXFP4 decomposition per 32-element K block (Sec. 3.2.1, Alg. 2) on the E2M1 grid
 * {0, .5, 1, 1.5, 2, 3, 4, 6} that block-scaled FP4 tensor cores multiply:
 *   alpha = smallest power of two with blockmax <= 4.5*alpha (exponent kept >= -123), q1 = rne_e2m1(x/alpha),
 *   r = x - alpha*q1 (exact), beta = alpha/16, q2 = rne_e2m1(r/beta), both saturating at +-6.
 *   q1/q2 [M, K/2] bytes, element 2i in bits 3:0 and 2i+1 in bits 7:4 (sign in bit 3 of the nibble);
 *   e8m0_1/e8m0_2 [M, K/32] bytes, value 2^(byte-127), row-major.
 * K % 32 == 0; pointers 16-byte aligned; ldx % 8 == 0.
 */
msd_status_t msd_decompose_mxfp4(const void* x_bf16, int64_t M, int64_t K, int64_t ldx, uint8_t* q1, uint8_t* q2,
                                 uint8_t* e8m0_1, uint8_t* e8m0_2, void* stream);

/*
 * W8A16 MSD linear layer (Alg. 1; pass fusion by stacking [X1; X2] along the rows, Sec. 3.9):
 *   y[i,n] = w_scale[n] * (alpha_i * sum_k q1[i,k] w[n,k] + beta_i * sum_k q2[i,k] w[n,k]),
 * the two sums exact in INT32, the combine in FP32.
 *   x_bf16 [M,K]; w [N,K] INT8, K contiguous; w_scale [N] FP32; y [M,N] BF16 or FP32 (ytype);
 *   acc_dbg nullable [2,M,N] INT32 (the two accumulators, for bit-exact checks).
 * K % 16 == 0; N % 8 == 0 when y is BF16; x, w, y 16-byte aligned.  K <= 131072 (beyond that the INT32 sums could
 * overflow: MSD_ERR_UNSUPPORTED).
 * M <= 128 (decode regime): the weight rows sit on the MMA M axis and the weights are streamed once.  M > 128
 * (prefill regime): tiles of 128 tokens x 256 weight rows, both components against the same weight tile, outputs
 * written by TMA stores (N % 4 == 0 also when y is FP32); with few output tiles K is split over the CTAs and the FP32
 * partial results are added in a fixed order (acc_dbg != NULL keeps K unsplit: the accumulators exist only then).
 * workspace: >= msd_gemm_w8a16_workspace_bytes(M,N,K) bytes, 1024-byte aligned.
 */
size_t msd_gemm_w8a16_workspace_bytes(int64_t M, int64_t N, int64_t K);
msd_status_t msd_gemm_w8a16(const void* x_bf16, const int8_t* w, const float* w_scale, int64_t M, int64_t N,
                            int64_t K, void* y, msd_out_t ytype, int32_t* acc_dbg, void* workspace,
                            size_t workspace_bytes, void* stream);
/* The same layer with the scaling constants of the activation decomposition chosen (Sec. 3.3); the weights, the
 * integer GEMM and the combine are unchanged. */
msd_status_t msd_gemm_w8a16_ex(const void* x_bf16, const int8_t* w, const float* w_scale, int64_t M, int64_t N,
                               int64_t K, void* y, msd_out_t ytype, int32_t* acc_dbg, msd_scaling_t scaling,
                               void* workspace, size_t workspace_bytes, void* stream);

/*
 * Grouped W8A16 MSD layer for mixture-of-experts blocks (Discussion, "Extension to MoE and Sparse
 * Architectures": the decomposition works per activation row, so it
 * carries over to grouped matrix multiplication unchanged).  The rows of x are sorted by expert; expert e owns the next
 * group_sizes[e] rows and multiplies them against its own weight:
 *   y[i,:] = msd_gemm_w8a16 row result of x[i,:] with w[e], w_scale[e]   for the rows i of group e.
 *   x_bf16 [M_total, K] (device), w [E, N, K] INT8, w_scale [E, N] FP32, y [M_total, N] (device);
 *   group_sizes_host [E] INT32 in HOST memory, each 0..128 (decode regime per expert), M_total = their sum.
 * Empty groups are skipped (their weights are not read).  One decomposition launch over all rows, then one stream-K
 * GEMM launch per 64 non-empty groups.  K % 16 == 0; N % 8 == 0 when y is BF16; E * N < 2^31.
 * workspace: >= msd_grouped_gemm_w8a16_workspace_bytes(M_total, largest group, E, N, K), 1024-byte aligned, zeroed once
 * (msd_workspace_init); the library leaves its counters zero after every call.
 */
size_t msd_grouped_gemm_w8a16_workspace_bytes(int64_t M_total, int32_t max_group_size, int32_t E, int64_t N, int64_t K);
msd_status_t msd_grouped_gemm_w8a16(const void* x_bf16, const int8_t* w, const float* w_scale, const int32_t* group_sizes_host,
                                    int32_t E, int64_t N, int64_t K, void* y, msd_out_t ytype, void* workspace,
                                    size_t workspace_bytes, void* stream);

/*
 * The same W8A16 layer for callers that cannot allocate device memory.  (The paper has no counterpart; this is a
 * packaging variant of msd_gemm_w8a16, not a step of the method.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits - a plug-in called from inside somebody else's serving
 * loop that forbids allocation on the hot path, a host whose memory pool is owned by another runtime and handed out
 * only as ready-made input/output tensors, or a latency-critical thread that must not take the allocator's lock.
 * Such a caller can still pass inputs and outputs, but has no way to obtain a workspace.  This entry point therefore
 * takes none: its scratch is a fixed array inside the library's device image (3 MB + 1 KB per GPU that loads the
 * library, held until the process exits).  It calls no cudaMalloc / cudaFree and no allocating library routine.
 *
 * Limits: 1 <= M <= 16, N <= 16384, K <= 16384 (and the shape rules of msd_gemm_w8a16); anything larger returns
 * MSD_ERR_UNSUPPORTED before any launch - use msd_gemm_w8a16 with your own workspace instead.
 * First use on a device resolves the array's device address (cudaGetSymbolAddress, with that device current); make
 * that first call outside any stream capture.  All calls on a device share the one array: it still holds the
 * previous call's contents (the parts that must start at zero - the arrival counters, and for shapes that split K
 * over CTAs through memory the meeting place of the partial sums, up to about 2 MB - are cleared on `stream` at the
 * start of every call), and
 * two calls that overlap on the GPU - different streams, or a graph replayed concurrently - race on it.  Results are
 * identical to msd_gemm_w8a16.
 */
msd_status_t msd_gemm_w8a16_noalloc(const void* x_bf16, const int8_t* w, const float* w_scale, int64_t M, int64_t N,
                                    int64_t K, void* y, msd_out_t ytype, void* stream);

/* Diagnostic hook: when `device_buffer` is non-NULL, every later msd_gemm_w8a16 launch writes 16 64-bit SM-clock
 * samples per CTA into it (entry, set-up done, producer / MMA / epilogue milestones); NULL switches it off.
 * The buffer must hold 16 * 8 bytes per SM-count CTA (256 CTAs at most). */
void msd_debug_set_trace(void* device_buffer);
/* Same for msd_attn_decode_int8kv: 32 samples per CTA for the first 1024 CTAs (entry, set-up done, then for the first
 * six tiles: scores ready, P written, O ready, O merged; loop end; exit). */
void msd_debug_set_attn_trace(void* device_buffer);

/* Same computation with the activations and the result in HOST memory (pinned for asynchronous copies):
 * copies x to the device workspace, runs msd_gemm_w8a16, copies y back; weights stay resident on the device.
 * workspace: >= msd_gemm_w8a16_host_workspace_bytes(M,N,K). */
size_t msd_gemm_w8a16_host_workspace_bytes(int64_t M, int64_t N, int64_t K);
msd_status_t msd_gemm_w8a16_host(const void* x_bf16_host, const int8_t* w, const float* w_scale, int64_t M,
                                 int64_t N, int64_t K, void* y_host, msd_out_t ytype, void* workspace,
                                 size_t workspace_bytes, void* stream);

/*
 * Comparison path the method replaces (Sec. 3.1 first equation): weights dequantized to BF16,
 * bf16(w_scale[n]*w[n,k]), then a BF16 x BF16 GEMM with FP32 accumulation.  Same shapes as msd_gemm_w8a16, M > 128
 * included (there K % 64 == 0, and N % 4 == 0 for FP32 output: the same many-row pipeline as msd_gemm_w8a16's, run as a
 * BF16 GEMM).  workspace: >= msd_gemm_dequant_bf16_workspace_bytes(M,N,K) (holds the dequantized weights).
 */
size_t msd_gemm_dequant_bf16_workspace_bytes(int64_t M, int64_t N, int64_t K);
msd_status_t msd_gemm_dequant_bf16(const void* x_bf16, const int8_t* w, const float* w_scale, int64_t M,
                                   int64_t N, int64_t K, void* y, msd_out_t ytype, void* workspace,
                                   size_t workspace_bytes, void* stream);

/*
 * The stronger comparison path: dequantization fused into the GEMM, as weight-only-quantization kernels do it
 * (Sec. 2.3).  The INT8 weights are read once, converted to BF16 inside the kernel (exact) and multiplied against the
 * BF16 activations with FP32 accumulation; the weight scale is applied to the sums:
 *   y[m,n] = w_scale[n] * sum_k x[m,k] * w[n,k].
 * No decomposition, no rounding of the weights: it is more accurate than msd_gemm_dequant_bf16 and moves the same
 * bytes as msd_gemm_w8a16.  Decode regime only: 1 <= M <= 128; K % 64 == 0; N % 8 == 0; pointers as for msd_gemm_w8a16.
 * workspace: >= msd_gemm_w8a16_fused_dequant_workspace_bytes(M,N,K) (FP32 partial results when K is split), 1024-byte
 * aligned, no initialisation needed.  Errors as msd_gemm_w8a16; shapes it cannot stage -> MSD_ERR_UNSUPPORTED.
 */
size_t msd_gemm_w8a16_fused_dequant_workspace_bytes(int64_t M, int64_t N, int64_t K);
msd_status_t msd_gemm_w8a16_fused_dequant(const void* x_bf16, const int8_t* w, const float* w_scale, int64_t M, int64_t N,
                                          int64_t K, void* y, msd_out_t ytype, void* workspace, size_t workspace_bytes,
                                          void* stream);

/*
 * W4A16 MSD linear layer (Alg. 2 + Tab. mxfp4-compute): both MXFP4 components are multiplied against the
 * MXFP4 weight by block-scaled FP4 MMAs accumulating in FP32,
 *   y[i,n] = sum_blocks 2^(e1+ew) <q1,w> + 2^(e2+ew) <q2,w>.
 *   x_bf16 [M,K]; w_fp4 [N,K/2] packed E2M1 (element 2i in bits 3:0); w_e8m0 [N,K/32]; y [M,N].
 * K % 128 == 0, N % 8 == 0; x, w_fp4, y 16-byte aligned, w_e8m0 4-byte aligned.
 */
size_t msd_gemm_w4a16_workspace_bytes(int64_t M, int64_t N, int64_t K);
msd_status_t msd_gemm_w4a16(const void* x_bf16, const uint8_t* w_fp4, const uint8_t* w_e8m0, int64_t M, int64_t N,
                            int64_t K, void* y, msd_out_t ytype, void* workspace, size_t workspace_bytes,
                            void* stream);

/*
 * Grouped W4A16 MSD layer for mixture-of-experts blocks (Discussion, "Extension to MoE and Sparse
 * Architectures"; the decomposition works per 32-element block of an
 * activation row, so it carries over unchanged).  The rows of x are sorted by expert; expert e owns the next
 * group_sizes[e] rows and multiplies them against its own MXFP4 weight:
 *   y[i,:] = msd_gemm_w4a16 row result of x[i,:] with w_fp4[e], w_e8m0[e]   for the rows i of group e.
 *   x_bf16 [M_total, K] (device), w_fp4 [E, N, K/2], w_e8m0 [E, N, K/32], y [M_total, N] (device);
 *   group_sizes_host [E] INT32 in HOST memory, each 0..128 (decode regime per expert), M_total = their sum.
 * Empty groups are skipped (their weights are not read).  Per 64 non-empty groups one decomposition launch (the first
 * also brings every expert's weight scales into the blocked layout) and one GEMM launch in which group g is token tile
 * g.  K % 128 == 0, N % 8 == 0, E * N < 2^31; x, w_fp4, y 16-byte aligned, w_e8m0 4-byte aligned.
 * workspace: >= msd_grouped_gemm_w4a16_workspace_bytes(E, N, K), 1024-byte aligned; no initialisation needed.
 */
size_t msd_grouped_gemm_w4a16_workspace_bytes(int32_t E, int64_t N, int64_t K);
msd_status_t msd_grouped_gemm_w4a16(const void* x_bf16, const uint8_t* w_fp4, const uint8_t* w_e8m0,
                                    const int32_t* group_sizes_host, int32_t E, int64_t N, int64_t K, void* y,
                                    msd_out_t ytype, void* workspace, size_t workspace_bytes, void* stream);

/*
 * Weight scales prepared once.  The block-scaled MMA (Sec. 3.2.1 / Sec. 3.8.3: two FP4 GEMMs with E8M0 block scales)
 * reads the scales of a weight tile as 512-byte blocks of 128 rows x 4 K blocks; msd_gemm_w4a16 and
 * msd_grouped_gemm_w4a16 bring the row-major w_e8m0 into that form on every call.  Weights do not change between calls,
 * so the relayout can be done when they are loaded:
 *   msd_prepare_w4a16_scales: w_e8m0 [E, N, K/32] (device, 4-byte aligned; E = 1 for one matrix) -> prepared (device,
 *     1024-byte aligned, >= msd_w4a16_prepared_scales_bytes(E, N, K) bytes, owned by the caller): the blocked scales
 *     for both tile widths the kernels use, about twice the size of w_e8m0.  Launches on `stream`, does not synchronise.
 *   msd_gemm_w4a16_prepared / msd_grouped_gemm_w4a16_prepared: as the entry points above with `prepared_scales` in the
 *     place of w_e8m0 (same N, K and, for the grouped call, the same E as at preparation); results are bit-identical
 *     to theirs.  Same status codes; a null `prepared_scales` -> MSD_ERR_NULL_POINTER, not 1024-byte aligned ->
 *     MSD_ERR_BAD_ALIGNMENT.
 */
size_t msd_w4a16_prepared_scales_bytes(int32_t E, int64_t N, int64_t K);
msd_status_t msd_prepare_w4a16_scales(const uint8_t* w_e8m0, int32_t E, int64_t N, int64_t K, uint8_t* prepared,
                                      void* stream);
msd_status_t msd_gemm_w4a16_prepared(const void* x_bf16, const uint8_t* w_fp4, const uint8_t* prepared_scales, int64_t M,
                                     int64_t N, int64_t K, void* y, msd_out_t ytype, void* workspace,
                                     size_t workspace_bytes, void* stream);
msd_status_t msd_grouped_gemm_w4a16_prepared(const void* x_bf16, const uint8_t* w_fp4, const uint8_t* prepared_scales,
                                             const int32_t* group_sizes_host, int32_t E, int64_t N, int64_t K, void* y,
                                             msd_out_t ytype, void* workspace, size_t workspace_bytes, void* stream);

/*
 * The paper-literal MXFP4 components (Sec. 3.2.1, Alg. 2; Tab. mxfp4-evolution): both passes round onto the E1M2 grid
 * {0, .25, ..., 1.75}, alpha = 2^ceil(log2(blockmax / 1.859375)) (exponent kept >= -123), beta = alpha / 16, error bound
 * alpha / 64.  Tensor cores have no E1M2 operand type; every E1M2 value is an E4M3 number, so the components are
 * emitted as E4M3 bytes and multiplied with tcgen05.mma kind::mxf8f6f4 (E4M3 x E2M1, block scales) at the FP8 rate.
 *   msd_decompose_mxfp4_e1m2: q1/q2 [M, K] E4M3 bytes, e8m0_1/e8m0_2 [M, K/32] row-major; K % 32 == 0.
 *   msd_gemm_w4a16_e1m2: same arguments and result layout as msd_gemm_w4a16; K % 128 == 0; w_fp4 32-byte aligned,
 *   w_e8m0 4-byte aligned.
 */
msd_status_t msd_decompose_mxfp4_e1m2(const void* x_bf16, int64_t M, int64_t K, int64_t ldx, uint8_t* q1_e4m3, uint8_t* q2_e4m3,
                                      uint8_t* e8m0_1, uint8_t* e8m0_2, void* stream);
size_t msd_gemm_w4a16_e1m2_workspace_bytes(int64_t M, int64_t N, int64_t K);
msd_status_t msd_gemm_w4a16_e1m2(const void* x_bf16, const uint8_t* w_fp4, const uint8_t* w_e8m0, int64_t M, int64_t N,
                                 int64_t K, void* y, msd_out_t ytype, void* workspace, size_t workspace_bytes, void* stream);

/*
 * Decode attention over an INT8 KV cache (Sec. 4, Alg. 3; tiled form Sec. 4.3) with one scale per token per
 * KV head, split over the context (flash-decoding) and merged with the log-sum-exp rule:
 *   Q row decomposed two-pass INT8; S_j = (alpha_Q S1_j + beta_Q S2_j) * k_scale[j] * softmax_scale;
 *   P = exp(S - running max); P~_j = P_j * v_scale[j] decomposed two-pass INT8 with the fixed scale
 *   alpha_P = max(tile's v_scale)/127; O += alpha_P P1 V + beta_P P2 V; O / sum(P) at the end.
 *   q_bf16 [B,Hq,D]; k_cache [T,Hkv,D] INT8; v_cache [T,Hkv,Dv] INT8 or NULL (V = first Dv entries of the K row);
 *   k_scale [T,Hkv] FP32; v_scale [T,Hkv] or NULL (= k_scale); cu_seqlens [B+1] INT32 token offsets (device);
 *   total_tokens = T, the number of token rows the caches hold (>= cu_seqlens[B]); max_seqlen >= every length;
 *   out_bf16 [B,Hq,Dv]; lse nullable [B,Hq] FP32 (natural-log sum of exp of the scaled scores).
 * Hq % Hkv == 0; D % 16 == 0, D <= 640; Dv % 16 == 0, Dv <= 512; Dv <= D when v_cache is NULL.
 * Empty sequences give zeros and lse = -inf.  A sequence longer than max_seqlen: tokens past max_seqlen may be left
 * out, and msd_last_device_status may report MSD_ERR_BAD_SHAPE (the workspace has no room for that sequence's partial
 * results; nothing is written outside it).
 */
size_t msd_attn_decode_int8kv_workspace_bytes(int32_t B, int32_t Hq, int32_t Hkv, int32_t D, int32_t Dv,
                                              int32_t max_seqlen);
msd_status_t msd_attn_decode_int8kv(const void* q_bf16, const int8_t* k_cache, const int8_t* v_cache,
                                    const float* k_scale, const float* v_scale, const int32_t* cu_seqlens,
                                    int64_t total_tokens, int32_t max_seqlen, int32_t B, int32_t Hq, int32_t Hkv, int32_t D, int32_t Dv,
                                    float softmax_scale, void* out_bf16, float* lse, void* workspace,
                                    size_t workspace_bytes, void* stream);

/*
 * The same attention with q_len query tokens per sequence (speculative / multi-token decode, Sec. 4.4: the stacked
 * query operand then has 2 * q_len * G rows per KV head).  The q_len tokens are the LAST q_len tokens of each sequence's
 * cache: query token s (0-based) attends to positions [0, L - q_len + s].  Every sequence must hold at least q_len
 * tokens.  q_bf16 [B, q_len, Hq, D]; out_bf16 [B, q_len, Hq, Dv]; lse nullable [B, q_len, Hq]; 1 <= q_len <= 64.
 * Workspace: msd_attn_decode_int8kv_workspace_bytes called with Hq * q_len in place of Hq; the schedule likewise.
 */
msd_status_t msd_attn_decode_int8kv_spec(const void* q_bf16, const int8_t* k_cache, const int8_t* v_cache,
                                         const float* k_scale, const float* v_scale, const int32_t* cu_seqlens,
                                         int64_t total_tokens, int32_t max_seqlen, int32_t B, int32_t q_len, int32_t Hq, int32_t Hkv,
                                         int32_t D, int32_t Dv, float softmax_scale, void* out_bf16, float* lse, void* workspace,
                                         size_t workspace_bytes, void* stream);

/*
 * The same attention over a PAGED cache (serving layouts; the paper's kernels read a contiguous cache, Alg. 3):
 *   k_cache [num_blocks * page_size, Hkv, D], v_cache [num_blocks * page_size, Hkv, Dv] or NULL, scales
 *   [num_blocks * page_size, Hkv]; block_table [B, max_blocks_per_seq] INT32 (device): logical token u of sequence b
 *   is row block_table[b][u / page_size] * page_size + u % page_size; seqlens [B] INT32 (device).
 * page_size: a power of two from 8 to 128.  Entries of block_table past ceil(seqlens[b] / page_size) are never read.
 * max_seqlen >= every seqlens[b] and <= max_blocks_per_seq * page_size.  Workspace, schedule, outputs and errors as for
 * msd_attn_decode_int8kv (same max_seqlen); an unsupported page size returns MSD_ERR_UNSUPPORTED.
 */
msd_status_t msd_attn_decode_int8kv_paged(const void* q_bf16, const int8_t* k_cache, const int8_t* v_cache,
                                          const float* k_scale, const float* v_scale, const int32_t* block_table,
                                          const int32_t* seqlens, int64_t num_blocks, int32_t page_size,
                                          int32_t max_blocks_per_seq, int32_t max_seqlen, int32_t B, int32_t Hq, int32_t Hkv,
                                          int32_t D, int32_t Dv, float softmax_scale, void* out_bf16, float* lse,
                                          void* workspace, size_t workspace_bytes, void* stream);

/* The split schedule msd_attn_decode_int8kv uses (so a checker can mirror it): writes the tile size, the largest
 * number of context splits a (sequence, query row) can have and the tokens per split.  With *split_tokens > 0 split s
 * of a sequence of length L covers tokens [s*split_tokens, min(L, (s+1)*split_tokens)) and is walked in tiles of
 * `tile` tokens (splits past L are empty).  *split_tokens = 0: the splits depend on the lengths of all sequences of
 * the call (Sec. 4.3 leaves the partition of the context open; head groups of up to 8 rows per KV head may cut the list
 * of all sequences' tiles into equal runs, as many as fit the machine at once, so that no SM is left with more work
 * than another) - msd_attn_decode_split_starts lists them. */
msd_status_t msd_attn_decode_schedule(int32_t B, int32_t Hq, int32_t Hkv, int32_t D, int32_t Dv, int32_t max_seqlen,
                                      int32_t* tile, int32_t* n_splits, int32_t* split_tokens);

/* The context splits of one call, for a checker (host arithmetic; needs the CUDA device only to ask how many CTAs of
 * the kernel are resident at once).  seqlens: HOST, [B] tokens per sequence (as the call's cu_seqlens / seqlens say).
 * q_len, Hq as for msd_attn_decode_int8kv_spec (q_len = 1 otherwise); paged / v_aliased: non-zero for a paged cache /
 * for v_cache == NULL.  starts: HOST, written, [B][Hkv][q_len * Hq / Hkv][n_splits + 1] INT32 with n_splits as
 * msd_attn_decode_schedule(B, q_len * Hq, ...) reports it: row r of a KV head (query token r / (Hq / Hkv), head
 * r % (Hq / Hkv) of the group) of sequence b has its split s over tokens [starts[..][s], starts[..][s + 1]) of the
 * sequence; every start is a multiple of the tile; trailing entries repeat the length (empty splits).  The partial
 * results are merged in this order.  Errors: MSD_ERR_NULL_POINTER, MSD_ERR_BAD_SHAPE, MSD_ERR_CUDA. */
msd_status_t msd_attn_decode_split_starts(int32_t B, int32_t q_len, int32_t Hq, int32_t Hkv, int32_t D, int32_t Dv,
                                          int32_t max_seqlen, int32_t paged, int32_t v_aliased, const int32_t* seqlens,
                                          int32_t* starts);

/* The same arithmetic with the number of resident CTAs given instead of asked of the device (no CUDA call at all: for
 * tests of the schedule on a host without a GPU).  resident_ctas >= 1, otherwise MSD_ERR_BAD_SHAPE. */
msd_status_t msd_debug_attn_split_starts(int32_t B, int32_t q_len, int32_t Hq, int32_t Hkv, int32_t D, int32_t Dv,
                                         int32_t max_seqlen, int32_t v_aliased, int32_t resident_ctas, const int32_t* seqlens,
                                         int32_t* starts);

/* The softmax references of the kernel that msd_attn_decode_int8kv (and _spec, _paged) runs for this shape, for a
 * checker that mirrors it (Sec. 4.3; Alg. 3 lines 6-8).  Head groups of up to 8 rows per KV head: *m_margin = 0,
 * *sv_growth = 0 - the running maximum itself and alpha_P = (the tile's largest v_scale) / 127.  Wider groups keep the
 * integer PV sums of consecutive tiles in one accumulator, so their references are held: per context split the
 * reference of a row moves only when a tile's maximum exceeds it, to that maximum + *m_margin (natural-log units), and
 * alpha_P = a_ref / 127 where a_ref is set to *sv_growth times the tile's largest v_scale whenever one exceeds it. */
msd_status_t msd_attn_decode_softmax_rule(int32_t B, int32_t Hq, int32_t Hkv, int32_t D, int32_t Dv, int32_t max_seqlen,
                                          float* m_margin, float* sv_growth);

/* Debug dumps for bit-exact checks of Alg. 3 lines 1-4.  While a pointer is non-NULL every later attention launch
 * writes: q_dbg [2, R, D] INT8, the two components of each query row (R = B * q_len * Hq rows in the order of q_bf16);
 * q_scale_dbg [2, R] FP32, alpha_Q then beta_Q; s_dbg [2, q_len * Hq, T] INT32, the raw sums S1, S2 of row (token s,
 * head h) -> s * Hq + h against cache row t (T = total_tokens; paged: T = num_blocks * page_size, t the physical row),
 * written for every token of the sequences, visible to the row or not.  NULL switches a dump off. */
void msd_debug_set_attn_dump(int8_t* q_dbg, float* q_scale_dbg, int32_t* s_dbg);

/* Comparison kernel, not part of the MSD path: the cache expansion that MSD attention removes (Sec. 2.3; the
 * "Dequant" arm of Sec. 6.4).  out[t,h,:] = bf16(scale[t,h] * cache[t,h,:]), FP32 product rounded to nearest even.
 * cache [T,H,D] INT8, scale [T,H] FP32, out [T,H,D] BF16, all device pointers; cache and out 16-byte aligned;
 * D % 16 == 0.  T = 0 is a no-op.  A BF16 attention kernel reading `out` completes the comparison arm. */
msd_status_t msd_kv_dequant_bf16(const int8_t* cache, const float* scale, int64_t T, int32_t H, int32_t D,
                                 void* out_bf16, void* stream);

/* Comparison kernel, not part of the MSD path: decode attention over a BF16 KV cache, the second half of the "Dequant"
 * arm of Sec. 6.4 (msd_kv_dequant_bf16 is the first).  out = softmax(softmax_scale * Q K^T) V per sequence and head
 * with Q, K, V and the probabilities as BF16 tensor-core operands and FP32 accumulation, split over the context and
 * merged like msd_attn_decode_int8kv; no decomposition anywhere.
 *   q_bf16 [B,Hq,D], k_bf16 [T,Hkv,D], v_bf16 [T,Hkv,Dv] BF16, 16-byte aligned; cu_seqlens [B+1] INT32 token offsets
 *   (device); total_tokens = T; max_seqlen >= every length; out_bf16 [B,Hq,Dv]; lse nullable [B,Hq] FP32.
 * Shapes: D = 64 or 128, Dv = 128, Hq % Hkv == 0, Hq / Hkv <= 16; anything else: MSD_ERR_UNSUPPORTED.  Workspace:
 * msd_attn_decode_bf16kv_workspace_bytes (0 for a shape it does not take), 1024-byte aligned, no initialisation.
 * Errors as msd_attn_decode_int8kv; empty sequences give zeros and lse = -inf. */
size_t msd_attn_decode_bf16kv_workspace_bytes(int32_t B, int32_t Hq, int32_t Hkv, int32_t D, int32_t Dv, int32_t max_seqlen);
msd_status_t msd_attn_decode_bf16kv(const void* q_bf16, const void* k_bf16, const void* v_bf16, const int32_t* cu_seqlens,
                                    int64_t total_tokens, int32_t max_seqlen, int32_t B, int32_t Hq, int32_t Hkv, int32_t D,
                                    int32_t Dv, float softmax_scale, void* out_bf16, float* lse, void* workspace,
                                    size_t workspace_bytes, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* MSD_H_ */
