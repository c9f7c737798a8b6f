/*
 * lowra.h -- C ABI of the B200 (sm_100a) hot path of LowRA's quantized-LoRA linear layer.
 *
 * Data model (paper Section 4.1): a frozen base weight W [N, K] (N output channels = rows,
 * K input features) is quantised per output channel: row r has its own precision
 * b_r in {1, 2, 4} bits ("Per-Output-Channel Quantization"), its own 2^b_r mapping values and
 * its own 2^b_r - 1 sorted thresholds ("Per-Output-Channel Thresholds and Mappings"), and is
 * normalised in blocks of 64 consecutive elements by the block's maximum magnitude
 * ("Groupwise Normalization").  The quantised state is: the per-row precisions (`Precs` in
 * Appendix A), the packed codes, one fp32 absmax per 64-block, the mapping table and the
 * threshold table.
 *
 * Storage order: rows are grouped by precision (all 1-bit rows, then 2-bit, then 4-bit),
 * ascending original index inside a group.  `perm[p]` is the original row of stored row p.
 * Stored row p of class c (bits b) with rank q inside its class starts at byte
 *     seg_off[c] + q * K * b / 8
 * of the packed buffer; element k of the row occupies bits [k*b, k*b + b) of the row's
 * little-endian bitstream (bit i of the stream = bit (i % 8) of byte i / 8).  No padding:
 * packed_bytes = K * (n_1 + 2 n_2 + 4 n_4) / 8.
 *
 * Tables: `maps` and `thresholds` are fp32 [N, 16], row r = original row r, first 2^b (resp.
 * 2^b - 1) entries valid.  `absmax` is fp32 [N, K / 64] in STORED row order.
 *
 * Conventions for every call:
 *   - pointers named *_dev are DEVICE pointers owned by the caller, 16-byte aligned; pointers
 *     named *_host are host pointers; the library never allocates, frees or synchronises
 *     (except lowra_device_status, which synchronises the given stream);
 *   - work is enqueued on `stream` (a cudaStream_t passed as void*; NULL = default stream);
 *   - the return value is a lowra_status; arguments are validated on the host before any launch;
 *   - inputs are read-only, outputs are fully overwritten;
 *   - there is no CPU fallback: on a device that is not sm_100 the calls return LOWRA_ERR_ARCH.
 * Not checked on the device (preconditions): precisions in {1,2,4}, thresholds non-decreasing in
 * their valid prefix, finite weights.
 */
#ifndef LOWRA_H
#define LOWRA_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    LOWRA_OK = 0,
    LOWRA_ERR_NULL = 1,      /* a required pointer is NULL */
    LOWRA_ERR_SHAPE = 2,     /* N < 1, K % 128 != 0, block != 64, M < 1, r not in {16,32,...,128} */
    LOWRA_ERR_ALIGN = 3,     /* a device pointer is not 16-byte aligned */
    LOWRA_ERR_PREC = 4,      /* a precision outside {1,2,4}, or counts that do not sum to N */
    LOWRA_ERR_WORKSPACE = 5, /* workspace smaller than lowra_workspace_bytes() */
    LOWRA_ERR_CUDA = 6,      /* a CUDA runtime / driver call failed */
    LOWRA_ERR_TIMEOUT = 7,   /* a bounded device-side wait ran out (read via lowra_device_status) */
    LOWRA_ERR_ARCH = 8,      /* current device is not compute capability 10.x */
    LOWRA_ERR_LIMIT = 9      /* problem larger than the built-in scratch of lowra_lora_forward_static */
} lowra_status;

const char* lowra_status_string(lowra_status st);

/* Immutable description of one quantised weight (host struct, device arrays inside). */
typedef struct {
    int32_t N, K, block;         /* block must be 64; K % 128 == 0; N >= 1 */
    int32_t counts[3];           /* rows with 1, 2, 4 bits */
    uint64_t seg_off[3];         /* byte offset of each precision class in the packed buffer */
    uint64_t packed_bytes;
    const uint8_t* precs_dev;    /* [N] bits per row, original order */
    const int32_t* perm_dev;     /* [N] stored position -> original row */
    const int32_t* inv_perm_dev; /* [N] original row -> stored position */
    const void* deal_dev;        /* NULL, or what lowra_deal_build wrote for this weight (see there) */
    const uint64_t* natural_offsets_dev;   /* NULL: packed codes and absmax rows in the grouped order described above.
                                    Otherwise [N + 1] byte offsets (a device copy of what lowra_natural_offsets
                                    writes): the packed buffer and the absmax rows are in the paper's own order
                                    (Appendix A.2) - rows in their ORIGINAL order, row r at byte natural_offsets[r],
                                    absmax row r = original row r - and every call that takes this layout (encode,
                                    decode, deal_build, forward, backward-input) reads or writes that buffer directly */
} lowra_layout;

/*
 * Storage planner (host only; Appendix A.1: packed rows are written "at the appropriate offset",
 * A.2: the offset follows from the channel's bit precision).  Reads precs_host[N]; writes
 * perm_host[N], inv_perm_host[N], counts[3], seg_off[3], *packed_bytes.  The caller uploads
 * perm / inv_perm / precs and fills a lowra_layout.
 * Errors: NULL pointer -> ERR_NULL; N < 1 or K % 128 != 0 -> ERR_SHAPE; bad precision -> ERR_PREC.
 */
lowra_status lowra_plan(int32_t N, int32_t K, const uint8_t* precs_host, int32_t* perm_host,
                        int32_t* inv_perm_host, int32_t counts[3], uint64_t seg_off[3],
                        uint64_t* packed_bytes);

/*
 * Quantize (Appendix A.1): for each 64-block of W compute the maximum magnitude and store it;
 * normalise each value with it (n = x * fl(1/absmax) in fp32, n = 0 for an all-zero block);
 * quantise n with the row's thresholds at the row's precision
 * (code = number of valid thresholds <= n, so a value on a threshold takes the upper bucket);
 * pack the codes and write them at the row's offset.
 *   W_dev          fp32 [N, K] row-major, original row order          (in)
 *   thresholds_dev fp32 [N, 16], original row order                   (in)
 *   packed_dev     uint8 [layout->packed_bytes]                       (out)
 *   absmax_dev     fp32 [N, K/64], stored row order                   (out)
 */
lowra_status lowra_encode(const lowra_layout* layout, const float* W_dev, const float* thresholds_dev,
                          uint8_t* packed_dev, float* absmax_dev, void* stream);

/*
 * Dequantize (Appendix A.2): unpack each row's 1/2/4-bit codes, look them up in the row's mapping
 * table, multiply by the block's absmax in fp32 and round to bf16 (nearest even).
 *   W_bf16_dev     bf16 bit patterns [N, K] row-major, original row order, 32-byte aligned   (out)
 */
lowra_status lowra_decode(const lowra_layout* layout, const uint8_t* packed_dev, const float* absmax_dev,
                          const float* maps_dev, uint16_t* W_bf16_dev, void* stream);

/*
 * Several matrices per launch (no counterpart in the paper; Appendix A.1 / A.2 describe one matrix): the weights of a
 * layer, or of a model, are quantised and dequantised together, and a launch per matrix spends a good part of a small
 * matrix's time (a 4096 x 4096 decode is 7 us of work) filling and draining the GPU.  lowra_encode_group and
 * lowra_decode_group hand the chunks of up to LOWRA_MAX_GROUP matrices - any shapes, any layouts - to the warps of ONE
 * launch, matrix after matrix in the order given (put the largest first).  Every member's result is bit for bit what the
 * single call gives.  The array of members is host memory and is read before the call returns; the pointers inside it
 * are device pointers with the meaning, layout and alignment of the arguments of lowra_encode / lowra_decode:
 *   encode: W_dev, tables_dev = thresholds (in);  packed_dev, absmax_dev (out);  W_bf16_dev unused
 *   decode: packed_dev, absmax_dev, tables_dev = mappings (in);  W_bf16_dev (out);  W_dev unused
 * Errors: as the single calls, for the first member that is at fault; count < 1 or > LOWRA_MAX_GROUP -> LOWRA_ERR_SHAPE.
 */
#define LOWRA_MAX_GROUP 8
typedef struct lowra_group_member {
    const lowra_layout* layout;
    const float* W_dev;
    const float* tables_dev;
    uint8_t* packed_dev;
    float* absmax_dev;
    uint16_t* W_bf16_dev;
} lowra_group_member;
lowra_status lowra_encode_group(const lowra_group_member* members_host, int32_t count, void* stream);
lowra_status lowra_decode_group(const lowra_group_member* members_host, int32_t count, void* stream);

/*
 * The paper's own buffer layout as a second storage variant (Appendix A.2: a thread of the
 * dequantisation kernel finds its offset into the quantised buffer from the channels' bit precisions):
 * rows in their ORIGINAL order, row r at byte offset sum_{i<r} K * b_i / 8; the absmax rows in original
 * order too.  A row's bytes are the same in both layouts, so converting is a row permutation.
 *
 * lowra_natural_offsets (host only): offsets_host[N + 1] from precs_host[N]; offsets_host[N] is the
 * buffer size (= the grouped layout's packed_bytes).  Errors as lowra_plan.
 *
 * Nothing has to be converted to use such a buffer: point layout->natural_offsets_dev at the offsets and every kernel
 * finds a row at its offset there (the perm / inv_perm / counts of the layout are still needed: work is still handed
 * out precision by precision).  lowra_reorder_rows converts an existing buffer from one order to the other:
 *
 * lowra_reorder_rows: to_natural != 0: grouped -> natural; to_natural == 0: natural -> grouped.
 *   offsets_dev     uint64 [N + 1], device copy of the offsets above                        (in)
 *   packed_src_dev  uint8 [packed_bytes], absmax_src_dev fp32 [N, K/64] in the source order (in)
 *   packed_dst_dev, absmax_dst_dev: the same in the destination order; not in place          (out)
 * Errors: as lowra_encode; source == destination -> LOWRA_ERR_SHAPE.
 */
lowra_status lowra_natural_offsets(int32_t N, int32_t K, const uint8_t* precs_host, uint64_t* offsets_host);
lowra_status lowra_reorder_rows(const lowra_layout* layout, int32_t to_natural, const uint64_t* offsets_dev,
                                const uint8_t* packed_src_dev, const float* absmax_src_dev,
                                uint8_t* packed_dst_dev, float* absmax_dst_dev, void* stream);

/*
 * Quantisation error per output channel (Section 5 and its footnote: the precision assigner minimises
 * the summed square error, SSE = sum_k (W[i,k] - W_hat[i,k])^2; Section 5.1 starts from every channel's
 * error under 1, 2 and 4 bits) and, optionally, the residual W - W_hat that an iterative low-rank
 * initialiser decomposes after quantising (appendix on the low-rank initialisers).  One fused pass
 * over W: W_hat is exactly what lowra_encode followed by lowra_decode gives for this layout and these
 * tables (bf16), but neither codes nor W_hat are written.
 *   W_dev          fp32 [N, K] row-major, original row order                        (in)
 *   maps_dev, thresholds_dev   fp32 [N, 16], original row order                     (in)
 *   sse_dev        fp64 [N], original row order: sum of the squared fp32 residuals (four at a time in
 *                  fp32, those partial sums in fp64, fixed order; within 2^-21 relative of the
 *                  exact sum)                                                       (out)
 *   residual_dev   fp32 [N, K] = fl32(W - W_hat), or NULL to skip it                (out)
 * For the error of every channel under each precision, call it once per uniform layout.
 * Errors: as lowra_encode.
 */
lowra_status lowra_quant_error(const lowra_layout* layout, const float* W_dev, const float* maps_dev,
                               const float* thresholds_dev, double* sse_dev, float* residual_dev,
                               void* stream);

/*
 * The same error for every channel under 1, 2 and 4 bits in one pass over W (Section 5.1, step 1: each
 * channel's error under 1-, 2- and 4-bit quantisation is what the channels are clustered by).  No
 * layout: every row is quantised three times, with its own three codebooks.
 *   W_dev            fp32 [N, K] row-major, K % 128 == 0                                        (in)
 *   maps3_dev, thresholds3_dev   fp32 [3][N][16]: plane 0 = the 1-bit tables of every row, plane 1 =
 *                    the 2-bit tables, plane 2 = the 4-bit tables (as lowra_learn_codebooks writes them
 *                    for a layout in which every row has that precision)                       (in)
 *   sse3_dev         fp64 [N][3], the three errors of a row side by side; arithmetic and accuracy as
 *                    lowra_quant_error                                                          (out)
 */
lowra_status lowra_channel_errors(int32_t N, int32_t K, const float* W_dev, const float* maps3_dev,
                                  const float* thresholds3_dev, double* sse3_dev, void* stream);

/* Bytes of device scratch that lowra_lora_forward / lowra_lora_backward_input need for M tokens and
 * LoRA rank r (0 if the arguments are invalid).  The first 256 bytes hold the device status word; the
 * rest: the down-projected activations, flags, the deal of the rows to the dequant warps and 19 MB for
 * the fp32 partial tiles that tiles cut between SMs are handed over in (about 21 MB for a 4096 x 11008
 * matrix at 4096 tokens). */
size_t lowra_workspace_bytes(const lowra_layout* layout, int32_t M, int32_t r);

/*
 * Once per weight instead of once per call (no counterpart in the paper; like the storage planner it depends
 * on the channels' precisions only).  The fused calls below hand the rows of every group of channels to their
 * dequantising warps sorted by precision.  With layout->deal_dev == NULL every call works that out again in
 * a small prologue launch, which also clears the status word and the flags in the workspace.  With
 * layout->deal_dev pointing at a buffer filled by lowra_deal_build the fused kernel is the only launch
 * of a call (3-6 us less per call on a B200); the workspace then has to be initialised once with
 * lowra_workspace_init before its first use, is written by these calls only, and its status word is no
 * longer cleared per call: lowra_device_status reports the first failure since the initialisation.
 *   lowra_deal_bytes   size of the buffer for this layout (0 if the layout is invalid); about 40 bytes per
 *                      channel (0.44 MB for 11008 channels)
 *   lowra_deal_build   fills deal_dev (256-byte aligned, >= lowra_deal_bytes(layout) bytes) for both the
 *                      forward and the backward-input call; reads layout->precs_dev / inv_perm_dev and
 *                      ignores layout->deal_dev.  The buffer is read-only afterwards and may serve any
 *                      number of calls, streams and workspaces.
 *   lowra_workspace_init   zero-fills the workspace (status word, call numbering, flags).
 * Errors: as lowra_lora_forward; LOWRA_ERR_WORKSPACE for a buffer that is too small or not 256-byte aligned
 * (lowra_deal_build: LOWRA_ERR_ALIGN for the alignment).
 */
size_t lowra_deal_bytes(const lowra_layout* layout);
lowra_status lowra_deal_build(const lowra_layout* layout, void* deal_dev, size_t deal_bytes, void* stream);
lowra_status lowra_workspace_init(void* workspace_dev, size_t workspace_bytes, void* stream);

/*
 * Forward of the quantized-LoRA linear layer (Section 3: the fine-tuning module recovers the base
 * weights with the dequantize kernel; frozen base plus trainable low-rank factors):
 *     Y = X . deq(Wq)^T + s * (X . A) . B
 * deq(Wq) is exactly what lowra_decode produces, formed on the fly in the operand stage of the
 * tensor-core contraction and never written to memory.  fp32 accumulation, bf16 output.
 *   X_dev bf16 [M, K];  A_dev bf16 [K, r];  B_dev bf16 [r, N];  Y_dev bf16 [M, N], original
 *   channel order; all row-major.  r in {16, 32, ..., 128}.  X . A is rounded to bf16 once.
 *   workspace_dev: >= lowra_workspace_bytes(layout, M, r) bytes, 256-byte aligned, contents
 *   overwritten.  Calls that share a workspace must not overlap on the device; and a call must have the
 *   device's SMs to itself while it runs: its grid is persistent (one CTA per SM) and its CTAs wait for one
 *   another, so they all have to be resident - do not run another kernel beside it on a second stream (the
 *   call would sit in its bounded waits and end with LOWRA_ERR_TIMEOUT).  With
 *   layout->deal_dev set: initialised by lowra_workspace_init and since then written by these calls only
 *   (any mix of forward / backward-input, weights and token counts).
 *   Limits (LOWRA_ERR_SHAPE otherwise): N % 8 == 0, N <= 524288, N * K / 64 < 2^32, M >= 1.
 */
lowra_status lowra_lora_forward(const lowra_layout* layout, const uint8_t* packed_dev,
                                const float* absmax_dev, const float* maps_dev, const uint16_t* X_dev,
                                int32_t M, const uint16_t* A_dev, const uint16_t* B_dev, int32_t r,
                                float s, uint16_t* Y_dev, void* workspace_dev, size_t workspace_bytes,
                                void* stream);

/*
 * Input gradient of the same layer (the base weights are frozen, Section 3, so the only gradient
 * through the quantised weight is the one with respect to the input):
 *     dX = dY . deq(Wq) + s * (dY . B^T) . A^T
 *   dY_dev bf16 [M, N];  dX_dev bf16 [M, K];  other arguments as in lowra_lora_forward.
 */
lowra_status lowra_lora_backward_input(const lowra_layout* layout, const uint8_t* packed_dev,
                                       const float* absmax_dev, const float* maps_dev,
                                       const uint16_t* dY_dev, int32_t M, const uint16_t* A_dev,
                                       const uint16_t* B_dev, int32_t r, float s, uint16_t* dX_dev,
                                       void* workspace_dev, size_t workspace_bytes, void* stream);

/*
 * (No counterpart in the paper: a packaging of the two calls above.)  Several weights of ONE shape in one launch -
 * the q, k and v projections of a layer, its gate and up projections - each with its own quantised state, low-rank
 * factors, input and output:
 *     forward:         Y_i  = X_i  . deq(Wq_i)^T + s * (X_i . A_i) . B_i
 *     backward-input:  dX_i = dY_i . deq(Wq_i)   + s * (dY_i . B_i^T) . A_i^T          i = 0 .. count - 1
 * The results are bit for bit those of `count` single calls.  What is saved is what a call costs beside its tiles:
 * the launch, the pipeline's fill and drain, the wait for the first down-projected tile and the ragged last row of
 * tiles are paid once for the group instead of once per weight (on a B200 about 12 us per weight left out; a
 * 4096 x 4096 call at 4096 tokens takes 155 us).  Members may share an input (q, k, v read the same X).
 *   members_host   HOST array of `count` members, 1 <= count <= LOWRA_MAX_BATCH; every layout has the same N
 *                  and K and carries a deal (layout->deal_dev, see lowra_deal_build); act_dev is X [M, K] (forward)
 *                  or dY [M, N] (backward-input), out_dev is Y [M, N] or dX [M, K]
 *   workspace_dev  >= lowra_batch_workspace_bytes(layout, count, M, r) bytes, 256-byte aligned, initialised once with
 *                  lowra_workspace_init; rules as for lowra_lora_forward
 * Errors: as lowra_lora_forward; count out of range or members of different shapes -> LOWRA_ERR_SHAPE; a member
 * without a deal -> LOWRA_ERR_NULL.
 */
#define LOWRA_MAX_BATCH 4
typedef struct {
    const lowra_layout* layout;
    const uint8_t* packed_dev;
    const float* absmax_dev;
    const float* maps_dev;
    const uint16_t* act_dev;
    const uint16_t* A_dev;
    const uint16_t* B_dev;
    uint16_t* out_dev;
} lowra_member;
size_t lowra_batch_workspace_bytes(const lowra_layout* layout, int32_t count, int32_t M, int32_t r);
lowra_status lowra_lora_forward_batch(const lowra_member* members_host, int32_t count, int32_t M, int32_t r, float s,
                                      void* workspace_dev, size_t workspace_bytes, void* stream);
lowra_status lowra_lora_backward_input_batch(const lowra_member* members_host, int32_t count, int32_t M, int32_t r,
                                             float s, void* workspace_dev, size_t workspace_bytes, void* stream);

/*
 * Forward pass for several adapters that share one quantised base weight (Section 4.1, "Adapting LowRA to Production
 * Use Cases": the thresholds are shared, so there is one packed buffer, and every adapter brings its own mapping
 * table and its own low-rank factors).  The tokens of the batch are sorted by adapter: adapter a owns the token rows
 * [group_start_host[a], group_start_host[a + 1]) of X and Y, and for those rows
 *     Y = X . deq_a(Wq)^T + s * (X . A_a) . B_a
 * with deq_a the dequantisation through adapter a's mappings.  One call routes every group to its tables.  Up to
 * LOWRA_MAX_BATCH groups run in one fused launch (their tiles dealt to the SMs together, so that small groups fill the
 * GPU between them) when the layout carries a deal and the workspace has lowra_batch_workspace_bytes(layout,
 * LOWRA_MAX_BATCH, M, r) bytes; otherwise every group is a launch of its own.  A dequantised weight tile depends on
 * the adapter's mappings, so groups never share tiles; empty groups are skipped.
 *   maps_dev         fp32 [n_adapters][N][16]
 *   A_dev            bf16 [n_adapters][K][r];   B_dev  bf16 [n_adapters][r][N]
 *   group_start_host int32 [n_adapters + 1], HOST, non-decreasing, [0] = 0, [n_adapters] = M
 *   X_dev bf16 [M, K];  Y_dev bf16 [M, N];  workspace_dev: at least as lowra_lora_forward for M tokens (see above);
 *   with a deal in the layout, initialised by lowra_workspace_init.
 * Errors: as lowra_lora_forward; n_adapters < 1 or group_start_host not as described -> LOWRA_ERR_SHAPE.
 */
lowra_status lowra_lora_forward_adapters(const lowra_layout* layout, const uint8_t* packed_dev, const float* absmax_dev,
                                         const float* maps_dev, int32_t n_adapters, const uint16_t* X_dev, int32_t M,
                                         const int32_t* group_start_host, const uint16_t* A_dev, const uint16_t* B_dev,
                                         int32_t r, float s, uint16_t* Y_dev, void* workspace_dev, size_t workspace_bytes,
                                         void* stream);

/* Bytes of device scratch that lowra_lora_backward_adapters needs for M tokens and rank r (0 if the
 * arguments are invalid).  The first 256 bytes hold the device status word. */
size_t lowra_adapter_workspace_bytes(int32_t M, int32_t r);

/*
 * Gradients of the trainable low-rank factors of the same layer (Section 3: the base weights stay
 * frozen, only the adapters are trained).  With Y = X . deq(Wq)^T + s * (X . A) . B:
 *     dA = s * X^T . (dY . B^T)      [K, r]
 *     dB = s * (X . A)^T . dY        [r, N]
 * The quantised weight does not enter.  The two down-projections s X A and s dY B^T are rounded to
 * bf16 once (as in the forward / backward-input calls), the contractions over the tokens accumulate
 * in fp32, the results are rounded to bf16.
 *   X_dev bf16 [M, K];  dY_dev bf16 [M, N];  A_dev bf16 [K, r];  B_dev bf16 [r, N];
 *   dA_dev bf16 [K, r] (out);  dB_dev bf16 [r, N] (out); all row-major, device, 16-byte aligned.
 *   r in {16, 32, ..., 128};  K % 8 == 0, N % 8 == 0, M >= 1 (LOWRA_ERR_SHAPE otherwise).
 *   workspace_dev: >= lowra_adapter_workspace_bytes(M, r) bytes, 256-byte aligned, contents
 *   overwritten; lowra_device_status reads its status word.
 */
lowra_status lowra_lora_backward_adapters(const uint16_t* X_dev, const uint16_t* dY_dev, int32_t M,
                                          int32_t K, int32_t N, const uint16_t* A_dev,
                                          const uint16_t* B_dev, int32_t r, float s, uint16_t* dA_dev,
                                          uint16_t* dB_dev, void* workspace_dev, size_t workspace_bytes,
                                          void* stream);

/*
 * The same gradients from the down-projections that the two calls above have already formed (Section 3: forward and
 * backward of the layer come before the factors' gradients in a training step): lowra_lora_forward leaves
 * T = bf16(s X A) in its workspace, lowra_lora_backward_input leaves U = bf16(s dY B^T) in its own, both [M, rp] with
 * rp = r rounded up to 64.  With them only dA = X^T U and dB = T^T dY remain: X and dY are read once instead of twice
 * and two of the four products fall away.
 *   lowra_workspace_projection  device pointer to that matrix inside a workspace of the fused calls (member: 0 for the
 *                               plain calls, the member's index for the batch calls); valid from the moment that call
 *                               has run (stream order) until the next call on the same workspace - so forward and
 *                               backward-input need a workspace each for both to survive.  NULL for invalid arguments.
 *   T_dev, U_dev                bf16 [M, rp] as above (any device memory: the caller may also keep copies)
 *   workspace_dev               256-byte aligned, >= 256 bytes (status word only)
 * Other arguments, limits and errors as lowra_lora_backward_adapters; A, B and s are not needed (T and U carry them).
 */
const uint16_t* lowra_workspace_projection(const void* workspace_dev, int32_t member, int32_t M, int32_t r);
lowra_status lowra_lora_backward_adapters_reuse(const uint16_t* X_dev, const uint16_t* dY_dev, int32_t M, int32_t K,
                                                int32_t N, const uint16_t* T_dev, const uint16_t* U_dev, int32_t r,
                                                uint16_t* dA_dev, uint16_t* dB_dev, void* workspace_dev,
                                                size_t workspace_bytes, void* stream);

/*
 * Synchronises `stream` and returns the status word that the last forward / backward call wrote
 * into its workspace: LOWRA_OK, or LOWRA_ERR_TIMEOUT if a bounded wait inside a kernel ran out
 * (the kernel then released its resources and returned; the output is not valid).
 */
lowra_status lowra_device_status(const void* workspace_dev, void* stream);

/*
 * (No counterpart in the paper.)  Every wait inside the tensor-core kernels - on a shared-memory barrier, on a
 * flag another SM raises - gives up after this long; the kernel then records LOWRA_ERR_TIMEOUT in the status
 * word, lets what it has in flight land, releases its resources and returns (the output of that call is not
 * valid; the GPU and the workspace stay usable).  Process-wide, read when a call is made; 1 s unless changed.
 *   nanoseconds: 1000 .. 10^10, or 0 for the default.  Errors: outside that range -> LOWRA_ERR_SHAPE.
 */
lowra_status lowra_set_wait_limit(uint64_t nanoseconds);

/*
 * (No counterpart in the paper: this is a packaging variant of lowra_lora_forward.)
 *
 * lowra_lora_forward for callers that cannot hand over scratch memory.  Some hosts of this library
 * never get to call cudaMalloc themselves: a plug-in running inside another process's CUDA context
 * whose allocator it must not touch, a real-time or safety-certified loop in which every allocation
 * was frozen at start-up, a sandbox in which only pre-registered buffers may be passed around.  For
 * them the scratch that lowra_lora_forward takes as `workspace_dev` lives inside the library itself,
 * in a fixed device array of LOWRA_STATIC_SCRATCH_BYTES bytes that every GPU holds from the moment the
 * library is loaded there until the process exits.  The call allocates nothing, frees nothing and
 * calls no allocating routine; inputs and outputs are still the caller's.
 *
 *   - Same arguments, results and errors as lowra_lora_forward, without the workspace.  If
 *     the scratch this entry needs (lowra_workspace_bytes(layout, M, r) less the partial tiles, which
 *     it does without: tiles are never cut here) exceeds LOWRA_STATIC_SCRATCH_BYTES the call launches
 *     nothing and returns LOWRA_ERR_LIMIT (for scale: N = K = 8192, M = 8192, r = 64 needs about 1.6 MB).
 *   - status_out_dev (optional, may be NULL): a device uint32 that receives the device status word
 *     (LOWRA_OK or LOWRA_ERR_TIMEOUT) once the call's kernels have run, since the built-in scratch cannot
 *     be given to lowra_device_status.  It is always this call's own status: the word is cleared at the start of
 *     every call, also when layout->deal_dev is set (unlike a caller's workspace, whose word is then sticky).
 *   - The first call on each device looks up the device address of the built-in array (once per device,
 *     with that device current).  Make that first call outside any CUDA stream capture.
 *   - All calls on a device share the one array, and it keeps what the previous call left in it (the call
 *     clears the words it relies on being zero).  Two calls that overlap on the GPU - from different
 *     streams or threads - race on it; serialise them.
 */
#define LOWRA_STATIC_SCRATCH_BYTES (8u << 20)
lowra_status lowra_lora_forward_static(const lowra_layout* layout, const uint8_t* packed_dev,
                                       const float* absmax_dev, const float* maps_dev, const uint16_t* X_dev,
                                       int32_t M, const uint16_t* A_dev, const uint16_t* B_dev, int32_t r,
                                       float s, uint16_t* Y_dev, uint32_t* status_out_dev, void* stream);

/*
 * Mapping and threshold learner (Section 5, "Weighted Lloyd's for LoRA Quantization"; appendix "Weighted
 * Lloyd-Max Algorithm"): for every output channel, at the channel's assigned precision, run `iterations` rounds
 * of weighted Lloyd-Max on the channel's normalised values (normalised per 64-block exactly as in lowra_encode;
 * the weight of a value is the absmax of its block):
 *     assign:  bucket of n = number of current thresholds <= n
 *     levels:  y_j <- sum(w n) / sum(w) over bucket j   (an empty bucket keeps its level)
 *     thresholds: t_j <- (y_j + y_{j+1}) / 2
 * in fp64.  Output tables, fp32 [N, 16], original row order: maps = (float) y (unused entries 0),
 * thresholds[j] = (float)(((double) maps[j] + (double) maps[j+1]) / 2) (unused entries +infinity) - directly
 * usable by lowra_encode / lowra_decode.
 *   W_dev                 fp32 [N, K] row-major, original row order                      (in)
 *   init_levels_host      fp64 [3][16] HOST: starting levels for 1-, 2-, 4-bit rows      (in; the appendix
 *   init_thresholds_host  fp64 [3][16] HOST: starting thresholds                          on initialisation)
 *   iterations            0 .. 1000 (the paper runs 2)
 * The sums are formed by a fixed parallel tree, not in index order: results are reproducible from run to run
 * and agree with a serial fp64 implementation to rounding.  K * 4 bytes must fit in shared memory
 * (K <= 40960), else LOWRA_ERR_SHAPE.  Uses layout->precs_dev only (perm / offsets are not needed).
 */
lowra_status lowra_learn_codebooks(const lowra_layout* layout, const float* W_dev, const double* init_levels_host,
                                   const double* init_thresholds_host, int32_t iterations, float* maps_dev,
                                   float* thresholds_dev, void* stream);

/*
 * The same learner for every channel at all three precisions (Section 5.1 learns each channel's mappings and
 * thresholds under 1, 2 and 4 bits before it assigns precisions): one read of W, the three runs work on the
 * one normalised copy of the row in shared memory.  No layout.
 *   maps3_dev, thresholds3_dev   fp32 [3][N][16]: plane 0 = the 1-bit tables of every row, plane 1 = the 2-bit
 *                                tables, plane 2 = the 4-bit tables - the input format of lowra_channel_errors;
 *                                plane c is bit for bit what lowra_learn_codebooks gives for a layout in which
 *                                every row has 2^c bits                                                  (out)
 * Other arguments, limits and errors as lowra_learn_codebooks (N >= 1, K % 128 == 0).
 */
lowra_status lowra_learn_codebooks_all(int32_t N, int32_t K, const float* W_dev, const double* init_levels_host,
                                       const double* init_thresholds_host, int32_t iterations, float* maps3_dev,
                                       float* thresholds3_dev, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* LOWRA_H */
