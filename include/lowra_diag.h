/*
 * lowra_diag.h -- diagnostic entry points of the library; not part of the method and not needed by a user of
 * the quantized-LoRA layer (the product ABI is lowra.h).
 */
#ifndef LOWRA_DIAG_H
#define LOWRA_DIAG_H

#include "lowra.h"

#ifdef __cplusplus
extern "C" {
#endif

/*
 * (No counterpart in the paper.)  C = P . Q^T with P bf16 [M, K], Q bf16 [N, K] (both row-major, K % 64 == 0),
 * C bf16 [M, N], run through the same tensor-core pipeline as the fused kernels but with both operands fetched as
 * plain bf16 tiles.  It separates what the pipeline costs from what the dequantisation costs ("decode, then a
 * dense product" against the fused call).
 *   P_dev, Q_dev, C_dev: device, 16-byte aligned.  workspace_dev: device, 256-byte aligned, >= 256 bytes; its
 *   first word is the device status word (lowra_device_status).  Nothing is allocated; the call enqueues on
 *   `stream` and returns.
 * Errors: NULL pointer -> LOWRA_ERR_NULL; M < 1, N < 1, K < 64 or K % 64 != 0 -> LOWRA_ERR_SHAPE; misaligned
 * operand -> LOWRA_ERR_ALIGN; workspace too small or misaligned -> LOWRA_ERR_WORKSPACE.
 */
lowra_status lowra_dense_nt(const uint16_t* P_dev, const uint16_t* Q_dev, int32_t M, int32_t N, int32_t K,
                            uint16_t* C_dev, void* workspace_dev, size_t workspace_bytes, void* stream);

/*
 * (No counterpart in the paper.)  Failure-detection self test, part 1: a one-warp kernel waits on a shared-memory
 * barrier on which nobody ever arrives and then on a flag in global memory that nobody ever raises, with the very
 * wait routines of the tensor-core kernels and the given limit.  Both waits run out; the kernel records
 * LOWRA_ERR_TIMEOUT in the status word (byte 0 of the workspace; read it with lowra_device_status) and returns.
 * Nothing traps, faults or spins without a limit.
 *   workspace_dev: device, 256-byte aligned, >= 256 bytes, overwritten.  Words 8, 9, 10 (uint32) receive: a bit
 *   mask of the waits that ran out (1: barrier, 2: flag, 4: the whole-warp form of the barrier wait), and the
 *   microseconds spent in the first two.
 *   limit_ns: 1000 .. 10^8.
 * Errors: LOWRA_ERR_NULL, LOWRA_ERR_WORKSPACE, LOWRA_ERR_SHAPE (limit out of range), LOWRA_ERR_ARCH, LOWRA_ERR_CUDA.
 */
lowra_status lowra_diag_wait_expiry(void* workspace_dev, size_t workspace_bytes, uint64_t limit_ns, void* stream);

/*
 * (No counterpart in the paper.)  Failure-detection self test, part 2, injected on the host: the next `calls`
 * calls of lowra_lora_forward / lowra_lora_backward_input (in this process, whatever their arguments) run with
 * the publication of their "down-projection ready" flags switched off.  Every SM that needs a down-projected
 * tile then waits for a flag that never comes, gives up after the limit set by lowra_set_wait_limit, and the
 * whole call leaves through its failure path: status word LOWRA_ERR_TIMEOUT, output not valid, GPU and workspace
 * usable afterwards.  Set the limit to a few milliseconds first.  calls: 0 .. 1000 (0 disarms).
 */
lowra_status lowra_diag_drop_t_flags(int32_t calls);

#ifdef __cplusplus
}
#endif
#endif /* LOWRA_DIAG_H */
