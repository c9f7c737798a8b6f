// Prologue of the fused forward / backward-input calls: one small launch that clears the device status
// word and the "T ready" flags, and deals the rows of every group of 128 (forward) or 64 (backward)
// consecutive output channels to the 256 dequant threads of the main kernel so that each warp only holds
// rows of one precision.
#include "gemm_params.cuh"
#include "ptx.cuh"

namespace lowra {

namespace {

// One warp per group of G rows (128 forward, 64 backward).  The rows are ordered by precision class
// (1 bit, 2 bits, 4 bits, rows past N; stable).
//   forward : entry i of the group is the i-th row in that order = the row held by tensor-memory lane i of
//             the main kernel, so that at most two precisions meet in a warp (32 consecutive lanes);
//   backward: the ordered rows are cut into chunks of 16 rows of one class (every row is handled by two
//             threads, one per 64-feature half), so that no warp ever sees two precisions.  At most
//             64 / 16 + 3 = 7 chunks exist and the kernel has 12 dequant warps: with n chunks, k = 12 / n warps
//             share a chunk and take turns (warp c + j * n serves chunk c in the groups congruent to j mod k).
__device__ void deal_rows(const PrepParams& P, int blk) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int G = P.group, per = G / 32;
    const int CH = (G == 128) ? 32 : 16;
    const int n_groups = (P.N + G - 1) / G;
    for (int grp = blk * (kPrepThreads / 32) + warp; grp < n_groups; grp += P.blocks * (kPrepThreads / 32)) {
        uint32_t* out = P.items + (size_t)grp * kItemStride;
#pragma unroll
        for (int i = 0; i < kItemStride / 32; ++i) out[i * 32 + lane] = 0xFFFFFFFFu;
        __syncwarp();
        int cls[4];
        unsigned mask[4][4];
        int total[4] = {0, 0, 0, 0};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            cls[i] = 3;
            if (i < per) {
                const int row = grp * G + i * 32 + lane;
                if (row < P.N) cls[i] = P.precs[row] >> 1;
            }
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                mask[i][c] = (i < per) ? __ballot_sync(0xffffffffu, cls[i] == c) : 0u;
                total[c] += __popc(mask[i][c]);
            }
        }
        int chunk_base[4];
        chunk_base[0] = 0;
#pragma unroll
        for (int c = 1; c < 4; ++c) chunk_base[c] = chunk_base[c - 1] + (total[c - 1] + CH - 1) / CH;
        int class_base[4];
        class_base[0] = 0;
#pragma unroll
        for (int c = 1; c < 4; ++c) class_base[c] = class_base[c - 1] + total[c - 1];
        const int n_chunks = chunk_base[3] + (total[3] + CH - 1) / CH;
        const int k = kProducerWarps / n_chunks;   // warps that share a chunk (backward)
        if (lane == 0) P.n_chunks[grp] = (uint32_t)n_chunks;
        int before[4] = {0, 0, 0, 0};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            if (i < per) {
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    if (cls[i] == c) {
                        const int q = before[c] + __popc(mask[i][c] & ((1u << lane) - 1u));  // rank inside the class
                        const int off = i * 32 + lane, row = grp * G + off;
                        const uint32_t p = (c < 3) ? (uint32_t)P.inv_perm[row] : 0u;
                        const uint32_t word = (uint32_t)off | ((uint32_t)c << 7) | (p << 9);
                        if (CH == 32) {
                            // forward: position in precision order = tensor-memory lane of the row
                            out[class_base[c] + q] = word;
                        } else {
                            // backward: the group index is the stage index; of the k warps that share the
                            // chunk, the one whose turn it is gets the row (for both feature halves).
                            // Inside the class the rows are taken round-robin over (row offset mod 8), so that
                            // eight neighbouring lanes hold eight different residues: their 16-byte stores into
                            // the swizzled operand tile then fall into eight different bank groups.
                            const unsigned res_mask = 0x01010101u << (lane & 7);
                            int b = 0;   // rank of this row among the rows of its class with the same residue
#pragma unroll
                            for (int i2 = 0; i2 < 4; ++i2)
                                if (i2 < i) b += __popc(mask[i2][c] & res_mask);
                            b += __popc(mask[i][c] & res_mask & ((1u << lane) - 1u));
                            int pos = 0;  // rows taken before this one
#pragma unroll
                            for (int res = 0; res < 8; ++res) {
                                int cnt = 0;
#pragma unroll
                                for (int i2 = 0; i2 < 4; ++i2)
                                    if (i2 < per) cnt += __popc(mask[i2][c] & (0x01010101u << res));
                                pos += min(cnt, b) + ((res < (lane & 7) && cnt > b) ? 1 : 0);
                            }
                            const int j = grp % k;
                            const int thread = (chunk_base[c] + pos / CH + j * n_chunks) * 32 + pos % CH;
                            out[thread] = word;
                            out[thread + 16] = word;
                        }
                    }
                }
#pragma unroll
                for (int c = 0; c < 4; ++c) before[c] += __popc(mask[i][c]);
            }
        }
    }
}

}  // namespace

__global__ void __launch_bounds__(kPrepThreads) prep_kernel(const PrepParams P) {
    if (blockIdx.x == 0) {
        if (threadIdx.x == 0) *P.status = 0u;
        for (int i = threadIdx.x; i < P.n_flags; i += kPrepThreads) P.flags[i] = 0u;
    }
    deal_rows(P, blockIdx.x);
}

lowra_status launch_prep(const PrepParams& P, cudaStream_t stream) {
    prep_kernel<<<P.blocks, kPrepThreads, 0, stream>>>(P);
    return cudaGetLastError() == cudaSuccess ? LOWRA_OK : LOWRA_ERR_CUDA;
}

}  // namespace lowra
