// Prologue of the fused forward / backward-input calls: one small launch that clears the device status
// word and the "T ready" flags, and deals the rows of every group of 128 (forward) or 64 (backward)
// consecutive output channels to the dequant threads of the main kernel so that a warp holds rows of one
// precision wherever the counts allow.
#include "gemm_params.cuh"
#include "ptx.cuh"

namespace lowra {

namespace {

// Forward: one warp per group of 128 consecutive output channels (one weight tile of the main kernel).  The
// rows are ordered by precision class (1 bit, 2 bits, 4 bits, rows past N); entry i of the group is the i-th row
// in that order = the row held by lane i % 32 of warp i / 32 of a dequant group of the main kernel, so that at
// most two precisions meet in a warp.
__device__ void deal_rows(const PrepParams& P, int blk) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    constexpr int G = 128, per = G / 32;
    const int n_groups = (P.N + G - 1) / G;
    for (int grp = blk * (kPrepThreads / 32) + warp; grp < n_groups; grp += P.blocks * (kPrepThreads / 32)) {
        uint32_t* out = P.items + (size_t)grp * kItemStride;
        int cls[per];
        uint32_t stored[per];   // stored position of the row (asked for now: the answer is needed last)
        unsigned mask[per][4];
#pragma unroll
        for (int i = 0; i < per; ++i) {
            const int row = grp * G + i * 32 + lane;
            stored[i] = (row < P.N) ? (uint32_t)P.inv_perm[row] : 0u;
        }
#pragma unroll
        for (int i = 0; i < per; ++i) {
            const int row = grp * G + i * 32 + lane;
            cls[i] = (row < P.N) ? (P.precs[row] >> 1) : 3;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                mask[i][c] = __ballot_sync(0xffffffffu, cls[i] == c);
            }
        }
        // Order: the rows with the same offset mod 8 (16 of them; a lane's rows all share its lane & 7) are ranked by
        // (class, offset), and entry 8 * rank + (offset mod 8) takes the row.  Eight neighbouring lanes of a dequant warp
        // therefore always hold eight different offsets mod 8 - their 16-byte stores into the swizzled operand tile fall
        // into eight different bank groups whatever the precisions are - and the entries still run from the lowest
        // class to the highest, exactly sorted wherever the classes are spread evenly over the eight residues.
        const unsigned res_mask = 0x01010101u << (lane & 7);
#pragma unroll
        for (int i = 0; i < per; ++i) {
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                if (cls[i] == c) {
                    int rank = 0;   // rows of the same residue that come before this one
#pragma unroll
                    for (int c2 = 0; c2 < 4; ++c2)
#pragma unroll
                        for (int i2 = 0; i2 < per; ++i2)
                            if (c2 < c || (c2 == c && i2 < i)) rank += __popc(mask[i2][c2] & res_mask);
                    rank += __popc(mask[i][c] & res_mask & ((1u << lane) - 1u));
                    const int off = i * 32 + lane;
                    const uint32_t p = (c < 3) ? stored[i] : 0u;
                    out[rank * 8 + (lane & 7)] = (uint32_t)off | ((uint32_t)c << 7) | (p << 9);
                }
            }
        }
    }
}

// Backward-input: every pipeline stage of the main kernel brings a group of 64 consecutive output channels.
// The CTAs of a cluster take the groups in turn (group g is dequantised by CTA g % kCluster, which then copies
// the finished operand tile to its peers).  The rows of a group are ordered by precision class (rows past N last)
// and cut into four chunks of 16 rows; a chunk is the work of one dequant warp on one stage (32 lanes = 16 rows x
// 2 halves of the tile's 128 features), so most warps see one precision and a few see two.  The chunks of the
// groups of one CTA are numbered through the whole matrix and chunk n goes to warp n % kProducerWarps of that
// CTA as entry n / kProducerWarps of the warp's work list, so a warp only ever visits the stages it has work on:
//   heads[e]         = group index (bits 0-23) | arrivals this entry owes the stage barrier (bits 24-27)
//   rows[e * 32 + l] = what lane l needs to find its row, ready to use (16 bytes):
//                      x = byte offset of the row in the packed buffer / 16, y = index of the row's first absmax,
//                      z = index of the row's first level in the maps table,
//                      w = channel inside the group (bits 0-5) | precision class (bits 8-9; 3 = row past N: zeros)
// with e = entry * kListWarps + warp * kCluster + CTA.  Every list ends with all-ones heads.
__device__ __forceinline__ uint32_t list_slot(uint32_t n, int cta) {
    return (n / kProducerWarps) * kListWarps + (n % kProducerWarps) * kCluster + (uint32_t)cta;
}
// The chunks of a group are sorted by precision, so its last chunk is the dearest one (it holds the group's 4-bit
// rows, usually next to 2-bit ones: two code paths).  Which of a group's four warps takes which chunk therefore
// rotates from one group pair to the next; a warp still gets one chunk of every second group of its CTA, in order.
__device__ __forceinline__ uint32_t chunk_slot(uint32_t n0, uint32_t ci, int cta) {
    const uint32_t pair = n0 / kProducerWarps;                    // n0 = 4 * (group's number within its CTA)
    return list_slot((n0 & ~3u) + ((ci + pair) & 3u), cta);
}

__device__ void deal_backward(const PrepParams& P, int blk) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, tid = threadIdx.x;
    constexpr int kWarps = kPrepThreads / 32;
    constexpr int kChunks = 4;   // per group of 64 rows
    const int n_groups = (P.N + 63) / 64;
    if (blk == 0) {   // end markers behind the last entry of every CTA's lists
        for (int cta = 0; cta < kCluster; ++cta) {
            const uint32_t total = (uint32_t)kChunks * (uint32_t)((n_groups - cta + kCluster - 1) / kCluster);
            for (int i = tid; i < kListSlack; i += kPrepThreads) P.heads[list_slot(total + (uint32_t)i, cta)] = 0xFFFFFFFFu;
        }
    }
    uint4* rows = reinterpret_cast<uint4*>(P.items);
    // one warp per group
    for (int grp = blk * kWarps + warp; grp < n_groups; grp += P.blocks * kWarps) {
        const int cta = grp % kCluster;
        const uint32_t n0 = (uint32_t)kChunks * (uint32_t)(grp / kCluster);   // number of the group's first chunk
        int cls[2];
        uint32_t stored[2];   // stored position of the row (asked for now: the answer is needed last)
        unsigned mask[2][4];
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            const int row = grp * 64 + i * 32 + lane;
            stored[i] = (row < P.N) ? (uint32_t)P.inv_perm[row] : 0u;
        }
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            const int row = grp * 64 + i * 32 + lane;
            cls[i] = (row < P.N) ? (P.precs[row] >> 1) : 3;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                mask[i][c] = __ballot_sync(0xffffffffu, cls[i] == c);
            }
        }
        if (lane < kChunks)
            P.heads[chunk_slot(n0, (uint32_t)lane, cta)] = (uint32_t)grp | ((uint32_t)(kStageArrivals / kChunks) << 24);
#pragma unroll
        for (int i = 0; i < 2; ++i) {
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                if (cls[i] == c) {
                    const int off = i * 32 + lane, row = grp * 64 + off;
                    uint4 rec = make_uint4(0u, 0u, 0u, (uint32_t)off | ((uint32_t)c << 8));
                    if (c < 3) {
                        const uint32_t sp = stored[i];   // stored position
                        rec.x = (uint32_t)(packed_row_offset(P.L, c, (int)sp, row) >> 4);
                        rec.y = (uint32_t)absmax_row_of(P.L, (int)sp, row) * (uint32_t)P.L.nb;
                        rec.z = (uint32_t)row * (uint32_t)kTableStride;
                    }
                    // the eight rows with the same offset mod 8 are ranked by (class, offset); position 8 * rank +
                    // (offset mod 8): eight neighbouring lanes always hold eight different residues, so their 16-byte
                    // stores into the swizzled operand tile fall into eight different bank groups whatever the
                    // precisions are, and the positions still run from the lowest class to the highest
                    const unsigned res_mask = 0x01010101u << (lane & 7);
                    int rank = 0;
#pragma unroll
                    for (int c2 = 0; c2 < 4; ++c2)
#pragma unroll
                        for (int i2 = 0; i2 < 2; ++i2)
                            if (c2 < c || (c2 == c && i2 < i)) rank += __popc(mask[i2][c2] & res_mask);
                    rank += __popc(mask[i][c] & res_mask & ((1u << lane) - 1u));
                    const int pos = rank * 8 + (lane & 7);
                    uint4* dst = rows + (size_t)chunk_slot(n0, (uint32_t)(pos / 16), cta) * 32 + pos % 16;
                    dst[0] = rec;
                    dst[16] = rec;
                }
            }
        }
    }
}

}  // namespace

__global__ void __launch_bounds__(kPrepThreads) prep_kernel(const PrepParams P) {
    pdl_enter();   // the fused kernel may set itself up meanwhile; it waits for this grid before it reads the deal
    if (blockIdx.x == 0) {
        if (threadIdx.x == 0 && P.status != nullptr) *P.status = 0u;   // null: keep what earlier launches recorded
        if (threadIdx.x == 0 && P.exits != nullptr) *P.exits = 0u;
        for (int i = threadIdx.x; i < P.n_flags; i += kPrepThreads) P.flags[i] = 0u;
    }
    if (P.group == 64) {
        deal_backward(P, blockIdx.x);
    } else {
        deal_rows(P, blockIdx.x);
    }
}

lowra_status launch_prep(const PrepParams& P, cudaStream_t stream) {
    return launch_pdl(prep_kernel, (unsigned)P.blocks, kPrepThreads, stream, P) == cudaSuccess ? LOWRA_OK : LOWRA_ERR_CUDA;
}

}  // namespace lowra
