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
        unsigned mask[per][4];
        int total[4] = {0, 0, 0, 0};
#pragma unroll
        for (int i = 0; i < per; ++i) {
            const int row = grp * G + i * 32 + lane;
            cls[i] = (row < P.N) ? (P.precs[row] >> 1) : 3;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                mask[i][c] = __ballot_sync(0xffffffffu, cls[i] == c);
                total[c] += __popc(mask[i][c]);
            }
        }
        int class_base[4];
        class_base[0] = 0;
#pragma unroll
        for (int c = 1; c < 4; ++c) class_base[c] = class_base[c - 1] + total[c - 1];
#pragma unroll
        for (int i = 0; i < per; ++i) {
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                if (cls[i] == c) {
                    // inside the class the rows are taken round-robin over (row offset mod 8), so that eight
                    // neighbouring lanes hold eight different residues: their 16-byte stores into the swizzled
                    // operand tile then fall into eight different bank groups
                    const unsigned res_mask = 0x01010101u << (lane & 7);
                    int b = 0;   // rank of this row among the rows of its class with the same residue
#pragma unroll
                    for (int i2 = 0; i2 < per; ++i2)
                        if (i2 < i) b += __popc(mask[i2][c] & res_mask);
                    b += __popc(mask[i][c] & res_mask & ((1u << lane) - 1u));
                    int q = 0;   // rows of the class taken before this one
#pragma unroll
                    for (int res = 0; res < 8; ++res) {
                        int cnt = 0;
#pragma unroll
                        for (int i2 = 0; i2 < per; ++i2) cnt += __popc(mask[i2][c] & (0x01010101u << res));
                        q += min(cnt, b) + ((res < (lane & 7) && cnt > b) ? 1 : 0);
                    }
                    const int off = i * 32 + lane, row = grp * G + off;
                    const uint32_t p = (c < 3) ? (uint32_t)P.inv_perm[row] : 0u;
                    out[class_base[c] + q] = (uint32_t)off | ((uint32_t)c << 7) | (p << 9);
                }
            }
        }
    }
}

// Backward-input: every pipeline stage of the main kernel brings a group of 64 consecutive output channels.
// The CTAs of a cluster take the groups in turn (group g is dequantised by CTA g % kCluster, which then copies
// the finished operand tile to its peers).  The rows of a group are ordered by precision class and cut into
// chunks of at most 16 rows of one class; a chunk is the work of one dequant warp on one stage (32 lanes =
// 16 rows x 2 halves of the tile's 128 features).  The chunks of the groups of one CTA are numbered through the
// whole matrix and chunk n goes to warp n % kProducerWarps of that CTA as entry n / kProducerWarps of the
// warp's work list, so a warp only ever visits the stages it has work on:
//   heads[e]         = group index (bits 0-23) | arrivals this entry owes the stage barrier (bits 24-27) |
//                      precision class of the chunk (bits 28-29; 3 = rows past N, to be zero-filled)
//   rows[e * 32 + l] = what lane l needs to find its row, ready to use (16 bytes):
//                      x = byte offset of the row in the packed buffer / 16, y = index of the row's first absmax,
//                      z = index of the row's first level in the maps table, w = channel inside the group
//                      (all ones: this lane has no row)
// with e = entry * kListWarps + warp * kCluster + CTA.  The stage barrier expects kStageArrivals arrivals; the
// first chunk of a group also arrives for the chunks the group does not have.  Every list ends with all-ones heads.
__device__ __forceinline__ uint32_t list_slot(uint32_t n, int cta) {
    return (n / kProducerWarps) * kListWarps + (n % kProducerWarps) * kCluster + (uint32_t)cta;
}

__device__ void deal_backward(const PrepParams& P, int blk, uint16_t* pre, uint32_t* wsum) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, tid = threadIdx.x;
    constexpr int kWarps = kPrepThreads / 32;
    const int n_groups = (P.N + 63) / 64;
    // ---- chunks per group (every block computes all of them: the numbering needs the running sums)
    for (int grp = warp; grp < n_groups; grp += kWarps) {
        const int r0 = grp * 64 + lane, r1 = r0 + 32;
        const int c0 = (r0 < P.N) ? (P.precs[r0] >> 1) : 3, c1 = (r1 < P.N) ? (P.precs[r1] >> 1) : 3;
        int n = 0;
#pragma unroll
        for (int c = 0; c < 4; ++c)
            n += (__popc(__ballot_sync(0xffffffffu, c0 == c)) + __popc(__ballot_sync(0xffffffffu, c1 == c)) + 15) / 16;
        if (lane == 0) pre[grp] = (uint16_t)n;
    }
    __syncthreads();
    // ---- exclusive running sums, one per CTA of the cluster (over the groups g with g % kCluster == cta)
    for (int cta = 0; cta < kCluster; ++cta) {
        const int n_mine = (n_groups - cta + kCluster - 1) / kCluster;   // groups of this CTA
        const int seg = (n_mine + kPrepThreads - 1) / kPrepThreads;
        const int begin = min(tid * seg, n_mine), end = min(begin + seg, n_mine);
        uint32_t mine = 0;
        for (int i = begin; i < end; ++i) mine += pre[i * kCluster + cta];
        uint32_t incl = mine;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const uint32_t v = __shfl_up_sync(0xffffffffu, incl, d);
            if (lane >= d) incl += v;
        }
        if (lane == 31) wsum[warp] = incl;
        __syncthreads();
        uint32_t run = incl - mine;
        uint32_t total = 0;
#pragma unroll
        for (int w2 = 0; w2 < kWarps; ++w2) {
            if (w2 < warp) run += wsum[w2];
            total += wsum[w2];
        }
        for (int i = begin; i < end; ++i) {
            const uint32_t n = pre[i * kCluster + cta];
            pre[i * kCluster + cta] = (uint16_t)run;
            run += n;
        }
        if (blk == 0)
            for (int i = tid; i < kListSlack; i += kPrepThreads) P.heads[list_slot(total + (uint32_t)i, cta)] = 0xFFFFFFFFu;
        __syncthreads();
    }

    // ---- the deal proper: one warp per group
    for (int grp = blk * kWarps + warp; grp < n_groups; grp += P.blocks * kWarps) {
        const uint32_t g0 = pre[grp];
        int cls[2];
        unsigned mask[2][4];
        int total_c[4] = {0, 0, 0, 0};
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            const int row = grp * 64 + i * 32 + lane;
            cls[i] = (row < P.N) ? (P.precs[row] >> 1) : 3;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                mask[i][c] = __ballot_sync(0xffffffffu, cls[i] == c);
                total_c[c] += __popc(mask[i][c]);
            }
        }
        int chunk_base[4];
        chunk_base[0] = 0;
#pragma unroll
        for (int c = 1; c < 4; ++c) chunk_base[c] = chunk_base[c - 1] + (total_c[c - 1] + 15) / 16;
        const int n_chunks = chunk_base[3] + (total_c[3] + 15) / 16;
        auto entry_of = [&](int ci) { return list_slot(g0 + (uint32_t)ci, grp % kCluster); };
        uint4* rows = reinterpret_cast<uint4*>(P.items);
        for (int ci = 0; ci < n_chunks; ++ci)
            rows[(size_t)entry_of(ci) * 32 + lane] = make_uint4(0u, 0u, 0u, 0xFFFFFFFFu);
        if (lane < n_chunks) {
            const int c = (lane >= chunk_base[1]) + (lane >= chunk_base[2]) + (lane >= chunk_base[3]);   // class of chunk `lane`
            P.heads[entry_of(lane)] = (uint32_t)grp | ((uint32_t)(lane == 0 ? kStageArrivals - n_chunks + 1 : 1) << 24) |
                                      ((uint32_t)c << 28);
        }
        __syncwarp();
#pragma unroll
        for (int i = 0; i < 2; ++i) {
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                if (cls[i] == c) {
                    const int off = i * 32 + lane, row = grp * 64 + off;
                    uint4 rec = make_uint4(0u, 0u, 0u, (uint32_t)off);
                    if (c < 3) {
                        const uint32_t sp = (uint32_t)P.inv_perm[row];   // stored position
                        const uint64_t row_bytes = ((uint64_t)P.L.K << c) >> 3;
                        rec.x = (uint32_t)((P.L.seg_off[c] + (uint64_t)(sp - (uint32_t)P.L.class_start[c]) * row_bytes) >> 4);
                        rec.y = sp * (uint32_t)P.L.nb;
                        rec.z = (uint32_t)row * (uint32_t)kTableStride;
                    }
                    // inside the class the rows are taken round-robin over (row offset mod 8), so that eight
                    // neighbouring lanes hold eight different residues: their 16-byte stores into the swizzled
                    // operand tile then fall into eight different bank groups
                    const unsigned res_mask = 0x01010101u << (lane & 7);
                    int b = 0;   // rank of this row among the rows of its class with the same residue
                    if (i == 1) b += __popc(mask[0][c] & res_mask);
                    b += __popc(mask[i][c] & res_mask & ((1u << lane) - 1u));
                    int pos = 0;  // rows taken before this one
#pragma unroll
                    for (int res = 0; res < 8; ++res) {
                        const int cnt = __popc(mask[0][c] & (0x01010101u << res)) + __popc(mask[1][c] & (0x01010101u << res));
                        pos += min(cnt, b) + ((res < (lane & 7) && cnt > b) ? 1 : 0);
                    }
                    uint4* dst = rows + (size_t)entry_of(chunk_base[c] + pos / 16) * 32 + pos % 16;
                    dst[0] = rec;
                    dst[16] = rec;
                }
            }
        }
    }
}


}  // namespace

__global__ void __launch_bounds__(kPrepThreads) prep_kernel(const PrepParams P) {
    ptx::grid_launch_dependents();   // the fused kernel may set itself up meanwhile; it waits for this grid before reading
    if (blockIdx.x == 0) {
        if (threadIdx.x == 0) *P.status = 0u;
        for (int i = threadIdx.x; i < P.n_flags; i += kPrepThreads) P.flags[i] = 0u;
    }
    if (P.group == 64) {
        __shared__ uint16_t pre[kMaxGroups64];
        __shared__ uint32_t wsum[kPrepThreads / 32];
        deal_backward(P, blockIdx.x, pre, wsum);
    } else {
        deal_rows(P, blockIdx.x);
    }
}

lowra_status launch_prep(const PrepParams& P, cudaStream_t stream) {
    prep_kernel<<<P.blocks, kPrepThreads, 0, stream>>>(P);
    return cudaGetLastError() == cudaSuccess ? LOWRA_OK : LOWRA_ERR_CUDA;
}

}  // namespace lowra
