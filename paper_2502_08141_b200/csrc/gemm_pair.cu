// Dense diagnostic with the two-CTA form of tcgen05.mma (cta_group::2): C [M, N] = P [M, K] . Q [N, K]^T, bf16.
//
// Two CTAs of a cluster (two neighbouring SMs) work on one 256 x 256 tile.  Each CTA holds half of either
// operand in its own shared memory - 128 rows of P and 128 rows of Q per 64-wide contraction block, 32 KB per
// stage instead of the 48 KB of the one-CTA 128 x 256 tile - and the accumulator of its own 128 rows of the tile in
// its own tensor memory; the MMA is issued by one thread of the even ("leader") CTA and runs on both SMs, each
// tensor core reading its half of P locally and both halves of Q.  Per FLOP that is two thirds of the one-CTA
// tile's shared-memory traffic and L2 traffic, which is what bounds the one-CTA pipeline of this library.
//   - TMA: both CTAs load their halves; the bytes of both are counted on the LEADER's "full" barrier
//     (tiled TMA loads with .cta_group::2 and the leader's barrier address; every CTA loads for itself).
//   - slot release and "accumulator complete": tcgen05.commit.cta_group::2 with a CTA mask, which arrives on the
//     barrier at the same offset in both CTAs.
//   - "accumulator drained": the epilogue warps of both CTAs arrive on the leader's barrier.
//   - tensor memory is allocated and freed by the same warp of both CTAs (cta_group::2 forms).
// warp 0 = TMA, warp 1 = MMA issue (leader) and TMEM owner, warps 2-5 = epilogue.  All waits are bounded.
// This entry point exists to measure what the two-CTA form is worth for this pipeline; the fused kernels still use
// the one-CTA form.
#include <cudaTypedefs.h>

#include "gemm_params.cuh"
#include "ptx.cuh"

namespace lowra {

namespace {

constexpr uint64_t kPairWaitNs = 1000ull * 1000ull * 1000ull;
constexpr int kPairThreads = 192;
constexpr int kPairStages = 6;
constexpr uint32_t kPairHalf = 128 * 64 * 2;                 // 16 KB: 128 rows x 64 contraction elements
constexpr uint32_t kPairStageBytes = 2 * kPairHalf;          // this CTA's halves of P and Q
constexpr uint32_t kPairSmemBytes = kPairStages * kPairStageBytes + 1024;
constexpr uint32_t kPairIdesc = ptx::umma_idesc_bf16(256, 256);

struct PairBarriers {
    uint64_t full[kPairStages];     // leader: both CTAs' TMA bytes of the stage have landed
    uint64_t empty[kPairStages];    // every CTA: the MMAs reading the stage are complete
    uint64_t tmem_full[2];          // every CTA: the accumulator is complete
    uint64_t tmem_empty[2];         // leader: the epilogue warps of both CTAs have drained the accumulator
    uint32_t tmem_base;
    uint32_t abort;
};

struct PairParams {
    uint16_t* C;
    uint32_t* status;
    int M, N, K;
    int tiles_m, tiles_n;
};

__device__ __forceinline__ void tma_load_2d_pair(void* dst, const CUtensorMap* map, int x, int y, uint32_t leader_bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(ptx::smem_u32(dst)),
        "l"(reinterpret_cast<uint64_t>(map)), "r"(leader_bar), "r"(x), "r"(y)
        : "memory");
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t* dst, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(ptx::smem_u32(dst)), "r"(ncols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void umma_bf16_pair(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t"
        ".reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5, %5, %5, %5, %5}, p;\n\t"
        "}\n"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(0u)
        : "memory");
}
// arrives (when the MMAs issued so far are complete) on the barrier at this offset in every CTA of the mask
__device__ __forceinline__ void umma_commit_pair(uint64_t* bar, uint16_t cta_mask) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(ptx::smem_u32(bar)), "h"(cta_mask)
                 : "memory");
}
__device__ __forceinline__ void mbar_arrive_release_cluster(uint32_t caddr) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(caddr) : "memory");
}

__global__ void __launch_bounds__(kPairThreads, 1)
pair_kernel(const PairParams P, const __grid_constant__ CUtensorMap tmP, const __grid_constant__ CUtensorMap tmQ) {
    extern __shared__ __align__(1024) unsigned char pair_smem[];
    unsigned char* base = pair_smem;
    PairBarriers* bars = reinterpret_cast<PairBarriers*>(base + kPairStages * kPairStageBytes);
    volatile uint32_t* abort_flag = &bars->abort;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t crank = ptx::cluster_ctarank();          // 0 = leader
    const bool leader = crank == 0;
    const bool aligned = (ptx::smem_u32(pair_smem) & 1023u) == 0u;
    const int cid = (int)blockIdx.x / 2, NC = (int)gridDim.x / 2;
    const int n_tiles = P.tiles_m * P.tiles_n;
    const int n_blocks = P.K / 64;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kPairStages; ++s) { ptx::mbar_init(&bars->full[s], 1); ptx::mbar_init(&bars->empty[s], 1); }
        for (int a = 0; a < 2; ++a) { ptx::mbar_init(&bars->tmem_full[a], 1); ptx::mbar_init(&bars->tmem_empty[a], 8); }
        bars->abort = aligned ? 0u : 1u;
        ptx::fence_barrier_init();
        ptx::prefetch_tensormap(&tmP);
        ptx::prefetch_tensormap(&tmQ);
    }
    __syncthreads();
    ptx::cluster_sync();   // both CTAs' barriers exist before anything is counted on them
    if (warp == 1) tmem_alloc_pair(&bars->tmem_base, 512);
    ptx::tc_fence_before();
    __syncthreads();
    ptx::cluster_sync();
    ptx::tc_fence_after();
    const uint32_t tmem_base = bars->tmem_base;
    bool failed = !aligned;

    if (failed) {
        // nothing is loaded or multiplied
    } else if (warp == 0) {
        if (lane == 0) {
            uint32_t it = 0;
            for (int g = cid; g < n_tiles && !failed; g += NC) {
                const int tm = g / P.tiles_n, tn = g - tm * P.tiles_n;
                const int m0 = tm * 256 + 128 * (int)crank, n0 = tn * 256 + 128 * (int)crank;
                for (int kb = 0; kb < n_blocks; ++kb, ++it) {
                    const int s = it % kPairStages;
                    if (!ptx::mbar_wait(&bars->empty[s], ((it / kPairStages) & 1u) ^ 1u, abort_flag, kPairWaitNs)) { failed = true; bars->abort = 1u; break; }
                    const uint32_t leader_bar = ptx::map_to_cta(ptx::smem_u32(&bars->full[s]), 0u);
                    if (leader) ptx::mbar_arrive_expect_tx(&bars->full[s], 2u * kPairStageBytes);   // both CTAs' bytes
                    unsigned char* p_s = base + s * kPairStageBytes;
                    tma_load_2d_pair(p_s, &tmP, kb * 64, m0, leader_bar);
                    tma_load_2d_pair(p_s + kPairHalf, &tmQ, kb * 64, n0, leader_bar);
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0 && leader) {
            uint32_t it = 0, tile_iter = 0;
            for (int g = cid; g < n_tiles && !failed; g += NC, ++tile_iter) {
                const uint32_t acc = tile_iter & 1u, aph = (tile_iter >> 1) & 1u;
                if (!ptx::mbar_wait(&bars->tmem_empty[acc], aph ^ 1u, abort_flag, kPairWaitNs)) { failed = true; bars->abort = 1u; break; }
                ptx::tc_fence_after();
                const uint32_t d_tmem = tmem_base + acc * 256u;
                for (int kb = 0; kb < n_blocks; ++kb, ++it) {
                    const int s = it % kPairStages;
                    if (!ptx::mbar_wait(&bars->full[s], (it / kPairStages) & 1u, abort_flag, kPairWaitNs)) { failed = true; bars->abort = 1u; break; }
                    ptx::tc_fence_after();
                    const uint32_t p_addr = ptx::smem_u32(base + s * kPairStageBytes);
                    const uint64_t adesc = ptx::umma_desc_k_sw128(p_addr);
                    const uint64_t bdesc = ptx::umma_desc_k_sw128(p_addr + kPairHalf);
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk)
                        umma_bf16_pair(d_tmem, adesc + 2u * kk, bdesc + 2u * kk, kPairIdesc, (kb | kk) != 0 ? 1u : 0u);
                    umma_commit_pair(&bars->empty[s], (uint16_t)3);
                }
                if (failed) break;
                umma_commit_pair(&bars->tmem_full[acc], (uint16_t)3);
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue: this CTA's 128 rows of the tile
        const int q = warp & 3;
        const uint32_t leader_empty0 = ptx::map_to_cta(ptx::smem_u32(&bars->tmem_empty[0]), 0u);
        const uint32_t leader_empty1 = ptx::map_to_cta(ptx::smem_u32(&bars->tmem_empty[1]), 0u);
        uint32_t tile_iter = 0;
        for (int g = cid; g < n_tiles && !failed; g += NC, ++tile_iter) {
            const int tm = g / P.tiles_n, tn = g - tm * P.tiles_n;
            const uint32_t acc = tile_iter & 1u, aph = (tile_iter >> 1) & 1u;
            if (!ptx::mbar_wait_warp(&bars->tmem_full[acc], aph, abort_flag, kPairWaitNs)) { failed = true; bars->abort = 1u; break; }
            ptx::tc_fence_after();
            const int row = tm * 256 + 128 * (int)crank + q * 32 + lane;
#pragma unroll 1
            for (int chunk = 0; chunk < 8; ++chunk) {
                uint32_t v[32];
                ptx::tmem_ld_32x32(tmem_base + ((uint32_t)(q * 32) << 16) + acc * 256u + (uint32_t)chunk * 32u, v);
                ptx::tmem_ld_wait();
                const int col = tn * 256 + chunk * 32;
                if (row < P.M) {
                    uint16_t* dst = P.C + (size_t)row * P.N + col;
                    if (col + 32 <= P.N && (P.N % 8) == 0) {
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            uint4 w;
                            w.x = pack_bf16x2(__uint_as_float(v[8 * j]), __uint_as_float(v[8 * j + 1]));
                            w.y = pack_bf16x2(__uint_as_float(v[8 * j + 2]), __uint_as_float(v[8 * j + 3]));
                            w.z = pack_bf16x2(__uint_as_float(v[8 * j + 4]), __uint_as_float(v[8 * j + 5]));
                            w.w = pack_bf16x2(__uint_as_float(v[8 * j + 6]), __uint_as_float(v[8 * j + 7]));
                            *reinterpret_cast<uint4*>(dst + 8 * j) = w;
                        }
                    } else {
                        for (int j = 0; j < 32 && col + j < P.N; ++j) dst[j] = (uint16_t)pack_bf16x2(__uint_as_float(v[j]), 0.0f);
                    }
                }
            }
            ptx::tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_release_cluster(acc ? leader_empty1 : leader_empty0);
        }
    }
    if (failed) atomicExch(P.status, aligned ? (uint32_t)LOWRA_ERR_TIMEOUT : (uint32_t)LOWRA_ERR_CUDA);
    ptx::tc_fence_before();
    __syncthreads();
    ptx::cluster_sync();   // no peer reads this CTA's shared memory or arrives on its barriers any more
    if (warp == 1) {
        ptx::tc_fence_after();
        tmem_dealloc_pair(tmem_base, 512);
    }
}

bool make_map_k(CUtensorMap* map, const void* ptr, uint64_t rows, uint64_t cols, uint32_t box_rows) {
    static PFN_cuTensorMapEncodeTiled_v12000 fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess || q != cudaDriverEntryPointSuccess)
            return false;
        fn = reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(p);
    }
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {cols * 2};
    cuuint32_t box[2] = {64, box_rows};
    cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

__global__ void pair_clear_status(uint32_t* status) { *status = 0u; }

}  // namespace
}  // namespace lowra

extern "C" lowra_status lowra_dense_nt_pair(const uint16_t* P_dev, const uint16_t* Q_dev, int32_t M, int32_t N, int32_t K,
                                            uint16_t* C_dev, void* workspace_dev, size_t workspace_bytes, void* stream_v) {
    using namespace lowra;
    if (!P_dev || !Q_dev || !C_dev || !workspace_dev) return LOWRA_ERR_NULL;
    if (M < 1 || N < 1 || K < 64 || K % 64 != 0) return LOWRA_ERR_SHAPE;
    if (!aligned16(P_dev) || !aligned16(Q_dev) || !aligned16(C_dev)) return LOWRA_ERR_ALIGN;
    if (workspace_bytes < 256 || (reinterpret_cast<uintptr_t>(workspace_dev) & 255u) != 0) return LOWRA_ERR_WORKSPACE;
    lowra_status st = check_device();
    if (st != LOWRA_OK) return st;
    cudaStream_t stream = (cudaStream_t)stream_v;
    uint32_t* status = reinterpret_cast<uint32_t*>(workspace_dev);
    pair_clear_status<<<1, 1, 0, stream>>>(status);
    PairParams P;
    P.C = C_dev;
    P.status = status;
    P.M = M;
    P.N = N;
    P.K = K;
    P.tiles_m = (M + 255) / 256;
    P.tiles_n = (N + 255) / 256;
    CUtensorMap tmP, tmQ;
    if (!make_map_k(&tmP, P_dev, (uint64_t)M, (uint64_t)K, 128) || !make_map_k(&tmQ, Q_dev, (uint64_t)N, (uint64_t)K, 128))
        return LOWRA_ERR_CUDA;
    static bool configured = false;
    static int max_clusters = kNumSMs / 2;
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.blockDim = dim3(kPairThreads, 1, 1);
    cfg.dynamicSmemBytes = kPairSmemBytes;
    cfg.stream = stream;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (!configured) {
        if (cudaFuncSetAttribute(pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kPairSmemBytes) != cudaSuccess)
            return LOWRA_ERR_CUDA;
        cfg.gridDim = dim3(kNumSMs / 2 * 2, 1, 1);
        int n = 0;
        if (cudaOccupancyMaxActiveClusters(&n, pair_kernel, &cfg) != cudaSuccess || n < 1) return LOWRA_ERR_CUDA;
        if (n < max_clusters) max_clusters = n;
        configured = true;
    }
    const int n_tiles = P.tiles_m * P.tiles_n;
    const int clusters = n_tiles < max_clusters ? n_tiles : max_clusters;
    cfg.gridDim = dim3((unsigned)(clusters * 2), 1, 1);
    return cudaLaunchKernelEx(&cfg, pair_kernel, P, tmP, tmQ) == cudaSuccess ? LOWRA_OK : LOWRA_ERR_CUDA;
}
