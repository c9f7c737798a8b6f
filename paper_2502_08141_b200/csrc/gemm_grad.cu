// The four skinny products behind the gradients of the low-rank factors:
//     T  = s X A          [M, rp]     U  = s dY B^T        [M, rp]      (down-projections, rank padded to 64)
//     dA = X^T U          [K, r]      dB = (dY^T T)^T      [r, N]
// All have the shape  D [R rows x rp columns] = sum over c < C of  P(row, c) * Q(c, column)  with rp <= 128 and a
// long contraction, so they are bound by reading P (X or dY) once from HBM, not by the tensor cores.
//
// One CTA computes a tile of 128 rows over a slice of the contraction: the S CTAs of a thread-block cluster share a
// tile, each streams its slice (TMA -> shared memory -> tcgen05.mma -> TMEM), dumps its fp32 partial tile into its own
// shared memory, and after a cluster barrier every CTA sums 128 / S rows of the tile over all S partials through
// distributed shared memory (fixed order: bit-reproducible) and writes them out in bf16.  S is chosen so that the
// grid covers the SMs about twice over; two CTAs fit on an SM (96 KB ring each), which keeps enough loads in flight.
//
// Either operand can lie either way in memory; a tile arrives by TMA exactly as it lies:
//     K-major  (the contraction index is contiguous: X for T, dY and B for U)   one box of [rows][64 c]
//     MN-major (the row / column index is contiguous: A for T; X, dY, U, T for the gradients)   boxes of [64 c][64 rows]
// warp 0 = TMA, warp 1 = MMA issue, warps 2-5 = epilogue and reduction.  All waits are bounded.
#include "gemm_params.cuh"
#include "ptx.cuh"

namespace lowra {

namespace {

constexpr int kSkinnyThreads = 192;                    // 6 warps
constexpr uint32_t kSkinnyRing = 96 * 1024;            // pipeline stages; afterwards the fp32 partial tile
constexpr uint32_t kSkinnySmemP = 128 * 64 * 2;        // 16 KB of P per stage
constexpr uint32_t kSkinnySmemBytes = kSkinnyRing + 256;
constexpr int kSkinnyMaxStages = 4;
constexpr int kSkinnyMaxSplit = 8;                     // portable cluster size
constexpr int kSkinnySlots = 2 * kNumSMs - 2 * 16;      // CTAs resident at once (two per SM, less what clusters leave unused)

struct SkinnyBarriers {
    uint64_t full[kSkinnyMaxStages];
    uint64_t empty[kSkinnyMaxStages];
    uint64_t tmem_full;
    uint32_t tmem_base;
    uint32_t abort;
};
static_assert(sizeof(SkinnyBarriers) <= 256, "barrier block");

__global__ void __launch_bounds__(kSkinnyThreads, 2)
skinny_kernel(const SkinnyArgs P, const int S, const __grid_constant__ CUtensorMap tmP, const __grid_constant__ CUtensorMap tmQ) {
    extern __shared__ __align__(1024) unsigned char skinny_smem[];
    unsigned char* base = skinny_smem;
    SkinnyBarriers* bars = reinterpret_cast<SkinnyBarriers*>(base + kSkinnyRing);
    volatile uint32_t* abort_flag = &bars->abort;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int r0 = blockIdx.x * 128;
    const uint32_t crank = ptx::cluster_ctarank();            // which slice of the contraction
    const int n_blocks = (P.C + 63) / 64;
    const int kb0 = (int)((long long)crank * n_blocks / S), kb1 = (int)((long long)(crank + 1) * n_blocks / S);
    const int n_my = kb1 - kb0;
    const uint32_t stage_bytes = kSkinnySmemP + (uint32_t)P.rp * 128u;   // 24 or 32 KB
    const int stages = (int)(kSkinnyRing / stage_bytes);                  // 4 or 3
    const uint32_t tmem_cols = 128;                                       // >= rp, a power of two
    const bool aligned = (ptx::smem_u32(skinny_smem) & 1023u) == 0u;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kSkinnyMaxStages; ++s) { ptx::mbar_init(&bars->full[s], 1); ptx::mbar_init(&bars->empty[s], 1); }
        ptx::mbar_init(&bars->tmem_full, 1);
        bars->abort = aligned ? 0u : 1u;
        ptx::fence_barrier_init();
        ptx::prefetch_tensormap(&tmP);
        ptx::prefetch_tensormap(&tmQ);
    }
    if (warp == 1) ptx::tmem_alloc(&bars->tmem_base, tmem_cols);
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem_base = bars->tmem_base;
    pdl_enter();   // the operands may come from the kernels launched before this one
    bool failed = !aligned;

    // fp32 partial tile [128 rows][rp + 4]: the padding spreads the rows of a warp over the banks
    float* part = reinterpret_cast<float*>(base);
    const int pstride = P.rp + 4;

    if (failed) {
        // shared memory not aligned as the swizzled tiles need: nothing is loaded or multiplied
    } else if (warp == 0) {
        if (lane == 0) {
            int issued = 0;
            for (int i = 0; i < n_my; ++i) {
                const int s = i % stages, kb = kb0 + i;
                if (!ptx::mbar_wait(&bars->empty[s], ((i / stages) & 1u) ^ 1u, abort_flag, P.wait_ns)) { failed = true; bars->abort = 1u; break; }
                unsigned char* p_s = base + s * stage_bytes;
                unsigned char* q_s = p_s + kSkinnySmemP;
                ptx::mbar_arrive_expect_tx(&bars->full[s], stage_bytes);
                // rows, columns and contraction indices past the end of a matrix read as zero
                if (P.a_mn) {
                    ptx::tma_load_2d(p_s, &tmP, r0, kb * 64, &bars->full[s]);
                    ptx::tma_load_2d(p_s + 8192, &tmP, r0 + 64, kb * 64, &bars->full[s]);
                } else {
                    ptx::tma_load_2d(p_s, &tmP, kb * 64, r0, &bars->full[s]);
                }
                if (P.b_mn) {
                    for (int h = 0; h < P.rp / 64; ++h) ptx::tma_load_2d(q_s + h * 8192, &tmQ, h * 64, kb * 64, &bars->full[s]);
                } else {
                    ptx::tma_load_2d(q_s, &tmQ, kb * 64, 0, &bars->full[s]);
                }
                issued = i + 1;
            }
            if (failed) {   // let the copies in flight land before the shared memory is given back
                for (int back = 1; back <= stages && back <= issued; ++back)
                    ptx::mbar_wait(&bars->full[(issued - back) % stages], ((issued - back) / stages) & 1u, nullptr, 2000000ull);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc = ptx::umma_idesc_bf16(128, P.rp) | (P.a_mn ? (1u << 15) : 0u) | (P.b_mn ? (1u << 16) : 0u);
            const uint32_t a_step = P.a_mn ? 128u : 2u, b_step = P.b_mn ? 128u : 2u;   // 16 contraction indices further
            for (int i = 0; i < n_my; ++i) {
                const int s = i % stages;
                if (!ptx::mbar_wait(&bars->full[s], (i / stages) & 1u, abort_flag, P.wait_ns)) { failed = true; bars->abort = 1u; break; }
                ptx::tc_fence_after();
                const uint32_t p_addr = ptx::smem_u32(base + s * stage_bytes);
                const uint32_t q_addr = p_addr + kSkinnySmemP;
                const uint64_t adesc = P.a_mn ? ptx::umma_desc_mn_sw128(p_addr, 8192u) : ptx::umma_desc_k_sw128(p_addr);
                const uint64_t bdesc = P.b_mn ? ptx::umma_desc_mn_sw128(q_addr, 8192u) : ptx::umma_desc_k_sw128(q_addr);
#pragma unroll
                for (int kk = 0; kk < 4; ++kk)
                    ptx::umma_bf16(tmem_base, adesc + a_step * kk, bdesc + b_step * kk, idesc, (i | kk) != 0 ? 1u : 0u);
                ptx::umma_commit(&bars->empty[s]);
            }
            if (!failed && n_my > 0) ptx::umma_commit(&bars->tmem_full);
        }
    } else {
        // ------------------------------------------------------------------ TMEM -> fp32 partial tile in shared memory
        const int q = warp & 3;
        const int row = q * 32 + lane;
        if (n_my > 0 && !ptx::mbar_wait_warp(&bars->tmem_full, 0u, abort_flag, P.wait_ns)) { failed = true; bars->abort = 1u; }
        if (!failed) {
            ptx::tc_fence_after();
            for (int c0 = 0; c0 < P.rp; c0 += 32) {
                uint32_t v[32];
                if (n_my > 0) {
                    ptx::tmem_ld_32x32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)c0, v);
                    ptx::tmem_ld_wait();
                } else {
#pragma unroll
                    for (int j = 0; j < 32; ++j) v[j] = 0u;
                }
                float4* dst = reinterpret_cast<float4*>(part + row * pstride + c0);
#pragma unroll
                for (int j = 0; j < 8; ++j)
                    dst[j] = make_float4(__uint_as_float(v[4 * j]), __uint_as_float(v[4 * j + 1]), __uint_as_float(v[4 * j + 2]),
                                         __uint_as_float(v[4 * j + 3]));
            }
            ptx::tc_fence_before();
        }
    }
    if (failed) atomicExch(P.status, aligned ? (uint32_t)LOWRA_ERR_TIMEOUT : (uint32_t)LOWRA_ERR_CUDA);
    __syncwarp();
    ptx::cluster_sync();   // every partial tile of the cluster is in place

    // ---------------------------------------------------------------------- sum over the slices, round, write
    if (warp >= 2 && bars->abort == 0u) {
        const int t = threadIdx.x - 64;
        const int rows_per = 128 / S, row_base = (int)crank * rows_per;
        const uint32_t part_addr = ptx::smem_u32(part);
        if (!P.transposed) {
            // out [R, ld_out]: four neighbouring columns per thread
            const int c4n = P.rp / 4;
            for (int u = t; u < rows_per * c4n; u += 128) {
                const int row = row_base + u / c4n, col = (u % c4n) * 4;
                const uint32_t addr = part_addr + (uint32_t)(row * pstride + col) * 4u;
                float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
                for (int p = 0; p < S; ++p) {
                    const float4 v = ptx::ld_cluster_f4(ptx::map_to_cta(addr, (uint32_t)p));
                    acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
                }
                const int grow = r0 + row;
                if (grow < P.R && col < P.n_cols) {
                    uint2 w;
                    w.x = pack_bf16x2(acc.x * P.scale, acc.y * P.scale);
                    w.y = pack_bf16x2(acc.z * P.scale, acc.w * P.scale);
                    *reinterpret_cast<uint2*>(P.out + (size_t)grow * P.ld_out + col) = w;
                }
            }
        } else {
            // out [n_cols, ld_out] = D^T.  A warp takes 8 rows x 16 columns of D: its loads read whole 64-byte runs of
            // a row, its stores write 8 neighbouring elements (rows of D) of 16 rows of out.
            const int c4n = P.rp / 4;
            const int lane_row = lane & 7, lane_c4 = lane >> 3;
            const int units = (rows_per / 8) * (c4n / 4);          // 8 x 16 patches of this CTA's rows
            for (int u = warp - 2; u < units; u += 4) {
                const int row = row_base + (u % (rows_per / 8)) * 8 + lane_row;
                const int col = ((u / (rows_per / 8)) * 4 + lane_c4) * 4;
                const uint32_t addr = part_addr + (uint32_t)(row * pstride + col) * 4u;
                float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
                for (int p = 0; p < S; ++p) {
                    const float4 v = ptx::ld_cluster_f4(ptx::map_to_cta(addr, (uint32_t)p));
                    acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
                }
                const int grow = r0 + row;
                if (grow < P.R && col < P.n_cols) {
                    uint16_t* dst = P.out + (size_t)col * P.ld_out + grow;
                    dst[0] = (uint16_t)pack_bf16x2(acc.x * P.scale, 0.0f);
                    dst[(size_t)P.ld_out] = (uint16_t)pack_bf16x2(acc.y * P.scale, 0.0f);
                    dst[2 * (size_t)P.ld_out] = (uint16_t)pack_bf16x2(acc.z * P.scale, 0.0f);
                    dst[3 * (size_t)P.ld_out] = (uint16_t)pack_bf16x2(acc.w * P.scale, 0.0f);
                }
            }
        }
    }
    ptx::cluster_sync();   // nobody leaves while a peer still reads its partial tile
    if (warp == 1) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc(tmem_base, tmem_cols);
    }
}

}  // namespace

// tmP: box of [64 c][64 rows] (a_mn) or [128 rows][64 c]; tmQ: box of [64 c][64 columns] (b_mn) or [rp columns][64 c].
lowra_status launch_skinny(const CUtensorMap& tmP, const CUtensorMap& tmQ, const SkinnyArgs& a, cudaStream_t stream) {
    static SmemLimit limit = {};
    if (ensure_smem_limit(reinterpret_cast<const void*>(skinny_kernel), kSkinnySmemBytes, &limit) != LOWRA_OK) return LOWRA_ERR_CUDA;
    const int tiles = (a.R + 127) / 128, n_blocks = (a.C + 63) / 64;
    // split of the contraction: the one with the shortest estimated run = waves of CTAs x (blocks per CTA + a fixed
    // cost of set-up, pipeline fill and reduction, about six blocks' worth); every slice keeps four blocks or more
    int S = 1;
    long best = -1;
    for (int c = 1; c <= kSkinnyMaxSplit && (c == 1 || n_blocks >= 4 * c); c *= 2) {
        const long waves = ((long)tiles * c + kSkinnySlots - 1) / kSkinnySlots;
        const long cost = waves * ((n_blocks + c - 1) / c + 6);
        if (best < 0 || cost < best) { best = cost; S = c; }
    }
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 1;
    attr[0].val.clusterDim.y = (unsigned)S;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.gridDim = dim3((unsigned)tiles, (unsigned)S, 1);
    cfg.blockDim = dim3(kSkinnyThreads, 1, 1);
    cfg.dynamicSmemBytes = kSkinnySmemBytes;
    cfg.stream = stream;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, skinny_kernel, a, S, tmP, tmQ) == cudaSuccess ? LOWRA_OK : LOWRA_ERR_CUDA;
}

}  // namespace lowra
