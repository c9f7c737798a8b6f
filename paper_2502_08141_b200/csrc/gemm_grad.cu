// Gradients of the low-rank factors: dA = X^T . U  [K, r]  and  dB = (dY^T . T)^T  [r, N], where
// U = s dY B^T and T = s X A (bf16, [tokens, rank padded to 64]) have been produced by the down-projection tiles
// of the fused kernels.  Both products contract over the tokens:
//     D [128 rows x rp ranks] = sum over tokens  P[token, row] * Q[token, rank]
// with P = X (rows = input features) or dY (rows = output channels) and Q = U or T.  Both operands of
// tcgen05.mma are therefore "MN-major": a contraction index (a token) is a 128-byte row of 64 consecutive rows
// (resp. ranks), exactly how the tiles lie in the row-major matrices, so TMA delivers them as they are.
//
// One CTA per tile of 128 rows; 64 tokens per pipeline stage, four stages; warp 0 = TMA, warp 1 = MMA issue,
// warps 2-5 = epilogue (TMEM -> bf16 -> global).  The products are skinny (2 M r (K + N) FLOPs, 2-3 % of the
// layer's), so this kernel is a plain single-CTA pipeline.  All waits are bounded.
#include "gemm_params.cuh"
#include "ptx.cuh"

namespace lowra {

namespace {

constexpr uint64_t kGradWaitNs = 1000ull * 1000ull * 1000ull;
constexpr int kGradStages = 4;
constexpr int kGradThreads = 192;                      // 6 warps
constexpr uint32_t kGradSmemA = 128 * 64 * 2;          // 16 KB: [row half][64 tokens][64 rows]
constexpr uint32_t kGradSmemB = 128 * 64 * 2;          // 16 KB: [rank half][64 tokens][64 ranks] (8 KB used when rp = 64)
constexpr uint32_t kGradSmemBytes = kGradStages * (kGradSmemA + kGradSmemB) + 1024;

struct GradBarriers {
    uint64_t full[kGradStages];
    uint64_t empty[kGradStages];
    uint64_t tmem_full;
    uint32_t tmem_base;
    uint32_t abort;
};

struct GradParams {
    uint16_t* out;        // dA [R, r] (transposed == 0) or dB [r, R] (transposed == 1), bf16
    uint32_t* status;
    int R;                // rows of P in total (K or N)
    int M;                // tokens
    int r, rp;            // rank, rank rounded up to 64
    int transposed;
};

__global__ void __launch_bounds__(kGradThreads, 1)
grad_kernel(const GradParams P, const __grid_constant__ CUtensorMap tmP, const __grid_constant__ CUtensorMap tmQ) {
    extern __shared__ __align__(1024) unsigned char grad_smem[];
    unsigned char* base = grad_smem;
    GradBarriers* bars = reinterpret_cast<GradBarriers*>(base + kGradStages * (kGradSmemA + kGradSmemB));
    volatile uint32_t* abort_flag = &bars->abort;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int r0 = blockIdx.x * 128;
    const int n_blocks = (P.M + 63) / 64;
    const uint32_t tmem_cols = 128;   // >= rp, power of two

    if ((ptx::smem_u32(grad_smem) & 1023u) != 0u) {
        if (threadIdx.x == 0) atomicExch(P.status, (uint32_t)LOWRA_ERR_CUDA);
        return;
    }
    if (threadIdx.x == 0) {
        for (int s = 0; s < kGradStages; ++s) { ptx::mbar_init(&bars->full[s], 1); ptx::mbar_init(&bars->empty[s], 1); }
        ptx::mbar_init(&bars->tmem_full, 1);
        bars->abort = 0u;
        ptx::fence_barrier_init();
        ptx::prefetch_tensormap(&tmP);
        ptx::prefetch_tensormap(&tmQ);
    }
    if (warp == 1) ptx::tmem_alloc(&bars->tmem_base, tmem_cols);
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem_base = bars->tmem_base;
    pdl_enter();   // T and U come from the kernels launched before this one
    bool failed = false;

    if (warp == 0) {
        if (lane == 0) {
            const uint32_t bytes = kGradSmemA + (uint32_t)(P.rp / 64) * 8192u;
            for (int kb = 0; kb < n_blocks; ++kb) {
                const int s = kb % kGradStages;
                if (!ptx::mbar_wait(&bars->empty[s], ((kb / kGradStages) & 1u) ^ 1u, abort_flag, kGradWaitNs)) { failed = true; bars->abort = 1u; break; }
                unsigned char* a_s = base + s * (kGradSmemA + kGradSmemB);
                unsigned char* b_s = a_s + kGradSmemA;
                ptx::mbar_arrive_expect_tx(&bars->full[s], bytes);
                // boxes of 64 columns x 64 tokens; rows / ranks past the end of the matrix read as zero
                ptx::tma_load_2d(a_s, &tmP, r0, kb * 64, &bars->full[s]);
                ptx::tma_load_2d(a_s + 8192, &tmP, r0 + 64, kb * 64, &bars->full[s]);
                for (int h = 0; h < P.rp / 64; ++h) ptx::tma_load_2d(b_s + h * 8192, &tmQ, h * 64, kb * 64, &bars->full[s]);
            }
            if (failed) {   // let the copies in flight land before the shared memory is given back
                for (int back = 1; back <= kGradStages && back <= n_blocks; ++back)
                    ptx::mbar_wait(&bars->full[(n_blocks - back) % kGradStages], ((n_blocks - back) / kGradStages) & 1u, nullptr, 2000000ull);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            // M = 128 rows, N = rp ranks, both operands MN-major
            const uint32_t idesc = ptx::umma_idesc_bf16(128, P.rp) | (1u << 15) | (1u << 16);
            for (int kb = 0; kb < n_blocks; ++kb) {
                const int s = kb % kGradStages;
                if (!ptx::mbar_wait(&bars->full[s], (kb / kGradStages) & 1u, abort_flag, kGradWaitNs)) { failed = true; bars->abort = 1u; break; }
                ptx::tc_fence_after();
                const uint32_t a_addr = ptx::smem_u32(base + s * (kGradSmemA + kGradSmemB));
                const uint64_t adesc = ptx::umma_desc_mn_sw128(a_addr, 8192u);
                const uint64_t bdesc = ptx::umma_desc_mn_sw128(a_addr + kGradSmemA, 8192u);
#pragma unroll
                for (int kk = 0; kk < 4; ++kk)   // 16 tokens = two 1024-byte groups per MMA
                    ptx::umma_bf16(tmem_base, adesc + 128u * kk, bdesc + 128u * kk, idesc, (kb | kk) != 0 ? 1u : 0u);
                ptx::umma_commit(&bars->empty[s]);
            }
            if (!failed) ptx::umma_commit(&bars->tmem_full);
        }
    } else {
        // ------------------------------------------------------------------ epilogue: thread = row, registers = ranks
        const int q = warp & 3;
        const int row = r0 + q * 32 + lane;
        if (!ptx::mbar_wait_warp(&bars->tmem_full, 0u, abort_flag, kGradWaitNs)) { failed = true; bars->abort = 1u; }
        if (!failed) {
            ptx::tc_fence_after();
            for (int c0 = 0; c0 < P.rp; c0 += 32) {
                uint32_t v[32];
                ptx::tmem_ld_32x32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)c0, v);
                ptx::tmem_ld_wait();
                if (row < P.R) {
                    if (!P.transposed) {
                        // dA [R, r]: this row's ranks are contiguous
#pragma unroll
                        for (int j = 0; j < 32; j += 2) {
                            if (c0 + j + 1 < P.r) {
                                *reinterpret_cast<uint32_t*>(P.out + (size_t)row * P.r + c0 + j) =
                                    pack_bf16x2(__uint_as_float(v[j]), __uint_as_float(v[j + 1]));
                            } else if (c0 + j < P.r) {
                                P.out[(size_t)row * P.r + c0 + j] = (uint16_t)pack_bf16x2(__uint_as_float(v[j]), 0.0f);
                            }
                        }
                    } else {
                        // dB [r, R]: the 32 lanes of the warp write 32 neighbouring columns of one rank
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            if (c0 + j < P.r) P.out[(size_t)(c0 + j) * P.R + row] = (uint16_t)pack_bf16x2(__uint_as_float(v[j]), 0.0f);
                    }
                }
            }
            ptx::tc_fence_before();
        }
    }
    if (failed) atomicExch(P.status, (uint32_t)LOWRA_ERR_TIMEOUT);
    __syncthreads();
    if (warp == 1) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc(tmem_base, tmem_cols);
    }
}

}  // namespace

// P: bf16 [M, R] row-major (X or dY); Q: bf16 [M, rp] row-major (U or T); out: dA [R, r] or dB [r, R].
lowra_status launch_grad(const CUtensorMap& tmP, const CUtensorMap& tmQ, uint16_t* out, uint32_t* status, int R, int M, int r,
                         int rp, bool transposed, cudaStream_t stream) {
    static bool configured = false;
    if (!configured) {
        if (cudaFuncSetAttribute(grad_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kGradSmemBytes) != cudaSuccess)
            return LOWRA_ERR_CUDA;
        configured = true;
    }
    GradParams P;
    P.out = out;
    P.status = status;
    P.R = R;
    P.M = M;
    P.r = r;
    P.rp = rp;
    P.transposed = transposed ? 1 : 0;
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.gridDim = dim3((unsigned)((R + 127) / 128), 1, 1);
    cfg.blockDim = dim3(kGradThreads, 1, 1);
    cfg.dynamicSmemBytes = kGradSmemBytes;
    cfg.stream = stream;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, grad_kernel, P, tmP, tmQ) == cudaSuccess ? LOWRA_OK : LOWRA_ERR_CUDA;
}

}  // namespace lowra
