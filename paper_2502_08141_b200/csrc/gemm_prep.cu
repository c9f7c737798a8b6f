// Prologue of the fused forward / backward-input calls: one launch that
//   (A) computes the LoRA down-projection  T = s * X . A   (forward)  or  U = s * dY . B^T  (backward)
//       with warp-level tensor-core MMAs, rounded once to bf16, zero-padded to a multiple of 64 columns;
//   (B) writes the other LoRA factor as a K-major, zero-padded bf16 matrix that TMA can fetch:
//       Bt[n, j] = B[j, n] (forward)  or  Ap[k, j] = A[k, j] (backward);
//   (C) deals the rows of every group of 128 (forward) or 64 (backward) consecutive output channels to the
//       256 dequant threads of the main kernel so that each warp only holds rows of one precision;
//   and clears the device status word.
#include "gemm_params.cuh"
#include "ptx.cuh"

namespace lowra {

namespace {

constexpr int kTM = kPrepTokens;   // tokens per CTA
constexpr int kDC = 128;           // contraction elements per pipeline stage
constexpr int kPrepStages = 3;
constexpr int kInPitch = kDC + 8;  // bf16 elements; +8 keeps ldmatrix rows on distinct banks

__device__ __forceinline__ int f_tile_elems(int rp, bool f_is_A) {
    return f_is_A ? kDC * (rp + 8) : rp * (kDC + 8);
}

// ------------------------------------------------------------------------------------------ role A
__device__ void down_projection(const PrepParams& P, int tile, unsigned char* smem_raw) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int m0 = tile * kTM;
    const int rp = P.rp;
    const int in_elems = kTM * kInPitch;
    const int f_elems = f_tile_elems(rp, P.f_is_A);
    const int stage_elems = in_elems + f_elems;
    uint16_t* smem = reinterpret_cast<uint16_t*>(smem_raw);
    const int n_chunks = (P.C + kDC - 1) / kDC;

    auto issue = [&](int chunk, int stage) {
        if (chunk < n_chunks) {
            const int c0 = chunk * kDC;
            uint16_t* in_s = smem + stage * stage_elems;
            uint16_t* f_s = in_s + in_elems;
            // In tile: kTM rows x 16 chunks of 8 elements
            for (int i = tid; i < kTM * (kDC / 8); i += kPrepThreads) {
                const int row = i / (kDC / 8), ch = i % (kDC / 8);
                const bool ok = (m0 + row < P.M) && (c0 + ch * 8 < P.C);
                const uint16_t* src = ok ? P.In + (size_t)(m0 + row) * P.C + c0 + ch * 8 : P.In;
                ptx::cp_async_16(ptx::smem_u32(in_s + row * kInPitch + ch * 8), src, ok);
            }
            if (P.f_is_A) {  // tile [c][j], pitch rp + 8; F(c, j) = F[c * r + j]
                const int cpr = rp / 8;
                for (int i = tid; i < kDC * cpr; i += kPrepThreads) {
                    const int c = i / cpr, j8 = i % cpr;
                    const bool ok = (c0 + c < P.C) && (j8 * 8 < P.r);
                    const uint16_t* src = ok ? P.F + (size_t)(c0 + c) * P.r + j8 * 8 : P.F;
                    ptx::cp_async_16(ptx::smem_u32(f_s + c * (rp + 8) + j8 * 8), src, ok);
                }
            } else {         // tile [j][c], pitch kDC + 8; F(c, j) = F[j * C + c]
                for (int i = tid; i < rp * (kDC / 8); i += kPrepThreads) {
                    const int j = i / (kDC / 8), ch = i % (kDC / 8);
                    const bool ok = (j < P.r) && (c0 + ch * 8 < P.C);
                    const uint16_t* src = ok ? P.F + (size_t)j * P.C + c0 + ch * 8 : P.F;
                    ptx::cp_async_16(ptx::smem_u32(f_s + j * (kDC + 8) + ch * 8), src, ok);
                }
            }
        }
        ptx::cp_async_commit();
    };

    const int nt_per_warp = rp / 32;  // n8 tiles per warp: 2 (rp = 64) or 4 (rp = 128)
    float acc[2][4][4];
#pragma unroll
    for (int a = 0; a < 2; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b)
#pragma unroll
            for (int c = 0; c < 4; ++c) acc[a][b][c] = 0.0f;

    for (int s = 0; s < kPrepStages - 1; ++s) issue(s, s);

    for (int chunk = 0; chunk < n_chunks; ++chunk) {
        issue(chunk + kPrepStages - 1, (chunk + kPrepStages - 1) % kPrepStages);
        ptx::cp_async_wait<kPrepStages - 1>();
        __syncthreads();
        const uint16_t* in_s = smem + (chunk % kPrepStages) * stage_elems;
        const uint16_t* f_s = in_s + in_elems;
#pragma unroll
        for (int kk = 0; kk < kDC / 16; ++kk) {
            const int k0 = kk * 16;
            uint32_t a[2][4];
#pragma unroll
            for (int mt = 0; mt < 2; ++mt) {
                const int row = mt * 16 + (lane & 7) + 8 * ((lane >> 3) & 1);
                const int col = k0 + 8 * (lane >> 4);
                ptx::ldmatrix_x4(ptx::smem_u32(in_s + row * kInPitch + col), a[mt][0], a[mt][1], a[mt][2], a[mt][3]);
            }
#pragma unroll
            for (int nt = 0; nt < 4; ++nt) {
                if (nt < nt_per_warp) {
                    const int n0 = (warp * nt_per_warp + nt) * 8;
                    uint32_t b0, b1;
                    if (P.f_is_A) {
                        const int krow = k0 + (lane & 15);
                        ptx::ldmatrix_x2_trans(ptx::smem_u32(f_s + krow * (rp + 8) + n0), b0, b1);
                    } else {
                        const int nrow = n0 + (lane & 7);
                        const int col = k0 + 8 * ((lane >> 3) & 1);
                        ptx::ldmatrix_x2(ptx::smem_u32(f_s + nrow * (kDC + 8) + col), b0, b1);
                    }
#pragma unroll
                    for (int mt = 0; mt < 2; ++mt)
                        ptx::mma_16816(acc[mt][nt], a[mt][0], a[mt][1], a[mt][2], a[mt][3], b0, b1);
                }
            }
        }
        __syncthreads();
    }
    ptx::cp_async_wait<0>();

    const int g = lane >> 2, t = lane & 3;
#pragma unroll
    for (int mt = 0; mt < 2; ++mt)
#pragma unroll
        for (int nt = 0; nt < 4; ++nt) {
            if (nt < nt_per_warp) {
                const int n = (warp * nt_per_warp + nt) * 8 + 2 * t;
                const int mA = m0 + mt * 16 + g, mB = mA + 8;
                if (mA < P.M)
                    *reinterpret_cast<uint32_t*>(P.T + (size_t)mA * rp + n) =
                        pack_bf16x2(P.s * acc[mt][nt][0], P.s * acc[mt][nt][1]);
                if (mB < P.M)
                    *reinterpret_cast<uint32_t*>(P.T + (size_t)mB * rp + n) =
                        pack_bf16x2(P.s * acc[mt][nt][2], P.s * acc[mt][nt][3]);
            }
        }
}

// ------------------------------------------------------------------------------------------ role B
// Dst [R, rp]: forward Dst[n, j] = Src[j * R + n] (Src = B [r, N]); backward Dst[k, j] = Src[k * r + j].
__device__ void pad_factor(const PrepParams& P, int blk) {
    const int rp = P.rp;
    const size_t total = (size_t)P.R * rp;
    for (size_t i = (size_t)blk * kPrepThreads + threadIdx.x; i < total; i += (size_t)P.blocksB * kPrepThreads) {
        uint16_t v = 0;
        if (P.src_transposed) {
            // consecutive threads walk along n so that the reads of Src are contiguous
            const int j = (int)(i / P.R), n = (int)(i % P.R);
            if (j < P.r) v = P.Src[(size_t)j * P.R + n];
            P.Dst[(size_t)n * rp + j] = v;
        } else {
            const int k = (int)(i / rp), j = (int)(i % rp);
            if (j < P.r) v = P.Src[(size_t)k * P.r + j];
            P.Dst[i] = v;
        }
    }
}

// ------------------------------------------------------------------------------------------ role C
// One warp per group of G rows (128 forward, 64 backward).  The rows are ordered by precision class
// (1 bit, 2 bits, 4 bits, rows past N; stable) and cut into chunks of CH rows of one class (32 forward;
// 16 backward, where every row is handled by two threads, one per 64-feature half), so that no warp of
// the main kernel ever sees two precisions.  At most G / CH + 3 = 7 chunks exist and the kernel has 8
// dequant warps: with n chunks, k = 8 / n warps share a chunk and take turns over the stages
// (warp c + j * n serves chunk c at the stages whose index is congruent to j mod k).
__device__ void deal_rows(const PrepParams& P, int blk) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int G = P.group, per = G / 32;
    const int CH = (G == 128) ? 32 : 16;
    const int n_groups = (P.N + G - 1) / G;
    for (int grp = blk * (kPrepThreads / 32) + warp; grp < n_groups; grp += P.blocksC * (kPrepThreads / 32)) {
        uint32_t* out = P.items + (size_t)grp * 256;
#pragma unroll
        for (int i = 0; i < 8; ++i) out[i * 32 + lane] = 0xFFFFFFFFu;
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
        const int n_chunks = chunk_base[3] + (total[3] + CH - 1) / CH;
        const int k = 8 / n_chunks;
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
                        for (int j = 0; j < k; ++j) {
                            // backward: the group index is the stage index, so only the warp whose turn it
                            // is gets the row; forward: all k warps get it and take turns over the stages
                            if (CH == 16 && j != (grp & (k - 1))) continue;
                            const int thread = (chunk_base[c] + q / CH + j * n_chunks) * 32 + q % CH;
                            out[thread] = word;
                            if (CH == 16) out[thread + 16] = word;
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
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int b = blockIdx.x;
    if (b == 0 && threadIdx.x == 0) *P.status = 0u;
    if (b < P.blocksA) down_projection(P, b, smem_raw);
    else if (b < P.blocksA + P.blocksB) pad_factor(P, b - P.blocksA);
    else deal_rows(P, b - P.blocksA - P.blocksB);
}

static size_t prep_smem_bytes(int rp) {
    const int f = (kDC * (rp + 8) > rp * (kDC + 8)) ? kDC * (rp + 8) : rp * (kDC + 8);
    return (size_t)kPrepStages * (kTM * kInPitch + f) * sizeof(uint16_t);
}

lowra_status launch_prep(const PrepParams& P, cudaStream_t stream) {
    static bool configured = false;
    if (!configured) {
        if (cudaFuncSetAttribute(prep_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)prep_smem_bytes(128)) != cudaSuccess)
            return LOWRA_ERR_CUDA;
        configured = true;
    }
    prep_kernel<<<P.blocksA + P.blocksB + P.blocksC, kPrepThreads, prep_smem_bytes(P.rp), stream>>>(P);
    return cudaGetLastError() == cudaSuccess ? LOWRA_OK : LOWRA_ERR_CUDA;
}

}  // namespace lowra
