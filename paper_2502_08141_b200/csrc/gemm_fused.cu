// Fused dequant + LoRA tensor-core kernel (forward, backward-input, and a dense diagnostic mode).
//
// One persistent CTA per SM walks over output tiles of 128 "operand rows" x 256 tokens:
//   forward : operand rows = output channels n;  Y^T tile [128 n x 256 m]  = W_hat[n, :] . X[m, :]
//   backward: operand rows = input features k;   dX^T tile [128 k x 256 m] = W_hat[:, k] . dY[m, :]
// The 128-row operand (the weights) is the A operand of tcgen05.mma and is produced in shared memory by
// eight dequant warps straight from the packed codes (never from HBM as bf16); the 256-token operand
// (activations / output gradients) is the B operand and arrives by TMA.  The accumulator lives in
// TMEM (two 128 x 256 fp32 buffers, so the epilogue of one tile overlaps the main loop of the next).
// The LoRA term is folded into the same accumulator as extra contraction blocks whose operands
// (the padded factor and the down-projected activations from the prologue) both arrive by TMA.
//
// Warp roles: 0 = TMA producer, 1 = MMA issuer (and TMEM owner), 2-5 = epilogue, 6-13 = dequant.
// All mbarrier waits are bounded; a wait that runs out sets the status word and every role leaves.
#include "gemm_params.cuh"
#include "ptx.cuh"

namespace lowra {

namespace {

constexpr uint64_t kWaitLimitNs = 1000ull * 1000ull * 1000ull;  // 1 s per wait
constexpr uint32_t kIdesc = ptx::umma_idesc_bf16(kTileR, kTileT);

struct Barriers {
    uint64_t full_x[kStages];   // TMA bytes of a stage have landed
    uint64_t full_w[kStages];   // dequant warps have written (or skipped) a stage
    uint64_t empty[kStages];    // the MMAs reading a stage have completed
    uint64_t tmem_full[2];
    uint64_t tmem_empty[2];
    uint64_t drain;
    uint32_t tmem_base;
    uint32_t abort;
};

// rowinfo word written by the prologue: bits 0-6 row offset inside its group, 7-8 class (3 = past N),
// 9-31 stored position.
__device__ __forceinline__ int info_row(uint32_t w) { return (int)(w & 127u); }
__device__ __forceinline__ int info_class(uint32_t w) { return (int)((w >> 7) & 3u); }
__device__ __forceinline__ int info_pos(uint32_t w) { return (int)(w >> 9); }

// ---- dequantisation of 8 consecutive elements to 8 bf16 (one 16-byte chunk) ----------------------
// 1 bit: LH = {level0 * absmax, level1 * absmax} as bf16x2; each output word picks two halves.
__device__ __forceinline__ uint4 deq8_b1(uint32_t bits8, uint32_t LH) {
    uint32_t o[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const uint32_t v = (bits8 >> (2 * j)) & 3u;
        const uint32_t sel = ((v * 0x1122u) & 0x2222u) | 0x1010u;
        o[j] = __byte_perm(LH, LH, sel);
    }
    return make_uint4(o[0], o[1], o[2], o[3]);
}

// 2 bits: E01 = {level0, level1} * absmax, E23 = {level2, level3} * absmax, bf16x2 each.
__device__ __forceinline__ uint4 deq8_b2(uint32_t bits16, uint32_t E01, uint32_t E23) {
    uint32_t o[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const uint32_t y = bits16 >> (4 * j);
        const uint32_t t = (y & 3u) | ((y << 6) & 0x300u);
        const uint32_t sel = t * 0x22u + 0x1010u;
        o[j] = __byte_perm(E01, E23, sel);
    }
    return make_uint4(o[0], o[1], o[2], o[3]);
}

// 4 bits: per-thread table of the 16 unscaled fp32 levels in shared memory (entry e at lut[e * stride]).
__device__ __forceinline__ uint4 deq8_b4(uint32_t bits32, const float* lut, int stride, float a) {
    uint32_t o[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const uint32_t c0 = (bits32 >> (8 * j)) & 15u;
        const uint32_t c1 = (bits32 >> (8 * j + 4)) & 15u;
        o[j] = pack_bf16x2(__fmul_rn(lut[c0 * stride], a), __fmul_rn(lut[c1 * stride], a));
    }
    return make_uint4(o[0], o[1], o[2], o[3]);
}

// Packed bits of `nbits` (32, 64 or 128) starting at p.
__device__ __forceinline__ uint4 load_bits(const uint8_t* p, int cls) {
    uint4 q = make_uint4(0u, 0u, 0u, 0u);
    if (cls == 0) {
        q.x = __ldg(reinterpret_cast<const uint32_t*>(p));
    } else if (cls == 1) {
        const uint2 t = __ldg(reinterpret_cast<const uint2*>(p));
        q.x = t.x;
        q.y = t.y;
    } else if (cls == 2) {
        q = __ldg(reinterpret_cast<const uint4*>(p));
    }
    return q;
}

// The 8 elements number x (0..3) of a thread's 32 elements.
__device__ __forceinline__ uint32_t chunk_bits(const uint4& q, int cls, int x) {
    if (cls == 0) return (q.x >> (8 * x)) & 0xFFu;
    if (cls == 1) return (((x & 2) ? q.y : q.x) >> ((x & 1) * 16)) & 0xFFFFu;
    return x == 0 ? q.x : x == 1 ? q.y : x == 2 ? q.z : q.w;
}

struct RowState {
    const uint8_t* bits_ptr;   // this thread's first packed byte of the row (block 0)
    const float* absmax_ptr;
    float m0, m1, m2, m3;      // levels for 1- and 2-bit rows
    int cls;                   // 0,1,2 = 1,2,4 bits; 3 = row past the end
};

__device__ __forceinline__ uint4 deq_chunk(const RowState& rs, const uint4& q, int x, float a, uint32_t LH,
                                           uint32_t E01, uint32_t E23, const float* lut, int lut_stride) {
    const uint32_t bits = chunk_bits(q, rs.cls, x);
    if (rs.cls == 0) return deq8_b1(bits, LH);
    if (rs.cls == 1) return deq8_b2(bits, E01, E23);
    if (rs.cls == 2) return deq8_b4(bits, lut, lut_stride, a);
    return make_uint4(0u, 0u, 0u, 0u);
}

}  // namespace

template <int MODE>
__global__ void __launch_bounds__(kGemmThreads, 1)
fused_kernel(const GemmParams P, const __grid_constant__ CUtensorMap tmB, const __grid_constant__ CUtensorMap tmB2,
             const __grid_constant__ CUtensorMap tmA2) {
    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw_addr = ptx::smem_u32(smem_raw);
    unsigned char* base = smem_raw + ((1024u - (raw_addr & 1023u)) & 1023u);
    unsigned char* out_s = base + kStages * kSmemStage;
    float* lut4 = reinterpret_cast<float*>(out_s + kSmemOut);
    Barriers* bars = reinterpret_cast<Barriers*>(out_s + kSmemOut + kSmemLut4);
    volatile uint32_t* abort_flag = &bars->abort;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int total_blocks = P.lora_blocks + P.main_blocks;
    const int n_tiles = P.tiles_r * P.tiles_t;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            ptx::mbar_init(&bars->full_x[s], 1);
            ptx::mbar_init(&bars->full_w[s], kProducerWarps);
            ptx::mbar_init(&bars->empty[s], 1);
        }
        for (int a = 0; a < 2; ++a) {
            ptx::mbar_init(&bars->tmem_full[a], 1);
            ptx::mbar_init(&bars->tmem_empty[a], 4);
        }
        ptx::mbar_init(&bars->drain, 1);
        bars->abort = 0u;
        ptx::fence_barrier_init();
        ptx::prefetch_tensormap(&tmB);
        if (P.lora_blocks > 0) ptx::prefetch_tensormap(&tmB2);
        if (P.lora_blocks > 0 || MODE == kModeDense) ptx::prefetch_tensormap(&tmA2);
    }
    if (warp == 1) ptx::tmem_alloc(&bars->tmem_base, kTmemCols);
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem_base = bars->tmem_base;

    bool failed = false;

    if (warp == 0) {
        // ================================================================== TMA producer
        if (lane == 0) {
            uint32_t it = 0;
            for (int tile = blockIdx.x; tile < n_tiles && !failed; tile += gridDim.x) {
                const int r0 = (tile % P.tiles_r) * kTileR, m0 = (tile / P.tiles_r) * kTileT;
                for (int kb = 0; kb < total_blocks; ++kb, ++it) {
                    const int s = it % kStages;
                    const uint32_t ph = (it / kStages) & 1u;
                    if (!ptx::mbar_wait(&bars->empty[s], ph ^ 1u, abort_flag, kWaitLimitNs)) { failed = true; bars->abort = 1u; break; }
                    unsigned char* a_s = base + s * kSmemStage;
                    unsigned char* b_s = a_s + kSmemA;
                    if (kb < P.lora_blocks) {
                        ptx::mbar_arrive_expect_tx(&bars->full_x[s], kSmemA + kSmemB);
                        ptx::tma_load_2d(a_s, &tmA2, kb * kTileC, r0, &bars->full_x[s]);
                        ptx::tma_load_2d(b_s, &tmB2, kb * kTileC, m0, &bars->full_x[s]);
                    } else {
                        const int c0 = (kb - P.lora_blocks) * kTileC;
                        if (MODE == kModeDense) {
                            ptx::mbar_arrive_expect_tx(&bars->full_x[s], kSmemA + kSmemB);
                            ptx::tma_load_2d(a_s, &tmA2, c0, r0, &bars->full_x[s]);
                        } else {
                            ptx::mbar_arrive_expect_tx(&bars->full_x[s], kSmemB);
                        }
                        ptx::tma_load_2d(b_s, &tmB, c0, m0, &bars->full_x[s]);
                    }
                }
            }
            if (failed) {
                // let this thread's own copies land before the CTA's shared memory is released
                for (uint32_t back = 1; back <= (uint32_t)kStages && back <= it; ++back) {
                    const uint32_t j = it - back;
                    ptx::mbar_wait(&bars->full_x[j % kStages], (j / kStages) & 1u, nullptr, 2000000ull);
                }
            }
        }
    } else if (warp == 1) {
        // ================================================================== MMA issuer
        if (lane == 0) {
            uint32_t it = 0, tile_iter = 0;
            for (int tile = blockIdx.x; tile < n_tiles && !failed; tile += gridDim.x, ++tile_iter) {
                const uint32_t acc = tile_iter & 1u, aph = (tile_iter >> 1) & 1u;
                if (!ptx::mbar_wait(&bars->tmem_empty[acc], aph ^ 1u, abort_flag, kWaitLimitNs)) { failed = true; bars->abort = 1u; break; }
                ptx::tc_fence_after();
                const uint32_t d_tmem = tmem_base + acc * kTileT;
                for (int kb = 0; kb < total_blocks; ++kb, ++it) {
                    const int s = it % kStages;
                    const uint32_t ph = (it / kStages) & 1u;
                    if (!ptx::mbar_wait(&bars->full_x[s], ph, abort_flag, kWaitLimitNs)) { failed = true; bars->abort = 1u; break; }
                    if (MODE != kModeDense)
                        if (!ptx::mbar_wait(&bars->full_w[s], ph, abort_flag, kWaitLimitNs)) { failed = true; bars->abort = 1u; break; }
                    ptx::tc_fence_after();
                    const uint32_t a_addr = ptx::smem_u32(base + s * kSmemStage);
                    const uint64_t adesc = ptx::umma_desc_k_sw128(a_addr);
                    const uint64_t bdesc = ptx::umma_desc_k_sw128(a_addr + kSmemA);
#pragma unroll
                    for (int kk = 0; kk < kTileC / 16; ++kk)  // 16 elements = 32 bytes along K per MMA
                        ptx::umma_bf16(d_tmem, adesc + 2u * kk, bdesc + 2u * kk, kIdesc, (kb | kk) != 0 ? 1u : 0u);
                    ptx::umma_commit(&bars->empty[s]);
                }
                if (failed) break;
                ptx::umma_commit(&bars->tmem_full[acc]);
            }
            if (failed) {
                ptx::umma_commit(&bars->drain);
                ptx::mbar_wait(&bars->drain, 0u, nullptr, 2000000ull);
            }
        }
    } else if (warp < kFirstProducerWarp) {
        // ================================================================== epilogue
        const int q = warp & 3;                 // TMEM lane quarter this warp may read
        const int et = (warp - kFirstEpilogueWarp) * 32 + lane;
        uint16_t* out16 = reinterpret_cast<uint16_t*>(out_s);
        const bool vec_ok = (P.ld_out % 8) == 0;
        uint32_t tile_iter = 0;
        for (int tile = blockIdx.x; tile < n_tiles && !failed; tile += gridDim.x, ++tile_iter) {
            const int r0 = (tile % P.tiles_r) * kTileR, m0 = (tile / P.tiles_r) * kTileT;
            const uint32_t acc = tile_iter & 1u, aph = (tile_iter >> 1) & 1u;
            // the four epilogue warps share named barriers, so they must agree on leaving
            if (!ptx::mbar_wait_warp(&bars->tmem_full[acc], aph, abort_flag, kWaitLimitNs)) bars->abort = 1u;
            ptx::named_barrier_sync(1, 128);
            if (*abort_flag != 0u) { failed = true; break; }
            ptx::tc_fence_after();
#pragma unroll 1
            for (int chunk = 0; chunk < kTileT / 32; ++chunk) {
                if (m0 + chunk * 32 >= P.M) break;
                uint32_t v[32];
                ptx::tmem_ld_32x32(tmem_base + ((uint32_t)(q * 32) << 16) + acc * kTileT + chunk * 32, v);
                ptx::tmem_ld_wait();
                // thread = operand row (channel), v[j] = token j: transpose through shared memory
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    const uint32_t two = pack_bf16x2(__uint_as_float(v[j]), 0.0f);
                    out16[j * kTileR + q * 32 + lane] = (uint16_t)two;
                }
                ptx::named_barrier_sync(1, 128);
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int idx = i * 128 + et;
                    const int row = idx >> 4, ch = idx & 15;
                    const int m = m0 + chunk * 32 + row, n = r0 + ch * 8;
                    if (m < P.M && n < P.R) {
                        const uint4 val = *reinterpret_cast<const uint4*>(out16 + row * kTileR + ch * 8);
                        uint16_t* dst = P.out + (size_t)m * P.ld_out + n;
                        if (vec_ok && n + 8 <= P.R) {
                            *reinterpret_cast<uint4*>(dst) = val;
                        } else {
                            const uint16_t* e = reinterpret_cast<const uint16_t*>(&val);
                            for (int t = 0; t < 8 && n + t < P.R; ++t) dst[t] = e[t];
                        }
                    }
                }
                ptx::named_barrier_sync(1, 128);
            }
            ptx::tc_fence_before();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(&bars->tmem_empty[acc]);
        }
    } else if (MODE != kModeDense) {
        // ================================================================== dequant producers
        const int pt = threadIdx.x - kFirstProducerWarp * 32;  // 0..255
        const float* lut = lut4 + pt;
        constexpr int kLutStride = kProducerWarps * 32;
        const int K = P.L.K;
        uint32_t it = 0;
        for (int tile = blockIdx.x; tile < n_tiles && !failed; tile += gridDim.x) {
            const int rt = tile % P.tiles_r;
            const int r0 = rt * kTileR;
            if (MODE == kModeForward) {
                // ------------------------------------------------------------ forward: row = channel
                // thread pair (2 lanes) per row, each 32 of the 64 elements of a stage
                const int slot = pt >> 1, h = pt & 1, jq = (lane >> 1) & 3;
                const uint32_t info = __ldg(P.rowinfo + (size_t)rt * kTileR + slot);
                const int row_local = info_row(info);
                RowState rs;
                rs.cls = info_class(info);
                rs.m0 = rs.m1 = rs.m2 = rs.m3 = 0.0f;
                rs.bits_ptr = P.packed;
                rs.absmax_ptr = P.absmax;
                int bits_stride = 0;  // packed bytes per 64-element block
                if (rs.cls < 3) {
                    const int p = info_pos(info);
                    const int b = 1 << rs.cls;
                    const int r = r0 + row_local;
                    bits_stride = 8 * b;
                    rs.bits_ptr = P.packed + P.L.seg_off[rs.cls] +
                                  (size_t)(p - P.L.class_start[rs.cls]) * ((size_t)K * b / 8) + h * (4 * b);
                    rs.absmax_ptr = P.absmax + (size_t)p * P.L.nb;
                    const float* mrow = P.maps + (size_t)r * kTableStride;
                    if (rs.cls == 0) {
                        rs.m0 = __ldg(mrow); rs.m1 = __ldg(mrow + 1);
                    } else if (rs.cls == 1) {
                        rs.m0 = __ldg(mrow); rs.m1 = __ldg(mrow + 1); rs.m2 = __ldg(mrow + 2); rs.m3 = __ldg(mrow + 3);
                    } else {
#pragma unroll
                        for (int e = 0; e < 16; ++e) lut4[e * kLutStride + pt] = __ldg(mrow + e);
                    }
                }
                const uint32_t row_off = (uint32_t)row_local * 128u;
                const int swz = row_local & 7;
                // two blocks of look-ahead
                uint4 q0 = make_uint4(0, 0, 0, 0), q1 = q0;
                float a0 = 0.0f, a1 = 0.0f;
                if (rs.cls < 3) {
                    q0 = load_bits(rs.bits_ptr, rs.cls);
                    a0 = __ldg(rs.absmax_ptr);
                    if (P.main_blocks > 1) {
                        q1 = load_bits(rs.bits_ptr + bits_stride, rs.cls);
                        a1 = __ldg(rs.absmax_ptr + 1);
                    }
                }
                for (int kb = 0; kb < total_blocks; ++kb, ++it) {
                    const int s = it % kStages;
                    const uint32_t ph = (it / kStages) & 1u;
                    if (!ptx::mbar_wait_warp(&bars->empty[s], ph ^ 1u, abort_flag, kWaitLimitNs)) { failed = true; bars->abort = 1u; break; }
                    if (kb >= P.lora_blocks) {
                        const int mb = kb - P.lora_blocks;
                        uint4 q2 = make_uint4(0, 0, 0, 0);
                        float a2 = 0.0f;
                        if (rs.cls < 3 && mb + 2 < P.main_blocks) {
                            q2 = load_bits(rs.bits_ptr + (size_t)(mb + 2) * bits_stride, rs.cls);
                            a2 = __ldg(rs.absmax_ptr + mb + 2);
                        }
                        const uint32_t a_s = ptx::smem_u32(base + s * kSmemStage) + row_off;
                        uint32_t LH = 0, E01 = 0, E23 = 0;
                        if (rs.cls == 0) {
                            LH = pack_bf16x2(__fmul_rn(rs.m0, a0), __fmul_rn(rs.m1, a0));
                        } else if (rs.cls == 1) {
                            E01 = pack_bf16x2(__fmul_rn(rs.m0, a0), __fmul_rn(rs.m1, a0));
                            E23 = pack_bf16x2(__fmul_rn(rs.m2, a0), __fmul_rn(rs.m3, a0));
                        }
#pragma unroll
                        for (int t = 0; t < 4; ++t) {
                            // rotate the chunk order so that the 8 lanes of a quarter-warp hit 8 distinct
                            // 16-byte bank groups whatever rows they own
                            const int x = ((jq + t) & 3) ^ (row_local & 3);
                            const uint4 val = deq_chunk(rs, q0, x, a0, LH, E01, E23, lut, kLutStride);
                            const int chunk_phys = (4 * h + x) ^ swz;
                            ptx::st_shared_v4(a_s + (uint32_t)chunk_phys * 16u, val);
                        }
                        q0 = q1; q1 = q2; a0 = a1; a1 = a2;
                        ptx::fence_proxy_async_smem();
                    }
                    __syncwarp();
                    if (lane == 0) ptx::mbar_arrive(&bars->full_w[s]);
                }
            } else {
                // ------------------------------------------------------------ backward: row = contraction index
                // every stage brings 64 new channels; 4 threads per channel, 32 input features each
                const int qslot = pt & 63, kq = pt >> 6;
                const int k_first = r0 + 32 * kq;       // first input feature of this thread
                const bool k_ok = k_first < K;          // K % 128 == 0, so all 32 are in range or none
                const uint32_t* infos = P.rowinfo;
                uint32_t info_next = (P.main_blocks > 0) ? __ldg(infos + qslot) : (3u << 7);
                for (int kb = 0; kb < total_blocks; ++kb, ++it) {
                    const int s = it % kStages;
                    const uint32_t ph = (it / kStages) & 1u;
                    uint4 q = make_uint4(0, 0, 0, 0);
                    float a = 0.0f;
                    RowState rs;
                    rs.cls = 3;
                    rs.m0 = rs.m1 = rs.m2 = rs.m3 = 0.0f;
                    int col = qslot;
                    if (kb >= P.lora_blocks) {
                        // fetch this stage's row before waiting for the slot (hides the load latency)
                        const int mb = kb - P.lora_blocks;
                        const uint32_t info = info_next;
                        if (mb + 1 < P.main_blocks) info_next = __ldg(infos + (size_t)(mb + 1) * kTileC + qslot);
                        col = info_row(info);
                        rs.cls = k_ok ? info_class(info) : 3;
                        if (rs.cls < 3) {
                            const int p = info_pos(info);
                            const int b = 1 << rs.cls;
                            const int n = mb * kTileC + col;
                            q = load_bits(P.packed + P.L.seg_off[rs.cls] +
                                              (size_t)(p - P.L.class_start[rs.cls]) * ((size_t)K * b / 8) +
                                              (size_t)k_first * b / 8,
                                          rs.cls);
                            a = __ldg(P.absmax + (size_t)p * P.L.nb + k_first / kBlock);
                            const float* mrow = P.maps + (size_t)n * kTableStride;
                            if (rs.cls == 0) {
                                rs.m0 = __ldg(mrow); rs.m1 = __ldg(mrow + 1);
                            } else if (rs.cls == 1) {
                                rs.m0 = __ldg(mrow); rs.m1 = __ldg(mrow + 1); rs.m2 = __ldg(mrow + 2); rs.m3 = __ldg(mrow + 3);
                            } else {
#pragma unroll
                                for (int e = 0; e < 16; ++e) lut4[e * kLutStride + pt] = __ldg(mrow + e);
                            }
                        }
                    }
                    if (!ptx::mbar_wait_warp(&bars->empty[s], ph ^ 1u, abort_flag, kWaitLimitNs)) { failed = true; bars->abort = 1u; break; }
                    if (kb >= P.lora_blocks) {
                        uint32_t LH = 0, E01 = 0, E23 = 0;
                        if (rs.cls == 0) {
                            LH = pack_bf16x2(__fmul_rn(rs.m0, a), __fmul_rn(rs.m1, a));
                        } else if (rs.cls == 1) {
                            E01 = pack_bf16x2(__fmul_rn(rs.m0, a), __fmul_rn(rs.m1, a));
                            E23 = pack_bf16x2(__fmul_rn(rs.m2, a), __fmul_rn(rs.m3, a));
                        }
                        // operand tile is [128 features][64 channels], K-major: this thread owns column `col`
                        const uint32_t a_s = ptx::smem_u32(base + s * kSmemStage);
                        const uint32_t col_chunk = (uint32_t)col >> 3, col_in = ((uint32_t)col & 7u) * 2u;
#pragma unroll
                        for (int x = 0; x < 4; ++x) {
                            const uint4 val = deq_chunk(rs, q, x, a, LH, E01, E23, lut, kLutStride);
                            const uint32_t w[4] = {val.x, val.y, val.z, val.w};
#pragma unroll
                            for (int e = 0; e < 8; ++e) {
                                const uint32_t krow = (uint32_t)(32 * kq + 8 * x + e);
                                const uint32_t addr = a_s + krow * 128u + ((col_chunk ^ (krow & 7u)) << 4) + col_in;
                                const uint16_t hv = (uint16_t)((e & 1) ? (w[e >> 1] >> 16) : (w[e >> 1] & 0xFFFFu));
                                asm volatile("st.shared.u16 [%0], %1;" ::"r"(addr), "h"(hv) : "memory");
                            }
                        }
                        ptx::fence_proxy_async_smem();
                    }
                    __syncwarp();
                    if (lane == 0) ptx::mbar_arrive(&bars->full_w[s]);
                }
            }
        }
    }

    if (failed) atomicExch(P.status, (uint32_t)LOWRA_ERR_TIMEOUT);
    // ---------------------------------------------------------------------- teardown
    ptx::tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc(tmem_base, kTmemCols);
    }
}

template <int MODE>
static lowra_status launch_mode(const GemmParams& G, const CUtensorMap& tmB, const CUtensorMap& tmB2,
                                const CUtensorMap& tmA2, cudaStream_t stream) {
    static bool configured = false;
    if (!configured) {
        if (cudaFuncSetAttribute(fused_kernel<MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)kGemmSmemBytes) != cudaSuccess)
            return LOWRA_ERR_CUDA;
        configured = true;
    }
    const int n_tiles = G.tiles_r * G.tiles_t;
    const int grid = n_tiles < kNumSMs ? n_tiles : kNumSMs;
    fused_kernel<MODE><<<grid, kGemmThreads, kGemmSmemBytes, stream>>>(G, tmB, tmB2, tmA2);
    return cudaGetLastError() == cudaSuccess ? LOWRA_OK : LOWRA_ERR_CUDA;
}

lowra_status launch_fused(int mode, const GemmParams& G, const CUtensorMap& tmB, const CUtensorMap& tmB2,
                          const CUtensorMap& tmA2, cudaStream_t stream) {
    if (mode == kModeForward) return launch_mode<kModeForward>(G, tmB, tmB2, tmA2, stream);
    if (mode == kModeBackward) return launch_mode<kModeBackward>(G, tmB, tmB2, tmA2, stream);
    return launch_mode<kModeDense>(G, tmB, tmB2, tmA2, stream);
}

}  // namespace lowra
