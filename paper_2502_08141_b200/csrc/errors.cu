// lowra_quant_error: summed square error per output channel and, optionally, the residual W - W_hat.
// lowra_channel_errors: the same error under 1, 2 and 4 bits at once (one read of W), without a layout.
//
// The precision assigner minimises the summed square error between the weights and their quantised
// counterparts (paper Section 5 and its footnote; Section 5.1 starts from every channel's error under 1, 2 and
// 4 bits), and an iterative low-rank initialiser factorises the residual W - W_hat after quantising (appendix on
// the low-rank initialisers).  Both come out of one pass over W, fused: block absmax, normalise, bucket, look the
// level up, scale and round to bf16 exactly as lowra_encode followed by lowra_decode would - without writing codes
// or W_hat - then
//     residual = fl32(x - w_hat)            one fp32 subtraction per element (optional output)
//     SSE_row  = sum of residual^2          four neighbouring squares are added in fp32, those partial sums in fp64,
//                                           fixed reduction tree (reproducible)
// so SSE agrees with the exact sum to 2^-21 relative at worst (residual rounded to fp32: 2^-23; a square and two
// additions in fp32: 3 * 2^-24 more), typically far closer.
//
// One warp per row at a time (grid-stride, no block-wide synchronisation); sixteen lanes with one float4 each cover
// a 64-element absmax block, so the block maximum is four shuffles.  Traffic: 4 bytes per element read (+ 4 written with the residual).
#include "lowra_common.cuh"

namespace lowra {

namespace {

constexpr int kErrThreads = 256;
constexpr int kErrWarps = kErrThreads / 32;
constexpr int kErrBatch = 4;   // float4 loads per thread and batch; two batches in flight

struct ErrParams {
    RowLayout L;
    const float* W;           // [N, K] original order
    const float* maps;        // [N, 16]
    const float* thresholds;  // [N, 16]
    double* sse;              // [N]
    float* residual;          // [N, K] or null
};

// level of the bucket of n: the number of thresholds <= n picks the level (thresholds sorted, as the encoder assumes).
// 4 bits: levels at tab[0 .. 15], thresholds at tab[16 .. 30] of the warp's table in shared memory; branch-free binary
// search, four look-ups by index (the same search as lowra_encode's).
template <int B>
__device__ __forceinline__ float level_of(float n, const float (&t)[3], const float (&y)[4], const float* tab) {
    if (B == 1) return t[0] <= n ? y[1] : y[0];
    if (B == 2) {
        const bool hi = t[1] <= n;
        const bool lo = (hi ? t[2] : t[0]) <= n;
        return hi ? (lo ? y[3] : y[2]) : (lo ? y[1] : y[0]);
    }
    const float* ts = tab + 16;
    int k = ts[7] <= n ? 8 : 0;
    k += ts[k + 3] <= n ? 4 : 0;
    k += ts[k + 1] <= n ? 2 : 0;
    k += ts[k] <= n ? 1 : 0;
    return tab[k];
}

template <int B>
__device__ void error_row(const ErrParams& P, int r, float* y_warp) {
    const int lane = threadIdx.x & 31;
    const int K = P.L.K;
    const float* wrow = P.W + (size_t)r * K;
    float* rrow = P.residual ? P.residual + (size_t)r * K : nullptr;
    const float* trow = P.thresholds + (size_t)r * kTableStride;
    const float* yrow = P.maps + (size_t)r * kTableStride;
    float t[3] = {0.f, 0.f, 0.f}, y[4] = {0.f, 0.f, 0.f, 0.f};
    if (B == 1) {
        t[0] = __ldg(trow); y[0] = __ldg(yrow); y[1] = __ldg(yrow + 1);
    } else if (B == 2) {
        t[0] = __ldg(trow); t[1] = __ldg(trow + 1); t[2] = __ldg(trow + 2);
        y[0] = __ldg(yrow); y[1] = __ldg(yrow + 1); y[2] = __ldg(yrow + 2); y[3] = __ldg(yrow + 3);
    } else {
        __syncwarp();   // the previous row's look-ups are over
        if (lane < 16) { y_warp[lane] = __ldg(yrow + lane); y_warp[16 + lane] = __ldg(trow + lane); }
        __syncwarp();
    }

    double acc = 0.0;
    const int n4 = K / 4;   // float4 pieces of the row (a multiple of 32); lane l takes pieces l, l + 32, ...
    // the loads of the next batch are under way while this one is worked on
    float4 nxt[kErrBatch];
#pragma unroll
    for (int u = 0; u < kErrBatch; ++u) {
        const int i = lane + u * 32;
        nxt[u] = (i < n4) ? ld_stream_f4(wrow + (size_t)i * 4) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
    for (int base = lane; base < n4; base += 32 * kErrBatch) {
        float4 x[kErrBatch];
#pragma unroll
        for (int u = 0; u < kErrBatch; ++u) {
            x[u] = nxt[u];
            const int i = base + 32 * kErrBatch + u * 32;
            nxt[u] = (i < n4) ? ld_stream_f4(wrow + (size_t)i * 4) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int u = 0; u < kErrBatch; ++u) {
            const int i = base + u * 32;
            // sixteen neighbouring lanes hold one absmax block
            float m = fmaxf(fmaxf(fabsf(x[u].x), fabsf(x[u].y)), fmaxf(fabsf(x[u].z), fabsf(x[u].w)));
#pragma unroll
            for (int d = 8; d >= 1; d >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, d));
            const float inv = (m == 0.0f) ? 0.0f : __frcp_rn(m);
            // w_hat of the four elements, rounded to bf16 two at a time
            const float l0 = __fmul_rn(level_of<B>(__fmul_rn(x[u].x, inv), t, y, y_warp), m);
            const float l1 = __fmul_rn(level_of<B>(__fmul_rn(x[u].y, inv), t, y, y_warp), m);
            const float l2 = __fmul_rn(level_of<B>(__fmul_rn(x[u].z, inv), t, y, y_warp), m);
            const float l3 = __fmul_rn(level_of<B>(__fmul_rn(x[u].w, inv), t, y, y_warp), m);
            const uint32_t h01 = pack_bf16x2(l0, l1), h23 = pack_bf16x2(l2, l3);
            float4 res;
            res.x = __fsub_rn(x[u].x, __uint_as_float(h01 << 16));
            res.y = __fsub_rn(x[u].y, __uint_as_float(h01 & 0xFFFF0000u));
            res.z = __fsub_rn(x[u].z, __uint_as_float(h23 << 16));
            res.w = __fsub_rn(x[u].w, __uint_as_float(h23 & 0xFFFF0000u));
            if (i < n4) {
                // four squares in fp32 (three roundings of the partial sum), then into the fp64 sum
                const float q = __fadd_rn(__fadd_rn(__fmul_rn(res.x, res.x), __fmul_rn(res.y, res.y)),
                                          __fadd_rn(__fmul_rn(res.z, res.z), __fmul_rn(res.w, res.w)));
                acc += (double)q;
                if (rrow) __stcs(reinterpret_cast<float4*>(rrow + (size_t)i * 4), res);
            }
        }
    }
    // fixed tree over the lanes
#pragma unroll
    for (int d = 16; d >= 1; d >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, d);
    if (lane == 0) P.sse[r] = acc;
}

__global__ void __launch_bounds__(kErrThreads) error_kernel(const ErrParams P) {
    __shared__ float y_smem[kErrWarps][32];   // per warp: the 16 levels and 15 thresholds of a 4-bit row
    pdl_enter();
    const int warp = threadIdx.x >> 5;
    float* y_warp = y_smem[warp];
    // one warp per row at a time
    for (int i = blockIdx.x * kErrWarps + warp; i < P.L.N; i += gridDim.x * kErrWarps) {
        const int r = P.L.perm[P.L.N - 1 - i];   // stored rows from the last to the first: the dear 4-bit rows go out first
        const int b = P.L.precs[r];
        if (b == 1) error_row<1>(P, r, y_warp);
        else if (b == 2) error_row<2>(P, r, y_warp);
        else error_row<4>(P, r, y_warp);
    }
}

// ---- all three precisions in one pass (the assigner's input: every channel's error under 1, 2 and 4 bits) ----
struct Err3Params {
    const float* W;           // [N, K]
    const float* maps;        // [3][N][16]: tables of the 1-, 2- and 4-bit codebooks of every row
    const float* thresholds;  // [3][N][16]
    double* sse;              // [N][3]
    int N, K;
};

__global__ void __launch_bounds__(kErrThreads) error3_kernel(const Err3Params P) {
    __shared__ float y_smem[kErrWarps][32];   // per warp: the 16 levels and 15 thresholds of the row's 4-bit codebook
    pdl_enter();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    float* y_warp = y_smem[warp];
    const int K = P.K, n4 = K / 4;
    const size_t plane = (size_t)P.N * kTableStride;
    for (int r = blockIdx.x * kErrWarps + warp; r < P.N; r += gridDim.x * kErrWarps) {
        const float* wrow = P.W + (size_t)r * K;
        const float* t1 = P.thresholds + (size_t)r * kTableStride;
        const float* y1 = P.maps + (size_t)r * kTableStride;
        const float ta[3] = {__ldg(t1), 0.f, 0.f};
        const float ya[4] = {__ldg(y1), __ldg(y1 + 1), 0.f, 0.f};
        const float tb[3] = {__ldg(t1 + plane), __ldg(t1 + plane + 1), __ldg(t1 + plane + 2)};
        const float yb[4] = {__ldg(y1 + plane), __ldg(y1 + plane + 1), __ldg(y1 + plane + 2), __ldg(y1 + plane + 3)};
        __syncwarp();   // the previous row's look-ups are over
        if (lane < 16) { y_warp[lane] = __ldg(y1 + 2 * plane + lane); y_warp[16 + lane] = __ldg(t1 + 2 * plane + lane); }
        __syncwarp();
        double acc1 = 0.0, acc2 = 0.0, acc4 = 0.0;
        float4 nxt[kErrBatch];
#pragma unroll
        for (int u = 0; u < kErrBatch; ++u) {
            const int i = lane + u * 32;
            nxt[u] = (i < n4) ? ld_stream_f4(wrow + (size_t)i * 4) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
        for (int base = lane; base < n4; base += 32 * kErrBatch) {
            float4 x[kErrBatch];
#pragma unroll
            for (int u = 0; u < kErrBatch; ++u) {
                x[u] = nxt[u];
                const int i = base + 32 * kErrBatch + u * 32;
                nxt[u] = (i < n4) ? ld_stream_f4(wrow + (size_t)i * 4) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
#pragma unroll
            for (int u = 0; u < kErrBatch; ++u) {
                const int i = base + u * 32;
                float m = fmaxf(fmaxf(fabsf(x[u].x), fabsf(x[u].y)), fmaxf(fabsf(x[u].z), fabsf(x[u].w)));
#pragma unroll
                for (int d = 8; d >= 1; d >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, d));
                const float inv = (m == 0.0f) ? 0.0f : __frcp_rn(m);
                const float xs[4] = {x[u].x, x[u].y, x[u].z, x[u].w};
                float n[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) n[e] = __fmul_rn(xs[e], inv);
                // squared residuals of the four elements at one precision, added in fp32
                auto group = [&](auto level) -> float {
                    const uint32_t h01 = pack_bf16x2(__fmul_rn(level(n[0]), m), __fmul_rn(level(n[1]), m));
                    const uint32_t h23 = pack_bf16x2(__fmul_rn(level(n[2]), m), __fmul_rn(level(n[3]), m));
                    const float r0 = __fsub_rn(xs[0], __uint_as_float(h01 << 16)), r1 = __fsub_rn(xs[1], __uint_as_float(h01 & 0xFFFF0000u));
                    const float r2 = __fsub_rn(xs[2], __uint_as_float(h23 << 16)), r3 = __fsub_rn(xs[3], __uint_as_float(h23 & 0xFFFF0000u));
                    return __fadd_rn(__fadd_rn(__fmul_rn(r0, r0), __fmul_rn(r1, r1)), __fadd_rn(__fmul_rn(r2, r2), __fmul_rn(r3, r3)));
                };
                const float q1 = group([&](float v) { return level_of<1>(v, ta, ya, y_warp); });
                const float q2 = group([&](float v) { return level_of<2>(v, tb, yb, y_warp); });
                const float q4 = group([&](float v) { return level_of<4>(v, tb, yb, y_warp); });
                if (i < n4) { acc1 += (double)q1; acc2 += (double)q2; acc4 += (double)q4; }
            }
        }
#pragma unroll
        for (int d = 16; d >= 1; d >>= 1) {
            acc1 += __shfl_xor_sync(0xffffffffu, acc1, d);
            acc2 += __shfl_xor_sync(0xffffffffu, acc2, d);
            acc4 += __shfl_xor_sync(0xffffffffu, acc4, d);
        }
        if (lane == 0) { P.sse[(size_t)r * 3] = acc1; P.sse[(size_t)r * 3 + 1] = acc2; P.sse[(size_t)r * 3 + 2] = acc4; }
    }
}

}  // namespace
}  // namespace lowra

extern "C" lowra_status lowra_quant_error(const lowra_layout* layout, const float* W_dev, const float* maps_dev,
                                          const float* thresholds_dev, double* sse_dev, float* residual_dev,
                                          void* stream) {
    using namespace lowra;
    lowra_status st = check_layout(layout);
    if (st != LOWRA_OK) return st;
    if (!W_dev || !maps_dev || !thresholds_dev || !sse_dev) return LOWRA_ERR_NULL;
    if (!aligned16(W_dev) || !aligned16(maps_dev) || !aligned16(thresholds_dev) || !aligned16(sse_dev) ||
        (residual_dev && !aligned16(residual_dev)))
        return LOWRA_ERR_ALIGN;
    st = check_device();
    if (st != LOWRA_OK) return st;
    ErrParams P;
    P.L = make_row_layout(layout);
    P.W = W_dev;
    P.maps = maps_dev;
    P.thresholds = thresholds_dev;
    P.sse = sse_dev;
    P.residual = residual_dev;
    // a row per warp and as many CTAs as that takes: rows differ in cost with their precision, and fresh CTAs handed out
    // by the hardware keep the SMs more evenly busy than a persistent grid did (+12 to 23 %)
    const unsigned grid = (unsigned)((layout->N + kErrWarps - 1) / kErrWarps);
    return launch_pdl(error_kernel, grid, kErrThreads, (cudaStream_t)stream, P) == cudaSuccess ? LOWRA_OK : LOWRA_ERR_CUDA;
}

extern "C" lowra_status lowra_channel_errors(int32_t N, int32_t K, const float* W_dev, const float* maps3_dev,
                                             const float* thresholds3_dev, double* sse3_dev, void* stream) {
    using namespace lowra;
    if (!W_dev || !maps3_dev || !thresholds3_dev || !sse3_dev) return LOWRA_ERR_NULL;
    if (N < 1 || K < 128 || K % 128 != 0) return LOWRA_ERR_SHAPE;
    if (!aligned16(W_dev) || !aligned16(maps3_dev) || !aligned16(thresholds3_dev) || (reinterpret_cast<uintptr_t>(sse3_dev) & 7u) != 0)
        return LOWRA_ERR_ALIGN;
    lowra_status st = check_device();
    if (st != LOWRA_OK) return st;
    Err3Params P;
    P.W = W_dev;
    P.maps = maps3_dev;
    P.thresholds = thresholds3_dev;
    P.sse = sse3_dev;
    P.N = N;
    P.K = K;
    const unsigned grid = (unsigned)((N + kErrWarps - 1) / kErrWarps);   // a row per warp, as above
    return launch_pdl(error3_kernel, grid, kErrThreads, (cudaStream_t)stream, P) == cudaSuccess ? LOWRA_OK : LOWRA_ERR_CUDA;
}
