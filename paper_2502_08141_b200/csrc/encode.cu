// lowra_encode: fp32 weights -> block absmax + packed 1/2/4-bit codes (paper Appendix A.1).
//
// HBM-bound on the 4 bytes read per element.  One warp handles 1024 consecutive elements of one
// stored row: eight 128-bit loads per lane are issued back to back, each group of 128 elements
// (two absmax blocks) is reduced with warp shuffles, normalised, pushed through a branch-free
// threshold search held in registers and packed with shuffles into whole 32-bit words.
//
// Bit-exactness with the definition rests on three things: the block maximum is exact in fp32; the
// reciprocal is the correctly rounded one (__frcp_rn) and the product a separate rounded multiply
// (__fmul_rn, never fused); the search returns the number of thresholds <= n, which for sorted
// thresholds is what the branch-free binary search below computes.
#include "lowra_common.cuh"

namespace lowra {

constexpr int kEncodeThreads = 256;
constexpr int kEncodeWarps = kEncodeThreads / 32;
constexpr int kEncodeChunk = 1024;  // elements per warp task
constexpr int kGroups = kEncodeChunk / 128;

struct EncodeParams {
    RowLayout L;
    const float* W;           // [N, K] original order
    const float* thresholds;  // [N, 16] original order
    uint8_t* packed;
    float* absmax;            // [N, nb] stored order
    uint32_t chunks_per_row;  // ceil(K / 1024)
    uint32_t n_tasks;
};

template <int B>
struct Thresholds;

template <>
struct Thresholds<1> {
    float t0;
    __device__ __forceinline__ void load(const float* t) { t0 = __ldg(t); }
    __device__ __forceinline__ uint32_t code(float n) const { return t0 <= n ? 1u : 0u; }
};

template <>
struct Thresholds<2> {
    float t[3];
    __device__ __forceinline__ void load(const float* p) {
#pragma unroll
        for (int j = 0; j < 3; ++j) t[j] = __ldg(p + j);
    }
    __device__ __forceinline__ uint32_t code(float n) const {
        const bool c1 = t[1] <= n;
        const float m = c1 ? t[2] : t[0];
        const bool c0 = m <= n;
        return (c1 ? 2u : 0u) | (c0 ? 1u : 0u);
    }
};

// selp keeps the 15 thresholds in registers (a C ternary tree is turned into an indexed local array)
__device__ __forceinline__ float sel(bool c, float a, float b) {
    float r;
    asm("{ .reg .pred p; setp.ne.u32 p, %3, 0; selp.f32 %0, %1, %2, p; }" : "=f"(r) : "f"(a), "f"(b), "r"((uint32_t)c));
    return r;
}

template <>
struct Thresholds<4> {
    float t0, t1, t2, t3, t4, t5, t6, t7, t8, t9, t10, t11, t12, t13, t14;
    __device__ __forceinline__ void load(const float* p) {
        const float4 a = __ldg(reinterpret_cast<const float4*>(p));
        const float4 b = __ldg(reinterpret_cast<const float4*>(p) + 1);
        const float4 c = __ldg(reinterpret_cast<const float4*>(p) + 2);
        const float4 d = __ldg(reinterpret_cast<const float4*>(p) + 3);
        t0 = a.x; t1 = a.y; t2 = a.z; t3 = a.w; t4 = b.x; t5 = b.y; t6 = b.z; t7 = b.w;
        t8 = c.x; t9 = c.y; t10 = c.z; t11 = c.w; t12 = d.x; t13 = d.y; t14 = d.z;
    }
    __device__ __forceinline__ uint32_t code(float n) const {
        const bool c3 = t7 <= n;
        const bool c2 = sel(c3, t11, t3) <= n;
        const float hi1 = sel(c2, t13, t9), lo1 = sel(c2, t5, t1);
        const bool c1 = sel(c3, hi1, lo1) <= n;
        const float q3 = sel(c1, t14, t12), q2 = sel(c1, t10, t8), q1 = sel(c1, t6, t4), q0 = sel(c1, t2, t0);
        const bool c0 = sel(c3, sel(c2, q3, q2), sel(c2, q1, q0)) <= n;
        return (c3 ? 8u : 0u) | (c2 ? 4u : 0u) | (c1 ? 2u : 0u) | (c0 ? 1u : 0u);
    }
};

template <int B>
__device__ __forceinline__ void encode_chunk(const EncodeParams& P, int p, int chunk, int lane) {
    constexpr int c = B >> 1;  // class index of B bits
    const int K = P.L.K;
    const int r = __ldg(P.L.perm + p);
    const float* wrow = P.W + (size_t)r * K;
    const int e0 = chunk * kEncodeChunk;
    int groups = (K - e0) / 128;
    if (groups > kGroups) groups = kGroups;

    float4 v[kGroups];
#pragma unroll
    for (int g = 0; g < kGroups; ++g)
        v[g] = (g < groups) ? ld_stream_f4(wrow + e0 + g * 128 + lane * 4) : make_float4(0.f, 0.f, 0.f, 0.f);

    Thresholds<B> thr;
    thr.load(P.thresholds + (size_t)r * kTableStride);

    const size_t row_bytes = (size_t)K * B / 8;
    uint8_t* prow = P.packed + P.L.seg_off[c] + (size_t)(p - P.L.class_start[c]) * row_bytes;
    float* arow = P.absmax + (size_t)p * P.L.nb;

#pragma unroll
    for (int g = 0; g < kGroups; ++g) {
        if (g < groups) {  // warp-uniform
            // block maximum over 64 elements = 16 lanes x 4
            float m = fmaxf(fmaxf(fabsf(v[g].x), fabsf(v[g].y)), fmaxf(fabsf(v[g].z), fabsf(v[g].w)));
#pragma unroll
            for (int d = 8; d >= 1; d >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, d));
            if ((lane & 15) == 0) arow[(e0 + g * 128) / kBlock + (lane >> 4)] = m;
            const float inv = (m == 0.0f) ? 0.0f : __frcp_rn(m);
            uint32_t piece = thr.code(__fmul_rn(v[g].x, inv));
            piece |= thr.code(__fmul_rn(v[g].y, inv)) << B;
            piece |= thr.code(__fmul_rn(v[g].z, inv)) << (2 * B);
            piece |= thr.code(__fmul_rn(v[g].w, inv)) << (3 * B);
            // 4*B bits per lane -> whole 32-bit words: 8 / B lanes per word
            uint32_t word = piece;
            word |= __shfl_down_sync(0xffffffffu, word, 1) << (4 * B);
            if constexpr (B <= 2) word |= __shfl_down_sync(0xffffffffu, word, 2) << (8 * B);
            if constexpr (B <= 1) word |= __shfl_down_sync(0xffffffffu, word, 4) << (16 * B);
            constexpr int kLanesPerWord = 8 / B;
            if ((lane % kLanesPerWord) == 0) {
                uint32_t* dst = reinterpret_cast<uint32_t*>(prow + (size_t)(e0 + g * 128) * B / 8);
                dst[lane / kLanesPerWord] = word;
            }
        }
    }
}

__global__ void __launch_bounds__(kEncodeThreads) encode_kernel(const EncodeParams P) {
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const uint32_t stride = gridDim.x * kEncodeWarps;
    for (uint32_t t = blockIdx.x * kEncodeWarps + warp; t < P.n_tasks; t += stride) {
        const int p = t / P.chunks_per_row;
        const int chunk = t - p * P.chunks_per_row;
        const int c = (p >= P.L.class_start[1]) + (p >= P.L.class_start[2]);
        if (c == 0) encode_chunk<1>(P, p, chunk, lane);
        else if (c == 1) encode_chunk<2>(P, p, chunk, lane);
        else encode_chunk<4>(P, p, chunk, lane);
    }
}

}  // namespace lowra

extern "C" lowra_status lowra_encode(const lowra_layout* layout, const float* W_dev, const float* thresholds_dev,
                                     uint8_t* packed_dev, float* absmax_dev, void* stream) {
    using namespace lowra;
    lowra_status st = check_layout(layout);
    if (st != LOWRA_OK) return st;
    if (!W_dev || !thresholds_dev || !packed_dev || !absmax_dev) return LOWRA_ERR_NULL;
    if (!aligned16(W_dev) || !aligned16(thresholds_dev) || !aligned16(packed_dev) || !aligned16(absmax_dev))
        return LOWRA_ERR_ALIGN;
    st = check_device();
    if (st != LOWRA_OK) return st;

    EncodeParams P;
    P.L = make_row_layout(layout);
    P.W = W_dev;
    P.thresholds = thresholds_dev;
    P.packed = packed_dev;
    P.absmax = absmax_dev;
    P.chunks_per_row = (uint32_t)((layout->K + kEncodeChunk - 1) / kEncodeChunk);
    const uint64_t tasks = (uint64_t)layout->N * P.chunks_per_row;
    if (tasks > 0xFFFFFFFFull) return LOWRA_ERR_SHAPE;
    P.n_tasks = (uint32_t)tasks;
    const uint64_t blocks_needed = (tasks + kEncodeWarps - 1) / kEncodeWarps;
    const uint64_t cap = (uint64_t)kNumSMs * 8;
    const unsigned grid = (unsigned)(blocks_needed < cap ? blocks_needed : cap);
    encode_kernel<<<grid, kEncodeThreads, 0, (cudaStream_t)stream>>>(P);
    return cudaGetLastError() == cudaSuccess ? LOWRA_OK : LOWRA_ERR_CUDA;
}
