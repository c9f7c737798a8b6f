// lowra_encode: fp32 weights -> block absmax + packed 1/2/4-bit codes (paper Appendix A.1).
//
// HBM-bound on the 4 bytes read per element, so the kernel has to get by on a handful of instructions per
// element.  One warp handles 1024 consecutive elements of one stored row.  Each lane issues eight 128-bit
// streaming loads back to back (coalesced) and parks them in the warp's slice of shared memory; lane l then
// owns elements 32 l .. 32 l + 31 (half an absmax block), which it reads back as eight 128-bit loads (the
// 32-element segments are 144 bytes apart, so neither the writes nor the reads collide on a bank).  The block
// maximum is one shuffle away; codes are accumulated as bit planes of sign bits:
//   "thresholds <= n" is counted through the sign of n - t (exact: a difference of two floats has the sign of
//   the exact difference, and equal values give +0, so a value on a threshold takes the upper bucket; n is
//   first passed through n + 0.0 so that a negative zero cannot come out below a threshold of +0),
//   1 bit : one subtract and one funnel shift per element,
//   2 bits: three sign planes (one per threshold; sorted thresholds) combined into the two code planes with
//           two logic ops per 32 elements, then interleaved,
//   4 bits: branch-free binary search over the row's 15 thresholds, which lie in the warp's slice of shared memory
//           (four look-ups by index per element; kept in registers and picked with selects, a search costs 20
//           instructions on the half-rate pipe).
// A lane ends up with 4, 8 or 16 packed bytes: the warp writes 128, 256 or 512 contiguous bytes.
//
// Bit-exactness with the definition rests on: the block maximum is exact in fp32; the reciprocal is the
// correctly rounded one (__frcp_rn) and the product a separate rounded multiply (__fmul_rn, never fused).
#include "lowra_common.cuh"

namespace lowra {

constexpr int kEncodeThreads = 256;
constexpr int kEncodeWarps = kEncodeThreads / 32;
constexpr int kEncodeChunk = 1024;  // elements per warp task
constexpr int kSegBytes = 144;      // 32 floats + 16 bytes of padding

struct EncodeParams {
    RowLayout L;
    const float* W;           // [N, K] original order
    const float* thresholds;  // [N, 16] original order
    uint8_t* packed;
    float* absmax;            // [N, nb] stored order
    uint32_t chunks_per_row;  // ceil(K / 1024)
    uint32_t n_tasks;
};

// sign bit of (n - t) pushed into `plane` from the right: after 32 pushes (elements 31 .. 0) bit i of the
// plane says "element i is below t"
__device__ __forceinline__ uint32_t push_below(uint32_t plane, float n, float t) {
    return __funnelshift_l(__float_as_uint(__fsub_rn(n, t)), plane, 1);
}

// bits of x (16 of them) spread to the even positions
__device__ __forceinline__ uint32_t spread16(uint32_t x) {
    x = (x | (x << 8)) & 0x00FF00FFu;
    x = (x | (x << 4)) & 0x0F0F0F0Fu;
    x = (x | (x << 2)) & 0x33333333u;
    x = (x | (x << 1)) & 0x55555555u;
    return x;
}

template <int B>
__device__ __forceinline__ void encode_chunk(const EncodeParams& P, int p, int chunk, int lane, unsigned char* stage) {
    constexpr int c = B >> 1;  // class index of B bits
    const int K = P.L.K;
    const int r = __ldg(P.L.perm + p);
    const float* wrow = P.W + (size_t)r * K;
    const int e0 = chunk * kEncodeChunk;
    const int valid = min(K - e0, kEncodeChunk);   // a multiple of 128

    // ---- coalesced loads, parked in shared memory: element e of the chunk at segment e / 32, offset e % 32
    float4 v[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int e = (i * 32 + lane) * 4;
        v[i] = (e < valid) ? ld_stream_f4(wrow + e0 + e) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
    const float* trow = P.thresholds + (size_t)r * kTableStride;
    float t0 = 0.f, t1 = 0.f, t2 = 0.f;
    float* ts = reinterpret_cast<float*>(stage + 32 * kSegBytes);   // 4 bits: the row's 15 thresholds, searched by index
    if (B == 1) {
        t0 = __ldg(trow);
    } else if (B == 2) {
        t0 = __ldg(trow); t1 = __ldg(trow + 1); t2 = __ldg(trow + 2);
    } else if (lane < 16) {
        t0 = __ldg(trow + lane);
    }
    __syncwarp();   // the previous task's reads of the stage are over
    if (B == 4 && lane < 16) ts[lane] = t0;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int e = (i * 32 + lane) * 4;
        *reinterpret_cast<float4*>(stage + (e >> 5) * kSegBytes + (e & 31) * 4) = v[i];
    }
    __syncwarp();

    // ---- this lane's 32 elements = half an absmax block
    float x[32];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const float4 f = *reinterpret_cast<const float4*>(stage + lane * kSegBytes + j * 16);
        x[4 * j] = f.x; x[4 * j + 1] = f.y; x[4 * j + 2] = f.z; x[4 * j + 3] = f.w;
    }
    float m = 0.0f;
#pragma unroll
    for (int i = 0; i < 32; ++i) m = fmaxf(m, fabsf(x[i]));
    m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 1));
    const bool live = lane * 32 < valid;
    if (live && (lane & 1) == 0) P.absmax[(size_t)absmax_row_of(P.L, p, r) * P.L.nb + (e0 >> 6) + (lane >> 1)] = m;
    const float inv = (m == 0.0f) ? 0.0f : __frcp_rn(m);

    uint8_t* dst = P.packed + packed_row_offset(P.L, c, p, r) + (size_t)(e0 + lane * 32) * B / 8;
    if (B == 1) {
        uint32_t below = 0u;
#pragma unroll
        for (int i = 31; i >= 0; --i) below = push_below(below, __fadd_rn(__fmul_rn(x[i], inv), 0.0f), t0);
        if (live) *reinterpret_cast<uint32_t*>(dst) = ~below;
    } else if (B == 2) {
        uint32_t s0 = 0u, s1 = 0u, s2 = 0u;   // element i is below threshold 0 / 1 / 2
#pragma unroll
        for (int i = 31; i >= 0; --i) {
            const float n = __fadd_rn(__fmul_rn(x[i], inv), 0.0f);
            s0 = push_below(s0, n, t0);
            s1 = push_below(s1, n, t1);
            s2 = push_below(s2, n, t2);
        }
        // sorted thresholds: code = number of thresholds <= n; high bit = not below t1, low bit = not below t2
        // (upper half) or not below t0 (lower half)
        const uint32_t hi = ~s1;
        const uint32_t lo = (hi & ~s2) | (s1 & ~s0);
        uint2 w;
        w.x = spread16(lo & 0xFFFFu) | (spread16(hi & 0xFFFFu) << 1);
        w.y = spread16(lo >> 16) | (spread16(hi >> 16) << 1);
        if (live) *reinterpret_cast<uint2*>(dst) = w;
    } else {
        uint32_t w[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            uint32_t acc = 0u;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                // number of thresholds <= n (sorted thresholds): branch-free binary search, four look-ups by index
                const float n = __fmul_rn(x[8 * q + i], inv);
                uint32_t k = ts[7] <= n ? 8u : 0u;
                k += ts[k + 3] <= n ? 4u : 0u;
                k += ts[k + 1] <= n ? 2u : 0u;
                k += ts[k] <= n ? 1u : 0u;
                acc |= k << (4 * i);
            }
            w[q] = acc;
        }
        if (live) *reinterpret_cast<uint4*>(dst) = make_uint4(w[0], w[1], w[2], w[3]);
    }
}

// The tasks of up to NM matrices, numbered through, matrix after matrix.
template <int NM>
struct EncodeGroup {
    EncodeParams m[NM];
    uint32_t first_task[NM + 1];   // first task of every member; [NM] (and the entries of unused members) = number of tasks
};

template <int NM>
__global__ void __launch_bounds__(kEncodeThreads, 3) encode_kernel(const __grid_constant__ EncodeGroup<NM> G) {
    __shared__ __align__(16) unsigned char stage_all[kEncodeWarps][32 * kSegBytes + 64];
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    unsigned char* stage = stage_all[warp];
    pdl_enter();
    const uint32_t stride = gridDim.x * kEncodeWarps;
    for (uint32_t t = blockIdx.x * kEncodeWarps + warp; t < G.first_task[NM]; t += stride) {
        int mi = 0;
#pragma unroll
        for (int i = 1; i < NM; ++i) mi += (t >= G.first_task[i]) ? 1 : 0;
        const EncodeParams& P = G.m[mi];
        const uint32_t local = t - G.first_task[mi];
        const int p = local / P.chunks_per_row;
        const int chunk = local - p * P.chunks_per_row;
        const int c = (p >= P.L.class_start[1]) + (p >= P.L.class_start[2]);
        if (c == 0) encode_chunk<1>(P, p, chunk, lane, stage);
        else if (c == 1) encode_chunk<2>(P, p, chunk, lane, stage);
        else encode_chunk<4>(P, p, chunk, lane, stage);
    }
}

namespace {

// checks one matrix's arguments and fills its entry
lowra_status encode_member(const lowra_layout* layout, const float* W_dev, const float* thresholds_dev, uint8_t* packed_dev,
                           float* absmax_dev, EncodeParams& P) {
    lowra_status st = check_layout(layout);
    if (st != LOWRA_OK) return st;
    if (!W_dev || !thresholds_dev || !packed_dev || !absmax_dev) return LOWRA_ERR_NULL;
    if (!aligned16(W_dev) || !aligned16(thresholds_dev) || !aligned16(packed_dev) || !aligned16(absmax_dev))
        return LOWRA_ERR_ALIGN;
    P.L = make_row_layout(layout);
    P.W = W_dev;
    P.thresholds = thresholds_dev;
    P.packed = packed_dev;
    P.absmax = absmax_dev;
    P.chunks_per_row = (uint32_t)((layout->K + kEncodeChunk - 1) / kEncodeChunk);
    const uint64_t tasks = (uint64_t)layout->N * P.chunks_per_row;
    if (tasks > 0xFFFFFFFFull) return LOWRA_ERR_SHAPE;
    P.n_tasks = (uint32_t)tasks;
    return LOWRA_OK;
}

template <int NM>
lowra_status launch_encode(const EncodeGroup<NM>& G, void* stream) {
    const uint64_t tasks = G.first_task[NM];
    const uint64_t blocks_needed = (tasks + kEncodeWarps - 1) / kEncodeWarps;
    const uint64_t cap = (uint64_t)kNumSMs * 3;   // three CTAs (80 registers, 36 KB of shared memory) are resident per SM
    const unsigned grid = (unsigned)(blocks_needed < cap ? blocks_needed : cap);
    return launch_pdl(encode_kernel<NM>, grid, kEncodeThreads, (cudaStream_t)stream, G) == cudaSuccess ? LOWRA_OK : LOWRA_ERR_CUDA;
}

}  // namespace

}  // namespace lowra

extern "C" lowra_status lowra_encode(const lowra_layout* layout, const float* W_dev, const float* thresholds_dev,
                                     uint8_t* packed_dev, float* absmax_dev, void* stream) {
    using namespace lowra;
    EncodeGroup<1> G;
    lowra_status st = encode_member(layout, W_dev, thresholds_dev, packed_dev, absmax_dev, G.m[0]);
    if (st != LOWRA_OK) return st;
    st = check_device();
    if (st != LOWRA_OK) return st;
    G.first_task[0] = 0;
    G.first_task[1] = G.m[0].n_tasks;
    return launch_encode<1>(G, stream);
}

extern "C" lowra_status lowra_encode_group(const lowra_group_member* members_host, int32_t count, void* stream) {
    using namespace lowra;
    if (!members_host) return LOWRA_ERR_NULL;
    if (count < 1 || count > LOWRA_MAX_GROUP) return LOWRA_ERR_SHAPE;
    EncodeGroup<LOWRA_MAX_GROUP> G;
    uint64_t total = 0;
    for (int i = 0; i < count; ++i) {
        const lowra_group_member& m = members_host[i];
        lowra_status st = encode_member(m.layout, m.W_dev, m.tables_dev, m.packed_dev, m.absmax_dev, G.m[i]);
        if (st != LOWRA_OK) return st;
        G.first_task[i] = (uint32_t)total;
        total += G.m[i].n_tasks;
        if (total > 0xFFFFFFFFull) return LOWRA_ERR_SHAPE;
    }
    for (int i = count; i <= LOWRA_MAX_GROUP; ++i) {
        if (i < LOWRA_MAX_GROUP) G.m[i] = G.m[0];
        G.first_task[i] = (uint32_t)total;
    }
    lowra_status st = check_device();
    if (st != LOWRA_OK) return st;
    return launch_encode<LOWRA_MAX_GROUP>(G, stream);
}
