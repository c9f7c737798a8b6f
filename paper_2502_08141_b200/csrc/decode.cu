// lowra_decode: packed 1/2/4-bit codes -> bf16 weights (paper Appendix A.2).
//
// HBM-bound: 2 bytes written per element against b/8 + 1/16 bytes read.  One warp handles one
// 512-byte piece of one stored row: every lane fetches 16 packed bytes with a single 128-bit load,
// the row's mapping table is staged in shared memory, and the codes are redistributed with warp
// shuffles so that every store instruction of the warp writes 512 contiguous bytes of the output.
#include "lowra_common.cuh"

namespace lowra {

constexpr int kDecodeThreads = 256;
constexpr int kDecodeWarps = kDecodeThreads / 32;

struct DecodeParams {
    RowLayout L;
    const uint8_t* packed;
    const float* absmax;   // [N, nb] stored order
    const float* maps;     // [N, 16] original order
    uint16_t* out;         // [N, K] bf16, original order
    uint32_t pieces_per_row[3];  // ceil(K * b / 4096)
    uint32_t task_start[4];      // first task of each class; [3] = number of tasks
};

// One 512-byte piece of a B-bit row: 4096 / B elements, written as 16 / B warp-wide stores.
template <int B>
__device__ __forceinline__ void decode_piece(const DecodeParams& P, int p, int piece, int lane, float* lut) {
    constexpr int c = B >> 1;         // class index of B bits
    constexpr int kElems = 4096 / B;  // elements in the piece
    constexpr int kIters = 16 / B;    // 256 elements (512 output bytes) per iteration
    constexpr int kUnits = 16 / B;    // 8-element units held by one lane's 16 bytes
    constexpr uint32_t kMask = (1u << B) - 1u;
    const int K = P.L.K;
    const int r = __ldg(P.L.perm + p);
    const size_t row_bytes = (size_t)K * B / 8;
    const uint8_t* row = P.packed + P.L.seg_off[c] + (size_t)(p - P.L.class_start[c]) * row_bytes;

    const size_t byte0 = (size_t)piece * 512 + (size_t)lane * 16;
    uint4 q = make_uint4(0u, 0u, 0u, 0u);
    if (byte0 < row_bytes) q = ld_stream_v4(row + byte0);

    if (lane < (1 << B)) lut[lane] = __ldg(P.maps + (size_t)r * kTableStride + lane);

    const int e0 = piece * kElems;  // first element of the piece
    const int blk0 = e0 / kBlock;
    const float* arow = P.absmax + (size_t)p * P.L.nb;
    float av0 = (blk0 + lane < P.L.nb) ? __ldg(arow + blk0 + lane) : 0.0f;
    float av1 = 0.0f;
    if (B == 1 && blk0 + 32 + lane < P.L.nb) av1 = __ldg(arow + blk0 + 32 + lane);
    __syncwarp();

    uint16_t* orow = P.out + (size_t)r * K;
#pragma unroll
    for (int j = 0; j < kIters; ++j) {
        // This lane writes elements e0 + 256 j + 8 lane .. +8, i.e. 8-element unit u = 32 j + lane
        // of the piece; that unit sits in lane u / kUnits, 32-bit word (u % kUnits) * B / 4.
        const int u = 32 * j + lane;
        const int src = u / kUnits;
        const int sub = u % kUnits;
        const int w = (sub * B) >> 2;
        const uint32_t x0 = __shfl_sync(0xffffffffu, q.x, src);
        const uint32_t x1 = __shfl_sync(0xffffffffu, q.y, src);
        const uint32_t x2 = __shfl_sync(0xffffffffu, q.z, src);
        const uint32_t x3 = __shfl_sync(0xffffffffu, q.w, src);
        const uint32_t word = (w == 0) ? x0 : (w == 1) ? x1 : (w == 2) ? x2 : x3;
        const uint32_t bits = word >> ((sub * 8 * B) & 31);
        // 256 elements = 4 absmax blocks per iteration, 8 lanes per block
        const int blk = 4 * j + (lane >> 3);
        const float a = __shfl_sync(0xffffffffu, (B == 1 && j >= 8) ? av1 : av0, blk & 31);
        uint32_t o[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const uint32_t c0 = (bits >> (2 * i * B)) & kMask;
            const uint32_t c1 = (bits >> ((2 * i + 1) * B)) & kMask;
            const float f0 = __fmul_rn(lut[c0], a);
            const float f1 = __fmul_rn(lut[c1], a);
            o[i] = pack_bf16x2(f0, f1);
        }
        const int e = e0 + 256 * j + 8 * lane;
        if (e < K) st_stream_v4(orow + e, make_uint4(o[0], o[1], o[2], o[3]));
    }
    __syncwarp();  // the table slot is reused by the warp's next piece
}

__global__ void __launch_bounds__(kDecodeThreads) decode_kernel(const DecodeParams P) {
    __shared__ float lut_all[kDecodeWarps][kTableStride];
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    float* lut = lut_all[warp];
    const uint32_t n_tasks = P.task_start[3];
    const uint32_t stride = gridDim.x * kDecodeWarps;
    for (uint32_t t = blockIdx.x * kDecodeWarps + warp; t < n_tasks; t += stride) {
        const int c = (t >= P.task_start[1]) + (t >= P.task_start[2]);
        const uint32_t local = t - P.task_start[c];
        const uint32_t ppr = P.pieces_per_row[c];
        const int q = local / ppr;
        const int piece = local - q * ppr;
        const int p = P.L.class_start[c] + q;
        if (c == 0) decode_piece<1>(P, p, piece, lane, lut);
        else if (c == 1) decode_piece<2>(P, p, piece, lane, lut);
        else decode_piece<4>(P, p, piece, lane, lut);
    }
}

}  // namespace lowra

extern "C" lowra_status lowra_decode(const lowra_layout* layout, const uint8_t* packed_dev,
                                     const float* absmax_dev, const float* maps_dev, uint16_t* W_bf16_dev,
                                     void* stream) {
    using namespace lowra;
    lowra_status st = check_layout(layout);
    if (st != LOWRA_OK) return st;
    if (!packed_dev || !absmax_dev || !maps_dev || !W_bf16_dev) return LOWRA_ERR_NULL;
    if (!aligned16(packed_dev) || !aligned16(absmax_dev) || !aligned16(maps_dev) || !aligned16(W_bf16_dev))
        return LOWRA_ERR_ALIGN;
    st = check_device();
    if (st != LOWRA_OK) return st;

    DecodeParams P;
    P.L = make_row_layout(layout);
    P.packed = packed_dev;
    P.absmax = absmax_dev;
    P.maps = maps_dev;
    P.out = W_bf16_dev;
    uint64_t tasks = 0;
    for (int c = 0; c < 3; ++c) {
        const uint64_t row_bytes = (uint64_t)layout->K * (1u << c) / 8u;
        P.pieces_per_row[c] = (uint32_t)((row_bytes + 511) / 512);
        P.task_start[c] = (uint32_t)tasks;
        tasks += (uint64_t)layout->counts[c] * P.pieces_per_row[c];
    }
    if (tasks > 0xFFFFFFFFull) return LOWRA_ERR_SHAPE;
    P.task_start[3] = (uint32_t)tasks;
    const uint64_t blocks_needed = (tasks + kDecodeWarps - 1) / kDecodeWarps;
    const uint64_t cap = (uint64_t)kNumSMs * 8;
    const unsigned grid = (unsigned)(blocks_needed < cap ? blocks_needed : cap);
    decode_kernel<<<grid, kDecodeThreads, 0, (cudaStream_t)stream>>>(P);
    return cudaGetLastError() == cudaSuccess ? LOWRA_OK : LOWRA_ERR_CUDA;
}
