// lowra_natural_offsets / lowra_reorder_rows: the paper's own buffer layout as a second storage variant.
//
// The paper's dequantisation kernel finds a thread's offset into the quantised buffer from the channels' bit
// precisions (Appendix A.2): the rows lie in their ORIGINAL order, row r at byte offset sum_{i<r} K b_i / 8.
// The kernels of this library work on rows grouped by precision; these two calls convert between the two orders
// (packed codes and absmax rows), so a buffer written by either convention can be used with the other.  A row's
// bytes are the same in both (LSB-first codes at the row's precision): the conversion is a row permutation.
//
// One warp per row: 16-byte vectors of packed codes (K % 128 == 0 makes every row a whole number of them and
// every offset a multiple of 16), 8-byte vectors of absmax.  Traffic: every byte read once and written once.
#include "lowra_common.cuh"

namespace lowra {

namespace {

constexpr int kMoveThreads = 256;

struct MoveParams {
    RowLayout L;
    const uint64_t* offsets;   // [N + 1] natural byte offsets
    const uint8_t* src_packed;
    const float* src_absmax;
    uint8_t* dst_packed;
    float* dst_absmax;
    int to_natural;
};

__global__ void __launch_bounds__(kMoveThreads) move_kernel(const MoveParams P) {
    pdl_enter();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int r = blockIdx.x * (kMoveThreads / 32) + warp; r < P.L.N; r += gridDim.x * (kMoveThreads / 32)) {
        const int b = P.L.precs[r], c = b >> 1;
        const int p = P.L.inv_perm[r];                                        // stored position in the grouped order
        const size_t row_bytes = (size_t)P.L.K * b / 8;
        const size_t grouped = P.L.seg_off[c] + (size_t)(p - P.L.class_start[c]) * row_bytes;
        const size_t natural = P.offsets[r];
        const uint4* src = reinterpret_cast<const uint4*>(P.src_packed + (P.to_natural ? grouped : natural));
        uint4* dst = reinterpret_cast<uint4*>(P.dst_packed + (P.to_natural ? natural : grouped));
        for (int i = lane; i < (int)(row_bytes / 16); i += 32) st_stream_v4(dst + i, ld_stream_v4(src + i));
        const float2* asrc = reinterpret_cast<const float2*>(P.src_absmax + (size_t)(P.to_natural ? p : r) * P.L.nb);
        float2* adst = reinterpret_cast<float2*>(P.dst_absmax + (size_t)(P.to_natural ? r : p) * P.L.nb);
        for (int i = lane; i < P.L.nb / 2; i += 32) adst[i] = asrc[i];
    }
}

}  // namespace
}  // namespace lowra

extern "C" lowra_status lowra_natural_offsets(int32_t N, int32_t K, const uint8_t* precs_host, uint64_t* offsets_host) {
    if (!precs_host || !offsets_host) return LOWRA_ERR_NULL;
    if (N < 1 || K < 128 || K % 128 != 0) return LOWRA_ERR_SHAPE;
    uint64_t off = 0;
    for (int32_t r = 0; r < N; ++r) {
        const int b = precs_host[r];
        if (b != 1 && b != 2 && b != 4) return LOWRA_ERR_PREC;
        offsets_host[r] = off;
        off += (uint64_t)K * (uint64_t)b / 8;
    }
    offsets_host[N] = off;
    return LOWRA_OK;
}

extern "C" lowra_status lowra_reorder_rows(const lowra_layout* layout, int32_t to_natural, const uint64_t* offsets_dev,
                                           const uint8_t* packed_src_dev, const float* absmax_src_dev,
                                           uint8_t* packed_dst_dev, float* absmax_dst_dev, void* stream) {
    using namespace lowra;
    lowra_status st = check_layout(layout);
    if (st != LOWRA_OK) return st;
    if (!offsets_dev || !packed_src_dev || !absmax_src_dev || !packed_dst_dev || !absmax_dst_dev) return LOWRA_ERR_NULL;
    if (!aligned16(packed_src_dev) || !aligned16(packed_dst_dev) || !aligned16(absmax_src_dev) || !aligned16(absmax_dst_dev) ||
        !aligned16(offsets_dev))
        return LOWRA_ERR_ALIGN;
    if (packed_src_dev == packed_dst_dev || absmax_src_dev == absmax_dst_dev) return LOWRA_ERR_SHAPE;   // not in place
    st = check_device();
    if (st != LOWRA_OK) return st;
    MoveParams P;
    P.L = make_row_layout(layout);
    P.offsets = offsets_dev;
    P.src_packed = packed_src_dev;
    P.src_absmax = absmax_src_dev;
    P.dst_packed = packed_dst_dev;
    P.dst_absmax = absmax_dst_dev;
    P.to_natural = to_natural ? 1 : 0;
    const int cap = kNumSMs * 8;
    const int want = (layout->N + kMoveThreads / 32 - 1) / (kMoveThreads / 32);
    return launch_pdl(move_kernel, (unsigned)(want < cap ? want : cap), kMoveThreads, (cudaStream_t)stream, P) == cudaSuccess
               ? LOWRA_OK : LOWRA_ERR_CUDA;
}
