// lowra_decode: packed 1/2/4-bit codes -> bf16 weights (paper Appendix A.2).
//
// HBM-bound: 2 bytes written per element against b/8 + 1/16 bytes read, so the kernel must spend very few
// instructions per element and every store instruction must fill whole 128-byte lines.
// One warp handles one 512-byte piece of one stored row.  Every lane fetches 16 packed bytes with a single
// 128-bit load; the piece and its absmax values are parked in the warp's slice of shared memory, and the warp
// then walks over the piece 512 elements at a time: lane l expands elements 16 l .. 16 l + 15 (four lanes
// per 64-element absmax block) and writes them with one 32-byte vector store, so a store instruction of
// the warp writes 1 KB of contiguous output.
//   1 bit : the two levels are scaled by the block's absmax and rounded to bf16 once; a pair of elements is
//           then one multiply-add (min + bit * |H - L| in both 16-bit halves);
//   2 bits: the four scaled levels sit in two registers, a pair of elements is one byte permute;
//   4 bits: the row's 16 fp32 levels are staged in shared memory; per element one load, one multiply,
//           half a convert.
// Results are bit-identical to table[code] * absmax rounded to bf16 (round to nearest even).
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

__device__ __forceinline__ void st_stream_v8(void* p, const uint32_t (&v)[8]) {
    asm volatile("st.global.cs.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(p), "r"(v[0]), "r"(v[1]), "r"(v[2]),
                 "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7])
                 : "memory");
}

struct WarpStage {
    uint4 packed[32];    // the 512-byte piece
    float absmax[64];    // absmax of the piece's blocks (64 at 1 bit, 32 at 2 bits, 16 at 4 bits)
    float lut[16];       // 4-bit rows: the row's levels
};

// What a warp fetches for its piece.
struct Fetched {
    uint4 packed;        // this lane's 16 packed bytes
    float a0, a1;        // absmax of blocks lane and lane + 32 of the piece
    float m0, m1, m2, m3;   // 1 bit: levels 0, 1; 2 bits: levels 0 .. 3; 4 bits: m0 = level `lane` (lanes 0 .. 15)
    int c, e0, K;        // class, first element of the piece, row length
    uint16_t* dst;       // where element e0 of the row goes
};

__device__ __forceinline__ void locate(const DecodeParams& P, uint32_t t, int& c, int& p, int& piece) {
    c = (t >= P.task_start[1]) + (t >= P.task_start[2]);
    const uint32_t local = t - P.task_start[c];
    const uint32_t ppr = P.pieces_per_row[c];
    const int q = local / ppr;
    piece = local - q * ppr;
    p = P.L.class_start[c] + q;
}

__device__ __forceinline__ void fetch_piece(const DecodeParams& P, uint32_t t, int lane, Fetched& f) {
    int c, p, piece;
    locate(P, t, c, p, piece);
    const int K = P.L.K;
    const int r = __ldg(P.L.perm + p);
    const size_t row_bytes = ((size_t)K << c) >> 3;
    const uint8_t* row = P.packed + packed_row_offset(P.L, c, p, r);
    const size_t byte0 = (size_t)piece * 512 + (size_t)lane * 16;
    const int e0 = piece * (4096 >> c);                          // first element of the piece
    const int kBlocks = 64 >> c;                                 // blocks in a full piece
    const float* arow = P.absmax + (size_t)absmax_row_of(P.L, p, r) * P.L.nb + e0 / kBlock;
    const int blocks_left = P.L.nb - e0 / kBlock;                // blocks of the row from e0 on
    const float* mrow = P.maps + (size_t)r * kTableStride;
    f.packed = (byte0 < row_bytes) ? ld_stream_v4(row + byte0) : make_uint4(0u, 0u, 0u, 0u);
    f.a0 = (lane < kBlocks && lane < blocks_left) ? __ldg(arow + lane) : 0.0f;
    f.a1 = (lane + 32 < kBlocks && lane + 32 < blocks_left) ? __ldg(arow + lane + 32) : 0.0f;
    f.m0 = f.m1 = f.m2 = f.m3 = 0.0f;
    if (c == 2) {
        if (lane < 16) f.m0 = __ldg(mrow + lane);
    } else {
        f.m0 = __ldg(mrow); f.m1 = __ldg(mrow + 1);
        if (c == 1) { f.m2 = __ldg(mrow + 2); f.m3 = __ldg(mrow + 3); }
    }
    f.c = c; f.e0 = e0; f.K = K;
    f.dst = P.out + (size_t)r * K + e0;
}

// Expands the piece parked in the warp's stage: lane l, in round j, elements e0 + 512 j + 16 l .. + 15.
template <int B>
__device__ __forceinline__ void expand_piece(const Fetched& f, int lane, const WarpStage* ws) {
    constexpr int kIters = 8 / B;          // 512 elements per iteration
    const int K = f.K;
    uint16_t* dst = f.dst + lane * 16;
    const unsigned char* bytes = reinterpret_cast<const unsigned char*>(ws->packed);
    const float m0 = f.m0, m1 = f.m1, m2 = f.m2, m3 = f.m3;
#pragma unroll
    for (int j = 0; j < kIters; ++j) {
        // lane l: elements e0 + 512 j + 16 l .. + 15, i.e. bits [(512 j + 16 l) B, + 16 B) of the piece
        const int e = f.e0 + 512 * j + 16 * lane;
        const float a = ws->absmax[8 * j + (lane >> 2)];
        uint32_t o[8];
        if (B == 1) {
            const uint32_t h = *reinterpret_cast<const uint16_t*>(bytes + 64 * j + 2 * lane);
            const uint32_t LH = pack_bf16x2(__fmul_rn(m0, a), __fmul_rn(m1, a));
            const uint32_t L = LH & 0xFFFFu, H = LH >> 16;
            const uint32_t lo = min(L, H);
            const uint32_t BB = lo * 0x10001u, d = max(L, H) - lo, fl = (L > H) ? 0x10001u : 0u;
            const uint32_t z = h | (h << 15);   // pair i at bits 0 and 16 of z >> 2i
#pragma unroll
            for (int i = 0; i < 8; ++i) o[i] = (((z >> (2 * i)) & 0x10001u) ^ fl) * d + BB;
        } else if (B == 2) {
            const uint32_t w = *reinterpret_cast<const uint32_t*>(bytes + 128 * j + 4 * lane);
            const uint32_t E01 = pack_bf16x2(__fmul_rn(m0, a), __fmul_rn(m1, a));
            const uint32_t E23 = pack_bf16x2(__fmul_rn(m2, a), __fmul_rn(m3, a));
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const uint32_t y = w >> (4 * i);
                const uint32_t t = (y & 3u) | ((y << 6) & 0x300u);
                o[i] = __byte_perm(E01, E23, t * 0x22u + 0x1010u);
            }
        } else {
            const uint2 w = *reinterpret_cast<const uint2*>(bytes + 256 * j + 8 * lane);
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const uint32_t x = ((i < 4) ? w.x : w.y) >> (8 * (i & 3));
                o[i] = pack_bf16x2(__fmul_rn(ws->lut[x & 15u], a), __fmul_rn(ws->lut[(x >> 4) & 15u], a));
            }
        }
        if (e < K) st_stream_v8(dst + 512 * j, o);
    }
}

// The tasks of up to NM matrices, numbered through: matrix after matrix, inside a matrix class after class.
template <int NM>
struct DecodeGroup {
    DecodeParams m[NM];
    uint32_t first_task[NM + 1];   // first task of every member; [NM] (and the entries of unused members) = number of tasks
};

template <int NM>
__device__ __forceinline__ void fetch_task(const DecodeGroup<NM>& G, uint32_t t, int lane, Fetched& f) {
    int mi = 0;
#pragma unroll
    for (int i = 1; i < NM; ++i) mi += (t >= G.first_task[i]) ? 1 : 0;
    fetch_piece(G.m[mi], t - G.first_task[mi], lane, f);
}

// One piece per warp, one CTA per eight pieces: the hardware hands fresh CTAs to the SMs as others finish, which keeps the
// SMs evenly loaded although the pieces differ in length by a factor of four (a persistent grid whose warps walked over
// several pieces each, the next one's loads in flight, was 8 % slower).
template <int NM>
__global__ void __launch_bounds__(kDecodeThreads, 5) decode_kernel(const __grid_constant__ DecodeGroup<NM> G) {
    __shared__ __align__(16) WarpStage stage_all[kDecodeWarps];
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    WarpStage* ws = &stage_all[warp];
    pdl_enter();
    const uint32_t t = blockIdx.x * kDecodeWarps + warp;
    if (t >= G.first_task[NM]) return;
    Fetched cur;
    fetch_task<NM>(G, t, lane, cur);
    ws->packed[lane] = cur.packed;
    ws->absmax[lane] = cur.a0;
    ws->absmax[lane + 32] = cur.a1;
    if (cur.c == 2 && lane < 16) ws->lut[lane] = cur.m0;
    __syncwarp();
    if (cur.c == 0) expand_piece<1>(cur, lane, ws);
    else if (cur.c == 1) expand_piece<2>(cur, lane, ws);
    else expand_piece<4>(cur, lane, ws);
}

namespace {

// checks one matrix's arguments and fills its entry; `tasks` receives the number of its tasks
lowra_status decode_member(const lowra_layout* layout, const uint8_t* packed_dev, const float* absmax_dev, const float* maps_dev,
                           uint16_t* W_bf16_dev, DecodeParams& P, uint64_t& tasks) {
    lowra_status st = check_layout(layout);
    if (st != LOWRA_OK) return st;
    if (!packed_dev || !absmax_dev || !maps_dev || !W_bf16_dev) return LOWRA_ERR_NULL;
    if (!aligned16(packed_dev) || !aligned16(absmax_dev) || !aligned16(maps_dev) ||
        (reinterpret_cast<uintptr_t>(W_bf16_dev) & 31u) != 0)
        return LOWRA_ERR_ALIGN;
    P.L = make_row_layout(layout);
    P.packed = packed_dev;
    P.absmax = absmax_dev;
    P.maps = maps_dev;
    P.out = W_bf16_dev;
    tasks = 0;
    for (int c = 0; c < 3; ++c) {
        const uint64_t row_bytes = (uint64_t)layout->K * (1u << c) / 8u;
        P.pieces_per_row[c] = (uint32_t)((row_bytes + 511) / 512);
        P.task_start[c] = (uint32_t)tasks;
        tasks += (uint64_t)layout->counts[c] * P.pieces_per_row[c];
    }
    if (tasks > 0xFFFFFFFFull) return LOWRA_ERR_SHAPE;
    P.task_start[3] = (uint32_t)tasks;
    return LOWRA_OK;
}

template <int NM>
lowra_status launch_decode(const DecodeGroup<NM>& G, void* stream) {
    const uint64_t tasks = G.first_task[NM];
    const unsigned grid = (unsigned)((tasks + kDecodeWarps - 1) / kDecodeWarps);   // < 2^29: the tasks were counted in 32 bits
    return launch_pdl(decode_kernel<NM>, grid, kDecodeThreads, (cudaStream_t)stream, G) == cudaSuccess ? LOWRA_OK : LOWRA_ERR_CUDA;
}

}  // namespace

}  // namespace lowra

extern "C" lowra_status lowra_decode(const lowra_layout* layout, const uint8_t* packed_dev,
                                     const float* absmax_dev, const float* maps_dev, uint16_t* W_bf16_dev,
                                     void* stream) {
    using namespace lowra;
    DecodeGroup<1> G;
    uint64_t tasks = 0;
    lowra_status st = decode_member(layout, packed_dev, absmax_dev, maps_dev, W_bf16_dev, G.m[0], tasks);
    if (st != LOWRA_OK) return st;
    st = check_device();
    if (st != LOWRA_OK) return st;
    G.first_task[0] = 0;
    G.first_task[1] = (uint32_t)tasks;
    return launch_decode<1>(G, stream);
}

extern "C" lowra_status lowra_decode_group(const lowra_group_member* members_host, int32_t count, void* stream) {
    using namespace lowra;
    if (!members_host) return LOWRA_ERR_NULL;
    if (count < 1 || count > LOWRA_MAX_GROUP) return LOWRA_ERR_SHAPE;
    DecodeGroup<LOWRA_MAX_GROUP> G;
    uint64_t total = 0;
    for (int i = 0; i < count; ++i) {
        const lowra_group_member& m = members_host[i];
        uint64_t tasks = 0;
        lowra_status st = decode_member(m.layout, m.packed_dev, m.absmax_dev, m.tables_dev, m.W_bf16_dev, G.m[i], tasks);
        if (st != LOWRA_OK) return st;
        G.first_task[i] = (uint32_t)total;
        total += tasks;
        if (total > 0xFFFFFFFFull) return LOWRA_ERR_SHAPE;
    }
    for (int i = count; i <= LOWRA_MAX_GROUP; ++i) {
        if (i < LOWRA_MAX_GROUP) G.m[i] = G.m[0];
        G.first_task[i] = (uint32_t)total;
    }
    lowra_status st = check_device();
    if (st != LOWRA_OK) return st;
    return launch_decode<LOWRA_MAX_GROUP>(G, stream);
}
