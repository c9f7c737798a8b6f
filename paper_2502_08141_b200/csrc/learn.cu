// lowra_learn_codebooks: weighted Lloyd-Max per output channel (paper Section 5, "Weighted Lloyd's for LoRA
// Quantization", and the appendix "Weighted Lloyd-Max Algorithm"; the appendix on the learner's initialisation
// gives the initial tables, which the caller passes in).
//
// For every row, at the row's assigned precision b: the data are the row's normalised values n_i (block
// absmax normalisation exactly as in lowra_encode), each weighted by the absmax of its block; starting from the
// given levels y and thresholds t, T times: assign every value to its bucket (number of thresholds <= n),
// replace every level by the weighted mean of its bucket (an empty bucket keeps its level), set the thresholds
// to the midpoints of neighbouring levels.  All of that in fp64.  Output: the levels rounded to fp32 and the
// midpoints of those fp32 levels (computed in fp64, rounded to fp32), in [N, 16] tables.
//
// One CTA per row (as many CTAs as rows): the row is read from HBM once (4 bytes per element, the
// kernel's only traffic), normalised on its way into shared memory; the T passes run out of shared memory.
// Every thread keeps private fp64 sums per bucket: in registers for 1 and 2 bits, in a bank-conflict-free
// slice of shared memory for 4 bits; the block's weight enters once per sixteen elements (they are added up exactly
// first); a fixed reduction tree adds the threads' sums up (a halving exchange inside a warp, then across warps), so
// results are reproducible from run to run - but the order of the fp64 operations is not the index order of a
// serial loop, so sums agree with a serial implementation to rounding only.  One barrier per round; every warp forms
// the new levels and thresholds itself; a row whose thresholds have settled (as fp32 numbers) skips its remaining rounds.
#include <string.h>

#include "lowra_common.cuh"

namespace lowra {

constexpr int kLearnThreads = 128;
constexpr int kLearnWarps = kLearnThreads / 32;
constexpr int kLoadsInFlight = 8;   // 128-bit loads a thread issues before it looks at the first one (a 4096-element row in one go)

struct LearnParams {
    RowLayout L;
    const float* W;       // [N, K] original order
    float* maps;          // [N, 16] original order ([3][N][16] in the three-precision form: plane c = 2^c bits)
    float* thresholds;    // likewise
    int iterations;
    int N, K;             // the three-precision form has no layout: every row is learnt at 1, 2 and 4 bits
    double init_y[3][16];  // initial levels per class (1, 2, 4 bits)
    double init_t[3][16];  // initial thresholds per class
};

// NV sums per lane (NV = 4, 8 or 16) added up over the warp: instead of NV butterflies over all 32 lanes, every step
// hands half of a lane's values to its partner and adds the partner's other half to its own, so that the number of
// values halves with the distance; once a lane holds one value the remaining steps are plain butterflies.  Afterwards
// the lanes whose low bits are zero hold the totals: value number lane / (32 / NV) in v[0].  A fixed order of additions.
template <int NV>
__device__ __forceinline__ void warp_sums(double (&v)[NV], int lane) {
    int d = 16;
#pragma unroll
    for (int n = NV; n > 1; n >>= 1, d >>= 1) {
        const bool upper = (lane & d) != 0;
#pragma unroll
        for (int k = 0; k < n / 2; ++k) {
            const double send = upper ? v[k] : v[k + n / 2];
            const double keep = upper ? v[k + n / 2] : v[k];
            v[k] = keep + __shfl_xor_sync(0xffffffffu, send, d);
        }
    }
#pragma unroll
    for (; d >= 1; d >>= 1) v[0] += __shfl_xor_sync(0xffffffffu, v[0], d);
}

// number of thresholds <= x among t[0 .. L-2] (sorted): branch-free binary search, L = 2, 4 or 16.
// x is an fp32 value and tf[j] is the least fp32 number >= the fp64 threshold t[j], so "t[j] <= x" (in fp64) and
// "tf[j] <= x" (in fp32) are the same statement.
template <int B>
__device__ __forceinline__ int bucket_of(float x, const float* tf) {
    if (B == 1) return tf[0] <= x ? 1 : 0;
    if (B == 2) {
        const int hi = tf[1] <= x ? 2 : 0;
        return hi + (tf[hi] <= x ? 1 : 0);
    }
    int c = tf[7] <= x ? 8 : 0;
    c += tf[c + 3] <= x ? 4 : 0;
    c += tf[c + 1] <= x ? 2 : 0;
    c += tf[c] <= x ? 1 : 0;
    return c;
}

// Where group of four elements number q of a row lies in shared memory (in units of 16 bytes).  The rounds read the row
// sixteen elements = four groups per thread at a time (eight in the 4-bit rounds); with the groups of every set of four
// exchanged among themselves by the number of the pair of sets they are in, the eight lanes that share a shared-memory
// wavefront fall into eight different 16-byte columns, in the rounds' reads and in the loader's writes alike.
__device__ __forceinline__ int quad_slot(int q) { return q ^ ((q >> 3) & 3); }

// The row: coalesced 128-bit loads (all of a thread's loads in flight together); sixteen neighbouring lanes hold one
// 64-element block between them, so the block's absmax is four shuffles away and the values go to shared memory
// already normalised (as in lowra_encode: reciprocal rounded to nearest, one multiplication).  Ends with a barrier.
__device__ void load_row(const LearnParams& P, int r, float* xs, float* ws) {
    const int K = P.K;
    const int tid = threadIdx.x;
    const float* wrow = P.W + (size_t)r * K;
    for (int i0 = 0; i0 < K; i0 += 4 * kLoadsInFlight * kLearnThreads) {
        float4 v[kLoadsInFlight];
#pragma unroll
        for (int u = 0; u < kLoadsInFlight; ++u) {
            const int i = i0 + 4 * (u * kLearnThreads + tid);
            v[u] = (i < K) ? ld_stream_f4(wrow + i) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int u = 0; u < kLoadsInFlight; ++u) {
            const int i = i0 + 4 * (u * kLearnThreads + tid);   // K is a multiple of 128: a warp is in or out as a whole
            float m = fmaxf(fmaxf(fabsf(v[u].x), fabsf(v[u].y)), fmaxf(fabsf(v[u].z), fabsf(v[u].w)));
#pragma unroll
            for (int d = 8; d >= 1; d >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, d));
            const float inv = (m == 0.0f) ? 0.0f : __frcp_rn(m);
            if (i < K) {
                *reinterpret_cast<float4*>(xs + 4 * quad_slot(i >> 2)) =
                    make_float4(__fmul_rn(v[u].x, inv), __fmul_rn(v[u].y, inv), __fmul_rn(v[u].z, inv), __fmul_rn(v[u].w, inv));
                if ((tid & 15) == 0) ws[i / kBlock] = m;
            }
        }
    }
    __syncthreads();
}

// T rounds on the row parked in shared memory, at B bits; tables to maps_out / thr_out ([16] each).
// One barrier per round: the warps leave their partial sums in shared memory (two buffers, used in turn), meet once, and
// then EVERY warp forms the new levels and thresholds for itself - lane j holds level j and threshold j in registers, the
// same numbers in every warp since they come from the same partial sums in the same order - so nobody waits for a
// first warp to publish them.
template <int B>
__device__ void learn_row(const LearnParams& P, const float* xs, const float* ws, double* acc, double* red2, float* tfw_all,
                          float* maps_out, float* thr_out) {
    constexpr int Lv = 1 << B;      // levels
    constexpr int c = B >> 1;       // class index
    const int K = P.K;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    float* tf = tfw_all + warp * 16;                      // 4 bits: this warp's copy of the thresholds (bucket search by index)
    double ylane = lane < Lv ? P.init_y[c][lane] : 0.0;   // level `lane`
    float tlane = lane + 1 < Lv ? __double2float_ru(P.init_t[c][lane]) : 0.0f;   // threshold `lane`: the least fp32 number >= it
    float th[B <= 2 ? Lv - 1 : 1];                        // 1 and 2 bits: all thresholds in registers
    if (B <= 2) {
#pragma unroll
        for (int j = 0; j < Lv - 1; ++j) th[j] = __double2float_ru(P.init_t[c][j]);
    } else {
        if (lane < 16) tf[lane] = tlane;
        __syncwarp();
    }

    for (int it = 0; it < P.iterations; ++it) {
        double* red = red2 + (it & 1) * (2 * 16 * kLearnWarps);
        // ---- one pass: private sums of w * n and w per bucket.  The weight is the same for the sixteen elements a thread
        // takes at a time (a quarter of a 64-element block), so the elements themselves are added up per bucket first
        // (exactly: sixteen fp32 values in fp64) and counted, and the weight enters once per sixteen elements and bucket.
        if (B <= 2) {
            // Few buckets: no bucket index at all.  cn[0] / cd[0] take the elements below the first threshold, cn[j] /
            // cd[j] (j >= 1) everything at or above threshold j - 1 - predicated adds - and a bucket's sums are the
            // difference of two neighbours (which were added up over the same elements in the same order wherever the
            // bucket is empty, so that an empty bucket has exactly zero weight).
            double cn[Lv], cd[Lv];
#pragma unroll
            for (int j = 0; j < Lv; ++j) cn[j] = cd[j] = 0.0;
            for (int run = tid; run < K / 16; run += kLearnThreads) {   // elements 16 run .. 16 run + 15, all in block run / 4
                const float4 xa = *reinterpret_cast<const float4*>(xs + 4 * quad_slot(4 * run));
                const float4 xb = *reinterpret_cast<const float4*>(xs + 4 * quad_slot(4 * run + 1));
                const float4 xc = *reinterpret_cast<const float4*>(xs + 4 * quad_slot(4 * run + 2));
                const float4 xd = *reinterpret_cast<const float4*>(xs + 4 * quad_slot(4 * run + 3));
                const double w = (double)ws[run >> 2];
                const float xf[16] = {xa.x, xa.y, xa.z, xa.w, xb.x, xb.y, xb.z, xb.w, xc.x, xc.y, xc.z, xc.w, xd.x, xd.y, xd.z, xd.w};
                double sq[Lv];
                int cq[Lv];
#pragma unroll
                for (int j = 0; j < Lv; ++j) { sq[j] = 0.0; cq[j] = 0; }
#pragma unroll
                for (int u = 0; u < 16; ++u) {
                    const double x = (double)xf[u];
                    if (th[0] <= xf[u]) { sq[1] += x; ++cq[1]; } else { sq[0] += x; ++cq[0]; }
#pragma unroll
                    for (int j = 2; j < Lv; ++j)
                        if (th[j - 1] <= xf[u]) { sq[j] += x; ++cq[j]; }
                }
#pragma unroll
                for (int j = 0; j < Lv; ++j) {
                    cn[j] = fma(w, sq[j], cn[j]);
                    cd[j] = fma(w, (double)cq[j], cd[j]);
                }
            }
            double v[2 * Lv];
#pragma unroll
            for (int j = 0; j < Lv; ++j) {
                v[2 * j] = (j == 0 || j == Lv - 1) ? cn[j] : cn[j] - cn[j + 1];
                v[2 * j + 1] = (j == 0 || j == Lv - 1) ? cd[j] : cd[j] - cd[j + 1];
            }
            warp_sums<2 * Lv>(v, lane);
            if ((lane & (32 / (2 * Lv) - 1)) == 0) red[(lane / (32 / (2 * Lv))) * kLearnWarps + warp] = v[0];
        } else {
            // 16 buckets: the sums live in shared memory, one (w n, w) pair per thread and bucket; eight elements at a
            // time, their bucket searches side by side
            double2* acc2 = reinterpret_cast<double2*>(acc);
#pragma unroll
            for (int j = 0; j < Lv; ++j) acc2[j * kLearnThreads + tid] = make_double2(0.0, 0.0);
            for (int run = tid; run < K / 8; run += kLearnThreads) {
                const float4 xa = *reinterpret_cast<const float4*>(xs + 4 * quad_slot(2 * run));
                const float4 xb = *reinterpret_cast<const float4*>(xs + 4 * quad_slot(2 * run + 1));
                const double w = (double)ws[run >> 3];
                const float xf[8] = {xa.x, xa.y, xa.z, xa.w, xb.x, xb.y, xb.z, xb.w};
                int b[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) b[u] = bucket_of<B>(xf[u], tf);
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    double2 a = acc2[b[u] * kLearnThreads + tid];
                    a.x = fma(w, (double)xf[u], a.x);
                    a.y += w;
                    acc2[b[u] * kLearnThreads + tid] = a;
                }
            }
#pragma unroll
            for (int half = 0; half < 2; ++half) {   // eight buckets = sixteen sums at a time
                double v[16];
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const double2 a = acc2[(8 * half + j) * kLearnThreads + tid];
                    v[2 * j] = a.x;
                    v[2 * j + 1] = a.y;
                }
                warp_sums<16>(v, lane);
                if ((lane & 1) == 0) red[(16 * half + lane / 2) * kLearnWarps + warp] = v[0];
            }
        }
        __syncthreads();
        // ---- new levels (an empty bucket keeps its level), then midpoints with a shuffle in between: every warp
        if (lane < Lv) {
            double sn = 0.0, sd = 0.0;
#pragma unroll
            for (int w2 = 0; w2 < kLearnWarps; ++w2) { sn += red[(2 * lane) * kLearnWarps + w2]; sd += red[(2 * lane + 1) * kLearnWarps + w2]; }
            if (sd > 0.0) ylane = sn / sd;
        }
        const double yn = __shfl_down_sync(0xffffffffu, ylane, 1);
        bool same = true;
        if (lane + 1 < Lv) {
            const float tn = __double2float_ru((ylane + yn) * 0.5);
            same = tn == tlane;
            tlane = tn;
        }
        if (B <= 2) {
#pragma unroll
            for (int j = 0; j < Lv - 1; ++j) th[j] = __shfl_sync(0xffffffffu, tlane, j);
        } else {
            if (lane < 16) tf[lane] = tlane;
            __syncwarp();
        }
        // thresholds that have not moved (as the fp32 numbers the elements are compared with) assign every element
        // as before: the next round would add the same sums up in the same order and change nothing, nor any later one
        if (__all_sync(0xffffffffu, same)) break;
    }

    // ---- tables: fp32 levels, midpoints of the fp32 levels; unused levels 0, unused thresholds +inf
    if (warp == 0) {
        const float m = (lane < Lv) ? (float)ylane : 0.0f;
        const float mn = __shfl_down_sync(0xffffffffu, m, 1);
        if (lane < kTableStride) {
            maps_out[lane] = m;
            thr_out[lane] = (lane + 1 < Lv) ? (float)(((double)m + (double)mn) * 0.5) : __int_as_float(0x7f800000);
        }
    }
    __syncthreads();   // the sums in shared memory are reused by the next run, the row buffer by the next row
}

// FOUR = false: for weights without 4-bit rows.  Only the 4-bit runs need the 32 KB of per-thread bucket sums in shared
// memory, and the rounds of a row are a chain of short phases between barriers, so what hides their latency is the number
// of CTAs per SM: without those 32 KB three times as many fit (all-1-bit rows: 0.52 -> 0.34 ms on 4096 x 11008 at ten
// rounds).  (Running the 4-bit rows of a mixed weight in a kernel of their own was slower: the few rows leave most SMs
// idle for the length of a row.)
template <bool ALL3, bool FOUR>
__global__ void __launch_bounds__(kLearnThreads) learn_kernel(const __grid_constant__ LearnParams P) {
    extern __shared__ __align__(16) unsigned char learn_smem[];
    // [2 x 2 * 16 * warps doubles partial sums][FOUR: 2 * 16 * threads doubles sums][K floats][nb floats][warps x 16 floats]
    double* red2 = reinterpret_cast<double*>(learn_smem);
    double* acc = red2 + 2 * 2 * 16 * kLearnWarps;
    float* xs = reinterpret_cast<float*>(acc + (FOUR ? 2 * 16 * kLearnThreads : 0));
    float* ws = xs + P.K;
    float* tfw = ws + P.K / kBlock;   // 4-bit runs: a copy of the thresholds (fp32 upper neighbours) per warp
    pdl_enter();
    for (int i = blockIdx.x; i < P.N; i += gridDim.x) {
        // with a layout: stored rows from the last to the first, i.e. the long 4-bit rows are handed out first and the
        // short 1-bit rows fill the gaps at the end
        const int r = ALL3 ? i : P.L.perm[P.N - 1 - i];
        load_row(P, r, xs, ws);
        float* m = P.maps + (size_t)r * kTableStride;
        float* h = P.thresholds + (size_t)r * kTableStride;
        if (ALL3) {
            // the row under every precision, from the one copy in shared memory
            const size_t plane = (size_t)P.N * kTableStride;
            learn_row<1>(P, xs, ws, acc, red2, tfw, m, h);
            learn_row<2>(P, xs, ws, acc, red2, tfw, m + plane, h + plane);
            if (FOUR) learn_row<4>(P, xs, ws, acc, red2, tfw, m + 2 * plane, h + 2 * plane);
        } else {
            const int b = P.L.precs[r];
            if (b == 1) learn_row<1>(P, xs, ws, acc, red2, tfw, m, h);
            else if (b == 2) learn_row<2>(P, xs, ws, acc, red2, tfw, m, h);
            else if (FOUR) learn_row<4>(P, xs, ws, acc, red2, tfw, m, h);
        }
    }
}

}  // namespace lowra

namespace lowra {
namespace {

// validation shared by the two entry points is done by the callers; this fills the tables and launches
template <bool ALL3, bool FOUR>
lowra_status launch_learn_kernel(const LearnParams& P, void* stream) {
    const size_t smem = (2 * 2 * 16 * kLearnWarps + (FOUR ? 2 * 16 * kLearnThreads : 0)) * sizeof(double) +
                        ((size_t)P.K + (size_t)P.K / kBlock + 16 * kLearnWarps) * sizeof(float);
    if (smem > 200 * 1024) return LOWRA_ERR_SHAPE;   // the row has to fit into shared memory (K <= 40960)
    static SmemLimit limit = {};
    if (ensure_smem_limit(reinterpret_cast<const void*>(learn_kernel<ALL3, FOUR>), smem, &limit) != LOWRA_OK) return LOWRA_ERR_CUDA;
    // a row per CTA and as many CTAs as rows: a 4-bit row takes five times as long as a 1-bit one, and fresh CTAs handed out
    // by the hardware keep the SMs evenly busy where a persistent grid (every CTA walking over its share of the rows) left
    // some of them waiting at the end (the 7B layer at 60/35/5: 2.05 -> 1.68 ms)
    const unsigned grid = (unsigned)P.N;
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.gridDim = dim3(grid, 1, 1);
    cfg.blockDim = dim3(kLearnThreads, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = (cudaStream_t)stream;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, learn_kernel<ALL3, FOUR>, P) == cudaSuccess ? LOWRA_OK : LOWRA_ERR_CUDA;
}

// validation shared by the two entry points is done by the callers; this fills the tables and launches (`four`: whether
// any run at 4 bits is asked for)
template <bool ALL3>
lowra_status launch_learn(LearnParams& P, const double* init_levels_host, const double* init_thresholds_host,
                          bool four, void* stream) {
    if (((size_t)P.K + (size_t)P.K / kBlock) * sizeof(float) > 160 * 1024) return LOWRA_ERR_SHAPE;   // K <= 40960: the row has to fit
    lowra_status st = check_device();
    if (st != LOWRA_OK) return st;
    for (int c = 0; c < 3; ++c)
        for (int j = 0; j < 16; ++j) {
            P.init_y[c][j] = init_levels_host[c * 16 + j];
            P.init_t[c][j] = init_thresholds_host[c * 16 + j];
        }
    return four ? launch_learn_kernel<ALL3, true>(P, stream) : launch_learn_kernel<ALL3, false>(P, stream);
}

}  // namespace
}  // namespace lowra

extern "C" lowra_status lowra_learn_codebooks(const lowra_layout* layout, const float* W_dev,
                                              const double* init_levels_host, const double* init_thresholds_host,
                                              int32_t iterations, float* maps_dev, float* thresholds_dev, void* stream) {
    using namespace lowra;
    lowra_status st = check_layout(layout);
    if (st != LOWRA_OK) return st;
    if (!W_dev || !init_levels_host || !init_thresholds_host || !maps_dev || !thresholds_dev) return LOWRA_ERR_NULL;
    if (iterations < 0 || iterations > 1000) return LOWRA_ERR_SHAPE;
    if (!aligned16(W_dev) || !aligned16(maps_dev) || !aligned16(thresholds_dev)) return LOWRA_ERR_ALIGN;
    LearnParams P;
    P.L = make_row_layout(layout);
    P.W = W_dev;
    P.maps = maps_dev;
    P.thresholds = thresholds_dev;
    P.iterations = iterations;
    P.N = layout->N;
    P.K = layout->K;
    return launch_learn<false>(P, init_levels_host, init_thresholds_host, layout->counts[2] > 0, stream);
}

extern "C" lowra_status lowra_learn_codebooks_all(int32_t N, int32_t K, const float* W_dev,
                                                  const double* init_levels_host, const double* init_thresholds_host,
                                                  int32_t iterations, float* maps3_dev, float* thresholds3_dev,
                                                  void* stream) {
    using namespace lowra;
    if (!W_dev || !init_levels_host || !init_thresholds_host || !maps3_dev || !thresholds3_dev) return LOWRA_ERR_NULL;
    if (N < 1 || K < 128 || K % 128 != 0 || iterations < 0 || iterations > 1000) return LOWRA_ERR_SHAPE;
    if (!aligned16(W_dev) || !aligned16(maps3_dev) || !aligned16(thresholds3_dev)) return LOWRA_ERR_ALIGN;
    LearnParams P;
    memset(&P.L, 0, sizeof(P.L));   // no layout: every row at every precision
    P.W = W_dev;
    P.maps = maps3_dev;
    P.thresholds = thresholds3_dev;
    P.iterations = iterations;
    P.N = N;
    P.K = K;
    return launch_learn<true>(P, init_levels_host, init_thresholds_host, true, stream);
}
