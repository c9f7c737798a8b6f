// Fused dequant + LoRA tensor-core kernel (forward, backward-input, and a dense diagnostic mode).
//
// Persistent CTAs, one per SM, in clusters of two, walk over output tiles of 128 "operand rows" x 256 tokens:
//   forward : operand rows = output channels n;  Y^T tile [128 n x 256 m]  = W_hat[n, :] . X[m, :]
//   backward: operand rows = input features k;   dX^T tile [128 k x 256 m] = W_hat[:, k] . dY[m, :]
// The 128-row operand (the weights) is the A operand of tcgen05.mma.  Eight dequant warps produce it in shared
// memory straight from the packed codes (never from HBM as bf16), one 128-byte row per 64-element absmax
// block: K-major in the forward pass (a thread keeps one output channel for the whole tile), MN-major in the
// backward pass (every stage brings 64 new channels, dealt to the warps by the prologue).  The two CTAs of a
// cluster work on the same weight rows and on neighbouring token tiles, in lock step: they take the stages in
// turn, and the CTA that has dequantised a stage's operand tile sends a copy into its peer's shared memory
// (one asynchronous 16 KB copy, counted on the peer's stage barrier), so every weight is dequantised once
// per 512 tokens.  The 256-token operand (activations / output gradients) is the B operand and arrives by
// TMA.  Shared memory holds five weight slots and four token slots.  Accumulators live in TMEM (two, so the
// epilogue of a tile overlaps the main loop of the next).
// The LoRA term is folded into the same accumulator as extra contraction blocks at the end of every
// tile: the up-projection factor comes by TMA straight from the caller's matrix, the down-projected
// activations T = s X A (resp. U = s dY B^T) by TMA from the workspace.  T itself is produced by this same
// kernel: for every token tile there is one extra "T tile" whose 128 operand rows are the LoRA ranks
// (factor fetched by TMA, no dequant); T tiles come first in the tile order, their epilogue publishes a
// per-token-tile flag, and the TMA producer of a regular tile waits (bounded) for that flag before it
// fetches T.  All CTAs are co-resident and a T tile waits for nothing, so the wait cannot deadlock.
// Schedule: whole tiles dealt round-robin to the clusters, or (launcher's choice) stream-K behind the first rows of
// whole tiles: equal consecutive ranges of the remaining weight tiles' contraction blocks per cluster, partial tiles
// handed over through a scratch slot and either preloaded into the accumulator of the cluster that starts the tile
// or added in its epilogue (see the schedule in the kernel).
//
// Warp roles: 0 = TMA producer, 1 = MMA issuer (and TMEM owner), 2-5 = epilogue, 6-8 / 10-12 / 14-15 = dequant.
// All mbarrier waits are bounded; a wait that runs out sets the status word and every role leaves.
#include <mutex>

#include "gemm_params.cuh"
#include "ptx.cuh"

namespace lowra {

namespace {

constexpr uint64_t kGraceNs = 50ull * 1000ull;   // after a failure: time for copies and MMAs still in flight to land
constexpr uint32_t kIdesc = ptx::umma_idesc_bf16(kTileR, kTileT);
constexpr uint32_t kIdescAmn = kIdesc | (1u << 15);   // A operand MN-major

struct Barriers {
    uint64_t full_x[kStages];   // TMA bytes of a stage have landed
    uint64_t full_w[kMaxStagesA];   // the weight operand of a stage is complete (dequant warps, or a copy from a peer CTA)
    uint64_t empty[kStages];    // the MMAs reading a shared-memory stage have completed
    uint64_t tmem_full[2];
    uint64_t tmem_empty[2];
    uint64_t drain;
    uint64_t part_full;   // stream-K: a partial tile has been copied into the (idle) operand ring
    uint32_t tmem_base;
    uint32_t abort;
    uint32_t epi_leave[2];             // the epilogue warps' common answer to "has somebody given up?"
    uint32_t produced[kMaxStagesA];    // arrivals of this CTA's dequant warps on the stage being filled
    uint32_t free_upto[kCluster];   // stages 0 .. free_upto[c] - 1 have been found free by the TMA
                                       // producer of CTA c of the cluster (every CTA holds a copy of all counters)
};

// fields of the forward row word written by the prologue: bits 0-6 row offset inside the tile, 7-8 class
// (0, 1, 2 = 1, 2, 4 bits; 3 = row past N, to be zero-filled), 9-31 stored position
__device__ __forceinline__ int info_row(uint32_t w) { return (int)(w & 127u); }
__device__ __forceinline__ int info_class(uint32_t w) { return (int)((w >> 7) & 3u); }
__device__ __forceinline__ int info_pos(uint32_t w) { return (int)(w >> 9); }

// ---- dequantisation of one 64-element block to 64 bf16 (one 128-byte operand row) -----------------
// Packed codes of one 64-element block (8, 16 or 32 bytes) plus the block's absmax.
struct Block {
    uint4 lo, hi;
    float a;
};

__device__ __forceinline__ void load_block(Block& blk, const uint8_t* p, const float* absmax, int cls) {
    if (cls == 0) {
        const uint2 t = __ldg(reinterpret_cast<const uint2*>(p));
        blk.lo.x = t.x;
        blk.lo.y = t.y;
    } else if (cls == 1) {
        blk.lo = __ldg(reinterpret_cast<const uint4*>(p));
    } else if (cls == 2) {
        blk.lo = __ldg(reinterpret_cast<const uint4*>(p));
        blk.hi = __ldg(reinterpret_cast<const uint4*>(p) + 1);
    }
    if (cls < 3) blk.a = __ldg(absmax);
}

struct Levels { float m0, m1, m2, m3; };

// ---- cores: one 64-element block -> 32 words of bf16 pairs (element 2i in the low half of o[i]) --------
// 1 bit.  L, H = bf16(level0 * absmax), bf16(level1 * absmax) as 16-bit patterns; BB = min(L,H) in both
// halves, d = |H - L|, f = 0x10001 if L > H else 0.  A half takes min + d exactly when its (possibly
// flipped) code bit is set, so one multiply-add forms two elements without any carry between halves.
// 16 code bits h are spread once (z = h | h << 15) so that pair j sits at bits 0 and 16 of z >> 2j.
__device__ __forceinline__ void deq64_1bit(uint32_t w0, uint32_t w1, float m0, float m1, float a, uint32_t (&o)[32]) {
    const uint32_t LH = pack_bf16x2(__fmul_rn(m0, a), __fmul_rn(m1, a));
    const uint32_t L = LH & 0xFFFFu, H = LH >> 16;
    const uint32_t lo = min(L, H);
    const uint32_t BB = lo * 0x10001u, d = max(L, H) - lo, f = (L > H) ? 0x10001u : 0u;
#pragma unroll
    for (int q = 0; q < 4; ++q) {  // 16 elements per iteration
        const uint32_t w = (q < 2) ? w0 : w1;
        const uint32_t h = (q & 1) ? (w >> 16) : (w & 0xFFFFu);
        const uint32_t z = h | (h << 15);
#pragma unroll
        for (int j = 0; j < 8; ++j) o[8 * q + j] = (((z >> (2 * j)) & 0x10001u) ^ f) * d + BB;
    }
}

// 2 bits: E01 = {level0, level1} * absmax, E23 = {level2, level3} * absmax, bf16x2 each; a byte
// permute picks the two 16-bit entries named by a pair of codes.
__device__ __forceinline__ void deq64_2bit(const uint4& w, const Levels& lv, float a, uint32_t (&o)[32]) {
    const uint32_t E01 = pack_bf16x2(__fmul_rn(lv.m0, a), __fmul_rn(lv.m1, a));
    const uint32_t E23 = pack_bf16x2(__fmul_rn(lv.m2, a), __fmul_rn(lv.m3, a));
#pragma unroll
    for (int q = 0; q < 4; ++q) {  // one 32-bit word = 16 elements
        const uint32_t x = q == 0 ? w.x : q == 1 ? w.y : q == 2 ? w.z : w.w;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const uint32_t y = x >> (4 * j);
            const uint32_t t = (y & 3u) | ((y << 6) & 0x300u);
            o[8 * q + j] = __byte_perm(E01, E23, t * 0x22u + 0x1010u);
        }
    }
}


// 4 bits: the row's 16 fp32 levels sit in shared memory, entry-major: level c of the row at `tab + c * kStride` bytes
// (forward: kStride = 128, the 32 lanes of a warp side by side, so a warp's 32 look-ups fall into 32 different banks
// whatever the codes are; backward: kStride = 64, the 16 rows of an entry side by side, the two lanes of a row read
// the same table: at most two lanes per bank).  Parked there for the whole tile in the forward pass, fetched
// asynchronously two visits ahead in the backward pass.  Every element is one table load, one multiply and half a
// convert - rounded exactly as the decode kernel does.  (Measured instead: the levels scaled and rounded once per
// block into eight registers and picked with byte permutes, seven per element pair, no table in shared memory: the
// visits of warps with 4-bit rows became so long that a 60/35/5 mix ran 14 % slower in the forward pass.)
template <int kStride>
__device__ __forceinline__ void deq64_4bit_direct(const uint4& lo, const uint4& hi, float a, uint32_t tab, uint32_t (&o)[32]) {
    constexpr int kShift = (kStride == 128) ? 7 : 6;     // byte offset of level c = c << kShift
    constexpr uint32_t kMask = 15u << kShift;
#pragma unroll
    for (int q = 0; q < 8; ++q) {  // one 32-bit word = 8 elements
        const uint32_t w = q == 0 ? lo.x : q == 1 ? lo.y : q == 2 ? lo.z : q == 3 ? lo.w
                         : q == 4 ? hi.x : q == 5 ? hi.y : q == 6 ? hi.z : hi.w;
        float f[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const uint32_t off = (4 * j < kShift) ? (w << (kShift - 4 * j)) : (w >> (4 * j - kShift));   // c = (w >> 4j) & 15
            asm volatile("ld.shared.f32 %0, [%1];" : "=f"(f[j]) : "r"(tab + (off & kMask)) : "memory");
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) o[4 * q + j] = pack_bf16x2(__fmul_rn(f[2 * j], a), __fmul_rn(f[2 * j + 1], a));
    }
}

// ---- shared-memory operand (backward): the block is one 128-byte row of the swizzled tile ----------
// Chunk t (elements 8t .. 8t+7) of the row goes to physical 16-byte slot t ^ swz (128B swizzle).
__device__ __forceinline__ void store_row(uint32_t row_addr, int swz, const uint32_t (&o)[32]) {
#pragma unroll
    for (int t = 0; t < 8; ++t)
        ptx::st_shared_v4(row_addr + (uint32_t)((t ^ swz) << 4), make_uint4(o[4 * t], o[4 * t + 1], o[4 * t + 2], o[4 * t + 3]));
}

}  // namespace

// One piece of work of the persistent schedule: a whole tile or, under the stream-K schedule, a slice of the
// contraction of a weight tile.
struct Seg {
    bool is_t;     // a LoRA down-projection tile (operand rows = ranks) rather than a weight tile
    bool part;     // the slice does not start its tile: its fp32 sums go to this cluster's partial-tile slot
    bool pre;      // the slice starts its tile but does not end it: the accumulator is preloaded with the partial
                   // tiles of the clusters that hold the rest
    int prob;      // which weight of the batch
    int rt, mt;    // row tile, token tile
    int kb0, kb1;  // contraction blocks [kb0, kb1) of the tile
    int tile;      // weight tile index (stream-K)
};

// WIDE: the weight has no 4-bit rows, so nobody needs the level tables and their 16 KB hold a sixth weight slot.
// NB: members the kernel's parameters have room for (1: the plain calls; kMaxBatch: the batch calls).
template <int MODE, bool WIDE, int NB>
__global__ void __launch_bounds__(kGemmThreads, 1)
fused_kernel(const __grid_constant__ KParams<NB> P, const __grid_constant__ KMaps<NB> TM) {
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    unsigned char* base = smem_raw;                   // operand ring (the swizzled tiles need 1024-byte alignment)
    unsigned char* out_s = base + kSmemRingMax;       // epilogue staging
    Barriers* bars = reinterpret_cast<Barriers*>(out_s + kSmemOut);
    volatile uint32_t* abort_flag = &bars->abort;
    const uint64_t wait_ns = P.wait_ns;                // limit of every wait below (lowra_set_wait_limit; 1 s by default)
    if ((ptx::smem_u32(smem_raw) & 1023u) != 0u) {    // never seen; without it the operand descriptors would be wrong
        if (threadIdx.x == 0) atomicExch(P.status, (uint32_t)LOWRA_ERR_CUDA);
        return;
    }

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // Backward: the CTAs of a cluster work on the same weight rows and on neighbouring token tiles, in lock step:
    // every dequantised weight tile is produced once per cluster and written into the shared memory of all its CTAs.
    constexpr int CL = (MODE == kModeDense) ? 1 : kCluster;
    const uint32_t crank = (CL > 1) ? ptx::cluster_ctarank() : 0u;
    // ring geometry: SA weight-operand slots of 16 KB, then SB token-operand slots of 32 KB
    constexpr int SA = (MODE == kModeDense) ? kStages : ((MODE == kModeForward) ? kStagesA_fwd : kStagesA_bwd) + (WIDE ? 1 : 0);
    constexpr int SB = (MODE == kModeDense) ? kStages : (MODE == kModeForward) ? kStagesB_fwd : kStagesB_bwd;
    unsigned char* tab_all = base + SA * kSmemA + SB * kSmemB;   // level tables of 4-bit rows, 2 KB per dequant warp
    auto a_slot = [&](uint32_t it) { return base + (it % SA) * kSmemA; };
    auto b_slot = [&](uint32_t it) { return base + SA * kSmemA + (it % SB) * kSmemB; };
    const int cid = (int)blockIdx.x / CL, NC = (int)gridDim.x / CL;   // this cluster, clusters in the grid
    const int super_t = P.super_total;                      // groups of CL token tiles, all members one after the other
    const int n_t_tiles = (MODE != kModeDense && P.lora_blocks > 0) ? super_t : 0;   // all members' T tiles come first
    const int n_tiles = n_t_tiles + P.tiles_r * super_t;    // per cluster
    // token-tile group gst of the call -> member and group inside the member
    auto member_of = [&](int gst, int& prob, int& st) {
        prob = 0;
        if (NB > 1) {
#pragma unroll
            for (int i = 1; i < NB; ++i)
                if (i < P.count && gst >= P.mem[i].st0) prob = i;
        }
        st = gst - P.mem[prob].st0;
    };
    const int B = P.main_blocks + P.lora_blocks;            // contraction blocks of a weight tile
    // Schedule.  The pieces of work are numbered g = 0, 1, ...: first the T tiles, then the weight tiles; cluster c
    // takes g = c, c + NC, c + 2 NC, ... ("rows" of NC pieces; the clusters then sweep the contraction in step and
    // share the token operand in time).  Whole tiles only: all rows, the last one partly empty.  Stream-K (tile
    // count not a multiple of NC): only the first sk_dp rows; the contraction blocks of the remaining weight tiles,
    // laid end to end, are cut into NC equal consecutive ranges, so a range starts and ends anywhere inside a tile.
    // A slice that does not start its tile leaves its fp32 sums in the cluster's partial-tile slot; the cluster
    // whose range starts the tile collects them: written into its accumulator before its MMAs begin (sk_late == 0:
    // hidden behind the whole tiles in between, which needs long ranges) or added in its epilogue (sk_late == 1).
    const bool sk = MODE != kModeDense && P.sk != 0;
    const int w_dp = sk ? P.sk_dp : 0;                      // rows of whole pieces before the ranges
    const int sk_first = w_dp * NC - n_t_tiles;             // first weight tile of the stream-K part
    auto sk_lo = [&](int c) -> long long { return ((long long)c * P.sk_total) / NC; };
    const long long lo = sk ? sk_lo(cid) : 0, hi = sk ? sk_lo(cid + 1) : 0;
    const int tile0 = sk ? (int)(lo / B) : 0;
    const int n_wsegs = (sk && hi > lo) ? (int)((hi - (long long)tile0 * B + B - 1) / B) : 0;
    const int n_segs = sk ? w_dp + n_wsegs : (n_tiles > cid ? (n_tiles - cid + NC - 1) / NC : 0);
    auto seg_at = [&](int i) {
        Seg t;
        t.part = t.pre = false;
        t.tile = 0;
        t.prob = 0;
        if (!sk || i < w_dp) {
            const int g = cid + i * NC;
            int st;
            if (g < n_t_tiles) {
                member_of(g, t.prob, st);
                t.is_t = true; t.rt = 0; t.mt = st * CL + (int)crank; t.kb0 = 0; t.kb1 = P.main_blocks;
            } else {
                const int idx = g - n_t_tiles;
                const int gst = idx / P.tiles_r;
                member_of(gst, t.prob, st);
                t.is_t = false; t.rt = idx - gst * P.tiles_r; t.mt = st * CL + (int)crank; t.kb0 = 0; t.kb1 = B;
            }
        } else {
            const int k = i - w_dp;
            t.tile = tile0 + k;                             // counted from the first tile of the stream-K part
            const long long first = (long long)t.tile * B;
            t.kb0 = (k == 0) ? (int)(lo - first) : 0;
            t.kb1 = (hi < first + B) ? (int)(hi - first) : B;
            const int idx = sk_first + t.tile;
            const int gst = idx / P.tiles_r;
            int st;
            member_of(gst, t.prob, st);
            t.is_t = false; t.rt = idx - gst * P.tiles_r; t.mt = st * CL + (int)crank;
            t.part = t.kb0 > 0;
            t.pre = t.kb0 == 0 && t.kb1 < B;
        }
        return t;
    };
    // the clusters cid + 1 .. c_end - 1 hold the rest of the tile that this cluster's range starts
    auto contributors_end = [&](int tile) {
        const long long tile_end = (long long)(tile + 1) * B;
        int c_end = cid + 1;
        while (c_end < NC && sk_lo(c_end) < tile_end) ++c_end;
        return c_end;
    };

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            ptx::mbar_init(&bars->full_x[s], 1);
            ptx::mbar_init(&bars->empty[s], 1);
        }
        for (int s = 0; s < kMaxStagesA; ++s) ptx::mbar_init(&bars->full_w[s], kStageArrivals);
        for (int a = 0; a < 2; ++a) {
            ptx::mbar_init(&bars->tmem_full[a], 1);
            ptx::mbar_init(&bars->tmem_empty[a], 4);
        }
        ptx::mbar_init(&bars->drain, 1);
        ptx::mbar_init(&bars->part_full, 1);
        bars->abort = 0u;
        for (int c = 0; c < kCluster; ++c) bars->free_upto[c] = 0u;
        for (int c = 0; c < kMaxStagesA; ++c) bars->produced[c] = 0u;
        ptx::fence_barrier_init();
        ptx::prefetch_tensormap(&TM.m[0].tmB);
        if (P.lora_blocks > 0) { ptx::prefetch_tensormap(&TM.m[0].tmT); ptx::prefetch_tensormap(&TM.m[0].tmFt); }
        if (P.lora_blocks > 0 || MODE == kModeDense) ptx::prefetch_tensormap(&TM.m[0].tmFl);
    }
    if (warp == 1) ptx::tmem_alloc(&bars->tmem_base, kTmemCols);
    ptx::tc_fence_before();
    __syncthreads();
    if (CL > 1) ptx::cluster_sync();   // the peers' barriers and counters exist before anybody touches them
    ptx::tc_fence_after();
    // Everything above overlapped the prologue kernel (programmatic dependent launch); what follows reads what
    // that kernel wrote (row deal, cleared flags and status word).
    if (MODE != kModeDense) pdl_enter();
    const uint32_t tmem_base = bars->tmem_base;
    // This call's number on the workspace: the value that means "up" in the flags (T ready, partial tile ready).
    uint32_t want = 1u;
    if (MODE != kModeDense) {
        want = *reinterpret_cast<const volatile uint32_t*>(P.epoch) + 1u;
        if (want == 0u) want = 1u;   // only on a workspace that was never initialised (its flags are cleared per call)
    }

    bool failed = false;

    if (warp == 0) {
        // ================================================================== TMA producer
        if (lane == 0) {
            uint32_t it = 0;
            for (int i = 0; i < n_segs && !failed; ++i) {
                const Seg t = seg_at(i);
                const int r0 = t.rt * kTileR, m0 = t.mt * kTileT;
                const MemberMaps& tm = TM.m[t.prob];
                for (int kb = t.kb0; kb < t.kb1; ++kb, ++it) {
                    const int s = it % SB;
                    const uint32_t ph = (it / SB) & 1u;
                    if (!ptx::mbar_wait(&bars->empty[s], ph ^ 1u, abort_flag, wait_ns)) { failed = true; bars->abort = 1u; break; }
                    if (MODE != kModeDense) {   // tell the dequant warps of every CTA of the cluster
#pragma unroll
                        for (int c = 0; c < CL; ++c)
                            ptx::st_relaxed_cluster(ptx::map_to_cta(ptx::smem_u32(&bars->free_upto[crank]), (uint32_t)c), it + 1u);
                    }
                    unsigned char* a_s = a_slot(it);   // free as well: its last readers were the MMAs of stage it - SA
                    unsigned char* b_s = b_slot(it);
                    uint64_t* bar = &bars->full_x[s];
                    if (t.is_t) {
                        const int c0 = kb * kTileC;
                        if (MODE == kModeForward) {   // ranks x features from A [K, r]: one 64x64 box per 64 ranks
                            ptx::mbar_arrive_expect_tx(bar, (uint32_t)P.lora_blocks * 8192u + kSmemB);
                            for (int jb = 0; jb < P.lora_blocks; ++jb) ptx::tma_load_2d(a_s + jb * 8192, &tm.tmFt, jb * 64, c0, bar);
                        } else {                      // ranks x channels from B [r, N]: one 64 x 128 box
                            ptx::mbar_arrive_expect_tx(bar, kSmemA + kSmemB);
                            ptx::tma_load_2d(a_s, &tm.tmFt, c0, 0, bar);
                        }
                        ptx::tma_load_2d(b_s, &tm.tmB, c0, m0, bar);
                    } else if (kb < P.main_blocks) {
                        const int c0 = kb * kTileC;
                        if (MODE == kModeDense) {
                            ptx::mbar_arrive_expect_tx(bar, kSmemA + kSmemB);
                            ptx::tma_load_2d(a_s, &tm.tmFl, c0, r0, bar);
                        } else {
                            ptx::mbar_arrive_expect_tx(bar, kSmemB);
                        }
                        ptx::tma_load_2d(b_s, &tm.tmB, c0, m0, bar);
                    } else {
                        const int lb = kb - P.main_blocks;
                        if (lb == 0 || kb == t.kb0) {
                            // T of this token tile is written by another CTA: wait for its flag, then make
                            // those generic-proxy writes visible to the TMA (async proxy) reads below
                            if (!ptx::flag_wait(P.mem[t.prob].flags + t.mt, want, abort_flag, wait_ns)) { failed = true; bars->abort = 1u; break; }
                            ptx::fence_proxy_async_all();
                        }
                        ptx::mbar_arrive_expect_tx(bar, kSmemA + kSmemB);
                        if (MODE == kModeForward) {   // channels x ranks from B [r, N]: two 64-channel boxes; the dequant
                                                      // warps move the rows into tensor memory in their own row order
                            ptx::tma_load_2d(a_s, &tm.tmFl, r0, lb * 64, bar);
                            ptx::tma_load_2d(a_s + 8192, &tm.tmFl, r0 + 64, lb * 64, bar);
                        } else {                      // features x ranks from A [K, r], K-major: one 64 x 128 box
                            ptx::tma_load_2d(a_s, &tm.tmFl, lb * 64, r0, bar);
                        }
                        ptx::tma_load_2d(b_s, &tm.tmT, lb * 64, m0, bar);
                    }
                }
            }
            if (failed) {
                // let this thread's own copies land before the CTA's shared memory is released
                for (uint32_t back = 1; back <= (uint32_t)SB && back <= it; ++back) {
                    const uint32_t j = it - back;
                    ptx::mbar_wait(&bars->full_x[j % SB], (j / SB) & 1u, nullptr, 2000000ull);
                }
            }
        }
    } else if (warp == 1) {
        // ================================================================== MMA issuer
        if (lane == 0) {
            uint32_t it = 0, tile_iter = 0;
            // A barrier probe takes about a hundred cycles to answer, ready or not, and this thread is the
            // pacemaker of the whole CTA: the two barriers of stage it + 1 are probed (non-blocking) before the
            // MMAs of stage it are issued, so the answers are back by the time they are needed.
            bool ready_x = false, ready_w = false;
            // slots and phases of the two rings, carried along (no division by the ring depths in this loop: the
            // thread's instructions are one dependent chain)
            uint32_t sb = 0, phb = 0, sa = 0, pha = 0;
            for (int i = 0; i < n_segs && !failed; ++i, ++tile_iter) {
                const Seg t = seg_at(i);
                const uint32_t acc = tile_iter & 1u;            // two accumulators take turns
                const uint32_t aph = (tile_iter >> 1) & 1u;
                // the epilogue warps hand the accumulator over, every time (empty, or preloaded with partial sums)
                if (!ptx::mbar_wait(&bars->tmem_empty[acc], aph, abort_flag, wait_ns)) { failed = true; bars->abort = 1u; break; }
                ptx::tc_fence_after();
                const uint32_t d_tmem = tmem_base + acc * kTileT;
                const int kb_fresh = (t.pre && !P.sk_late) ? -1 : t.kb0;   // the block whose first MMA overwrites the accumulator
                for (int kb = t.kb0; kb < t.kb1; ++kb, ++it) {
                    const int s = (int)sb;                      // token slot
                    const uint32_t ph = phb;
                    const int sw = (int)sa;                     // weight slot
                    const uint32_t phw = pha;
                    if (!ready_x)
                        if (!ptx::mbar_wait(&bars->full_x[s], ph, abort_flag, wait_ns)) { failed = true; bars->abort = 1u; break; }
                    if (MODE != kModeDense && !ready_w)
                        if (!ptx::mbar_wait(&bars->full_w[sw], phw, abort_flag, wait_ns)) { failed = true; bars->abort = 1u; break; }
                    ptx::tc_fence_after();
                    // probe the next stage now (its slots depend on the running stage index only)
                    const uint32_t a_addr = ptx::smem_u32(base + sa * kSmemA);
                    const uint64_t bdesc = ptx::umma_desc_k_sw128(ptx::smem_u32(base + SA * kSmemA + sb * kSmemB));
                    if (++sb == (uint32_t)SB) { sb = 0; phb ^= 1u; }
                    if (++sa == (uint32_t)SA) { sa = 0; pha ^= 1u; }
                    ready_x = ptx::mbar_test_wait(&bars->full_x[sb], phb);
                    ready_w = (MODE == kModeDense) || ptx::mbar_test_wait(&bars->full_w[sa], pha);
                    // which weight-operand tiles are MN-major (a contraction index is a 128-byte row of 64 operand
                    // rows): forward - the factor tiles, fetched from A [K, r] (T tiles) and B [r, N] (LoRA blocks);
                    // backward - the dequantised weight tile
                    const bool lora_blk = !t.is_t && kb >= P.main_blocks;
                    const bool a_mn = (MODE == kModeForward) ? (t.is_t || lora_blk) : (MODE == kModeBackward && !t.is_t && !lora_blk);
                    if (a_mn) {
                        // 16 contraction rows = two 1024-byte groups per MMA
                        const uint64_t adesc = ptx::umma_desc_mn_sw128(a_addr, 8192u);
#pragma unroll
                        for (int kk = 0; kk < kTileC / 16; ++kk)
                            ptx::umma_bf16(d_tmem, adesc + 128u * kk, bdesc + 2u * kk, kIdescAmn, (kb != kb_fresh || kk != 0) ? 1u : 0u);
                    } else {
                        const uint64_t adesc = ptx::umma_desc_k_sw128(a_addr);
#pragma unroll
                        for (int kk = 0; kk < kTileC / 16; ++kk)  // 16 elements = 32 bytes along K per MMA
                            ptx::umma_bf16(d_tmem, adesc + 2u * kk, bdesc + 2u * kk, kIdesc, (kb != kb_fresh || kk != 0) ? 1u : 0u);
                    }
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
        uint16_t* stage16 = reinterpret_cast<uint16_t*>(out_s) + (warp - kFirstEpilogueWarp) * (kEpilogueTokens * 32);   // this warp's staging
        const int my_row = q * 32 + lane;
        // The four epilogue warps share named barriers, so they must leave together: one thread reads the abort
        // flag (any role may raise it at any time), the others take its answer after the barrier.  Two slots in
        // turn, so that the next question cannot overwrite an answer that a slow warp has not read yet.
        uint32_t agree_turn = 0;
        auto agree_abort = [&]() -> bool {
            if (et == 0) bars->epi_leave[agree_turn & 1u] = *abort_flag;
            ptx::named_barrier_sync(1, 128);
            const bool leave = *reinterpret_cast<volatile uint32_t*>(&bars->epi_leave[agree_turn & 1u]) != 0u;
            ++agree_turn;
            return leave;
        };
        // Hand the accumulator of piece i to the MMA warp (four arrivals, one per warp).  A piece that starts a tile
        // whose later blocks belong to other clusters first gets their partial sums written into the accumulator;
        // the MMAs then add on top.  `wait` false: look at the partial tiles' flags once and come back later if one
        // is missing (returns false); true: wait for them (bounded).
        auto hand_over = [&](int i, bool wait) -> bool {
            if (i >= n_segs) return true;
            const Seg t = seg_at(i);
            const uint32_t acc = (uint32_t)i & 1u;
            if (t.pre && !P.sk_late) {
                const int c_end = contributors_end(t.tile);
                for (int c = cid + 1; c < c_end; ++c) {
                    uint32_t ok = 1u;
                    if (lane == 0) {
                        if (wait) {
                            if (!ptx::flag_wait(P.sk_flags + c * CL + (int)crank, want, abort_flag, wait_ns)) { bars->abort = 1u; ok = 2u; }
                        } else {
                            ok = ptx::flag_test(P.sk_flags + c * CL + (int)crank, want) ? 1u : 0u;
                        }
                    }
                    ok = __shfl_sync(0xffffffffu, ok, 0);
                    if (ok == 0u) return false;
                    if (ok == 2u) return true;                        // timed out: the abort flag ends the loop below
                    (void)ptx::flag_test(P.sk_flags + c * CL + (int)crank, want);   // every lane's own acquire before its loads
                }
                const int m0 = t.mt * kTileT;
#pragma unroll 1
                for (int chunk = 0; chunk < kTileT / 32; ++chunk) {
                    if (m0 + chunk * 32 >= P.mem[t.prob].M) break;
                    float sum[32];
#pragma unroll
                    for (int j = 0; j < 32; ++j) sum[j] = 0.0f;
                    for (int c = cid + 1; c < c_end; ++c) {
                        const float* src = P.sk_part + ((size_t)c * CL + crank) * ((size_t)kTileT * kTileR) +
                                           (size_t)(chunk * 32) * kTileR + my_row;
#pragma unroll
                        for (int j = 0; j < 32; ++j) sum[j] += __ldcg(src + j * kTileR);
                    }
                    uint32_t v[32];
#pragma unroll
                    for (int j = 0; j < 32; ++j) v[j] = __float_as_uint(sum[j]);
                    ptx::tmem_st_32x32(tmem_base + ((uint32_t)(q * 32) << 16) + acc * kTileT + chunk * 32, v);
                }
                ptx::tmem_st_wait();
            }
            ptx::tc_fence_before();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(&bars->tmem_empty[acc]);
            return true;
        };
        // bit a: accumulator a not handed over yet (its partial tiles were not there at the first look)
        uint32_t owed = (hand_over(0, false) ? 0u : 1u) | (hand_over(1, false) ? 0u : 2u);
        uint32_t tile_iter = 0;
        for (int i = 0; i < n_segs && !failed; ++i, ++tile_iter) {
            const Seg t = seg_at(i);
            const int r0 = t.rt * kTileR, m0 = t.mt * kTileT;
            // a T tile writes the down-projected activations [M, rp] (scaled by s); a weight tile writes Y / dX
            uint16_t* out = t.is_t ? P.mem[t.prob].T : P.mem[t.prob].out;
            const int ld = t.is_t ? P.rp : P.ld_out;
            const int R = t.is_t ? P.rp : P.R;
            const float scale = t.is_t ? P.s : 1.0f;
            const bool vec_ok = (ld % 8) == 0;
            const uint32_t acc = tile_iter & 1u;
            const uint32_t aph = (tile_iter >> 1) & 1u;
            // everything before this piece is drained, so nobody waits for this warp: now the wait may block
            if (owed & (1u << acc)) { hand_over(i, true); owed &= ~(1u << acc); }
            // the four epilogue warps share named barriers, so they must agree on leaving
            if (!ptx::mbar_wait_warp(&bars->tmem_full[acc], aph, abort_flag, wait_ns)) bars->abort = 1u;
            if (agree_abort()) { failed = true; break; }
            ptx::tc_fence_after();
            float* part = P.sk_part + ((size_t)cid * CL + crank) * ((size_t)kTileT * kTileR) + my_row;
            // A piece that starts a tile which other clusters finish (sk_late): their partial tiles are added here.
            // The piece is this cluster's last one and its MMAs are complete, so the operand ring is idle: every
            // partial tile (128 KB, [token][row] fp32) is copied into it in one go and read from there.
            const float* add = nullptr;
            if (t.pre && P.sk_late) {
                const int c_end = contributors_end(t.tile);
                const float* ring = reinterpret_cast<const float*>(base) + my_row;
                bool leave = false;
                for (int c = cid + 1; c < c_end; ++c) {
                    if (lane == 0 && !ptx::flag_wait(P.sk_flags + c * CL + (int)crank, want, abort_flag, wait_ns)) bars->abort = 1u;
                    leave = agree_abort();             // also: everybody is done with the previous partial tile in the ring
                    if (leave) break;
                    if (et == 0) {
                        constexpr uint32_t kBytes = (uint32_t)(kTileT * kTileR * 4), kPiece = 16384u;
                        const unsigned char* src = reinterpret_cast<const unsigned char*>(
                            P.sk_part + ((size_t)c * CL + crank) * ((size_t)kTileT * kTileR));
                        // the slices were written with ordinary stores by other SMs and acquired through the flag by
                        // this very thread: make them visible to the copy engine (async proxy) as well
                        ptx::fence_proxy_async_all();
                        ptx::mbar_arrive_expect_tx(&bars->part_full, kBytes);
                        for (uint32_t off = 0; off < kBytes; off += kPiece)
                            ptx::bulk_copy_g2s(ptx::smem_u32(base) + off, src + off, kPiece, &bars->part_full);
                    }
                    if (!ptx::mbar_wait_warp(&bars->part_full, (uint32_t)(c - cid - 1) & 1u, abort_flag, wait_ns)) bars->abort = 1u;
                    leave = agree_abort();
                    if (leave) break;
                    if (c + 1 == c_end) { add = ring; break; }          // the last one is added on the way out, below
#pragma unroll 1
                    for (int chunk = 0; chunk < kTileT / 32; ++chunk) {   // the others go into the accumulator
                        if (m0 + chunk * 32 >= P.mem[t.prob].M) break;
                        uint32_t v[32];
                        const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + acc * kTileT + chunk * 32;
                        ptx::tmem_ld_32x32(taddr, v);
                        ptx::tmem_ld_wait();
#pragma unroll
                        for (int j = 0; j < 32; ++j) v[j] = __float_as_uint(__uint_as_float(v[j]) + ring[(chunk * 32 + j) * kTileR]);
                        ptx::tmem_st_32x32(taddr, v);
                    }
                    ptx::tmem_st_wait();
                }
                if (leave) { failed = true; break; }
            }
#pragma unroll 1
            for (int chunk = 0; chunk < kTileT / 32; ++chunk) {
                if (m0 + chunk * 32 >= P.mem[t.prob].M) break;
                uint32_t v[32];
                ptx::tmem_ld_32x32(tmem_base + ((uint32_t)(q * 32) << 16) + acc * kTileT + chunk * 32, v);
                ptx::tmem_ld_wait();
                if (add != nullptr) {
#pragma unroll
                    for (int j = 0; j < 32; ++j) v[j] = __float_as_uint(__uint_as_float(v[j]) + add[(chunk * 32 + j) * kTileR]);
                }
                if (t.part) {
                    // fp32 sums of a slice: [token][row], so that a warp writes 128 consecutive bytes
#pragma unroll
                    for (int j = 0; j < 32; ++j) __stcg(part + (size_t)(chunk * 32 + j) * kTileR, __uint_as_float(v[j]));
                    continue;
                }
                // thread = operand row (channel), v[j] = token j: transposed through the warp's own 512 bytes of shared
                // memory, eight tokens at a time (8 tokens x 32 channels; every lane then stores one 16-byte piece of a
                // token's 64 bytes) - no barrier between the warps
#pragma unroll
                for (int rnd = 0; rnd < 32 / kEpilogueTokens; ++rnd) {
#pragma unroll
                    for (int j = 0; j < kEpilogueTokens; ++j) {
                        const uint32_t two = pack_bf16x2(scale * __uint_as_float(v[rnd * kEpilogueTokens + j]), 0.0f);
                        stage16[j * 32 + lane] = (uint16_t)two;
                    }
                    __syncwarp();
                    {
                        const int tok = lane >> 2, piece = lane & 3;
                        const int m = m0 + chunk * 32 + rnd * kEpilogueTokens + tok, n = r0 + q * 32 + piece * 8;
                        if (m < P.mem[t.prob].M && n < R) {
                            const uint4 val = *reinterpret_cast<const uint4*>(stage16 + tok * 32 + piece * 8);
                            uint16_t* dst = out + (size_t)m * ld + n;
                            if (vec_ok && n + 8 <= R) {
                                *reinterpret_cast<uint4*>(dst) = val;
                            } else {
                                const uint16_t* e = reinterpret_cast<const uint16_t*>(&val);
                                for (int k = 0; k < 8 && n + k < R; ++k) dst[k] = e[k];
                            }
                        }
                    }
                    __syncwarp();
                }
            }
            // the accumulator goes to the piece after next (preloaded if that one collects partial tiles)
            if (!hand_over(i + 2, false)) owed |= 1u << acc;
            if (t.is_t || t.part) {
                // publish T of this token tile, resp. this cluster's partial tile: every writer fences, then one
                // thread raises the flag
                __threadfence();
                ptx::named_barrier_sync(1, 128);
                if (et == 0) {
                    if (t.is_t) {
                        ptx::fence_proxy_async_all();
                        if (!P.diag_drop_t_flags) ptx::flag_release(P.mem[t.prob].flags + t.mt, want);   // (diagnostic: the waits for T run out)
                    } else {
                        ptx::flag_release(P.sk_flags + cid * CL + (int)crank, want);   // one flag per CTA: its half of the slot
                    }
                }
            }
        }
    } else if (MODE != kModeDense && (warp & 3) != 1) {
        // ================================================================== dequant producers
        // The prologue has dealt the rows to these warps (see gemm_prep.cu).  Each thread dequantises one
        // 64-element absmax block per visit of a stage.
        // Warps 6-8, 10-12, 14, 15: warps 9 and 13 would share the MMA warp's scheduler and idle instead (the MMA
        // warp's instruction latency is what paces the CTA).
        const int pw = (warp - kFirstProducerWarp) - (warp > 9 ? 1 : 0) - (warp > 13 ? 1 : 0);   // 0 .. kProducerWarps - 1
        const uint32_t tab_warp = ptx::smem_u32(tab_all) + (uint32_t)pw * 2048u;   // this warp's 2 KB of level tables (4-bit rows)
        const uint32_t tab_lane = tab_warp + (uint32_t)lane * 4u;                   // forward: level c of this lane's row at tab_lane + 128 c
        uint32_t it0 = 0;                                       // running stage index at the start of the tile
        // Backward: a warp only visits the stages it has work on, so it can be several ring revolutions behind
        // or ahead of a stage's "empty" barrier, where a parity wait says nothing.  The TMA producer visits every
        // stage in order and publishes how many stages it has found free (bars->free_upto); the dequant warps
        // follow that counter instead (lane 0 polls, bounded).
        uint32_t seen_free = 0;
        auto stage_free = [&](uint32_t it) -> bool {
            if (it < seen_free) return true;
            uint32_t v = 0;
            if (lane == 0) {
                uint64_t t_start = 0;
#pragma unroll 1
                for (uint32_t spin = 0;; ++spin) {
                    v = ptx::ld_relaxed_cluster(&bars->free_upto[0]);
#pragma unroll
                    for (int c = 1; c < CL; ++c) v = min(v, ptx::ld_relaxed_cluster(&bars->free_upto[c]));
                    if (v + (uint32_t)(SA - SB) > it) break;
                    if (MODE == kModeForward || spin > 64u) __nanosleep(20);
                    if ((spin & 255u) == 255u) {
                        if (t_start == 0) t_start = ptx::globaltimer_ns();
                        if (*abort_flag != 0u || ptx::globaltimer_ns() - t_start > wait_ns) { v = 0; break; }
                    }
                }
            }
            v = __shfl_sync(0xffffffffu, v, 0);
            if (v + (uint32_t)(SA - SB) <= it) return false;
            seen_free = v + (uint32_t)(SA - SB);
            return true;
        };
        // One lane per visit: `cnt` arrivals on the stage's barrier of this CTA.  The warp that completes the
        // operand tile of the stage (kStageArrivals arrivals in all) hands a copy to every peer CTA of the cluster:
        // one asynchronous 16 KB copy per peer, counted in bytes on the peer's stage barrier, plus the arrivals
        // that barrier expects.
        auto finish_stage = [&](uint32_t it, int s, uint32_t cnt) {
            const bool last = CL > 1 && ptx::atom_add_acq_rel_shared(&bars->produced[s], cnt) + cnt == (uint32_t)kStageArrivals;
            if (last) bars->produced[s] = 0u;   // for the next use of the slot (ordered by the arrival below)
            ptx::mbar_arrive_n(&bars->full_w[s], cnt);
            if (last) {
                ptx::fence_proxy_async_smem();
                const uint32_t tile = ptx::smem_u32(a_slot(it));
                const uint32_t bar = ptx::smem_u32(&bars->full_w[s]);
#pragma unroll
                for (int c = 1; c < CL; ++c) {
                    const uint32_t peer = (crank + (uint32_t)c) % CL;
                    const uint32_t rbar = ptx::map_to_cta(bar, peer);
                    ptx::mbar_expect_tx_cluster(rbar, kSmemA);
                    ptx::bulk_copy_to_cta(ptx::map_to_cta(tile, peer), tile, kSmemA, rbar);
                    ptx::mbar_arrive_cluster(rbar, (uint32_t)kStageArrivals);
                }
            }
        };
        for (int i = 0; i < n_segs && !failed; ++i) {
            const Seg t = seg_at(i);
            const int r0 = t.rt * kTileR;
            const Member& W = P.mem[t.prob];                    // the weight this piece belongs to
            const uint32_t itb = it0 - (uint32_t)t.kb0;         // running stage index of block kb: itb + kb
            const int kb_end = min(t.kb1, P.main_blocks);       // end of this piece's dequantised blocks
            if (t.is_t) {
                // nothing to dequantise (the operand comes by TMA): the warps take the stages in turn and arrive
                // for everybody
                for (int kb = pw; kb < t.kb1; kb += kProducerWarps) {
                    const uint32_t it = itb + (uint32_t)kb;
                    if (!stage_free(it)) { failed = true; bars->abort = 1u; break; }
                    if (lane == 0) ptx::mbar_arrive_n(&bars->full_w[it % SA], kStageArrivals);
                }
            } else if (MODE == kModeForward) {
                // ---------------------------------------------------------------- forward
                // The operand tile of a stage is [128 channels][64 input features], K-major: a channel's
                // 64-element absmax block is one 128-byte row.  The CTAs of the cluster take the stages in turn
                // (stage kb is produced by CTA kb % CL and copied to the peers); inside the CTA the groups
                // of four warps take this CTA's stages in turn, and warp q of a group holds rows 32 q .. 32 q + 31
                // of the tile, roughly in precision order (see the deal in gemm_prep.cu).  A thread keeps its
                // channel for the whole tile; the packed codes of its next two blocks are already in registers.
                const int q = pw & 3, wgrp = pw >> 2;
                const uint32_t item = __ldg(W.items + (size_t)t.rt * kItemStride + q * 32 + lane);
                const int cls = info_class(item);
                const int row_local = info_row(item);
                Levels lv = {0.f, 0.f, 0.f, 0.f};
                const uint8_t* bits_ptr = W.packed;
                const float* absmax_ptr = W.absmax;
                const float* mrow = W.maps;
                int bits_stride = 0;  // packed bytes per 64-element block
                if (cls < 3) {
                    const int p = info_pos(item);
                    const int b = 1 << cls;
                    bits_stride = 8 * b;
                    bits_ptr = W.packed + packed_row_offset(W.L, cls, p, r0 + row_local);
                    absmax_ptr = W.absmax + (size_t)absmax_row_of(W.L, p, r0 + row_local) * W.L.nb;
                    mrow = W.maps + (size_t)(r0 + row_local) * kTableStride;
                    if (cls == 0) {
                        lv.m0 = __ldg(mrow); lv.m1 = __ldg(mrow + 1);
                    } else if (cls == 1) {
                        lv.m0 = __ldg(mrow); lv.m1 = __ldg(mrow + 1); lv.m2 = __ldg(mrow + 2); lv.m3 = __ldg(mrow + 3);
                    } else if (!WIDE) {
                        // the 16 levels of a 4-bit row: parked in shared memory for the whole tile (entry-major: the warp's
                        // 32 tables interleaved word by word; only this lane reads its own)
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const float4 f = __ldg(reinterpret_cast<const float4*>(mrow) + e);
                            ptx::st_shared_f32(tab_lane + 128u * (4 * e), f.x);
                            ptx::st_shared_f32(tab_lane + 128u * (4 * e + 1), f.y);
                            ptx::st_shared_f32(tab_lane + 128u * (4 * e + 2), f.z);
                            ptx::st_shared_f32(tab_lane + 128u * (4 * e + 3), f.w);
                        }
                    }
                }
                constexpr int kStep = CL * (kProducerWarps / 4);     // distance between two stages of this warp
                int kb_first = (int)crank + CL * wgrp;               // this warp's blocks: kb = kb_first (mod kStep)
                if (kb_first < t.kb0) kb_first += (t.kb0 - kb_first + kStep - 1) / kStep * kStep;
                // The block is dequantised into registers BEFORE the wait for the stage (the warps wait most of
                // the time): once the slot is free only the eight 16-byte stores remain on the critical path.
                Block cur, nxt;   // codes of this visit and of the next one
                cur.lo = cur.hi = nxt.lo = nxt.hi = make_uint4(0u, 0u, 0u, 0u);
                cur.a = nxt.a = 0.0f;
                if (cls < 3 && kb_first < kb_end)
                    load_block(cur, bits_ptr + (size_t)kb_first * bits_stride, absmax_ptr + kb_first, cls);
                if (cls < 3 && kb_first + kStep < kb_end)
                    load_block(nxt, bits_ptr + (size_t)(kb_first + kStep) * bits_stride, absmax_ptr + kb_first + kStep, cls);
#pragma unroll 1
                for (int kb = kb_first; kb < kb_end && !failed; kb += kStep) {
                    uint32_t o[32];
                    if (cls == 0) {
                        deq64_1bit(cur.lo.x, cur.lo.y, lv.m0, lv.m1, cur.a, o);
                    } else if (cls == 1) {
                        deq64_2bit(cur.lo, lv, cur.a, o);
                    } else if (!WIDE && cls == 2) {
                        deq64_4bit_direct<128>(cur.lo, cur.hi, cur.a, tab_lane, o);
                    } else {
#pragma unroll
                        for (int i = 0; i < 32; ++i) o[i] = 0u;
                    }
                    cur = nxt;
                    const int nb = kb + 2 * kStep;
                    if (cls < 3 && nb < kb_end)
                        load_block(nxt, bits_ptr + (size_t)nb * bits_stride, absmax_ptr + nb, cls);
                    const uint32_t it = itb + (uint32_t)kb;
                    const int s = it % SA;
                    if (!stage_free(it)) { failed = true; bars->abort = 1u; break; }
                    store_row(ptx::smem_u32(a_slot(it)) + (uint32_t)row_local * 128u, row_local & 7, o);
                    ptx::fence_proxy_async_smem();   // the tensor core and the copy to the peers read the row
                    __syncwarp();
                    if (lane == 0) finish_stage(it, s, kStageArrivals / 4);
                }
                // LoRA blocks: operands come by TMA; the warps take the stages in turn and arrive for everybody
                for (int kb = P.main_blocks + pw; kb < t.kb1 && !failed; kb += kProducerWarps) {
                    if (kb < t.kb0) continue;
                    const uint32_t it = itb + (uint32_t)kb;
                    if (!stage_free(it)) { failed = true; bars->abort = 1u; break; }
                    if (lane == 0) ptx::mbar_arrive_n(&bars->full_w[it % SA], kStageArrivals);
                }
            } else {
                // ---------------------------------------------------------------- backward
                // every stage brings 64 new channels (the contraction index); thread = one channel x 64 of
                // the tile's 128 input features = one absmax block.  Operand tile is MN-major:
                // [feature half][64 channels][64 features], so the block is one 128-byte row.
                // The warp walks its own work list (written by the prologue): entry = (stage, 16 rows of one
                // precision); entries two ahead are already in registers (codes, absmax, levels), in a
                // two-deep ring with static indices so that no load is waited on early.
                const int half = (lane >> 4) & 1;
                const int k_first = r0 + 64 * half;
                const int list = pw * CL + (int)crank;                      // this warp's work list among the cluster's
                // the piece's first group of this CTA, and the warp's first entry at or behind that group's first chunk
                const int g_first = t.kb0 + (((int)crank - t.kb0) % CL + CL) % CL;
                const uint32_t n_first = 4u * (uint32_t)(g_first / CL);
                const uint32_t j_first = n_first > (uint32_t)pw ? (n_first - (uint32_t)pw + kProducerWarps - 1) / kProducerWarps : 0u;
                const uint32_t* heads = W.heads + list + (size_t)j_first * kListWarps;   // entry j of the piece: heads[j * kListWarps]
                const uint4* rows = reinterpret_cast<const uint4*>(W.items) + ((size_t)list + (size_t)j_first * kListWarps) * 32 + lane;
                constexpr uint32_t kEnd = 0xFFFFFFFFu;
                // entry of this visit (0) and of the next one (1): head, row record, codes + absmax, 1/2-bit levels
                uint32_t head0, head1;
                uint4 rec0, rec1;
                Block blk0, blk1;
                Levels lv0 = {0.f, 0.f, 0.f, 0.f}, lv1 = {0.f, 0.f, 0.f, 0.f};
                blk0.lo = blk0.hi = blk1.lo = blk1.hi = make_uint4(0u, 0u, 0u, 0u);
                blk0.a = blk1.a = 0.0f;

                // fetch what an entry needs: codes, absmax, 1/2-bit levels in registers; the 16 fp32 levels of a 4-bit
                // row travel asynchronously into this warp's table cache (two slots of 16 rows x 64 bytes, one per
                // entry in flight; the two lanes of a row read the same 64 bytes)
                auto fetch = [&](Block& blk, Levels& lv, uint32_t head, const uint4& rec, uint32_t tab_slot) {
                    const int cls = (head == kEnd) ? 4 : (int)((rec.w >> 8) & 3u);   // this lane's row
                    if (cls < 3) {
                        load_block(blk, W.packed + ((size_t)rec.x << 4) + (((size_t)k_first << cls) >> 3),
                                   W.absmax + rec.y + (k_first >> 6), cls);
                        const float* mrow = W.maps + rec.z;
                        if (cls == 0) {
                            lv.m0 = __ldg(mrow); lv.m1 = __ldg(mrow + 1);
                        } else if (cls == 1) {
                            lv.m0 = __ldg(mrow); lv.m1 = __ldg(mrow + 1); lv.m2 = __ldg(mrow + 2); lv.m3 = __ldg(mrow + 3);
                        } else if (!WIDE) {
                            // entry-major: level c of row (lane & 15) at tab_slot + 64 c + 4 (lane & 15); the two lanes of
                            // a row fetch eight levels each
                            const uint32_t c0 = (uint32_t)(lane >> 4) * 8u;
#pragma unroll
                            for (uint32_t e = 0; e < 8; ++e)
                                ptx::cp_async_4(tab_slot + 64u * (c0 + e) + 4u * (uint32_t)(lane & 15), mrow + c0 + e);
                        }
                    }
                    ptx::cp_async_commit();   // one group per entry, empty or not
                };

                head0 = __ldg(heads);
                rec0 = __ldg(rows);
                head1 = __ldg(heads + kListWarps);
                rec1 = __ldg(rows + (size_t)kListWarps * 32);
                fetch(blk0, lv0, head0, rec0, tab_warp);
                fetch(blk1, lv1, head1, rec1, tab_warp + 1024u);
#pragma unroll 1
                for (uint32_t j = 0; !failed; ++j) {
                    const uint32_t head = head0;
                    if ((int)(head & 0xFFFFFFu) >= kb_end) break;   // behind the piece (the end markers are all ones)
                    const uint32_t col = rec0.w & 63u;             // channel inside the stage = K index of the tile
                    const int cls = (int)((rec0.w >> 8) & 3u);     // precision class of this lane's row (3: zeros)
                    // head and row record of the entry after next are asked for now and consumed after this visit;
                    // the lists end with kListSlack all-ones heads
                    const uint32_t head2 = __ldg(heads + (size_t)(j + 2) * kListWarps);
                    const uint4 rec2 = __ldg(rows + (size_t)(j + 2) * kListWarps * 32);
                    // the block is dequantised into registers BEFORE the wait for the stage, so that only the eight
                    // 16-byte stores remain once the slot is free (rows of two precisions may meet in the warp)
                    const uint32_t tab_slot = tab_warp + ((j & 1u) << 10);
                    ptx::cp_async_wait<1>();   // this entry's 4-bit tables have landed (the next entry's may still be under way)
                    __syncwarp();
                    uint32_t o[32];
                    if (cls == 0) {
                        deq64_1bit(blk0.lo.x, blk0.lo.y, lv0.m0, lv0.m1, blk0.a, o);
                    } else if (cls == 1) {
                        deq64_2bit(blk0.lo, lv0, blk0.a, o);
                    } else if (!WIDE && cls == 2) {
                        deq64_4bit_direct<64>(blk0.lo, blk0.hi, blk0.a, tab_slot + (lane & 15u) * 4u, o);
                    } else {
#pragma unroll
                        for (int i = 0; i < 32; ++i) o[i] = 0u;
                    }
                    const uint32_t it = itb + (head & 0xFFFFFFu);
                    const int s = it % SA;
                    if (!stage_free(it)) { failed = true; bars->abort = 1u; break; }
                    store_row(ptx::smem_u32(a_slot(it)) + (uint32_t)half * 8192u + col * 128u, (int)(col & 7u), o);
                    ptx::fence_proxy_async_smem();   // the tensor core and the copy to the peers read the row
                    __syncwarp();
                    if (lane == 0) finish_stage(it, s, (head >> 24) & 15u);
                    // shift, and fetch the data of the entry after next
                    head0 = head1; rec0 = rec1; blk0 = blk1; lv0 = lv1;
                    head1 = head2; rec1 = rec2;
                    fetch(blk1, lv1, head1, rec1, tab_slot);   // entry j + 2 takes over the table slot of entry j
                }
                // LoRA blocks: operands come by TMA; the warps take the stages in turn and arrive for everybody
                for (int kb = P.main_blocks + pw; kb < t.kb1 && !failed; kb += kProducerWarps) {
                    if (kb < t.kb0) continue;
                    const uint32_t it = itb + (uint32_t)kb;
                    if (!stage_free(it)) { failed = true; bars->abort = 1u; break; }
                    if (lane == 0) ptx::mbar_arrive_n(&bars->full_w[it % SA], kStageArrivals);
                }
            }
            it0 += (uint32_t)(t.kb1 - t.kb0);
        }
    }

    if (failed) {
        atomicExch(P.status, (uint32_t)LOWRA_ERR_TIMEOUT);
        // tell the peers as well, so that the CTAs of the cluster agree below on how they leave
#pragma unroll
        for (int c = 1; c < CL; ++c)
            ptx::st_relaxed_cluster(ptx::map_to_cta(ptx::smem_u32(&bars->abort), (crank + (uint32_t)c) % CL), 1u);
    }
    // ---------------------------------------------------------------------- teardown
    ptx::tc_fence_before();
    __syncthreads();
    if (CL > 1) ptx::cluster_sync();   // no peer writes into this CTA's shared memory (or arrives on its barriers) any more
    if (*abort_flag != 0u) {
        // Somebody gave up (the same answer in every CTA of the cluster: the flag was exchanged before the barrier).
        // Roles that were not waiting on them may have left bulk copies, TMA loads or MMAs in flight; they need
        // microseconds.  Every role has stopped issuing, so a fixed grace period covers them before shared and
        // tensor memory are given back.
        if (threadIdx.x == 0) {
            const uint64_t t0 = ptx::globaltimer_ns();
            while (ptx::globaltimer_ns() - t0 < kGraceNs) __nanosleep(1000);
        }
        __syncthreads();
        if (CL > 1) ptx::cluster_sync();
    }
    if (warp == 1) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc(tmem_base, kTmemCols);
    }
    if (MODE != kModeDense && threadIdx.x == 0) {
        // the last CTA to leave records the call's number; every CTA has read the old one long before.  Just before
        // the numbering wraps around, it clears the flags and starts again from zero.
        __threadfence();
        if (atomicAdd(P.exits, 1u) == gridDim.x - 1u) {
            if (want == 0xFFFFFFFFu) {
                for (int i = 0; i < P.n_flags; ++i) P.flags[i] = 0u;
                want = 0u;
            }
            *P.epoch = want;
            *P.exits = 0u;
        }
    }
}

template <int MODE, bool WIDE, int NB>
static lowra_status launch_mode(const GemmParams& G, const BatchMaps& TM, cudaStream_t stream) {
    constexpr int CL = (MODE == kModeDense) ? 1 : kCluster;
    // per device: the kernel attribute has been set there, and so many clusters (CL = 1: CTAs) can be resident at once
    static std::mutex mutex;
    static bool configured[kMaxDevices] = {false};
    static int max_clusters_of[kMaxDevices] = {0};
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = CL;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    // start while the prologue kernel (the previous launch in the stream) is still running; the kernel waits for
    // it before it reads anything that kernel writes
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.blockDim = dim3(kGemmThreads, 1, 1);
    cfg.dynamicSmemBytes = kGemmSmemBytes;
    cfg.stream = stream;
    cfg.attrs = attr;
    cfg.numAttrs = (MODE == kModeDense) ? 1 : 2;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return LOWRA_ERR_CUDA;
    int max_clusters = 0;
    {
        std::lock_guard<std::mutex> lock(mutex);
        if (!configured[dev]) {
            const int sms = device_sm_count();
            if (sms < CL) return LOWRA_ERR_CUDA;
            if (cudaFuncSetAttribute(fused_kernel<MODE, WIDE, NB>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     (int)kGemmSmemBytes) != cudaSuccess)
                return LOWRA_ERR_CUDA;
            int most = sms / CL;
            if (CL > 1) {
                // the persistent schedule needs every cluster of the grid resident (a tile waits for T of another)
                cfg.gridDim = dim3(sms / CL * CL, 1, 1);
                int n = 0;
                if (cudaOccupancyMaxActiveClusters(&n, fused_kernel<MODE, WIDE, NB>, &cfg) != cudaSuccess || n < 1) return LOWRA_ERR_CUDA;
                if (n < most) most = n;
            }
            max_clusters_of[dev] = most;
            configured[dev] = true;
        }
        max_clusters = max_clusters_of[dev];
    }
    const int super_t = G.super_total;
    const int n_t = (MODE != kModeDense && G.lora_blocks > 0) ? super_t : 0;
    const int n_tiles = G.tiles_r * super_t + n_t;
    const int clusters = n_tiles < max_clusters ? n_tiles : max_clusters;
    cfg.gridDim = dim3((unsigned)(clusters * CL), 1, 1);
    GemmParams Q = G;
    Q.sk = 0;
    if (MODE != kModeDense && G.sk_part != nullptr && clusters == max_clusters && n_t <= clusters && n_tiles % clusters != 0) {
        // stream-K for the last rows of pieces.  The clusters' sweeps over the contraction fall out of step inside
        // the ranges, so the token operand has to stay in L2 there.  If the whole operand does (<= 48 MB) and there
        // are three rows or more, only the first row stays whole and the partial tiles are preloaded - hidden
        // behind the whole tiles of the range.  Otherwise all full rows stay whole, only the last, incomplete row
        // is cut into ranges (little of the operand is live then), and the partial tiles are added in the
        // epilogue.  (Ranges from the start on a 90 MB operand: 6.5 times the DRAM reads, and no gain.)
        const int blocks = G.main_blocks + G.lora_blocks;
        const int rows = n_tiles / clusters;
        const int n_last = n_tiles - rows * clusters;                  // pieces of the last, incomplete row
        const size_t slab = (size_t)CL * kTileT * (size_t)G.C * 2u;    // token operand of one group of token tiles
        const bool operand_fits_l2 = (size_t)G.operand_bytes <= ((size_t)48 << 20);
        int dp = 0, late = 1;
        if (operand_fits_l2 && rows >= 3) {
            dp = 1; late = 0;
        } else if (2 * n_last >= clusters) {
            dp = rows;                    // two or three clusters per tile of the last row
        } else if (rows >= 2 && (size_t)((n_last + clusters) / G.tiles_r + 2) * slab <= ((size_t)40 << 20)) {
            dp = rows - 1;                // few tiles in the last row: every tile would be cut into many slices, each of
                                          // which the collecting cluster adds one after the other; cut the last two rows
        }
        const long long n_rest = (long long)n_tiles - (long long)dp * clusters;       // weight tiles behind the whole rows
        // adding partial tiles in the epilogue costs about as much as 14 blocks (flag, 128 KB copy, one more pass over
        // the accumulator): cutting the last row must save more than that over running it as one more row of whole tiles
        const bool pays = late == 0 || (long long)n_last * blocks / clusters + 14 < blocks;
        if (dp >= 1 && pays && n_rest * blocks >= clusters) {
            Q.sk = 1;
            Q.sk_dp = dp;
            Q.sk_late = late;
            Q.sk_total = n_rest * blocks;
        }
    }
    KParams<NB> QP;
    KMaps<NB> QM;
    static_cast<GemmCommon&>(QP) = static_cast<const GemmCommon&>(Q);
    for (int i = 0; i < NB; ++i) { QP.mem[i] = Q.mem[i]; QM.m[i] = TM.m[i]; }
    if (cudaLaunchKernelEx(&cfg, fused_kernel<MODE, WIDE, NB>, QP, QM) != cudaSuccess) return LOWRA_ERR_CUDA;
    return LOWRA_OK;
}

template <int MODE>
static lowra_status launch_variant(const GemmParams& G, const BatchMaps& TM, cudaStream_t stream) {
    bool wide = MODE != kModeDense;   // no member has 4-bit rows: the table cache becomes a weight slot
    for (int i = 0; i < G.count; ++i) wide = wide && G.mem[i].L.class_start[3] == G.mem[i].L.class_start[2];
    if constexpr (MODE == kModeDense) {
        return launch_mode<kModeDense, false, 1>(G, TM, stream);
    } else {
        if (G.count == 1)
            return wide ? launch_mode<MODE, true, 1>(G, TM, stream) : launch_mode<MODE, false, 1>(G, TM, stream);
        return wide ? launch_mode<MODE, true, kMaxBatch>(G, TM, stream) : launch_mode<MODE, false, kMaxBatch>(G, TM, stream);
    }
}

lowra_status launch_fused(int mode, const GemmParams& G, const BatchMaps& TM, cudaStream_t stream) {
    if (mode == kModeForward) return launch_variant<kModeForward>(G, TM, stream);
    if (mode == kModeBackward) return launch_variant<kModeBackward>(G, TM, stream);
    return launch_variant<kModeDense>(G, TM, stream);
}

}  // namespace lowra
