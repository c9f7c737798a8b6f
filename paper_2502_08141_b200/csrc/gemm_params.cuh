// Launch parameters shared by the prologue kernel, the fused tensor-core kernel and their host code.
#pragma once

#include <cuda.h>

#include "lowra_common.cuh"

namespace lowra {

// ---- prologue ------------------------------------------------------------------------------
constexpr int kPrepThreads = 128;
constexpr int kProducerWarps = 8;             // dequant warps of the main kernel
constexpr int kItemStride = 128;              // forward: entries per group of 128 rows in the deal table
constexpr int kStageArrivals = 8;             // arrivals a weight-slot barrier expects from the dequant warps (backward: four chunks x 2)
constexpr int kCluster = 2;                   // CTAs per cluster; they share every dequantised weight tile
constexpr int kListWarps = kProducerWarps * kCluster;   // backward: work lists (one per dequant warp of the cluster)
constexpr int kListSlack = 4 * kProducerWarps;  // backward: all-ones heads written behind the last entry of a CTA's lists
constexpr int kMaxGroups64 = 8192;            // backward: at most this many groups of 64 output channels (N <= 524288)

struct PrepParams {
    // deal of the rows to the dequant threads of the main kernel.  Row word = row offset inside its group
    // (bits 0-6) | class (bits 7-8, 3 = row past N) | stored position (bits 9-31), all ones for "no row".
    //   forward (group 128): items[g * kItemStride + i] = i-th row of group g in precision order
    //   backward (group 64): per-warp work lists, see deal_backward
    RowLayout L;
    const uint8_t* precs;
    const int32_t* inv_perm;
    uint32_t* items;      // forward: row words; backward: 16-byte row records of the work-list entries
    uint32_t* heads;      // backward: [7 * ceil(N / 64) + kListSlack] work-list heads
    int N, group;
    uint32_t* status;     // device status word, cleared (null: left alone)
    uint32_t* exits;      // the fused kernel's count of CTAs that have left, cleared (null: left alone)
    uint32_t* flags;      // [n_flags] "T of this token tile is ready" flags, cleared
    int n_flags;
    int blocks;
};

lowra_status launch_prep(const PrepParams& P, cudaStream_t stream);

// ---- fused kernel --------------------------------------------------------------------------
constexpr int kTileR = 128;       // rows of the MMA A operand per tile (output channels fwd, input features bwd)
constexpr int kTileT = 256;       // tokens per tile (MMA N)
constexpr int kTileC = 64;        // contraction elements per pipeline stage (= one absmax block, = 128 bytes of bf16)
constexpr int kStages = 4;        // dense diagnostic: four stages of one weight slot + one token slot
// Forward / backward: the dequant warps (and the copies between the CTAs of a cluster) need to run further ahead
// of the tensor core than the TMA loads do, so the ring is split into 16 KB weight slots and 32 KB token slots:
// five + four in both passes, plus 16 KB for the level tables of 4-bit rows (the token slots hide the L2
// latency of the TMA loads; a fifth weight slot was worth +9..13 % in the forward pass; a sixth is worth another
// +3..5 % and takes the place of the table cache in calls on weights without 4-bit rows; reading the tables through
// L1 instead, or keeping the levels in registers, cost more than the sixth slot gives).  A weight slot
// is free once the MMAs of that many stages earlier are complete; the weight ring must not be shallower than the
// token ring (the TMA warp also loads factor tiles into weight slots).
constexpr int kStagesA_fwd = 5, kStagesA_bwd = 5;
constexpr int kStagesB_fwd = 4, kStagesB_bwd = 4;
constexpr int kMaxStagesA = 6;
constexpr int kFirstEpilogueWarp = 2;
constexpr int kFirstProducerWarp = 6;
// 16 warps, of which two idle (the two that would share the MMA warp's scheduler): at most four per scheduler,
// so 128 registers per thread.
constexpr int kGemmWarps = 16;
constexpr int kGemmThreads = 32 * kGemmWarps;
static_assert(kProducerWarps == 8, "the warp map above places eight dequant warps");
constexpr int kTmemCols = 512;    // two 128 x 256 fp32 accumulators

constexpr int kModeForward = 0, kModeBackward = 1, kModeDense = 2;

constexpr int kMaxBatch = 4;      // weights of the same shape that one launch can walk (lowra_lora_*_batch)

// One weight of a call: its quantised state, the deal of its rows, its output, its down-projected activations.
struct Member {
    RowLayout L;
    const uint8_t* packed;
    const float* absmax;
    const float* maps;
    const uint32_t* items;    // from the deal: row words (forward: per tile; backward: per work-list entry)
    const uint32_t* heads;    // from the deal (backward): work-list heads
    uint16_t* out;            // [M, ld_out] bf16
    uint16_t* T;              // [M, rp] bf16: s * X . A (forward) or s * dY . B^T (backward), written by the T tiles
    uint32_t* flags;          // [tiles_t + kCluster] set to the call's number when T of a token tile is complete
    int M;                    // this member's tokens (the batch calls: the same for all; several adapters: a group's)
    int st0;                  // token-tile groups (kCluster tiles each) of the members before this one
};

// Tensor maps of one member: token operand, T, factor of the T tiles, factor of the LoRA blocks.
struct MemberMaps {
    CUtensorMap tmB, tmT, tmFt, tmFl;
};
template <int NB>
struct KMaps {
    MemberMaps m[NB];
};
using BatchMaps = KMaps<kMaxBatch>;

// What a launch needs beside its members.  (The kernel is instantiated for one member and for kMaxBatch members: a
// plain call then carries 0.7 KB of kernel parameters instead of 2.8 KB, which its launch latency shows.)
struct GemmCommon {
    int count;              // members (1 for the plain calls); all of one shape
    uint32_t* flags;        // all flags of the workspace (the members' T flags, then the partial-tile flags)
    uint32_t* status;
    // Calls on one workspace are numbered: `epoch` holds the number of the last call that ran on it, a call's own
    // number is that + 1, and a flag is up when it holds the call's number - so flags left over from earlier calls
    // never need clearing.  The last CTA to leave (counted in `exits`) writes the call's number back.
    uint32_t* epoch;
    uint32_t* exits;
    int n_flags;            // all flags of the workspace (T ready + partial tile ready), for the wrap of the numbering
    float s;
    int rp;                 // LoRA rank rounded up to 64
    int r;                  // LoRA rank
    int M;                  // tokens of the largest member (host: schedule choice)
    int super_total;        // token-tile groups (kCluster tiles each) of all members
    int R;                  // A-operand rows in total: N (forward, dense) or K (backward)
    int C;                  // main contraction length: K (forward, dense) or N (backward)
    int ld_out;             // = R
    int main_blocks;        // ceil(C / 64)
    int lora_blocks;        // rp / 64 (0 in dense mode)
    int tiles_r;            // row tiles of a member (all members have one shape)
    long long operand_bytes;   // token operands of the call, each distinct one counted once (host: schedule choice)
    // stream-K schedule (set by the launcher; sk == 0: whole tiles, dealt round-robin to the clusters)
    float* sk_part;         // fp32 partial tiles, one [kCluster][kTileT][kTileR] slot per cluster
    uint32_t* sk_flags;     // [clusters] raised when a cluster's partial tile is complete
    int sk;
    int sk_dp;              // rows of whole pieces (T tiles, then weight tiles, round-robin) before the ranges
    int sk_late;            // 1: partial tiles are added in the collecting piece's epilogue; 0: preloaded into its accumulator
    long long sk_total;     // contraction blocks of the weight tiles behind the whole rows
    unsigned long long wait_ns;   // limit of every device-side wait (lowra_set_wait_limit)
    int diag_drop_t_flags;  // diagnostic (lowra_diag_drop_t_flags): the T tiles do not raise their flags, so the waits
                            // for them run out and the call ends with LOWRA_ERR_TIMEOUT
};
template <int NB>
struct KParams : GemmCommon {
    Member mem[NB];
};
using GemmParams = KParams<kMaxBatch>;
unsigned long long wait_limit_ns();   // the process-wide limit, 1 s unless lowra_set_wait_limit changed it
constexpr int kMaxClusters = kNumSMs / kCluster;
constexpr size_t kSkSlotFloats = (size_t)kCluster * kTileT * kTileR;

constexpr uint32_t kSmemA = kTileR * kTileC * 2;   // 16 KB
constexpr uint32_t kSmemB = kTileT * kTileC * 2;   // 32 KB
constexpr uint32_t kSmemStage = kSmemA + kSmemB;
constexpr uint32_t kSmemRingMax = 224 * 1024;   // operand ring + table cache
static_assert(kStages * kSmemStage <= kSmemRingMax, "the dense ring fits into the same space");
constexpr int kEpilogueTokens = 8;                           // tokens per transposition round of the epilogue
constexpr uint32_t kSmemOut = kEpilogueTokens * kTileR * 2;  // epilogue staging: 8 tokens x 128 channels bf16
constexpr uint32_t kSmemBarriers = 1024;
constexpr uint32_t kSmemTab = kProducerWarps * 2048;         // fp32 level tables of the dequant warps' 4-bit rows
static_assert(kStagesA_bwd * kSmemA + kStagesB_bwd * kSmemB + kSmemTab <= kSmemRingMax, "the backward ring and its table cache fit");
static_assert(kStagesA_fwd * kSmemA + kStagesB_fwd * kSmemB + kSmemTab <= kSmemRingMax, "the forward ring and its table cache fit");
// no alignment slack: the dynamic shared memory of a kernel without static shared memory starts 1024-byte
// aligned (checked by the kernel, which the swizzled operand tiles need)
constexpr uint32_t kGemmSmemBytes = kSmemRingMax + kSmemOut + kSmemBarriers;
static_assert(kGemmSmemBytes <= 232448, "227 KB of shared memory per CTA");

lowra_status launch_fused(int mode, const GemmParams& G, const BatchMaps& TM, cudaStream_t stream);

// One skinny product D [R, rp] = P . Q (see gemm_grad.cu), written in bf16 as out [R, ld_out] or, transposed,
// as out [n_cols, ld_out].
struct SkinnyArgs {
    uint16_t* out;
    uint32_t* status;
    int R;            // rows of D
    int C;            // length of the contraction
    int rp;           // columns of D (64 or 128)
    int n_cols;       // columns of D that are written (a multiple of 16)
    int ld_out;
    int a_mn, b_mn;   // 1: the row (column) index of P (Q) is the contiguous one in memory
    int transposed;
    float scale;
    unsigned long long wait_ns;   // limit of every device-side wait
};
lowra_status launch_skinny(const CUtensorMap& tmP, const CUtensorMap& tmQ, const SkinnyArgs& a, cudaStream_t stream);

}  // namespace lowra
