// Host side of lowra_lora_forward / lowra_lora_backward_input / lowra_dense_nt: validation, workspace
// carve-up, TMA descriptors, launches.
#include <cudaTypedefs.h>

#include <atomic>
#include <mutex>
#include <string.h>

#include "gemm_params.cuh"
#include "lowra_diag.h"
#include "ptx.cuh"

namespace lowra {

namespace {
constexpr unsigned long long kDefaultWaitNs = 1000ull * 1000ull * 1000ull;   // 1 s per device-side wait
std::atomic<unsigned long long> g_wait_ns{kDefaultWaitNs};
std::atomic<int> g_drop_t_flags{0};   // diagnostic: so many fused calls to come do not publish their "T ready" flags
}  // namespace

unsigned long long wait_limit_ns() { return g_wait_ns.load(std::memory_order_relaxed); }

namespace {

constexpr size_t kStatusBytes = 256;   // status word at byte 0, then the two words that number the calls:
constexpr size_t kEpochOffset = 64;    //   number of the last call that ran on this workspace
constexpr size_t kExitsOffset = 128;   //   CTAs of the running call that have left

size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }

struct Workspace {
    size_t off_T[kMaxBatch];      // per member: its down-projected activations
    int flag0[kMaxBatch];         // per member: index of its first "T ready" flag
    size_t off_flags, off_items, off_meta, off_part, total;
    int rp, n_flags, sk_flag0;
};

bool rank_ok(int r) { return r >= 16 && r <= 128 && r % 16 == 0; }

// Sizes of the row deal (see gemm_prep.cu).  Forward: 128 row words per group of 128 channels; backward: 4 work-list
// entries (a head and 32 row records of 16 bytes each) per group of 64 channels, plus the end markers.
struct DealSizes {
    size_t fwd_bytes, rows_bytes, heads_bytes;
};
DealSizes deal_sizes(int N) {
    const size_t groups_per_cta = ((size_t)(N + 63) / 64 + kCluster - 1) / kCluster;
    const size_t entries = kCluster * (4 * groups_per_cta + kListSlack + kProducerWarps);
    DealSizes d;
    d.fwd_bytes = (size_t)((N + 127) / 128) * kItemStride * 4;
    d.rows_bytes = entries * 32 * 16;
    d.heads_bytes = entries * 4;
    return d;
}
// A deal kept by the caller (lowra_deal_build): forward row words | backward row records | backward heads
struct DealBuffer {
    size_t off_fwd, off_rows, off_heads, total;
};
DealBuffer plan_deal(int N) {
    const DealSizes z = deal_sizes(N);
    DealBuffer d;
    d.off_fwd = 0;
    d.off_rows = align256(z.fwd_bytes);
    d.off_heads = d.off_rows + align256(z.rows_bytes);
    d.total = d.off_heads + align256(z.heads_bytes);
    return d;
}

// Ms: the members' token counts (the plain and the batch calls: all equal).
Workspace plan_workspace(int N, int K, const int* Ms, int count, int r, bool stream_k) {
    (void)K;
    Workspace w;
    memset(&w, 0, sizeof(w));
    w.rp = (r + 63) / 64 * 64;
    const DealSizes z = deal_sizes(N);   // room for the deal of one direction, rebuilt by every call that brings none
    size_t off = kStatusBytes;
    int flags = 0;
    for (int i = 0; i < count; ++i) {
        w.off_T[i] = off;
        off += align256((size_t)Ms[i] * w.rp * 2);
        // the member's "T ready" flags (a cluster's last token tiles may lie past its tokens)
        w.flag0[i] = flags;
        flags += (Ms[i] + kTileT - 1) / kTileT + kCluster;
    }
    w.off_flags = off;
    w.sk_flag0 = flags;                                  // then one "partial tile ready" flag per CTA
    w.n_flags = flags + kMaxClusters * kCluster;
    w.off_items = w.off_flags + align256((size_t)w.n_flags * 4);
    w.off_meta = w.off_items + align256(z.rows_bytes > z.fwd_bytes ? z.rows_bytes : z.fwd_bytes);
    w.off_part = w.off_meta + align256(z.heads_bytes);
    w.total = w.off_part + (stream_k ? align256((size_t)kMaxClusters * kSkSlotFloats * 4) : 0);   // stream-K partial tiles
    return w;
}
Workspace plan_workspace(int N, int K, int M, int r, bool stream_k, int count = 1) {
    int Ms[kMaxBatch];
    for (int i = 0; i < kMaxBatch; ++i) Ms[i] = M;
    return plan_workspace(N, K, Ms, count, r, stream_k);
}

PFN_cuTensorMapEncodeTiled_v12000 encode_fn() {
    static PFN_cuTensorMapEncodeTiled_v12000 fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(p);
    }
    return fn;
}

// bf16 matrix [rows, cols] row-major with pitch `ld` elements; box = 64 columns x box_rows rows,
// 128-byte swizzle, out-of-range elements read as zero.
bool make_map(CUtensorMap* map, const void* ptr, uint64_t rows, uint64_t cols, uint64_t ld, uint32_t box_rows) {
    PFN_cuTensorMapEncodeTiled_v12000 fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {ld * 2};
    cuuint32_t box[2] = {(cuuint32_t)kTileC, box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult rc = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return rc == CUDA_SUCCESS;
}

// One weight of a fused call, as the entry points receive it.
struct MemberArgs {
    const lowra_layout* layout;
    const uint8_t* packed;
    const float* absmax;
    const float* maps;
    const uint16_t* act;   // X (forward) or dY (backward-input)
    const uint16_t* A;
    const uint16_t* B;
    uint16_t* out;
    int32_t M;             // tokens of this member
};

// Forward / backward-input for `count` weights of one shape in one launch (count == 1: the plain calls).  The members
// may have different token counts (several adapters on one weight: one member per token group).
lowra_status run_members(bool backward, const MemberArgs* mem, int count, int32_t r, float s, void* workspace,
                         size_t workspace_bytes, void* stream_v, bool stream_k = true) {
    if (count < 1 || count > kMaxBatch) return LOWRA_ERR_SHAPE;
    for (int i = 0; i < count; ++i) {
        lowra_status st = check_layout(mem[i].layout);
        if (st != LOWRA_OK) return st;
        if (!mem[i].packed || !mem[i].absmax || !mem[i].maps || !mem[i].act || !mem[i].A || !mem[i].B || !mem[i].out) return LOWRA_ERR_NULL;
    }
    if (!workspace) return LOWRA_ERR_NULL;
    const int N = mem[0].layout->N, K = mem[0].layout->K;
    if (!rank_ok(r) || N % 8 != 0 || N > 64 * kMaxGroups64 || (uint64_t)N * (uint64_t)(K / 64) >= (1ull << 32))
        return LOWRA_ERR_SHAPE;
    int Ms[kMaxBatch], M = 0;
    for (int i = 0; i < count; ++i) {
        const MemberArgs& m = mem[i];
        if (m.M < 1) return LOWRA_ERR_SHAPE;
        Ms[i] = m.M;
        M = m.M > M ? m.M : M;
        if (m.layout->N != N || m.layout->K != K) return LOWRA_ERR_SHAPE;                 // one shape per launch
        if (count > 1 && m.layout->deal_dev == nullptr) return LOWRA_ERR_NULL;            // a batch has no prologue launch
        if (!aligned16(m.packed) || !aligned16(m.absmax) || !aligned16(m.maps) || !aligned16(m.act) || !aligned16(m.A) ||
            !aligned16(m.B) || !aligned16(m.out) || (reinterpret_cast<uintptr_t>(m.layout->deal_dev) & 255u) != 0)
            return LOWRA_ERR_ALIGN;
    }
    const Workspace w = plan_workspace(N, K, Ms, count, r, stream_k);
    if (workspace_bytes < w.total || (reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return LOWRA_ERR_WORKSPACE;
    lowra_status st = check_device();
    if (st != LOWRA_OK) return st;
    cudaStream_t stream = (cudaStream_t)stream_v;

    unsigned char* ws = static_cast<unsigned char*>(workspace);
    uint32_t* status = reinterpret_cast<uint32_t*>(ws);
    uint32_t* flags = reinterpret_cast<uint32_t*>(ws + w.off_flags);

    GemmParams G;
    memset(&G, 0, sizeof(G));
    BatchMaps TM;
    memset(&TM, 0, sizeof(TM));
    G.count = count;
    for (int i = 0; i < count; ++i) {
        const MemberArgs& m = mem[i];
        Member& g = G.mem[i];
        g.L = make_row_layout(m.layout);
        g.packed = m.packed;
        g.absmax = m.absmax;
        g.maps = m.maps;
        g.out = m.out;
        g.T = reinterpret_cast<uint16_t*>(ws + w.off_T[i]);
        g.flags = flags + w.flag0[i];
        g.M = m.M;
        g.st0 = G.super_total;
        G.super_total += ((m.M + kTileT - 1) / kTileT + kCluster - 1) / kCluster;
        if (m.layout->deal_dev != nullptr) {
            // the rows were dealt once for this weight (lowra_deal_build) and the workspace numbers its calls
            // (lowra_workspace_init): nothing to prepare, the fused kernel is the only launch
            const DealBuffer d = plan_deal(N);
            const unsigned char* deal = static_cast<const unsigned char*>(m.layout->deal_dev);
            g.items = reinterpret_cast<const uint32_t*>(deal + (backward ? d.off_rows : d.off_fwd));
            g.heads = reinterpret_cast<const uint32_t*>(deal + d.off_heads);
        } else {
            // ---- prologue: clear status and flags, deal the rows (plain calls only)
            uint32_t* items = reinterpret_cast<uint32_t*>(ws + w.off_items);
            uint32_t* heads = reinterpret_cast<uint32_t*>(ws + w.off_meta);
            PrepParams P;
            memset(&P, 0, sizeof(P));
            P.L = g.L;
            P.precs = m.layout->precs_dev;
            P.inv_perm = m.layout->inv_perm_dev;
            P.items = items;
            P.heads = heads;
            P.N = N;
            P.group = backward ? 64 : 128;
            P.status = status;
            P.exits = reinterpret_cast<uint32_t*>(ws + kExitsOffset);
            P.flags = flags;
            P.n_flags = w.n_flags;
            P.blocks = ((N + P.group - 1) / P.group + 3) / 4;
            st = launch_prep(P, stream);
            if (st != LOWRA_OK) return st;
            g.items = items;
            g.heads = heads;
        }
    }

    // ---- fused kernel (its first tiles compute T = s X A, resp. U = s dY B^T, of every member)
    G.flags = flags;
    G.status = status;
    G.epoch = reinterpret_cast<uint32_t*>(ws + kEpochOffset);
    G.exits = reinterpret_cast<uint32_t*>(ws + kExitsOffset);
    G.n_flags = w.n_flags;
    G.s = s;
    G.rp = w.rp;
    G.r = r;
    G.M = M;
    G.R = backward ? K : N;
    G.C = backward ? N : K;
    G.ld_out = G.R;
    G.main_blocks = (G.C + kTileC - 1) / kTileC;
    G.lora_blocks = w.rp / kTileC;
    G.tiles_r = (G.R + kTileR - 1) / kTileR;
    for (int i = 0; i < count; ++i) {   // token operands: every distinct one once (q, k, v share X in the forward pass)
        bool seen = false;
        for (int j = 0; j < i; ++j) seen = seen || mem[j].act == mem[i].act;
        if (!seen) G.operand_bytes += (long long)mem[i].M * G.C * 2;
    }
    G.sk_part = stream_k ? reinterpret_cast<float*>(ws + w.off_part) : nullptr;   // null: whole tiles only
    G.sk_flags = flags + w.sk_flag0;
    G.wait_ns = wait_limit_ns();
    {   // diagnostic, armed by lowra_diag_drop_t_flags: take one of the calls it asked for
        int left = g_drop_t_flags.load(std::memory_order_relaxed);
        while (left > 0 && !g_drop_t_flags.compare_exchange_weak(left, left - 1, std::memory_order_relaxed)) {}
        G.diag_drop_t_flags = left > 0 ? 1 : 0;
    }
    for (int i = 0; i < count; ++i) {
        const MemberArgs& m = mem[i];
        MemberMaps& t = TM.m[i];
        if (!make_map(&t.tmB, m.act, (uint64_t)m.M, (uint64_t)G.C, (uint64_t)G.C, kTileT)) return LOWRA_ERR_CUDA;
        if (!make_map(&t.tmT, G.mem[i].T, (uint64_t)m.M, (uint64_t)w.rp, (uint64_t)w.rp, kTileT)) return LOWRA_ERR_CUDA;
        if (!backward) {
            // T tiles take ranks x features from A [K, r] (64 x 64 boxes); LoRA blocks take channels x ranks from B [r, N]
            if (!make_map(&t.tmFt, m.A, (uint64_t)K, (uint64_t)r, (uint64_t)r, 64)) return LOWRA_ERR_CUDA;
            if (!make_map(&t.tmFl, m.B, (uint64_t)r, (uint64_t)N, (uint64_t)N, 64)) return LOWRA_ERR_CUDA;
        } else {
            // T tiles take ranks x channels from B [r, N]; LoRA blocks take features x ranks from A [K, r] (64 x 128 boxes)
            if (!make_map(&t.tmFt, m.B, (uint64_t)r, (uint64_t)N, (uint64_t)N, kTileR)) return LOWRA_ERR_CUDA;
            if (!make_map(&t.tmFl, m.A, (uint64_t)K, (uint64_t)r, (uint64_t)r, kTileR)) return LOWRA_ERR_CUDA;
        }
    }
    return launch_fused(backward ? kModeBackward : kModeForward, G, TM, stream);
}

lowra_status run_lora(bool backward, const lowra_layout* layout, const uint8_t* packed, const float* absmax,
                      const float* maps, const uint16_t* act, int32_t M, const uint16_t* A, const uint16_t* B,
                      int32_t r, float s, uint16_t* out, void* workspace, size_t workspace_bytes, void* stream_v,
                      bool stream_k = true) {
    const MemberArgs m = {layout, packed, absmax, maps, act, A, B, out, M};
    return run_members(backward, &m, 1, r, s, workspace, workspace_bytes, stream_v, stream_k);
}

// scratch of the adapter-gradient call: status word | T = s X A | U = s dY B^T  (bf16 [M, rp] each)
struct AdapterWorkspace {
    size_t off_T, off_U, total;
    int rp;
};
AdapterWorkspace plan_adapter_workspace(int M, int r) {
    AdapterWorkspace w;
    w.rp = (r + 63) / 64 * 64;
    w.off_T = kStatusBytes;
    w.off_U = w.off_T + align256((size_t)M * w.rp * 2);
    w.total = w.off_U + align256((size_t)M * w.rp * 2);
    return w;
}

__global__ void clear_status_kernel(uint32_t* status) { *status = 0u; }

}  // namespace
}  // namespace lowra

extern "C" size_t lowra_workspace_bytes(const lowra_layout* layout, int32_t M, int32_t r) {
    using namespace lowra;
    if (!layout || layout->N < 1 || layout->K < 1 || M < 1 || !rank_ok(r)) return 0;
    return plan_workspace(layout->N, layout->K, M, r, true).total;
}

extern "C" size_t lowra_deal_bytes(const lowra_layout* layout) {
    using namespace lowra;
    if (!layout || layout->N < 1) return 0;
    return plan_deal(layout->N).total;
}

extern "C" lowra_status lowra_deal_build(const lowra_layout* layout, void* deal_dev, size_t deal_bytes, void* stream) {
    using namespace lowra;
    lowra_status st = check_layout(layout);
    if (st != LOWRA_OK) return st;
    if (!deal_dev) return LOWRA_ERR_NULL;
    const int N = layout->N;
    if (N % 8 != 0 || N > 64 * kMaxGroups64) return LOWRA_ERR_SHAPE;
    if ((reinterpret_cast<uintptr_t>(deal_dev) & 255u) != 0) return LOWRA_ERR_ALIGN;
    const DealBuffer d = plan_deal(N);
    if (deal_bytes < d.total) return LOWRA_ERR_WORKSPACE;
    st = check_device();
    if (st != LOWRA_OK) return st;
    unsigned char* deal = static_cast<unsigned char*>(deal_dev);
    for (int backward = 0; backward < 2; ++backward) {
        PrepParams P;
        memset(&P, 0, sizeof(P));   // no status word, no flags: this launch only deals
        P.L = make_row_layout(layout);
        P.precs = layout->precs_dev;
        P.inv_perm = layout->inv_perm_dev;
        P.items = reinterpret_cast<uint32_t*>(deal + (backward ? d.off_rows : d.off_fwd));
        P.heads = reinterpret_cast<uint32_t*>(deal + d.off_heads);
        P.N = N;
        P.group = backward ? 64 : 128;
        P.blocks = ((N + P.group - 1) / P.group + 3) / 4;
        st = launch_prep(P, (cudaStream_t)stream);
        if (st != LOWRA_OK) return st;
    }
    return LOWRA_OK;
}

extern "C" lowra_status lowra_workspace_init(void* workspace_dev, size_t workspace_bytes, void* stream) {
    if (!workspace_dev) return LOWRA_ERR_NULL;
    if (workspace_bytes < lowra::kStatusBytes || (reinterpret_cast<uintptr_t>(workspace_dev) & 255u) != 0)
        return LOWRA_ERR_WORKSPACE;
    // status word, call numbering and every flag start from zero; the rest of the scratch needs no initial value
    return cudaMemsetAsync(workspace_dev, 0, workspace_bytes, (cudaStream_t)stream) == cudaSuccess ? LOWRA_OK
                                                                                                   : LOWRA_ERR_CUDA;
}

extern "C" lowra_status lowra_lora_forward(const lowra_layout* layout, const uint8_t* packed_dev,
                                           const float* absmax_dev, const float* maps_dev, const uint16_t* X_dev,
                                           int32_t M, const uint16_t* A_dev, const uint16_t* B_dev, int32_t r, float s,
                                           uint16_t* Y_dev, void* workspace_dev, size_t workspace_bytes, void* stream) {
    return lowra::run_lora(false, layout, packed_dev, absmax_dev, maps_dev, X_dev, M, A_dev, B_dev, r, s, Y_dev,
                           workspace_dev, workspace_bytes, stream);
}

extern "C" lowra_status lowra_lora_backward_input(const lowra_layout* layout, const uint8_t* packed_dev,
                                                  const float* absmax_dev, const float* maps_dev,
                                                  const uint16_t* dY_dev, int32_t M, const uint16_t* A_dev,
                                                  const uint16_t* B_dev, int32_t r, float s, uint16_t* dX_dev,
                                                  void* workspace_dev, size_t workspace_bytes, void* stream) {
    return lowra::run_lora(true, layout, packed_dev, absmax_dev, maps_dev, dY_dev, M, A_dev, B_dev, r, s, dX_dev,
                           workspace_dev, workspace_bytes, stream);
}

static_assert(LOWRA_MAX_BATCH == lowra::kMaxBatch, "header and kernel agree on the batch limit");

extern "C" size_t lowra_batch_workspace_bytes(const lowra_layout* layout, int32_t count, int32_t M, int32_t r) {
    using namespace lowra;
    if (!layout || layout->N < 1 || layout->K < 1 || M < 1 || !rank_ok(r) || count < 1 || count > kMaxBatch) return 0;
    return plan_workspace(layout->N, layout->K, M, r, true, count).total;
}

namespace lowra {
namespace {
lowra_status run_batch(bool backward, const lowra_member* members, int32_t count, int32_t M, int32_t r, float s,
                       void* workspace, size_t workspace_bytes, void* stream) {
    if (!members) return LOWRA_ERR_NULL;
    if (count < 1 || count > kMaxBatch) return LOWRA_ERR_SHAPE;
    MemberArgs mem[kMaxBatch];
    for (int i = 0; i < count; ++i) {
        const lowra_member& m = members[i];
        mem[i] = MemberArgs{m.layout, m.packed_dev, m.absmax_dev, m.maps_dev, m.act_dev, m.A_dev, m.B_dev, m.out_dev, M};
        if (m.layout != nullptr && m.layout->deal_dev == nullptr) return LOWRA_ERR_NULL;   // also for a batch of one
    }
    return run_members(backward, mem, count, r, s, workspace, workspace_bytes, stream);
}
}  // namespace
}  // namespace lowra

extern "C" lowra_status lowra_lora_forward_batch(const lowra_member* members_host, int32_t count, int32_t M, int32_t r,
                                                 float s, void* workspace_dev, size_t workspace_bytes, void* stream) {
    return lowra::run_batch(false, members_host, count, M, r, s, workspace_dev, workspace_bytes, stream);
}

extern "C" lowra_status lowra_lora_backward_input_batch(const lowra_member* members_host, int32_t count, int32_t M,
                                                        int32_t r, float s, void* workspace_dev, size_t workspace_bytes,
                                                        void* stream) {
    return lowra::run_batch(true, members_host, count, M, r, s, workspace_dev, workspace_bytes, stream);
}

extern "C" lowra_status lowra_lora_forward_adapters(const lowra_layout* layout, const uint8_t* packed_dev,
                                                    const float* absmax_dev, const float* maps_dev, int32_t n_adapters,
                                                    const uint16_t* X_dev, int32_t M, const int32_t* group_start_host,
                                                    const uint16_t* A_dev, const uint16_t* B_dev, int32_t r, float s,
                                                    uint16_t* Y_dev, void* workspace_dev, size_t workspace_bytes,
                                                    void* stream) {
    using namespace lowra;
    lowra_status st = check_layout(layout);
    if (st != LOWRA_OK) return st;
    if (!maps_dev || !X_dev || !A_dev || !B_dev || !Y_dev || !group_start_host) return LOWRA_ERR_NULL;
    if (n_adapters < 1 || M < 1 || !rank_ok(r) || group_start_host[0] != 0 || group_start_host[n_adapters] != M)
        return LOWRA_ERR_SHAPE;
    for (int a = 0; a < n_adapters; ++a)
        if (group_start_host[a + 1] < group_start_host[a]) return LOWRA_ERR_SHAPE;
    const size_t N = (size_t)layout->N, K = (size_t)layout->K;
    if (workspace_bytes < lowra_workspace_bytes(layout, M, r)) return LOWRA_ERR_WORKSPACE;
    // Up to kMaxBatch token groups go into one launch (one member per group: the same packed weight, the group's
    // mappings, factors and token rows) when the layout carries a deal and the workspace has room for it; otherwise
    // every group is a launch of its own.
    const bool together = layout->deal_dev != nullptr &&
                          workspace_bytes >= plan_workspace(layout->N, layout->K, M, r, true, kMaxBatch).total;
    MemberArgs mem[kMaxBatch];
    int n = 0;
    for (int a = 0; a <= n_adapters; ++a) {
        if (a < n_adapters) {
            const int m0 = group_start_host[a], m = group_start_host[a + 1] - m0;
            if (m == 0) continue;
            mem[n++] = MemberArgs{layout, packed_dev, absmax_dev, maps_dev + (size_t)a * N * kTableStride, X_dev + (size_t)m0 * K,
                                  A_dev + (size_t)a * K * (size_t)r, B_dev + (size_t)a * (size_t)r * N, Y_dev + (size_t)m0 * N, m};
        }
        if (n > 0 && (a == n_adapters || n == (together ? kMaxBatch : 1))) {
            st = run_members(false, mem, n, r, s, workspace_dev, workspace_bytes, stream);
            if (st != LOWRA_OK) return st;
            n = 0;
        }
    }
    return LOWRA_OK;
}

// ---------------------------------------------------------------------------------------------------
// Forward without caller-provided scratch, for callers that may not allocate device memory.
// The scratch is this fixed array: part of the library image, present on every GPU that loads it.
// In host code `g_static_scratch` is only a handle for the symbol, never a device address; the address
// is looked up once per device with cudaGetSymbolAddress and that pointer is what the kernels get.
static __device__ __align__(256) unsigned char g_static_scratch[LOWRA_STATIC_SCRATCH_BYTES];

namespace lowra {
namespace {
std::mutex g_static_mutex;
void* g_static_ptr[kMaxDevices] = {nullptr};

// Device address of the built-in scratch on the current device (looked up on first use).
lowra_status static_scratch(void** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return LOWRA_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_ptr[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) return LOWRA_ERR_CUDA;
        g_static_ptr[dev] = p;
    }
    *out = g_static_ptr[dev];
    return LOWRA_OK;
}
}  // namespace
}  // namespace lowra

extern "C" lowra_status lowra_lora_forward_static(const lowra_layout* layout, const uint8_t* packed_dev,
                                                  const float* absmax_dev, const float* maps_dev,
                                                  const uint16_t* X_dev, int32_t M, const uint16_t* A_dev,
                                                  const uint16_t* B_dev, int32_t r, float s, uint16_t* Y_dev,
                                                  uint32_t* status_out_dev, void* stream) {
    using namespace lowra;
    if (!layout) return LOWRA_ERR_NULL;
    if (layout->N < 1 || layout->K < 1 || M < 1 || !rank_ok(r)) return LOWRA_ERR_SHAPE;
    const size_t need = plan_workspace(layout->N, layout->K, M, r, false).total;   // no room for partial tiles
    if (need > (size_t)LOWRA_STATIC_SCRATCH_BYTES) return LOWRA_ERR_LIMIT;
    lowra_status st = check_device();
    if (st != LOWRA_OK) return st;
    void* scratch = nullptr;
    st = static_scratch(&scratch);
    if (st != LOWRA_OK) return st;
    // The scratch starts zero-filled (a static array) and only these calls write it, so the numbering of the
    // calls holds whether or not the layout brings a deal; without one the prologue kernel rewrites the status
    // word, the flags and the deal on every call.  With one there is no prologue, and nobody could otherwise reset
    // the status word of the built-in array: clear it here, in stream order, so that the word handed back below is
    // this call's own.
    if (layout->deal_dev != nullptr) {
        clear_status_kernel<<<1, 1, 0, (cudaStream_t)stream>>>(static_cast<uint32_t*>(scratch));
        if (cudaGetLastError() != cudaSuccess) return LOWRA_ERR_CUDA;
    }
    st = run_lora(false, layout, packed_dev, absmax_dev, maps_dev, X_dev, M, A_dev, B_dev, r, s, Y_dev, scratch,
                  (size_t)LOWRA_STATIC_SCRATCH_BYTES, stream, false);
    if (st != LOWRA_OK) return st;
    if (status_out_dev &&
        cudaMemcpyAsync(status_out_dev, scratch, sizeof(uint32_t), cudaMemcpyDeviceToDevice, (cudaStream_t)stream) !=
            cudaSuccess)
        return LOWRA_ERR_CUDA;
    return LOWRA_OK;
}

extern "C" size_t lowra_adapter_workspace_bytes(int32_t M, int32_t r) {
    using namespace lowra;
    if (M < 1 || !rank_ok(r)) return 0;
    return plan_adapter_workspace(M, r).total;
}

namespace lowra {
namespace {
// dA = X^T U and dB = (dY^T T)^T, with the down-projections T = s X A and U = s dY B^T either computed here (T_in ==
// nullptr: four skinny products, X and dY read twice) or taken from the caller (two products, X and dY read once).
lowra_status run_adapters(const uint16_t* X_dev, const uint16_t* dY_dev, int32_t M, int32_t K, int32_t N, const uint16_t* A_dev,
                          const uint16_t* B_dev, int32_t r, float s, const uint16_t* T_in, const uint16_t* U_in, uint16_t* dA_dev,
                          uint16_t* dB_dev, void* workspace_dev, size_t workspace_bytes, void* stream_v) {
    const bool reuse = T_in != nullptr;
    if (!X_dev || !dY_dev || !dA_dev || !dB_dev || !workspace_dev) return LOWRA_ERR_NULL;
    if (reuse ? !U_in : (!A_dev || !B_dev)) return LOWRA_ERR_NULL;
    if (M < 1 || K < 8 || N < 8 || K % 8 != 0 || N % 8 != 0 || !rank_ok(r)) return LOWRA_ERR_SHAPE;
    if (!aligned16(X_dev) || !aligned16(dY_dev) || !aligned16(A_dev) || !aligned16(B_dev) || !aligned16(dA_dev) ||
        !aligned16(dB_dev) || !aligned16(T_in) || !aligned16(U_in))
        return LOWRA_ERR_ALIGN;
    const AdapterWorkspace w = plan_adapter_workspace(M, r);
    if (workspace_bytes < (reuse ? kStatusBytes : w.total) || (reinterpret_cast<uintptr_t>(workspace_dev) & 255u) != 0)
        return LOWRA_ERR_WORKSPACE;
    lowra_status st = check_device();
    if (st != LOWRA_OK) return st;
    cudaStream_t stream = (cudaStream_t)stream_v;
    unsigned char* ws = static_cast<unsigned char*>(workspace_dev);
    uint32_t* status = reinterpret_cast<uint32_t*>(ws);
    const uint16_t* T = reuse ? T_in : reinterpret_cast<uint16_t*>(ws + w.off_T);
    const uint16_t* U = reuse ? U_in : reinterpret_cast<uint16_t*>(ws + w.off_U);
    clear_status_kernel<<<1, 1, 0, stream>>>(status);
    const int rp = w.rp;
    CUtensorMap tmX, tmXt, tmdY, tmdYt, tmA, tmB, tmT, tmU;
    if (!make_map(&tmXt, X_dev, (uint64_t)M, (uint64_t)K, (uint64_t)K, 64) ||      // 64 tokens x 64 features (MN-major)
        !make_map(&tmdYt, dY_dev, (uint64_t)M, (uint64_t)N, (uint64_t)N, 64) ||
        !make_map(&tmT, T, (uint64_t)M, (uint64_t)rp, (uint64_t)rp, 64) ||
        !make_map(&tmU, U, (uint64_t)M, (uint64_t)rp, (uint64_t)rp, 64))
        return LOWRA_ERR_CUDA;
    if (!reuse &&
        (!make_map(&tmX, X_dev, (uint64_t)M, (uint64_t)K, (uint64_t)K, 128) ||      // rows of 64 features (K-major)
         !make_map(&tmdY, dY_dev, (uint64_t)M, (uint64_t)N, (uint64_t)N, 128) ||
         !make_map(&tmA, A_dev, (uint64_t)K, (uint64_t)r, (uint64_t)r, 64) ||       // 64 features x 64 ranks (MN-major)
         !make_map(&tmB, B_dev, (uint64_t)r, (uint64_t)N, (uint64_t)N, (uint32_t)rp)))   // ranks x 64 channels (K-major)
        return LOWRA_ERR_CUDA;
    SkinnyArgs a;
    memset(&a, 0, sizeof(a));
    a.status = status;
    a.wait_ns = wait_limit_ns();
    a.rp = rp;
    // Four skinny products; X and dY are each needed by two of them.  The two uses of the larger operand run back to
    // back, so that its second reading can come from L2, and the smaller operand is read first and last: T, U, dB, dA
    // when dY is the larger one, U, T, dA, dB otherwise.  With the caller's T and U only the two gradients are left.
    auto down_T = [&]() {   // T = s X A: rows = tokens, contraction over the K input features
        a.out = const_cast<uint16_t*>(T); a.R = M; a.C = K; a.n_cols = rp; a.ld_out = rp; a.a_mn = 0; a.b_mn = 1; a.transposed = 0; a.scale = s;
        return launch_skinny(tmX, tmA, a, stream);
    };
    auto down_U = [&]() {   // U = s dY B^T: rows = tokens, contraction over the N output channels
        a.out = const_cast<uint16_t*>(U); a.R = M; a.C = N; a.n_cols = rp; a.ld_out = rp; a.a_mn = 0; a.b_mn = 0; a.transposed = 0; a.scale = s;
        return launch_skinny(tmdY, tmB, a, stream);
    };
    auto grad_A = [&]() {   // dA = X^T U: rows = input features, contraction over the tokens
        a.out = dA_dev; a.R = K; a.C = M; a.n_cols = r; a.ld_out = r; a.a_mn = 1; a.b_mn = 1; a.transposed = 0; a.scale = 1.0f;
        return launch_skinny(tmXt, tmU, a, stream);
    };
    auto grad_B = [&]() {   // dB = (dY^T T)^T: rows = output channels, written transposed
        a.out = dB_dev; a.R = N; a.C = M; a.n_cols = r; a.ld_out = N; a.a_mn = 1; a.b_mn = 1; a.transposed = 1; a.scale = 1.0f;
        return launch_skinny(tmdYt, tmT, a, stream);
    };
    if (reuse) {
        if ((st = grad_A()) != LOWRA_OK) return st;
        return grad_B();
    }
    if (N > K) {
        if ((st = down_T()) != LOWRA_OK || (st = down_U()) != LOWRA_OK || (st = grad_B()) != LOWRA_OK) return st;
        return grad_A();
    }
    if ((st = down_U()) != LOWRA_OK || (st = down_T()) != LOWRA_OK || (st = grad_A()) != LOWRA_OK) return st;
    return grad_B();
}
}  // namespace
}  // namespace lowra

extern "C" lowra_status lowra_lora_backward_adapters(const uint16_t* X_dev, const uint16_t* dY_dev, int32_t M, int32_t K,
                                                     int32_t N, const uint16_t* A_dev, const uint16_t* B_dev, int32_t r,
                                                     float s, uint16_t* dA_dev, uint16_t* dB_dev, void* workspace_dev,
                                                     size_t workspace_bytes, void* stream) {
    return lowra::run_adapters(X_dev, dY_dev, M, K, N, A_dev, B_dev, r, s, nullptr, nullptr, dA_dev, dB_dev, workspace_dev,
                               workspace_bytes, stream);
}

extern "C" lowra_status lowra_lora_backward_adapters_reuse(const uint16_t* X_dev, const uint16_t* dY_dev, int32_t M, int32_t K,
                                                           int32_t N, const uint16_t* T_dev, const uint16_t* U_dev, int32_t r,
                                                           uint16_t* dA_dev, uint16_t* dB_dev, void* workspace_dev,
                                                           size_t workspace_bytes, void* stream) {
    if (!T_dev || !U_dev) return LOWRA_ERR_NULL;
    return lowra::run_adapters(X_dev, dY_dev, M, K, N, nullptr, nullptr, r, 1.0f, T_dev, U_dev, dA_dev, dB_dev, workspace_dev,
                               workspace_bytes, stream);
}

extern "C" const uint16_t* lowra_workspace_projection(const void* workspace_dev, int32_t member, int32_t M, int32_t r) {
    using namespace lowra;
    if (!workspace_dev || member < 0 || member >= kMaxBatch || M < 1 || !rank_ok(r)) return nullptr;
    const size_t t_bytes = align256((size_t)M * (size_t)((r + 63) / 64 * 64) * 2);   // as plan_workspace lays equal members out
    return reinterpret_cast<const uint16_t*>(static_cast<const unsigned char*>(workspace_dev) + kStatusBytes + (size_t)member * t_bytes);
}

extern "C" lowra_status lowra_device_status(const void* workspace_dev, void* stream) {
    if (!workspace_dev) return LOWRA_ERR_NULL;
    if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return LOWRA_ERR_CUDA;
    uint32_t word = 0;
    if (cudaMemcpy(&word, workspace_dev, sizeof(word), cudaMemcpyDeviceToHost) != cudaSuccess) return LOWRA_ERR_CUDA;
    return (lowra_status)word;
}

extern "C" lowra_status lowra_set_wait_limit(uint64_t nanoseconds) {
    using namespace lowra;
    if (nanoseconds == 0) nanoseconds = kDefaultWaitNs;
    if (nanoseconds < 1000ull || nanoseconds > 10ull * kDefaultWaitNs) return LOWRA_ERR_SHAPE;
    g_wait_ns.store(nanoseconds, std::memory_order_relaxed);
    return LOWRA_OK;
}

extern "C" lowra_status lowra_diag_drop_t_flags(int32_t calls) {
    if (calls < 0 || calls > 1000) return LOWRA_ERR_SHAPE;
    lowra::g_drop_t_flags.store(calls, std::memory_order_relaxed);
    return LOWRA_OK;
}

namespace lowra {
namespace {
// One CTA, one warp: lane 0 waits on a shared-memory barrier that nobody ever arrives on, then on a global flag that
// nobody ever raises, each with the given limit; whatever ran out is recorded and the kernel returns.
__global__ void wait_expiry_kernel(uint32_t* status, uint32_t* never_raised, uint32_t* report, unsigned long long limit_ns) {
    __shared__ uint64_t bar;
    if (threadIdx.x == 0) {
        ptx::mbar_init(&bar, 1);
        ptx::fence_barrier_init();
    }
    __syncwarp();
    uint32_t expired = 0;
    if (threadIdx.x == 0) {
        const uint64_t t0 = ptx::globaltimer_ns();
        if (!ptx::mbar_wait(&bar, 0u, nullptr, limit_ns)) expired |= 1u;
        const uint64_t t1 = ptx::globaltimer_ns();
        if (!ptx::flag_wait(never_raised, 0xFFFFFFFFu, nullptr, limit_ns)) expired |= 2u;
        const uint64_t t2 = ptx::globaltimer_ns();
        report[0] = expired;
        report[1] = (uint32_t)((t1 - t0) / 1000ull);   // microseconds spent in either wait
        report[2] = (uint32_t)((t2 - t1) / 1000ull);
        if (expired != 0u) atomicExch(status, (uint32_t)LOWRA_ERR_TIMEOUT);
    }
    expired = __shfl_sync(0xffffffffu, expired, 0);
    if (!ptx::mbar_wait_warp(&bar, 0u, nullptr, limit_ns) && threadIdx.x == 0) report[0] |= 4u;
}
}  // namespace
}  // namespace lowra

extern "C" lowra_status lowra_diag_wait_expiry(void* workspace_dev, size_t workspace_bytes, uint64_t limit_ns, void* stream) {
    using namespace lowra;
    if (!workspace_dev) return LOWRA_ERR_NULL;
    if (workspace_bytes < kStatusBytes || (reinterpret_cast<uintptr_t>(workspace_dev) & 255u) != 0) return LOWRA_ERR_WORKSPACE;
    if (limit_ns < 1000ull || limit_ns > 100ull * 1000ull * 1000ull) return LOWRA_ERR_SHAPE;   // 1 us .. 100 ms
    lowra_status st = check_device();
    if (st != LOWRA_OK) return st;
    uint32_t* w = reinterpret_cast<uint32_t*>(workspace_dev);
    if (cudaMemsetAsync(workspace_dev, 0, kStatusBytes, (cudaStream_t)stream) != cudaSuccess) return LOWRA_ERR_CUDA;
    wait_expiry_kernel<<<1, 32, 0, (cudaStream_t)stream>>>(w, w + 4, w + 8, limit_ns);
    return cudaGetLastError() == cudaSuccess ? LOWRA_OK : LOWRA_ERR_CUDA;
}

extern "C" lowra_status lowra_dense_nt(const uint16_t* P_dev, const uint16_t* Q_dev, int32_t M, int32_t N, int32_t K,
                                       uint16_t* C_dev, void* workspace_dev, size_t workspace_bytes, void* stream_v) {
    using namespace lowra;
    if (!P_dev || !Q_dev || !C_dev || !workspace_dev) return LOWRA_ERR_NULL;
    if (M < 1 || N < 1 || K < 64 || K % 64 != 0) return LOWRA_ERR_SHAPE;
    if (!aligned16(P_dev) || !aligned16(Q_dev) || !aligned16(C_dev)) return LOWRA_ERR_ALIGN;
    if (workspace_bytes < kStatusBytes || (reinterpret_cast<uintptr_t>(workspace_dev) & 255u) != 0)
        return LOWRA_ERR_WORKSPACE;
    lowra_status st = check_device();
    if (st != LOWRA_OK) return st;
    cudaStream_t stream = (cudaStream_t)stream_v;
    uint32_t* status = reinterpret_cast<uint32_t*>(workspace_dev);
    clear_status_kernel<<<1, 1, 0, stream>>>(status);

    GemmParams G;
    memset(&G, 0, sizeof(G));
    BatchMaps TM;
    memset(&TM, 0, sizeof(TM));
    G.count = 1;
    G.mem[0].out = C_dev;
    G.status = status;
    G.M = M;
    G.R = N;
    G.C = K;
    G.ld_out = N;
    G.main_blocks = K / kTileC;
    G.lora_blocks = 0;
    G.tiles_r = (N + kTileR - 1) / kTileR;
    G.super_total = (M + kTileT - 1) / kTileT;     // one CTA per "cluster" in the dense mode
    G.mem[0].M = M;
    G.wait_ns = wait_limit_ns();
    if (!make_map(&TM.m[0].tmB, P_dev, (uint64_t)M, (uint64_t)K, (uint64_t)K, kTileT)) return LOWRA_ERR_CUDA;
    if (!make_map(&TM.m[0].tmFl, Q_dev, (uint64_t)N, (uint64_t)K, (uint64_t)K, kTileR)) return LOWRA_ERR_CUDA;
    TM.m[0].tmT = TM.m[0].tmB;
    TM.m[0].tmFt = TM.m[0].tmB;
    return launch_fused(kModeDense, G, TM, stream);
}
