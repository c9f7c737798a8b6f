// Host side of the C ABI: status strings, the storage planner and argument validation.
#include <string.h>

#include <mutex>

#include "lowra_common.cuh"

namespace lowra {

lowra_status check_layout(const lowra_layout* L) {
    if (!L) return LOWRA_ERR_NULL;
    if (!L->precs_dev || !L->perm_dev || !L->inv_perm_dev) return LOWRA_ERR_NULL;
    if (L->N < 1 || L->K < 128 || L->K % 128 != 0 || L->block != kBlock) return LOWRA_ERR_SHAPE;
    int64_t n = 0;
    for (int c = 0; c < 3; ++c) {
        if (L->counts[c] < 0) return LOWRA_ERR_PREC;
        n += L->counts[c];
    }
    if (n != L->N) return LOWRA_ERR_PREC;
    const uint64_t K = (uint64_t)L->K;
    const uint64_t o1 = (uint64_t)L->counts[0] * K / 8, o2 = o1 + (uint64_t)L->counts[1] * K / 4;
    const uint64_t total = o2 + (uint64_t)L->counts[2] * K / 2;
    if (L->seg_off[0] != 0 || L->seg_off[1] != o1 || L->seg_off[2] != o2 || L->packed_bytes != total)
        return LOWRA_ERR_PREC;
    if (!aligned16(L->perm_dev) || !aligned16(L->inv_perm_dev)) return LOWRA_ERR_ALIGN;
    if ((reinterpret_cast<uintptr_t>(L->natural_offsets_dev) & 7u) != 0) return LOWRA_ERR_ALIGN;
    return LOWRA_OK;
}

lowra_status check_device() {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return LOWRA_ERR_CUDA;
    int major = 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess)
        return LOWRA_ERR_CUDA;
    return major == 10 ? LOWRA_OK : LOWRA_ERR_ARCH;
}

lowra_status ensure_smem_limit(const void* kernel, size_t bytes, SmemLimit* state) {
    static std::mutex mutex;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return LOWRA_ERR_CUDA;
    std::lock_guard<std::mutex> lock(mutex);
    if (bytes > state->set[dev]) {
        if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes) != cudaSuccess)
            return LOWRA_ERR_CUDA;
        state->set[dev] = bytes;
    }
    return LOWRA_OK;
}

int device_sm_count() {
    static std::mutex mutex;
    static int count[kMaxDevices] = {0};
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return 0;
    std::lock_guard<std::mutex> lock(mutex);
    if (count[dev] == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) return 0;
        count[dev] = n < kNumSMs ? n : kNumSMs;
    }
    return count[dev];
}

RowLayout make_row_layout(const lowra_layout* L) {
    RowLayout R;
    R.N = L->N;
    R.K = L->K;
    R.nb = L->K / kBlock;
    R.class_start[0] = 0;
    R.class_start[1] = L->counts[0];
    R.class_start[2] = L->counts[0] + L->counts[1];
    R.class_start[3] = L->N;
    for (int c = 0; c < 3; ++c) R.seg_off[c] = L->seg_off[c];
    R.precs = L->precs_dev;
    R.perm = L->perm_dev;
    R.inv_perm = L->inv_perm_dev;
    R.nat = L->natural_offsets_dev;
    return R;
}

}  // namespace lowra

extern "C" const char* lowra_status_string(lowra_status st) {
    switch (st) {
        case LOWRA_OK: return "ok";
        case LOWRA_ERR_NULL: return "null pointer";
        case LOWRA_ERR_SHAPE: return "unsupported shape";
        case LOWRA_ERR_ALIGN: return "pointer not 16-byte aligned";
        case LOWRA_ERR_PREC: return "bad precision or inconsistent layout";
        case LOWRA_ERR_WORKSPACE: return "workspace too small or misaligned";
        case LOWRA_ERR_CUDA: return "CUDA call failed";
        case LOWRA_ERR_TIMEOUT: return "device-side wait timed out";
        case LOWRA_ERR_ARCH: return "device is not sm_100";
        case LOWRA_ERR_LIMIT: return "problem exceeds the built-in scratch of the no-allocation entry point";
    }
    return "unknown status";
}

extern "C" lowra_status lowra_plan(int32_t N, int32_t K, const uint8_t* precs_host, int32_t* perm_host,
                                   int32_t* inv_perm_host, int32_t counts[3], uint64_t seg_off[3],
                                   uint64_t* packed_bytes) {
    if (!precs_host || !perm_host || !inv_perm_host || !counts || !seg_off || !packed_bytes)
        return LOWRA_ERR_NULL;
    if (N < 1 || K < 128 || K % 128 != 0) return LOWRA_ERR_SHAPE;
    int32_t cnt[3] = {0, 0, 0};
    for (int32_t r = 0; r < N; ++r) {
        const uint8_t b = precs_host[r];
        if (b != 1 && b != 2 && b != 4) return LOWRA_ERR_PREC;
        ++cnt[b >> 1];  // 1 -> 0, 2 -> 1, 4 -> 2
    }
    int32_t next[3] = {0, cnt[0], cnt[0] + cnt[1]};  // counting sort keeps original order per class
    for (int32_t r = 0; r < N; ++r) {
        const int c = precs_host[r] >> 1;
        const int32_t p = next[c]++;
        perm_host[p] = r;
        inv_perm_host[r] = p;
    }
    uint64_t off = 0;
    for (int c = 0; c < 3; ++c) {
        counts[c] = cnt[c];
        seg_off[c] = off;
        off += (uint64_t)cnt[c] * (uint64_t)K * (uint64_t)(1 << c) / 8u;
    }
    *packed_bytes = off;
    return LOWRA_OK;
}
