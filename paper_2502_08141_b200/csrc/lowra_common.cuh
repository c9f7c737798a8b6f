// Shared declarations of the CUDA path: launch-parameter structs, host-side validation helpers and
// a few device intrinsics.  Nothing in here is used by, or taken from, the CPU oracle.
#pragma once
#include <utility>

#include <cuda_runtime.h>
#include <stdint.h>

#include "lowra.h"

namespace lowra {

constexpr int kBlock = 64;        // elements per absmax block (Section 4.1, groupwise normalisation)
constexpr int kTableStride = 16;  // fp32 entries per row in the mapping / threshold tables
constexpr int kNumSMs = 148;      // B200: what grids and scratch are sized for; launches use min(this, the device's count)
constexpr int kMaxDevices = 64;   // per-device host state (launch configuration, built-in scratch) is kept for this many

// Everything a kernel needs to find a stored row; passed by value as a kernel argument.
struct RowLayout {
    int32_t N, K, nb;             // nb = K / 64
    int32_t class_start[4];       // first stored row of each precision class; [3] = N
    uint64_t seg_off[3];          // byte offset of each class in the packed buffer
    const uint8_t* precs;         // [N] original order
    const int32_t* perm;          // stored -> original
    const int32_t* inv_perm;      // original -> stored
    const uint64_t* nat;          // null: grouped order; else [N + 1] byte offsets of the rows in the natural-order buffer
};

lowra_status check_layout(const lowra_layout* L);
lowra_status check_device();
// Raises the dynamic shared-memory limit of `kernel` to `bytes` on the current device unless it already is that high
// there.  `state`: the caller's record per kernel (a zero-initialised static).  Thread-safe.
struct SmemLimit { size_t set[kMaxDevices]; };
lowra_status ensure_smem_limit(const void* kernel, size_t bytes, SmemLimit* state);
int device_sm_count();            // SMs of the current device, capped at kNumSMs (looked up once per device); 0 on error
RowLayout make_row_layout(const lowra_layout* L);

static inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// -------------------------------------------------------------------------------------------
// programmatic dependent launch: every kernel of the library lets its successor in the stream start launching
// right away (so the successor's launch latency and set-up overlap this kernel) and itself waits, before it
// touches global memory, until its predecessor has completed and flushed - stream order is preserved.
// -------------------------------------------------------------------------------------------
__device__ __forceinline__ void pdl_enter() {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
}
template <typename... KArgs, typename... Args>
static inline cudaError_t launch_pdl(void (*kernel)(KArgs...), unsigned grid, unsigned block, cudaStream_t stream, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.gridDim = dim3(grid, 1, 1);
    cfg.blockDim = dim3(block, 1, 1);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}

// -------------------------------------------------------------------------------------------
// device helpers
// -------------------------------------------------------------------------------------------
// Where stored row p (original row r, class c) lies: byte offset of its codes in the packed buffer, and its absmax row.
__device__ __forceinline__ size_t packed_row_offset(const RowLayout& L, int c, int p, int r) {
    return L.nat != nullptr ? (size_t)__ldg(L.nat + r) : (size_t)L.seg_off[c] + (size_t)(p - L.class_start[c]) * (((size_t)L.K << c) >> 3);
}
__device__ __forceinline__ int absmax_row_of(const RowLayout& L, int p, int r) { return L.nat != nullptr ? r : p; }

__device__ __forceinline__ int class_of_stored_row(const RowLayout& L, int p) {
    return (p >= L.class_start[1]) + (p >= L.class_start[2]);
}

// Two fp32 -> packed bf16x2, round to nearest even; `lo` lands in bits [0,16).
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

__device__ __forceinline__ uint4 ld_stream_v4(const void* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

__device__ __forceinline__ float4 ld_stream_f4(const void* p) {
    float4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.f32 {%0,%1,%2,%3}, [%4];"
                 : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(p));
    return v;
}

__device__ __forceinline__ void st_stream_v4(void* p, uint4 v) {
    asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w)
                 : "memory");
}

}  // namespace lowra
