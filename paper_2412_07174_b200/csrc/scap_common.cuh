// Shared device/host helpers of the SCAP sm_100a library (internal; the public ABI is scap.h).
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <type_traits>

#include "scap.h"

namespace scap {

constexpr int SCAP_MAX_K = 1 << 20;  // input channels per FC (keeps every index comfortably inside 32 bits)

struct Tuning {
    int split_k;  // 0 = automatic
    int pdl;      // programmatic dependent launch between the kernels of one call
    int tc;       // batch 3..16 on the tcgen05 kernel (0: the mma.sync variants)
    int host_direct;  // scap_sparse_fc_host moves device-addressable pinned host buffers with its own kernels
    int fma_rows;     // largest batch that takes the fp32-FMA body (2 or 4); larger batches take a tensor-core variant
    int cal_strip;    // channels per CTA of the calibration histogram kernel: 16 or 32
    int l2_hints;     // batch 1..4 FC kernel: L2 eviction hints (keep activations and modes, stream weights)
    int tile;         // columns per CTA of the FC kernel: 0 = automatic, else 128 or 256
    int tc_spin;      // tcgen05 kernel: polls before a barrier wait gives up (0 = the built-in limit)
    int head_rows;    // batch 1..4 FC kernel: 32-channel chunks per CTA whose weight rows are asked into L2 before the kept set is known
    int dense_stream; // batch 5..16: 1 = the dense-stream tcgen05 kernel (TMA box loads of all rows), 0 = the gather kernels, 2 = from batch 3
};
extern Tuning g_tune;

// ---- status helpers -------------------------------------------------------------------------
scap_status check_device();  // SCAP_OK on compute capability 10.x
int sm_count();              // multiprocessors of the current device (148 when no device is present)

inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

inline scap_status cuda_status(cudaError_t e) {
    if (e == cudaSuccess) return SCAP_OK;
    cudaGetLastError();
    return SCAP_ERR_CUDA;
}

// Opt-in to more than 48 KB of dynamic shared memory, once per kernel and device (the attribute belongs to the
// device's copy of the function, so a process that drives several devices sets it on each).
struct SmemOptIn {
    unsigned long long done = 0;  // bit d: set on device d (devices beyond 63 are set every time)
};
template <typename Kern>
inline cudaError_t ensure_dynamic_smem(Kern kern, int bytes, SmemOptIn &state) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64 && ((state.done >> dev) & 1ull)) return cudaSuccess;
    e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (e == cudaSuccess && dev >= 0 && dev < 64) state.done |= 1ull << dev;
    return e;
}

// ---- programmatic dependent launch ----------------------------------------------------------
// wait: blocks until every kernel this grid depends on has finished and its writes are visible
// (returns at once when the launch carried no programmatic dependency).
__device__ __forceinline__ void griddep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
// launch_dependents: lets the next kernel in the stream begin its launch early; that kernel still
// calls griddep_wait() before touching anything this grid produces.
__device__ __forceinline__ void griddep_launch_dependents() {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

template <typename... KArgs, typename... Args>
inline cudaError_t launch(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream, bool pdl,
                          Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = pdl ? 1 : 0;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// ---- storage dtype widening -------------------------------------------------------------------
// Two 16-bit values packed in one 32-bit word -> two floats (exact).
template <bool BF16>
__device__ __forceinline__ void widen2(uint32_t u, float &lo, float &hi) {
    if constexpr (BF16) {
        lo = __uint_as_float(u << 16);
        hi = __uint_as_float(u & 0xffff0000u);
    } else {
        __half2 h = *reinterpret_cast<__half2 *>(&u);
        float2 f = __half22float2(h);
        lo = f.x;
        hi = f.y;
    }
}

__device__ __forceinline__ float widen1(const __nv_bfloat16 &v) { return __bfloat162float(v); }
__device__ __forceinline__ float widen1(const __half &v) { return __half2float(v); }
__device__ __forceinline__ float widen1(const float &v) { return v; }

template <bool BF16>
__device__ __forceinline__ float widen_at(const void *p, size_t i) {
    if constexpr (BF16) return widen1(reinterpret_cast<const __nv_bfloat16 *>(p)[i]);
    else return widen1(reinterpret_cast<const __half *>(p)[i]);
}

// One 16-bit storage pattern -> float (exact).
template <bool BF16>
__device__ __forceinline__ float widen_bits(unsigned short u) {
    if constexpr (BF16) return __uint_as_float((uint32_t)u << 16);
    else return __half2float(__ushort_as_half(u));
}

// 16-byte streaming load of weights: read-only path, no L1 allocation (each byte is used once).
__device__ __forceinline__ uint4 ld_stream16(const void *p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

// Ordered read-only loads: being volatile asm, they are issued where they are written (the compiler neither
// sinks them towards their first use nor reorders them), which is what keeps a batch of them in flight together.
__device__ __forceinline__ float ld_nc(const float *p) {
    float v;
    asm volatile("ld.global.nc.f32 %0, [%1];" : "=f"(v) : "l"(p));
    return v;
}
__device__ __forceinline__ __nv_bfloat16 ld_nc(const __nv_bfloat16 *p) {
    unsigned short v;
    asm volatile("ld.global.nc.u16 %0, [%1];" : "=h"(v) : "l"(p));
    return __ushort_as_bfloat16(v);
}
__device__ __forceinline__ __half ld_nc(const __half *p) {
    unsigned short v;
    asm volatile("ld.global.nc.u16 %0, [%1];" : "=h"(v) : "l"(p));
    return __ushort_as_half(v);
}

// Activation loads.  With programmatic dependent launch a kernel is resident on an SM while its predecessor is
// still writing the activations, and the non-coherent path may serve a line that an earlier kernel left in that
// SM's L1; activations are therefore read through L2 (.cg), in issue order like ld_nc.
__device__ __forceinline__ float ld_act(const float *p) {
    float v;
    asm volatile("ld.global.cg.f32 %0, [%1];" : "=f"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ __nv_bfloat16 ld_act(const __nv_bfloat16 *p) {
    unsigned short v;
    asm volatile("ld.global.cg.u16 %0, [%1];" : "=h"(v) : "l"(p) : "memory");
    return __ushort_as_bfloat16(v);
}
__device__ __forceinline__ __half ld_act(const __half *p) {
    unsigned short v;
    asm volatile("ld.global.cg.u16 %0, [%1];" : "=h"(v) : "l"(p) : "memory");
    return __ushort_as_half(v);
}
// Predicated forms: the load is issued only where `on` holds and the result is 0 elsewhere.  No branch, so a batch
// of them still goes out together; and - unlike clamping the address of an unused slot to element 0 - the unused
// slots of all CTAs do not converge on one L2 sector (which serialises them there).
__device__ __forceinline__ float ld_nc_if(const float *p, bool on) {
    float v;
    asm volatile("{ .reg .pred q; setp.ne.u32 q, %2, 0; mov.f32 %0, 0f00000000; @q ld.global.nc.f32 %0, [%1]; }"
                 : "=f"(v) : "l"(p), "r"((unsigned)on));
    return v;
}
__device__ __forceinline__ float ld_act_if(const float *p, bool on) {
    float v;
    asm volatile("{ .reg .pred q; setp.ne.u32 q, %2, 0; mov.f32 %0, 0f00000000; @q ld.global.cg.f32 %0, [%1]; }"
                 : "=f"(v) : "l"(p), "r"((unsigned)on) : "memory");
    return v;
}
__device__ __forceinline__ unsigned short ld_act_if_u16(const void *p, bool on) {
    unsigned short v;
    asm volatile("{ .reg .pred q; setp.ne.u32 q, %2, 0; mov.u16 %0, 0; @q ld.global.cg.u16 %0, [%1]; }"
                 : "=h"(v) : "l"(p), "r"((unsigned)on) : "memory");
    return v;
}
__device__ __forceinline__ __nv_bfloat16 ld_act_if(const __nv_bfloat16 *p, bool on) { return __ushort_as_bfloat16(ld_act_if_u16(p, on)); }
__device__ __forceinline__ __half ld_act_if(const __half *p, bool on) { return __ushort_as_half(ld_act_if_u16(p, on)); }

// 16-byte activation / parameter load through L2, predicated (zeros where off).
__device__ __forceinline__ uint4 ld_act16_if(const void *p, bool on) {
    uint4 v;
    asm volatile(
        "{ .reg .pred q; setp.ne.u32 q, %5, 0; mov.u32 %0, 0; mov.u32 %1, 0; mov.u32 %2, 0; mov.u32 %3, 0;"
        " @q ld.global.cg.v4.u32 {%0,%1,%2,%3}, [%4]; }"
        : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
        : "l"(p), "r"((unsigned)on)
        : "memory");
    return v;
}

__device__ __forceinline__ uint4 ld_act16_if(const void *p, bool on, uint64_t pol) {
    uint4 v;
    asm volatile(
        "{ .reg .pred q; setp.ne.u32 q, %5, 0; mov.u32 %0, 0; mov.u32 %1, 0; mov.u32 %2, 0; mov.u32 %3, 0;"
        " @q ld.global.cg.L2::cache_hint.v4.u32 {%0,%1,%2,%3}, [%4], %6; }"
        : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
        : "l"(p), "r"((unsigned)on), "l"(pol)
        : "memory");
    return v;
}

// L2 eviction policies for loads that carry a cache hint.  keep: small data every column tile of a call reads again
// (activations, modes); stream: weight rows, read once.
__device__ __forceinline__ uint64_t l2_policy_keep() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ uint64_t l2_policy_stream() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ uint64_t l2_policy_normal() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_normal.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ uint4 ld_stream16(const void *p, uint64_t pol) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.L2::cache_hint.v4.u32 {%0,%1,%2,%3}, [%4], %5;"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p), "l"(pol));
    return v;
}
// Predicated form: zeros where `on` does not hold (no request goes out).
__device__ __forceinline__ uint4 ld_stream16_if(const void *p, bool on, uint64_t pol) {
    uint4 v;
    asm volatile(
        "{ .reg .pred q; setp.ne.u32 q, %5, 0; mov.u32 %0, 0; mov.u32 %1, 0; mov.u32 %2, 0; mov.u32 %3, 0;"
        " @q ld.global.nc.L1::no_allocate.L2::cache_hint.v4.u32 {%0,%1,%2,%3}, [%4], %6; }"
        : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
        : "l"(p), "r"((unsigned)on), "l"(pol));
    return v;
}
__device__ __forceinline__ float ld_nc_if(const float *p, bool on, uint64_t pol) {
    float v;
    asm volatile("{ .reg .pred q; setp.ne.u32 q, %2, 0; mov.f32 %0, 0f00000000; @q ld.global.nc.L2::cache_hint.f32 %0, [%1], %3; }"
                 : "=f"(v) : "l"(p), "r"((unsigned)on), "l"(pol));
    return v;
}
__device__ __forceinline__ float ld_act_if(const float *p, bool on, uint64_t pol) {
    float v;
    asm volatile("{ .reg .pred q; setp.ne.u32 q, %2, 0; mov.f32 %0, 0f00000000; @q ld.global.cg.L2::cache_hint.f32 %0, [%1], %3; }"
                 : "=f"(v) : "l"(p), "r"((unsigned)on), "l"(pol) : "memory");
    return v;
}
__device__ __forceinline__ unsigned short ld_act_if_u16(const void *p, bool on, uint64_t pol) {
    unsigned short v;
    asm volatile("{ .reg .pred q; setp.ne.u32 q, %2, 0; mov.u16 %0, 0; @q ld.global.cg.L2::cache_hint.u16 %0, [%1], %3; }"
                 : "=h"(v) : "l"(p), "r"((unsigned)on), "l"(pol) : "memory");
    return v;
}
__device__ __forceinline__ __nv_bfloat16 ld_act_if(const __nv_bfloat16 *p, bool on, uint64_t pol) { return __ushort_as_bfloat16(ld_act_if_u16(p, on, pol)); }
__device__ __forceinline__ __half ld_act_if(const __half *p, bool on, uint64_t pol) { return __ushort_as_half(ld_act_if_u16(p, on, pol)); }

// ---- shared-memory barriers and cluster addressing (split-K exchange of the FC kernel) ---------------------
__device__ __forceinline__ uint32_t smem_addr(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
// Address of the same shared-memory location in the CTA with rank `rank` of this cluster.
__device__ __forceinline__ uint32_t cluster_addr(uint32_t local, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local), "r"(rank));
    return r;
}
__device__ __forceinline__ void mbarrier_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
// One arrival that also announces `bytes` of asynchronous stores still to land on the barrier.
__device__ __forceinline__ void mbarrier_arrive_expect(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbarrier_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile("{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Asynchronous 4-byte store into another CTA of the cluster; the store itself counts 4 bytes down on that CTA's
// barrier when it lands, so data and notification travel together (no acknowledgement, no cluster barrier).
__device__ __forceinline__ void st_async_f32(uint32_t remote_addr, float v, uint32_t remote_bar) {
    asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.b32 [%0], %1, [%2];" ::"r"(remote_addr),
                 "r"(__float_as_uint(v)), "r"(remote_bar) : "memory");
}
// Split cluster barrier: arrive early, wait where the guarantee is needed.
__device__ __forceinline__ void cluster_arrive() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
// Arrival without memory ordering of its own: enough after mbarrier_init, whose fence publishes the barriers, and it
// does not wait for loads that are under way.
__device__ __forceinline__ void cluster_arrive_relaxed() { asm volatile("barrier.cluster.arrive.relaxed.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }

// 16-byte read-only load that asks L2 to keep the line (the calibration tensor is read again by the following passes).
__device__ __forceinline__ uint4 ld_keep16(const void *p, uint64_t pol) {
    uint4 v;
    asm volatile("ld.global.nc.L2::cache_hint.v4.u32 {%0,%1,%2,%3}, [%4], %5;"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p), "l"(pol));
    return v;
}

// Hint: bring the line that holds *p into L2 (no register result, no ordering effect).
__device__ __forceinline__ void prefetch_l2(const void *p) { asm volatile("prefetch.global.L2 [%0];" ::"l"(p)); }
// The same, and L2 is asked to keep the line (small data that many CTAs and later calls read again).
__device__ __forceinline__ void prefetch_l2_keep(const void *p) { asm volatile("prefetch.global.L2::evict_last [%0];" ::"l"(p)); }

}  // namespace scap
