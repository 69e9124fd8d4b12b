// Shared device helpers of the RAC kernels (sm_100a): bulk-copy / mbarrier PTX wrappers,
// packed binary32 arithmetic, small utilities.  Nothing in here is used by the CPU oracle.
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/rac.h"

namespace rac {

// ---------------------------------------------------------------------------------------------
// shared-memory addresses, mbarriers, 1-D bulk copies (TMA without a tensor map)
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void *p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_init_fence() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
// one arrival that also announces `bytes` of asynchronous copies
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// one poll; the hardware may park the thread for up to about a microsecond before answering
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity), "r"(1000u)
        : "memory");
    return ok != 0;
}
// Bounded wait: gives up after a fixed number of polls (well under a second) and reports it, so a copy
// that never lands cannot hang the GPU.
constexpr uint32_t kWaitPolls = 1u << 16;   // ~0.2 s of polling; a copy normally lands within microseconds
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity) {
    for (uint32_t i = 0; i < kWaitPolls; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
    }
    return false;
}

// global -> shared, completion counted on an mbarrier.  Addresses 16-byte aligned, bytes % 16 == 0.
__device__ __forceinline__ void bulk_load(uint32_t dst_smem, const void *src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst_smem), "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}
// shared -> global, tracked by the issuing thread's bulk groups
__device__ __forceinline__ void bulk_store(void *dst, uint32_t src_smem, uint32_t bytes) {
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst), "r"(src_smem), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void bulk_wait_read() {
    asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
// make this thread's ordinary shared-memory writes visible to the copy engine
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

__device__ __forceinline__ uint4 lds128(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}
__device__ __forceinline__ uint32_t lds32(uint32_t addr) {
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
}
__device__ __forceinline__ void sts128(uint32_t addr, uint4 v) {
    asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

// ---------------------------------------------------------------------------------------------
// packed binary32 arithmetic (two IEEE round-to-nearest operations per instruction on sm_100)
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ uint64_t pk(float2 v) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(v.x), "f"(v.y));
    return r;
}
__device__ __forceinline__ float2 upk(uint64_t r) {
    float2 v;
    asm("mov.b64 {%0, %1}, %2;" : "=f"(v.x), "=f"(v.y) : "l"(r));
    return v;
}
__device__ __forceinline__ float2 fma2(float2 a, float2 b, float2 c) {
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(pk(a)), "l"(pk(b)), "l"(pk(c)));
    return upk(d);
}
__device__ __forceinline__ float2 add2(float2 a, float2 b) {
    uint64_t d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(pk(a)), "l"(pk(b)));
    return upk(d);
}
__device__ __forceinline__ float2 sub2(float2 a, float2 b) {
    uint64_t d;
    asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(pk(a)), "l"(pk(b)));
    return upk(d);
}
__device__ __forceinline__ float2 mul2(float2 a, float2 b) {
    uint64_t d;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(pk(a)), "l"(pk(b)));
    return upk(d);
}

// a 32-bit word holding two bf16 -> (even channel, odd channel) as binary32 (exact)
__device__ __forceinline__ float2 bf16x2_to_f2(uint32_t w) {
    return make_float2(__uint_as_float(w << 16), __uint_as_float(w & 0xffff0000u));
}
// two binary32 -> packed bf16 (round to nearest even), first argument in the low half
__device__ __forceinline__ uint32_t f2_to_bf16x2(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&v);
}
__device__ __forceinline__ float bf16_round(float v) { return __bfloat162float(__float2bfloat16_rn(v)); }

__device__ __forceinline__ float half_bits_to_float(uint32_t h16) {
    return __half2float(__ushort_as_half(static_cast<unsigned short>(h16)));
}
// binary32 -> binary16 bits, round to nearest even, saturating at +-65504
__device__ __forceinline__ uint32_t float_to_half_bits_sat(float v) {
    v = fminf(fmaxf(v, -65504.0f), 65504.0f);
    return static_cast<uint32_t>(__half_as_ushort(__float2half_rn(v)));
}

// ---------------------------------------------------------------------------------------------
// host-side configuration helpers (defined in rac_codec.cu)
// ---------------------------------------------------------------------------------------------
struct Geometry {
    int d, group, bits, topk;
    int J;          // alignment groups per token
    int lpg;        // lanes per alignment group (group / 32)
    int nthreads;   // threads per CTA: one per 32 channels, rounded up to whole warps
    int code_bytes; // d*bits/8
    int scale_mode; // 0: static per-channel step table, 1: binary16 scales in the record (Eq. 8)
    int qgroup;     // channels per quantisation group (scale_mode 1; == group in mode 0)
    int Jq;         // quantisation groups per token
    int lpq;        // lanes per quantisation group, 0 when the group is the whole token and d/32 is no power of two <= 32
    int qgen;       // lanes per quantisation group when that is neither a power of two nor the token (then lpq == 0), else 0
    int topk_group; // outliers per quantisation group (scale_mode 1)
    int coef_fmt;   // 0: coefficient words in the record; 1: shared per segment, outside the record (scale_mode 1)
    int scale_off;  // byte offset of the scales in a record: 4*J, or 0 when the record holds no coefficients
    int codes_off;  // byte offset of the codes in a record: after the coefficient words and the scales
    int goff_off;   // byte offset of the per-group outlier offsets (Jq*topk_group bytes, padded to 2)
    int gval_off;   // byte offset of the per-group outlier values (Jq*topk_group binary16)
    int rec;        // record stride in bytes
};
int make_geometry(const rac_codec_cfg *cfg, Geometry *g);  // RAC_OK or an error

}  // namespace rac
