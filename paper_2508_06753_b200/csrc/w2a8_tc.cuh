// PTX wrappers shared by the tensor-core (tcgen05) kernels: mbarriers with bounded waits, TMA
// loads, tensor-memory allocation and loads, MMA issue and commit, shared-memory descriptors.
#pragma once

#include <cuda.h>

#include "w2a8_common.cuh"

namespace w2a8 {

constexpr unsigned kPfWaitPolls = 1u << 20;   // bound of every barrier wait (polls)

// ---- PTX wrappers ------------------------------------------------------------------
__device__ __forceinline__ uint32_t pf_smem_u32(const void *p) {
    return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void pf_mbar_init(uint32_t bar, unsigned count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void pf_mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void pf_mbar_arrive_expect_tx(uint32_t bar, unsigned bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool pf_mbar_try_wait(uint32_t bar, unsigned parity) {
    unsigned ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait; also gives up as soon as another role has raised the abort flag.
__device__ __forceinline__ bool pf_wait(uint32_t bar, unsigned parity, volatile int *abort_flag) {
    for (unsigned i = 0; i < kPfWaitPolls; ++i) {
        if (pf_mbar_try_wait(bar, parity)) return true;
        if ((i & 63u) == 63u && *abort_flag) return false;
    }
    *abort_flag = 1;
    return false;
}
// Whole-warp wait: only lane 0 polls the barrier (32 lanes polling one shared-memory
// word would compete with the tensor core for shared-memory bandwidth).
__device__ __forceinline__ bool pf_wait_warp(uint32_t bar, unsigned parity, volatile int *abort_flag) {
    int ok = 0;
    if ((threadIdx.x & 31) == 0) ok = pf_wait(bar, parity, abort_flag) ? 1 : 0;
    return __shfl_sync(0xFFFFFFFFu, ok, 0) != 0;
}
__device__ __forceinline__ void pf_tma_load_2d(uint32_t dst, const CUtensorMap *map, int x, int y, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar) : "memory");
}
// 16-byte store to a shared-space address
__device__ __forceinline__ void pf_st_shared_v4(uint32_t addr, uint32_t x, uint32_t y, uint32_t z, uint32_t w) {
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(x), "r"(y), "r"(z), "r"(w) : "memory");
}
__device__ __forceinline__ void pf_fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void pf_tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void pf_tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void pf_tmem_alloc(uint32_t dst_smem, uint32_t cols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void pf_tmem_dealloc(uint32_t taddr, uint32_t cols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void pf_mma_i8(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                          uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// mbarrier arrive once all MMAs issued so far by this thread have completed
__device__ __forceinline__ void pf_mma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void pf_tmem_ld32(uint32_t taddr, int (&v)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
          "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
          "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr) : "memory");
}
// (acc0, acc1) += (x0, x1) * sc as one packed fp32 instruction (one issue slot for two FMAs)
__device__ __forceinline__ void pf_fma2(float &acc0, float &acc1, float x0, float x1, float sc) {
    asm("{\n\t.reg .b64 a, b, c;\n\t"
        "mov.b64 a, {%2, %3};\n\t"
        "mov.b64 b, {%4, %4};\n\t"
        "mov.b64 c, {%0, %1};\n\t"
        "fma.rn.f32x2 c, a, b, c;\n\t"
        "mov.b64 {%0, %1}, c;\n\t}"
        : "+f"(acc0), "+f"(acc1) : "f"(x0), "f"(x1), "f"(sc));
}
// (acc0, acc1) += (float(d0), float(d1)) * sc for int32 d0, d1.  MAGIC (|d| < 2^22 only): the
// float is built as bits(d + 0x4B400000) = 12582912 + d (exact: below 2^24 in magnitude, one unit
// in the last place is 1) and the offset is taken off again by one packed subtraction, which is
// exact too: the result equals float(d) bit for bit, from full-rate integer and float
// instructions instead of the int-to-float conversion, which issues at a quarter of their rate.
template <bool MAGIC>
__device__ __forceinline__ void pf_cvt_fma2(float &acc0, float &acc1, int d0, int d1, float sc) {
    if constexpr (MAGIC) {
        const float x0 = __int_as_float(d0 + 0x4B400000), x1 = __int_as_float(d1 + 0x4B400000);
        asm("{\n\t.reg .b64 a, b, c, m;\n\t"
            "mov.b64 a, {%2, %3};\n\t"
            "mov.b64 m, {%5, %5};\n\t"
            "add.rn.f32x2 a, a, m;\n\t"
            "mov.b64 b, {%4, %4};\n\t"
            "mov.b64 c, {%0, %1};\n\t"
            "fma.rn.f32x2 c, a, b, c;\n\t"
            "mov.b64 {%0, %1}, c;\n\t}"
            : "+f"(acc0), "+f"(acc1) : "f"(x0), "f"(x1), "f"(sc), "f"(-12582912.0f));
    } else {
        pf_fma2(acc0, acc1, (float)d0, (float)d1, sc);
    }
}
__device__ __forceinline__ void pf_tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor of a K-major [rows][128 B] tile stored with the
// 128-byte swizzle: start address, 8-row stride of 1024 B, descriptor version 1,
// layout type 2 (128-byte swizzle).  A K step of 32 bytes inside the 128-byte row
// is taken by adding 32 to the start address.
__device__ __forceinline__ uint64_t pf_smem_desc(uint32_t addr) {
    uint64_t d = 0;
    d |= (uint64_t)((addr & 0x3FFFFu) >> 4);            // bits 0-13: start address / 16
    d |= (uint64_t)1 << 16;                              // bits 16-29: leading byte offset / 16 (unused here)
    d |= (uint64_t)(1024 >> 4) << 32;                    // bits 32-45: stride byte offset / 16
    d |= (uint64_t)1 << 46;                              // bits 46-47: descriptor version
    d |= (uint64_t)2 << 61;                              // bits 61-63: 128-byte swizzle
    return d;
}
// Instruction descriptor: int32 accumulate, signed 8-bit A and B, both K-major, M x N.
__host__ __device__ constexpr uint32_t pf_instr_desc(int m, int n) {
    return (2u << 4)                      // D format: S32
         | (1u << 7) | (1u << 10)         // A, B format: signed 8-bit
         | ((uint32_t)(n >> 3) << 17)     // N / 8
         | ((uint32_t)(m >> 4) << 24);    // M / 16
}

// The same for 16-bit floating-point operands (kind::f16): A and B bf16, both K-major, fp32
// accumulate; one instruction covers K = 16.
__host__ __device__ constexpr uint32_t pf_instr_desc_bf16(int m, int n) {
    return (1u << 4)                      // D format: F32
         | (1u << 7) | (1u << 10)         // A, B format: BF16
         | ((uint32_t)(n >> 3) << 17)     // N / 8
         | ((uint32_t)(m >> 4) << 24);    // M / 16
}
__device__ __forceinline__ void pf_mma_f16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                           uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}

// Driver entry point for building tensor maps (the library links the runtime only).
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);
inline EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *sym = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(sym);
    }
    return fn;
}

}  // namespace w2a8
