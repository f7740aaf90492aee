// The inner step shared by the streaming kernels: asynchronous-copy wrappers and the
// "cell" -- one 16-channel tile x one 256-k block of packed weights against 8 * MT tokens
// (up-convert and int8 multiply-accumulate of Sec. II-C, one scale group at a time).
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "w2a8_common.cuh"

namespace w2a8 {

// Kernel parameters of the one-shot streaming kernel; the cell reads the parity-export and
// ragged-tail fields from it (unused, and dropped by the compiler, in the full-block instances).
struct DecodeParams {
    const int8_t *a;
    const float *a_scale;
    const uint32_t *packed;
    const float *w_scale;
    float *y;
    int32_t *partials;
    float *ws;            // [chunks][M][N] partial outputs (chunks > 1)
    unsigned *counters;   // [grid.z][tile groups] arrival counters (chunks > 1)
    int *status;          // device status word (0 = ok)
    int M, N, K, G, group;
    int blocks, tail_slices, words_per_row;
    int chunks, blocks_per_chunk;
    int cluster;          // chunks > 1 and the chunks of a tile form one thread-block cluster
    int blocks_per_group; // 256-k blocks per scale group (groups of 256 and more)
    int s_vec;            // the scales of a cell and channel can be copied as one unit (16/8 B fp32, 8/4 B binary16)
    int h16;              // w_scale holds IEEE binary16 values (16-bit instances)
    int a16;              // a holds bf16 activations, a_scale is unused (16-bit-activation instances)
    int ldy;              // elements between consecutive token rows of y (>= N)
    int y16;              // 16-bit instances only: y holds bf16 instead of fp32
};

// ---- PTX wrappers ------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void *p) {
    return (uint32_t)__cvta_generic_to_shared(p);
}
// per-thread asynchronous copies into shared memory
__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async8(uint32_t dst, const void *src) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async4(uint32_t dst, const void *src) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait_group() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
// n is a constant after unrolling
__device__ __forceinline__ void cp_async_wait_pending(int n) {
    switch (n) {
        case 0: cp_async_wait_group<0>(); break;
        case 1: cp_async_wait_group<1>(); break;
        case 2: cp_async_wait_group<2>(); break;
        case 3: cp_async_wait_group<3>(); break;
        case 4: cp_async_wait_group<4>(); break;
        case 5: cp_async_wait_group<5>(); break;
        case 6: cp_async_wait_group<6>(); break;
        default: cp_async_wait_group<7>(); break;
    }
}

__device__ __forceinline__ uint4 ld_act16(const int8_t *p) {
    // plain (L1-allocating) load: the activations are written by the previous kernel of the
    // stream and are only read after the wait for it, so the read-only path is not used
    uint4 v;
    asm volatile("ld.global.ca.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

// The same 16 bytes from a staged copy of the activations in shared memory: `p` carries a 32-bit
// shared-window address in its low bits (see act_ptr), so pointer arithmetic stays plain adds.
__device__ __forceinline__ uint4 ld_act16_smem(const int8_t *p) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "r"((uint32_t)(uintptr_t)p));
    return v;
}
__device__ __forceinline__ const int8_t *act_ptr(uint32_t smem_addr) {
    return reinterpret_cast<const int8_t *>((uintptr_t)smem_addr);
}

// One cell: 4 slices x (unpack, 2 MMAs per token slab, promotion at group ends).
// w0s/w1s: this lane's four words (one per slice) of channels n0+gq and n0+gq+8;
// sc0/sc1: the cell's scales of the same channels (shared memory, 16 bytes each);
// brow[mt]: this lane's 16 activation bytes of slice 0 of the cell, token row of slab mt.
// H16: the scales in shared memory are IEEE binary16 (2 bytes each) instead of fp32.
// ASMEM: brow[] are shared-memory addresses made by act_ptr (activations staged per CTA).
template <int MT, int SPP, bool ONE, bool PARTIALS, bool FULL, bool H16, bool ASMEM = false>
__device__ __forceinline__ void compute_cell(const DecodeParams &p, const uint32_t (&w0s)[4],
                                             const uint32_t (&w1s)[4], const unsigned char *sc0,
                                             const unsigned char *sc1,
                                             const int8_t *const (&brow)[MT], int kb, int n0, int m0,
                                             int gq, int t, float (&acc)[MT][4]) {
    // FULL: the block has all four slices (always, except possibly the last block of K)
    const int R = FULL ? 4 : p.tail_slices;
    const int magic[4] = {kMagicInt, kMagicInt, kMagicInt, kMagicInt};
    int D[MT][4];   // int32 accumulators of the current group; a group never outlives a cell
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int i = 0; i < 4; ++i) D[mt][i] = kMagicInt;
    float s0s[4 / SPP], s1s[4 / SPP];
    if constexpr (!PARTIALS && H16) {
        if constexpr (SPP == 4) {
            s0s[0] = __half2float(*reinterpret_cast<const __half *>(sc0));
            s1s[0] = __half2float(*reinterpret_cast<const __half *>(sc1));
        } else if constexpr (SPP == 2) {
            const float2 v0 = __half22float2(*reinterpret_cast<const __half2 *>(sc0));
            const float2 v1 = __half22float2(*reinterpret_cast<const __half2 *>(sc1));
            s0s[0] = v0.x; s0s[1] = v0.y; s1s[0] = v1.x; s1s[1] = v1.y;
        } else {
            const uint2 r0 = *reinterpret_cast<const uint2 *>(sc0), r1 = *reinterpret_cast<const uint2 *>(sc1);
            const float2 v0 = __half22float2(*reinterpret_cast<const __half2 *>(&r0.x));
            const float2 v1 = __half22float2(*reinterpret_cast<const __half2 *>(&r0.y));
            const float2 v2 = __half22float2(*reinterpret_cast<const __half2 *>(&r1.x));
            const float2 v3 = __half22float2(*reinterpret_cast<const __half2 *>(&r1.y));
            s0s[0] = v0.x; s0s[1] = v0.y; s0s[2] = v1.x; s0s[3] = v1.y;
            s1s[0] = v2.x; s1s[1] = v2.y; s1s[2] = v3.x; s1s[3] = v3.y;
        }
    } else if constexpr (!PARTIALS) {
        if constexpr (SPP == 4) {
            s0s[0] = *reinterpret_cast<const float *>(sc0);
            s1s[0] = *reinterpret_cast<const float *>(sc1);
        } else if constexpr (SPP == 2) {
            const float2 v0 = *reinterpret_cast<const float2 *>(sc0);
            const float2 v1 = *reinterpret_cast<const float2 *>(sc1);
            s0s[0] = v0.x; s0s[1] = v0.y; s1s[0] = v1.x; s1s[1] = v1.y;
        } else {
            const float4 v0 = *reinterpret_cast<const float4 *>(sc0);
            const float4 v1 = *reinterpret_cast<const float4 *>(sc1);
            s0s[0] = v0.x; s0s[1] = v0.y; s0s[2] = v0.z; s0s[3] = v0.w;
            s1s[0] = v1.x; s1s[1] = v1.y; s1s[2] = v1.z; s1s[3] = v1.w;
        }
    }
#pragma unroll
    for (int s = 0; s < 4; ++s) {
        if (s < R) {
            const uint32_t w0 = w0s[s], w1 = w1s[s];
            const uint32_t a0 = lane_codes(w0, 0), a1 = lane_codes(w1, 0);
            const uint32_t a2 = lane_codes(w0, 1), a3 = lane_codes(w1, 1);
            const uint32_t a4 = lane_codes(w0, 2), a5 = lane_codes(w1, 2);
            const uint32_t a6 = lane_codes(w0, 3), a7 = lane_codes(w1, 3);
            const bool first = (s % SPP) == 0;
            const bool last = ((s + 1) % SPP) == 0 || s == R - 1;
#pragma unroll
            for (int mt = 0; mt < MT; ++mt) {
                const uint4 b = ASMEM ? ld_act16_smem(brow[mt] + s * kSliceK) : ld_act16(brow[mt] + s * kSliceK);
                if (first) mma_s8_16x8x32(D[mt], a0, a1, a2, a3, b.x, b.y, magic);
                else       mma_s8_16x8x32(D[mt], a0, a1, a2, a3, b.x, b.y, D[mt]);
                mma_s8_16x8x32(D[mt], a4, a5, a6, a7, b.z, b.w, D[mt]);
                if (last) {
                    if constexpr (PARTIALS) {
                        const int gi = (SPP == 1) ? 4 * kb + s
                                     : (SPP == 2) ? 2 * kb + (s >> 1)
                                                  : (int)(((long long)kb * kBlockK) / p.group);
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const int mm = m0 + 8 * mt + 2 * t + (i & 1);
                            const int nn = n0 + gq + 8 * (i >> 1);
                            if (mm < p.M)
                                atomicAdd(p.partials + ((size_t)mm * p.N + nn) * p.G + gi,
                                          (D[mt][i] - kMagicInt) >> 6);
                        }
                    } else {
                        const float s0 = s0s[s / SPP], s1 = s1s[s / SPP];
                        if constexpr (ONE) {
                            acc[mt][0] = fmaf(s0, __int_as_float(D[mt][0]) - kMagicFloat, acc[mt][0]);
                            acc[mt][2] = fmaf(s1, __int_as_float(D[mt][2]) - kMagicFloat, acc[mt][2]);
                        } else if constexpr (MT == 1) {
                            // packed fp32 pairs: measured faster for one slab, slower for more
                            promote2(acc[mt][0], acc[mt][1], D[mt][0], D[mt][1], s0);
                            promote2(acc[mt][2], acc[mt][3], D[mt][2], D[mt][3], s1);
                        } else {
                            acc[mt][0] = fmaf(s0, __int_as_float(D[mt][0]) - kMagicFloat, acc[mt][0]);
                            acc[mt][1] = fmaf(s0, __int_as_float(D[mt][1]) - kMagicFloat, acc[mt][1]);
                            acc[mt][2] = fmaf(s1, __int_as_float(D[mt][2]) - kMagicFloat, acc[mt][2]);
                            acc[mt][3] = fmaf(s1, __int_as_float(D[mt][3]) - kMagicFloat, acc[mt][3]);
                        }
                    }
                }
            }
        }
    }
}

// One cell against 8 * MT tokens whose activation bytes are already in registers: B[mt][s] holds
// this lane's 16 bytes of slice s (token row gq of slab mt).  A warp that owns the same block of
// every tile it works on loads them once per launch.  fp32 scales, whole blocks, acc as in
// compute_cell.
template <int MT, int SPP, bool ONE>
__device__ __forceinline__ void compute_cell_breg(const uint4 &wa, const uint4 &wb, const unsigned char *sc0,
                                                  const unsigned char *sc1, const uint4 (&B)[MT][4],
                                                  float (&acc)[MT][4]) {
    const uint32_t w0s[4] = {wa.x, wa.y, wa.z, wa.w};
    const uint32_t w1s[4] = {wb.x, wb.y, wb.z, wb.w};
    const int magic[4] = {kMagicInt, kMagicInt, kMagicInt, kMagicInt};
    float s0s[4 / SPP], s1s[4 / SPP];
    if constexpr (SPP == 4) {
        s0s[0] = *reinterpret_cast<const float *>(sc0);
        s1s[0] = *reinterpret_cast<const float *>(sc1);
    } else if constexpr (SPP == 2) {
        const float2 v0 = *reinterpret_cast<const float2 *>(sc0);
        const float2 v1 = *reinterpret_cast<const float2 *>(sc1);
        s0s[0] = v0.x; s0s[1] = v0.y; s1s[0] = v1.x; s1s[1] = v1.y;
    } else {
        const float4 v0 = *reinterpret_cast<const float4 *>(sc0);
        const float4 v1 = *reinterpret_cast<const float4 *>(sc1);
        s0s[0] = v0.x; s0s[1] = v0.y; s0s[2] = v0.z; s0s[3] = v0.w;
        s1s[0] = v1.x; s1s[1] = v1.y; s1s[2] = v1.z; s1s[3] = v1.w;
    }
    int D[MT][4];
#pragma unroll
    for (int s = 0; s < 4; ++s) {
        const uint32_t w0 = w0s[s], w1 = w1s[s];
        const uint32_t a0 = lane_codes(w0, 0), a1 = lane_codes(w1, 0);
        const uint32_t a2 = lane_codes(w0, 1), a3 = lane_codes(w1, 1);
        const uint32_t a4 = lane_codes(w0, 2), a5 = lane_codes(w1, 2);
        const uint32_t a6 = lane_codes(w0, 3), a7 = lane_codes(w1, 3);
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) {
            if ((s % SPP) == 0) mma_s8_16x8x32_pure(D[mt], a0, a1, a2, a3, B[mt][s].x, B[mt][s].y, magic);
            else                mma_s8_16x8x32_pure(D[mt], a0, a1, a2, a3, B[mt][s].x, B[mt][s].y, D[mt]);
            mma_s8_16x8x32_pure(D[mt], a4, a5, a6, a7, B[mt][s].z, B[mt][s].w, D[mt]);
            if (((s + 1) % SPP) == 0) {
                const float s0 = s0s[s / SPP], s1 = s1s[s / SPP];
                if constexpr (ONE) {
                    acc[mt][0] = fmaf(s0, __int_as_float(D[mt][0]) - kMagicFloat, acc[mt][0]);
                    acc[mt][2] = fmaf(s1, __int_as_float(D[mt][2]) - kMagicFloat, acc[mt][2]);
                } else {
                    promote2(acc[mt][0], acc[mt][1], D[mt][0], D[mt][1], s0);
                    promote2(acc[mt][2], acc[mt][3], D[mt][2], D[mt][3], s1);
                }
            }
        }
    }
}

}  // namespace w2a8
