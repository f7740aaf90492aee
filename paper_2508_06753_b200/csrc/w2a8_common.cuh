// Shared device/host helpers of the W2A8 CUDA library (sm_100a only).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "w2a8.h"

namespace w2a8 {

// ---- W2P layout constants (see w2_pack in w2a8.h) -------------------------
constexpr int kSliceK = 64;    // k per slice = smallest scale group
constexpr int kBlockK = 256;   // k per block = four slices
constexpr int kWordK = 16;     // codes per 32-bit word

// The unpack puts each 2-bit code into the two top bits of an int8 lane:
//   lane = ((word << (6 - 2 j)) & 0xC0C0C0C0) ^ 0x80808080  =  64 * (code - 2)
// (offset binary -> two's complement is the XOR of the top bit).  All integer
// sums therefore carry an exact factor 64 that the epilogue removes.
constexpr uint32_t kTopMask = 0xC0C0C0C0u;
constexpr uint32_t kSignFlip = 0x80808080u;
constexpr int kCodeGain = 64;

// int32 accumulators start at the bit pattern of 1.5 * 2^23; as long as the
// accumulated integer stays below 2^22 in magnitude, reinterpreting the
// accumulator as fp32 and subtracting 1.5 * 2^23 converts it exactly, with no
// integer-to-float instruction.
constexpr int kMagicInt = 0x4B400000;
constexpr float kMagicFloat = 12582912.0f;

__device__ __forceinline__ uint32_t lane_codes(uint32_t word, int j) {
    // j is a compile-time constant after unrolling; (x & mask) ^ flip is one LOP3 (LUT 0x6A)
    const uint32_t x = (j == 3) ? word : (word << (6 - 2 * j));
    uint32_t r;
    asm("lop3.b32 %0, %1, 0xC0C0C0C0, 0x80808080, 0x6A;" : "=r"(r) : "r"(x));
    return r;
}

// (acc0, acc1) += sc * (float(d0), float(d1)) for two accumulators in the magic-number form:
// one packed subtract and one packed fused multiply-add (two issue slots for two values).
__device__ __forceinline__ void promote2(float &acc0, float &acc1, int d0, int d1, float sc) {
    asm("{\n\t.reg .b64 a, b, c, m;\n\t"
        "mov.b64 a, {%2, %3};\n\t"
        "mov.b64 m, {%5, %5};\n\t"
        "add.rn.f32x2 a, a, m;\n\t"
        "mov.b64 b, {%4, %4};\n\t"
        "mov.b64 c, {%0, %1};\n\t"
        "fma.rn.f32x2 c, a, b, c;\n\t"
        "mov.b64 {%0, %1}, c;\n\t}"
        : "+f"(acc0), "+f"(acc1) : "r"(d0), "r"(d1), "f"(sc), "f"(-kMagicFloat));
}

// Thread-block clusters: barrier over all threads of all CTAs of the cluster (release /
// acquire), this CTA's rank, and a read of another CTA's shared memory.
__device__ __forceinline__ void cluster_sync() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// The two halves of a cluster barrier, for a phase whose only purpose is "every CTA of the
// cluster has started": arrive early, wait late.
__device__ __forceinline__ void cluster_arrive_relaxed() {
    asm volatile("barrier.cluster.arrive.relaxed.aligned;" ::: "memory");
}
__device__ __forceinline__ void cluster_wait() {
    asm volatile("barrier.cluster.wait.aligned;" ::: "memory");
}
__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ float ld_cluster_f32(uint32_t local_smem_addr, uint32_t rank) {
    uint32_t remote;
    float v;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local_smem_addr), "r"(rank));
    asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(remote) : "memory");
    return v;
}

__device__ __forceinline__ void st_cluster_f32(uint32_t local_smem_addr, uint32_t rank, float v) {
    uint32_t remote;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local_smem_addr), "r"(rank));
    asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(remote), "f"(v) : "memory");
}

// Programmatic dependent launch: wait until the previous kernel of the stream
// has completed and its writes are visible / let the next kernel start early.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

// D = A (16 x 32, int8, row) * B (32 x 8, int8, col) + C, int32 accumulate.
__device__ __forceinline__ void mma_s8_16x8x32(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2,
                                               uint32_t a3, uint32_t b0, uint32_t b1,
                                               const int (&c)[4]) {
    asm volatile(
        "mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
        "{%10,%11,%12,%13};"
        : "=r"(d[0]), "=r"(d[1]), "=r"(d[2]), "=r"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "r"(c[0]), "r"(c[1]), "r"(c[2]),
          "r"(c[3]));
}

// The same instruction as a pure function of its operands (not `volatile`): the compiler may
// interleave independent MMAs with the unpack arithmetic of neighbouring slices.
__device__ __forceinline__ void mma_s8_16x8x32_pure(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2,
                                                    uint32_t a3, uint32_t b0, uint32_t b1,
                                                    const int (&c)[4]) {
    asm("mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
        "{%10,%11,%12,%13};"
        : "=r"(d[0]), "=r"(d[1]), "=r"(d[2]), "=r"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "r"(c[0]), "r"(c[1]), "r"(c[2]),
          "r"(c[3]));
}

// D = A (16 x 16, bf16, row) * B (16 x 8, bf16, col) + C, fp32 accumulate.
__device__ __forceinline__ void mma_bf16_16x8x16(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2,
                                                 uint32_t a3, uint32_t b0, uint32_t b1,
                                                 const float (&c)[4]) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
        "{%10,%11,%12,%13};"
        : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "f"(c[0]), "f"(c[1]), "f"(c[2]),
          "f"(c[3]));
}

// ---- host side --------------------------------------------------------------
struct ShapeInfo {
    int slices;        // K / 64
    int blocks;        // ceil(K / 256)
    int tail_slices;   // slices in the last block (1..4)
    int words_per_row; // K / 16
    int G;             // K / group
    int spp;           // slices per scale group, capped at 4 (1, 2 or 4)
};

inline bool shape_ok(int M, int N, int K, int group, ShapeInfo *out) {
    if (M < 1 || N < 16 || K < 64 || group < 64) return false;
    if (K % 64 != 0 || N % 16 != 0 || K % group != 0) return false;
    if (!(group == 64 || group == 128 || group % 256 == 0 || group == K)) return false;
    if ((long long)M * N >= (1ll << 40)) return false;
    if (out) {
        out->slices = K / 64;
        out->blocks = (K + 255) / 256;
        out->tail_slices = out->slices - 4 * (out->blocks - 1);
        out->words_per_row = K / 16;
        out->G = K / group;
        out->spp = group == 64 ? 1 : (group == 128 ? 2 : 4);
    }
    return true;
}

inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// cluster_y > 1 launches thread-block clusters of (1, cluster_y, 1) CTAs (grid.y must be a multiple)
template <typename... KArgs, typename... Args>
inline cudaError_t launch_kernel_cluster(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                                         cudaStream_t stream, bool pdl, unsigned cluster_y, Args &&...args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    unsigned n = 0;
    if (pdl) {
        attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[n].val.programmaticStreamSerializationAllowed = 1;
        ++n;
    }
    if (cluster_y > 1) {
        attr[n].id = cudaLaunchAttributeClusterDimension;
        attr[n].val.clusterDim.x = 1;
        attr[n].val.clusterDim.y = cluster_y;
        attr[n].val.clusterDim.z = 1;
        ++n;
    }
    cfg.attrs = attr;
    cfg.numAttrs = n;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

template <typename... KArgs, typename... Args>
inline cudaError_t launch_kernel(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                                 cudaStream_t stream, bool pdl, Args &&...args) {
    return launch_kernel_cluster(kernel, grid, block, smem, stream, pdl, 1u, static_cast<Args &&>(args)...);
}

bool pdl_enabled();
int check_device();  // W2A8_OK or W2A8_ERR_ARCH / W2A8_ERR_CUDA

// ---- per-device state -------------------------------------------------------
// One process may drive several GPUs, and function attributes, the SM count and
// the architecture check belong to a device, not to the process: everything that
// is looked up once is kept per device ordinal.
constexpr int kMaxDevices = 64;
int current_device();   // ordinal of the current device, or -1
int sm_count();         // multiprocessors of the current device (148 on B200), >= 1

// Raise the dynamic shared-memory limit of `kernel` once per device.  `done` is a
// table owned by the caller (one per kernel instantiation); two threads racing on
// the same entry both make the (idempotent) call.
struct PerDeviceFlags {
    std::atomic<bool> done[kMaxDevices];
};
template <typename... KArgs>
inline cudaError_t allow_dynamic_smem(void (*kernel)(KArgs...), PerDeviceFlags &flags, int bytes) {
    const int dev = current_device();
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    if (flags.done[dev].load(std::memory_order_acquire)) return cudaSuccess;
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (e == cudaSuccess) flags.done[dev].store(true, std::memory_order_release);
    return e;
}

}  // namespace w2a8
