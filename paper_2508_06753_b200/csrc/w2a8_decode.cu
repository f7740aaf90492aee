// Memory-bound W2A8 kernel for small token counts (decode): streams the packed
// 2-bit weights once, unpacks them in registers and feeds int8 tensor-core
// MMAs (mma.sync m16n8k32) whose A operand is a 16-channel x 32-k weight tile
// and whose B operand is 32 k x 8 tokens.  The up-convert-and-compute idea is
// that of Sec. II-C, the K-splitting that of Sec. II-D; the thread/tile mapping
// and the asynchronous staging are specific to sm_100a.
//
// Work split: a CTA of 4 warps owns 64 output channels (one 16-channel tile per
// warp) and one chunk of up to 8 consecutive 256-k blocks; grid.y walks the
// chunks (split-K), grid.z walks 8*MT-token slabs.  A "cell" is one tile x one
// block: 1 KB of packed weights + its scales.
//
// Pipeline: every lane posts the cp.async copies of ALL its cells into a
// lane-private shared-memory FIFO before it waits for the previous kernel of
// the stream (weights and scales are frozen, only activations depend on it),
// so the whole chunk is in flight at once and, under programmatic dependent
// launch, while the previous kernel is still draining.  The activations of the
// chunk are then staged once per CTA and shared by its four warps.
//
// In the W2P layout one 128-bit unit per lane and channel holds word t of each
// of the four 64-k slices of a block -- exactly what the four lanes of an MMA
// quad must supply so that every MMA sums k of a single scale group.
#include "w2a8_common.cuh"

namespace w2a8 {

constexpr int kCellsMax = 8;                   // FIFO depth = cells per chunk
constexpr int kDecodeWarps = 4;
constexpr int kDecodeThreads = kDecodeWarps * 32;
constexpr int kTileGroupRows = 16 * kDecodeWarps;
constexpr int kFifoWBytes = kCellsMax * 2 * 32 * 16;   // per warp: weights
constexpr int kFifoSBytes = kCellsMax * 2 * 8 * 16;    // per warp: scales (<= 4 floats / row)
constexpr int kActPad = 64;                    // row stride = chunk bytes + 64: conflict-free LDS.128

struct DecodeParams {
    const int8_t *a;
    const float *a_scale;
    const uint32_t *packed;
    const float *w_scale;
    float *y;
    int32_t *partials;
    float *ws;            // [chunks][M][N] partial outputs (chunks > 1)
    unsigned *counters;   // [grid.z][N/16] arrival counters (chunks > 1)
    int M, N, K, G, group;
    int blocks, tail_slices, words_per_row;
    int chunks, cells_per_chunk;
    int act_stride;       // bytes per staged token row
};

__device__ __forceinline__ uint32_t smem_u32(const void *p) {
    return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async4(uint32_t dst, const void *src) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

template <int MT, int SPP, bool PARTIALS>
__global__ void __launch_bounds__(kDecodeThreads)
w2a8_decode_kernel(const DecodeParams p) {
    extern __shared__ __align__(128) unsigned char smem[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int gq = lane >> 2, t = lane & 3;
    const int tile = blockIdx.x * kDecodeWarps + warp;
    const bool tile_ok = tile * 16 < p.N;
    const int n0 = tile * 16;
    const int chunk = blockIdx.y;
    const int kb0 = chunk * p.cells_per_chunk;
    const int ncells = min(p.cells_per_chunk, p.blocks - kb0);
    const int m0 = blockIdx.z * (8 * MT);
    const int mrows = min(8 * MT, p.M - m0);

    unsigned char *fifo_w = smem + warp * (kFifoWBytes + kFifoSBytes);
    unsigned char *fifo_s = fifo_w + kFifoWBytes;
    unsigned char *acts = smem + kDecodeWarps * (kFifoWBytes + kFifoSBytes);
    constexpr int SPB = 4 / SPP;               // scales per block and channel

    // ---- post every cell of the chunk (independent of the previous kernel) ----
#pragma unroll
    for (int c = 0; c < kCellsMax; ++c) {
        if (tile_ok && c < ncells) {
            const int kb = kb0 + c;
            const int R = (kb == p.blocks - 1) ? p.tail_slices : 4;
#pragma unroll
            for (int r = 0; r < 2; ++r) {
                const size_t row = (size_t)(n0 + gq + 8 * r);
                const uint32_t *wp = p.packed + row * p.words_per_row + 16 * kb;
                unsigned char *dst = fifo_w + ((c * 2 + r) * 32 + lane) * 16;
                if (R == 4) {
                    cp_async16(smem_u32(dst), wp + 4 * t);
                } else {   // trailing block with fewer slices: words t*R .. t*R+R-1
                    uint4 v = make_uint4(0u, 0u, 0u, 0u);
                    v.x = __ldg(wp + t * R);
                    if (R > 1) v.y = __ldg(wp + t * R + 1);
                    if (R > 2) v.z = __ldg(wp + t * R + 2);
                    *reinterpret_cast<uint4 *>(dst) = v;
                }
                // scales of this block: lane t brings scale t of channel row (the parity
                // export has no scales: w_scale is null there)
                const int nsc = (SPP == 4) ? 1 : (R + SPP - 1) / SPP;
                const float *sp = (SPP == 4)
                    ? p.w_scale + row * p.G + (int)(((long long)kb * kBlockK) / p.group)
                    : p.w_scale + row * p.G + SPB * kb;
                if (!PARTIALS && t < nsc) cp_async4(smem_u32(fifo_s + ((c * 2 + r) * 8 + gq) * 16 + 4 * t), sp + t);
            }
        }
        cp_async_commit();
    }
    pdl_launch_dependents();
    pdl_wait();

    // ---- stage the activations of this chunk: [mrows][ncells * 256 (+pad)] ----
    {
        const int row_units = ncells * (kBlockK / 16);
        const int klen = min(ncells * kBlockK, p.K - kb0 * kBlockK);   // trailing block may be short
        for (int u = threadIdx.x; u < mrows * row_units; u += kDecodeThreads) {
            const int r = u / row_units, cu = u % row_units;
            uint4 v = make_uint4(0u, 0u, 0u, 0u);
            if (cu * 16 < klen)
                v = *reinterpret_cast<const uint4 *>(p.a + (size_t)(m0 + r) * p.K + (size_t)kb0 * kBlockK + cu * 16);
            *reinterpret_cast<uint4 *>(acts + r * p.act_stride + cu * 16) = v;
        }
    }
    __syncthreads();
    if (!tile_ok) return;

    float acc[MT][4];
    int D[MT][4];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int i = 0; i < 4; ++i) { acc[mt][i] = 0.f; D[mt][i] = kMagicInt; }

#pragma unroll
    for (int c = 0; c < kCellsMax; ++c) {
        if (c < ncells) {
            switch (c) {   // groups are committed in cell order
                case 0: cp_async_wait<kCellsMax - 1>(); break;
                case 1: cp_async_wait<kCellsMax - 2>(); break;
                case 2: cp_async_wait<kCellsMax - 3>(); break;
                case 3: cp_async_wait<kCellsMax - 4>(); break;
                case 4: cp_async_wait<kCellsMax - 5>(); break;
                case 5: cp_async_wait<kCellsMax - 6>(); break;
                case 6: cp_async_wait<kCellsMax - 7>(); break;
                default: cp_async_wait<0>(); break;
            }
            __syncwarp();   // scales were brought by the other lanes of the quad
            const int kb = kb0 + c;
            const int R = (kb == p.blocks - 1) ? p.tail_slices : 4;
            const uint4 wa = *reinterpret_cast<const uint4 *>(fifo_w + ((c * 2 + 0) * 32 + lane) * 16);
            const uint4 wb = *reinterpret_cast<const uint4 *>(fifo_w + ((c * 2 + 1) * 32 + lane) * 16);
            const float4 sa = *reinterpret_cast<const float4 *>(fifo_s + ((c * 2 + 0) * 8 + gq) * 16);
            const float4 sb = *reinterpret_cast<const float4 *>(fifo_s + ((c * 2 + 1) * 8 + gq) * 16);
            const uint32_t w0s[4] = {wa.x, wa.y, wa.z, wa.w};
            const uint32_t w1s[4] = {wb.x, wb.y, wb.z, wb.w};
            const float s0s[4] = {sa.x, sa.y, sa.z, sa.w};
            const float s1s[4] = {sb.x, sb.y, sb.z, sb.w};
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
                        uint4 b = make_uint4(0u, 0u, 0u, 0u);
                        if (8 * mt + gq < mrows)
                            b = *reinterpret_cast<const uint4 *>(acts + (8 * mt + gq) * p.act_stride +
                                                                 c * kBlockK + s * kSliceK + t * 16);
                        if (first) {
#pragma unroll
                            for (int i = 0; i < 4; ++i) D[mt][i] = kMagicInt;
                        }
                        mma_s8_16x8x32(D[mt], a0, a1, a2, a3, b.x, b.y);
                        mma_s8_16x8x32(D[mt], a4, a5, a6, a7, b.z, b.w);
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

    if constexpr (!PARTIALS) {
        // lane (gq, t) holds channels n0+gq, n0+gq+8 for tokens 2t, 2t+1 of each slab
        if (p.chunks == 1) {
#pragma unroll
            for (int mt = 0; mt < MT; ++mt)
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int mm = m0 + 8 * mt + 2 * t + (i & 1);
                    const int nn = n0 + gq + 8 * (i >> 1);
                    if (mm < p.M)
                        p.y[(size_t)mm * p.N + nn] = acc[mt][i] * (p.a_scale[mm] * (1.0f / kCodeGain));
                }
            return;
        }
        // split-K: park the partial outputs; the last warp to arrive for this tile
        // and slab sums all chunks in chunk order (repeatable to the bit).
        const size_t MN = (size_t)p.M * p.N;
#pragma unroll
        for (int mt = 0; mt < MT; ++mt)
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int mm = m0 + 8 * mt + 2 * t + (i & 1);
                const int nn = n0 + gq + 8 * (i >> 1);
                if (mm < p.M) __stcg(p.ws + chunk * MN + (size_t)mm * p.N + nn, acc[mt][i]);
            }
        __threadfence();
        __syncwarp();
        unsigned *counter = p.counters + (size_t)blockIdx.z * (p.N / 16) + tile;
        unsigned ticket = 0;
        if (lane == 0) ticket = atomicAdd(counter, 1u);
        ticket = __shfl_sync(0xFFFFFFFFu, ticket, 0);
        if (ticket != (unsigned)p.chunks - 1u) return;
        __threadfence();
#pragma unroll
        for (int mt = 0; mt < MT; ++mt)
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int mm = m0 + 8 * mt + 2 * t + (i & 1);
                const int nn = n0 + gq + 8 * (i >> 1);
                if (mm < p.M) {
                    float v = 0.f;
                    for (int ch = 0; ch < p.chunks; ++ch) v += __ldcg(p.ws + ch * MN + (size_t)mm * p.N + nn);
                    p.y[(size_t)mm * p.N + nn] = v * (p.a_scale[mm] * (1.0f / kCodeGain));
                }
            }
        if (lane == 0) *counter = 0u;   // leave the workspace reusable
    }
}

// ---- host side -----------------------------------------------------------------
int env_int(const char *name, int dflt);

// Number of K-chunks (grid.y).  At least ceil(blocks / 8) because a chunk holds at
// most 8 blocks; more when the grid would otherwise leave SMs idle.
int decode_chunks(int M, int N, const ShapeInfo &si) {
    const int min_chunks = (si.blocks + kCellsMax - 1) / kCellsMax;
    const int forced = env_int("W2A8_SPLITS", 0);
    int c;
    if (forced > 0) {
        c = forced;
    } else {
        const int groups = (N + kTileGroupRows - 1) / kTileGroupRows;
        const int slabs = M > 32 ? (M + 31) / 32 : 1;
        c = (296 + groups * slabs - 1) / (groups * slabs);
    }
    if (c < min_chunks) c = min_chunks;
    if (c > si.blocks) c = si.blocks;
    // equalise: the smallest chunk count that gives the same cells per chunk
    const int cells = (si.blocks + c - 1) / c;
    return (si.blocks + cells - 1) / cells;
}

static inline int decode_mt(int M) { return M > 32 ? 4 : (M + 7) / 8; }

size_t decode_workspace_bytes(int M, int N, const ShapeInfo &si) {
    const int mt = decode_mt(M);
    const int slabs = (M + 8 * mt - 1) / (8 * mt);
    size_t counters = ((size_t)4 * (N / 16) * slabs + 255) / 256 * 256;
    // room for one partial output per block of K: covers every chunk count
    size_t part = (size_t)si.blocks * M * N * sizeof(float);
    const int chunks = decode_chunks(M, N, si);
    if (env_int("W2A8_SPLITS", 0) <= 0) part = (size_t)(chunks > 1 ? chunks : 0) * M * N * sizeof(float);
    return counters + part;
}

template <int MT, int SPP, bool PARTIALS>
static cudaError_t launch_decode_inst(const DecodeParams &p, dim3 grid, size_t smem, cudaStream_t st) {
    static bool configured = false;   // one attribute call per instantiation and process
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(w2a8_decode_kernel<MT, SPP, PARTIALS>,
                                             cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
        if (e != cudaSuccess) return e;
        configured = true;
    }
    return launch_kernel(w2a8_decode_kernel<MT, SPP, PARTIALS>, grid, dim3(kDecodeThreads), smem, st,
                         pdl_enabled(), p);
}

template <int MT, int SPP>
static cudaError_t launch_decode_mt(const DecodeParams &p, bool want_partials, dim3 grid, size_t smem,
                                    cudaStream_t st) {
    return want_partials ? launch_decode_inst<MT, SPP, true>(p, grid, smem, st)
                         : launch_decode_inst<MT, SPP, false>(p, grid, smem, st);
}

template <int SPP>
static cudaError_t launch_decode_spp(DecodeParams &p, bool want_partials, cudaStream_t st) {
    const int mt = decode_mt(p.M);
    const int mrows = p.M < 8 * mt ? p.M : 8 * mt;
    p.act_stride = p.cells_per_chunk * kBlockK + kActPad;
    const size_t smem = (size_t)kDecodeWarps * (kFifoWBytes + kFifoSBytes) + (size_t)mrows * p.act_stride;
    dim3 grid((p.N + kTileGroupRows - 1) / kTileGroupRows, p.chunks, (p.M + 8 * mt - 1) / (8 * mt));
    switch (mt) {
        case 1: return launch_decode_mt<1, SPP>(p, want_partials, grid, smem, st);
        case 2: return launch_decode_mt<2, SPP>(p, want_partials, grid, smem, st);
        case 3: return launch_decode_mt<3, SPP>(p, want_partials, grid, smem, st);
        default: return launch_decode_mt<4, SPP>(p, want_partials, grid, smem, st);
    }
}

// Enqueue the decode kernel.  `partials` != nullptr selects the parity export.
int launch_decode(const int8_t *a, const float *a_scale, const uint32_t *packed,
                  const float *w_scale, float *y, int32_t *partials, int M, int N, int K,
                  int group, const ShapeInfo &si, void *workspace, cudaStream_t st) {
    DecodeParams p;
    p.a = a; p.a_scale = a_scale; p.packed = packed; p.w_scale = w_scale;
    p.y = y; p.partials = partials;
    p.M = M; p.N = N; p.K = K; p.G = si.G; p.group = group;
    p.blocks = si.blocks; p.tail_slices = si.tail_slices; p.words_per_row = si.words_per_row;
    p.chunks = decode_chunks(M, N, si);
    p.cells_per_chunk = (si.blocks + p.chunks - 1) / p.chunks;
    const int mt = decode_mt(M);
    const int slabs = (M + 8 * mt - 1) / (8 * mt);
    size_t counters = ((size_t)4 * (N / 16) * slabs + 255) / 256 * 256;
    p.counters = reinterpret_cast<unsigned *>(workspace);
    p.ws = reinterpret_cast<float *>(reinterpret_cast<char *>(workspace) + counters);
    if (partials) {
        // several warps add their share of a large group: start from zero
        if (cudaMemsetAsync(partials, 0, (size_t)M * N * si.G * sizeof(int32_t), st) != cudaSuccess)
            return W2A8_ERR_CUDA;
    }
    cudaError_t e = si.spp == 1 ? launch_decode_spp<1>(p, partials != nullptr, st)
                  : si.spp == 2 ? launch_decode_spp<2>(p, partials != nullptr, st)
                                : launch_decode_spp<4>(p, partials != nullptr, st);
    return e == cudaSuccess ? W2A8_OK : W2A8_ERR_CUDA;
}

}  // namespace w2a8
