// Memory-bound W2A8 kernel for small token counts (decode): streams the packed
// 2-bit weights once, unpacks them in registers and feeds int8 tensor-core
// MMAs (mma.sync m16n8k32) whose A operand is a 16-channel x 32-k weight tile
// and whose B operand is 32 k x 8 tokens.  The up-convert-and-compute idea is
// that of Sec. II-C; the thread/tile mapping is specific to sm_100a.
//
// Work split: a CTA owns 16 output channels; its 8 warps take interleaved
// 256-k blocks of the contraction (and CTAs along grid.y take interleaved
// sets of blocks: split-K, Sec. II-D).  In the W2P layout one 128-bit load per
// lane and channel brings word t of each of the four 64-k slices of a block,
// which is exactly what the four lanes of an MMA quad must hold so that every
// MMA sums k of a single scale group.
#include "w2a8_common.cuh"

namespace w2a8 {

struct DecodeParams {
    const int8_t *a;
    const float *a_scale;
    const uint32_t *packed;
    const float *w_scale;
    float *y;
    int32_t *partials;
    float *ws;            // [splits][M][N] partial outputs (splits > 1)
    unsigned *counters;   // [grid.z][N/16] arrival counters (splits > 1)
    int M, N, K, G, group;
    int blocks, tail_slices, words_per_row;
    int splits;
    int vec_ok;           // K % 256 == 0: scale rows are 16-byte aligned
};

constexpr int kDecodeWarps = 8;
constexpr int kDecodeThreads = kDecodeWarps * 32;

__device__ __forceinline__ uint4 ld_stream_v4(const uint32_t *p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

template <int SPP>
struct Cell {
    uint32_t w[2][4];                 // [channel g / g+8][slice]
    float sc[2][4 / SPP];             // [channel][scale group inside the block]
};

template <int SPP>
__device__ __forceinline__ void load_cell(const DecodeParams &p, Cell<SPP> &c, int n0, int gq,
                                          int t, int kb) {
    const int R = (kb == p.blocks - 1) ? p.tail_slices : 4;
#pragma unroll
    for (int r = 0; r < 2; ++r) {
        const size_t row = (size_t)(n0 + gq + 8 * r);
        const uint32_t *wp = p.packed + row * p.words_per_row + 16 * kb;
        if (R == 4) {
            uint4 v = ld_stream_v4(wp + 4 * t);
            c.w[r][0] = v.x; c.w[r][1] = v.y; c.w[r][2] = v.z; c.w[r][3] = v.w;
        } else {
#pragma unroll
            for (int s = 0; s < 4; ++s) c.w[r][s] = (s < R) ? __ldg(wp + t * R + s) : 0u;
        }
        if constexpr (SPP == 1) {
            const float *sp = p.w_scale + row * p.G + 4 * kb;
            if (R == 4 && p.vec_ok) {
                float4 v = __ldg(reinterpret_cast<const float4 *>(sp));
                c.sc[r][0] = v.x; c.sc[r][1] = v.y; c.sc[r][2] = v.z; c.sc[r][3] = v.w;
            } else {
#pragma unroll
                for (int s = 0; s < 4; ++s) c.sc[r][s] = (s < R) ? __ldg(sp + s) : 0.f;
            }
        } else if constexpr (SPP == 2) {
            const float *sp = p.w_scale + row * p.G + 2 * kb;
            if (R == 4 && p.vec_ok) {
                float2 v = __ldg(reinterpret_cast<const float2 *>(sp));
                c.sc[r][0] = v.x; c.sc[r][1] = v.y;
            } else {
#pragma unroll
                for (int s = 0; s < 2; ++s) c.sc[r][s] = (2 * s < R) ? __ldg(sp + s) : 0.f;
            }
        } else {
            c.sc[r][0] = __ldg(p.w_scale + row * p.G + (int)(((long long)kb * kBlockK) / p.group));
        }
    }
}

template <int MT, int SPP, bool PARTIALS>
__global__ void __launch_bounds__(kDecodeThreads)
w2a8_decode_kernel(const DecodeParams p) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int gq = lane >> 2, t = lane & 3;
    const int n0 = blockIdx.x * 16;
    const int split = blockIdx.y;
    const int m0 = blockIdx.z * (8 * MT);
    const int stride = kDecodeWarps * p.splits;

    float acc[MT][4];
    int D[MT][4];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int i = 0; i < 4; ++i) { acc[mt][i] = 0.f; D[mt][i] = kMagicInt; }

    // Weights and their scales never depend on the previous kernel: fetch the
    // first block before waiting for it, and let the next kernel start.
    int kb = split * kDecodeWarps + warp;
    Cell<SPP> cur, nxt;
    if (kb < p.blocks) load_cell<SPP>(p, cur, n0, gq, t, kb);
    pdl_launch_dependents();
    pdl_wait();

    while (kb < p.blocks) {
        const int kn = kb + stride;
        if (kn < p.blocks) load_cell<SPP>(p, nxt, n0, gq, t, kn);
        const int R = (kb == p.blocks - 1) ? p.tail_slices : 4;
#pragma unroll
        for (int s = 0; s < 4; ++s) {
            if (s < R) {
                const uint32_t w0 = cur.w[0][s], w1 = cur.w[1][s];
                const uint32_t a0 = lane_codes(w0, 0), a1 = lane_codes(w1, 0);
                const uint32_t a2 = lane_codes(w0, 1), a3 = lane_codes(w1, 1);
                const uint32_t a4 = lane_codes(w0, 2), a5 = lane_codes(w1, 2);
                const uint32_t a6 = lane_codes(w0, 3), a7 = lane_codes(w1, 3);
                const bool first = (s % SPP) == 0;
                const bool last = ((s + 1) % SPP) == 0 || s == R - 1;
#pragma unroll
                for (int mt = 0; mt < MT; ++mt) {
                    const int m = m0 + 8 * mt + gq;
                    uint4 b = make_uint4(0u, 0u, 0u, 0u);
                    if (m < p.M)
                        b = *reinterpret_cast<const uint4 *>(p.a + (size_t)m * p.K + kBlockK * kb +
                                                             kSliceK * s + 16 * t);
                    if (first) {
#pragma unroll
                        for (int i = 0; i < 4; ++i) D[mt][i] = kMagicInt;
                    }
                    mma_s8_16x8x32(D[mt], a0, a1, a2, a3, b.x, b.y);
                    mma_s8_16x8x32(D[mt], a4, a5, a6, a7, b.z, b.w);
                    if (last) {
                        if (PARTIALS) {
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
                            const float s0 = cur.sc[0][s / SPP];
                            const float s1 = cur.sc[1][s / SPP];
                            acc[mt][0] = fmaf(s0, __int_as_float(D[mt][0]) - kMagicFloat, acc[mt][0]);
                            acc[mt][1] = fmaf(s0, __int_as_float(D[mt][1]) - kMagicFloat, acc[mt][1]);
                            acc[mt][2] = fmaf(s1, __int_as_float(D[mt][2]) - kMagicFloat, acc[mt][2]);
                            acc[mt][3] = fmaf(s1, __int_as_float(D[mt][3]) - kMagicFloat, acc[mt][3]);
                        }
                    }
                }
            }
        }
        cur = nxt;
        kb = kn;
    }
    if constexpr (!PARTIALS) {
    // ---- reduce the 8 warps of the CTA in a fixed order ---------------------
    __shared__ float red[kDecodeWarps][MT * 4][32];
    __shared__ int is_last;
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int i = 0; i < 4; ++i) red[warp][mt * 4 + i][lane] = acc[mt][i];
    __syncthreads();

    const size_t MN = (size_t)p.M * p.N;
    for (int e = threadIdx.x; e < MT * 128; e += kDecodeThreads) {
        const int el = e & 31, ei = e >> 5;          // lane, (mt, i)
        const int mt = ei >> 2, i = ei & 3;
        float v = 0.f;
#pragma unroll
        for (int w = 0; w < kDecodeWarps; ++w) v += red[w][ei][el];
        const int mm = m0 + 8 * mt + 2 * (el & 3) + (i & 1);
        const int nn = n0 + (el >> 2) + 8 * (i >> 1);
        if (mm < p.M) {
            if (p.splits == 1)
                p.y[(size_t)mm * p.N + nn] = v * (p.a_scale[mm] * (1.0f / kCodeGain));
            else
                p.ws[split * MN + (size_t)mm * p.N + nn] = v;
        }
    }
    if (p.splits == 1) return;

    // ---- split-K: the last CTA to arrive sums the partial outputs in order ---
    __threadfence();
    __syncthreads();
    unsigned *counter = p.counters + blockIdx.z * gridDim.x + blockIdx.x;
    if (threadIdx.x == 0) is_last = (atomicAdd(counter, 1u) == (unsigned)p.splits - 1u);
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    for (int e = threadIdx.x; e < MT * 128; e += kDecodeThreads) {
        const int el = e & 31, ei = e >> 5;
        const int mt = ei >> 2, i = ei & 3;
        const int mm = m0 + 8 * mt + 2 * (el & 3) + (i & 1);
        const int nn = n0 + (el >> 2) + 8 * (i >> 1);
        if (mm < p.M) {
            float v = 0.f;
            for (int sp = 0; sp < p.splits; ++sp) v += __ldcg(p.ws + sp * MN + (size_t)mm * p.N + nn);
            p.y[(size_t)mm * p.N + nn] = v * (p.a_scale[mm] * (1.0f / kCodeGain));
        }
    }
    if (threadIdx.x == 0) *counter = 0u;   // leave the workspace reusable
    }  // !PARTIALS
}

// ---- host side -----------------------------------------------------------------
int env_int(const char *name, int dflt);

int decode_splits(int M, int N, const ShapeInfo &si) {
    if (M > 32) return 1;
    const int forced = env_int("W2A8_SPLITS", 0);
    const int max_splits = (si.blocks + kDecodeWarps - 1) / kDecodeWarps;
    int s = forced > 0 ? forced : 592 / (N / 16);
    if (s < 1) s = 1;
    if (s > max_splits) s = max_splits;
    return s;
}

size_t decode_workspace_bytes(int M, int N, const ShapeInfo &si) {
    const int zchunks = (M + 31) / 32;
    size_t counters = ((size_t)4 * (N / 16) * zchunks + 255) / 256 * 256;
    const int splits = decode_splits(M, N, si);
    size_t part = splits > 1 ? (size_t)splits * M * N * sizeof(float) : 0;
    return counters + part;
}

template <int MT, int SPP>
static cudaError_t launch_decode_mt(const DecodeParams &p, bool want_partials, dim3 grid,
                                    cudaStream_t st) {
    if (want_partials)
        return launch_kernel(w2a8_decode_kernel<MT, SPP, true>, grid, dim3(kDecodeThreads), 0, st,
                             pdl_enabled(), p);
    return launch_kernel(w2a8_decode_kernel<MT, SPP, false>, grid, dim3(kDecodeThreads), 0, st,
                         pdl_enabled(), p);
}

template <int SPP>
static cudaError_t launch_decode_spp(const DecodeParams &p, bool want_partials, cudaStream_t st) {
    const int mt = p.M > 32 ? 4 : (p.M + 7) / 8;
    dim3 grid(p.N / 16, p.splits, (p.M + 8 * mt - 1) / (8 * mt));
    switch (mt) {
        case 1: return launch_decode_mt<1, SPP>(p, want_partials, grid, st);
        case 2: return launch_decode_mt<2, SPP>(p, want_partials, grid, st);
        case 3: return launch_decode_mt<3, SPP>(p, want_partials, grid, st);
        default: return launch_decode_mt<4, SPP>(p, want_partials, grid, st);
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
    p.splits = partials ? 1 : decode_splits(M, N, si);
    p.vec_ok = (K % 256 == 0) ? 1 : 0;
    const int zchunks = (M + 31) / 32;
    size_t counters = ((size_t)4 * (N / 16) * zchunks + 255) / 256 * 256;
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
