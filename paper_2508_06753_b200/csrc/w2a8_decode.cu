// Memory-bound W2A8 kernel for small token counts (decode): streams the packed
// 2-bit weights once, unpacks them in registers and feeds int8 tensor-core
// MMAs (mma.sync m16n8k32) whose A operand is a 16-channel x 32-k weight tile
// and whose B operand is 32 k x 8 tokens.  The up-convert-and-compute idea is
// that of Sec. II-C, the K-splitting that of Sec. II-D; the staging, the
// thread/tile mapping and the launch overlap are specific to sm_100a.
//
// Work split.  A "cell" is one 16-channel tile x one 256-k block: 1 KB of packed
// weights plus its scales.  A CTA of 4 warps owns TG tiles and one chunk of the
// contraction; its warps are arranged TG tiles x KS = 4 / TG K-lanes, and the
// K-lanes take interleaved blocks of the chunk.  The K-lanes of a tile are
// summed through shared memory in a fixed order; chunks (grid.y, only used when
// the shape would otherwise leave SMs idle or the data would not fit in shared
// memory) are summed through the workspace by the last CTA to arrive, also in a
// fixed order.  grid.z walks 8*MT-token slabs.
//
// Pipeline.  A warp works in rounds of up to four cells.  Each lane requests the
// weights of a whole round with 128-bit loads into registers; the first half of
// the first round is requested before the kernel waits for the previous kernel
// of the stream (weights and scales are frozen; only activations depend on it),
// so under programmatic dependent launch the weight stream of this kernel
// overlaps the tail of the previous one.  The activations of the chunk are
// requested right behind that first half (so that they do not queue behind the
// whole weight stream), then the second half.  Scales and activations are
// staged once per CTA in shared memory by per-thread asynchronous copies.
//
// One 128-bit unit per lane and channel holds word t of each of the four 64-k
// slices of a block -- exactly what the four lanes of an MMA quad must supply
// so that every MMA sums k of a single scale group.
#include "w2a8_common.cuh"

namespace w2a8 {

constexpr int kDecodeWarps = 4;
constexpr int kDecodeThreads = kDecodeWarps * 32;
constexpr int kActPad = 64;                    // activation row stride = chunk bytes + 64
constexpr int kSmemBudget = 64 * 1024;         // per CTA: scales + activations
#ifndef W2A8_MINB
#define W2A8_MINB(MT) ((MT) == 1 ? 7 : 3)
#endif
constexpr int kRound = 4;                      // cells a lane keeps in flight (ring depth, power of 2)

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
    int tiles_per_warp;   // tiles a warp walks when it owns whole tiles (TG == 4)
    int s_stride;         // bytes per staged scale row
    int act_stride;       // bytes per staged token row
    int s_vec;            // scale rows can be copied in 16-byte units
    int off_a;            // byte offset of the activation area in shared memory
    int off_ring;         // byte offset of the per-lane weight rings
};

// ---- PTX wrappers ------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void *p) {
    return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ uint4 ld_stream_v4(const uint32_t *p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}
// per-thread asynchronous copies (activations, and scales that bulk copies cannot take)
__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async4(uint32_t dst, const void *src) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait_group() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// Optional timeline trace (build with -DW2A8_TRACE): every warp records the
// global timer at a few points of the kernel into a caller-provided buffer.
#ifdef W2A8_TRACE
__device__ unsigned long long *g_trace = nullptr;
__device__ __forceinline__ unsigned long long global_ns() {
    unsigned long long v;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(v));
    return v;
}
#define W2A8_TRACE_POINT(i)                                                                      \
    do {                                                                                         \
        if (g_trace && (threadIdx.x & 31) == 0)                                                  \
            g_trace[((((size_t)blockIdx.z * gridDim.y + blockIdx.y) * gridDim.x + blockIdx.x) *  \
                         kDecodeWarps + (threadIdx.x >> 5)) * 8 + (i)] = global_ns();            \
    } while (0)
#else
#define W2A8_TRACE_POINT(i) do { } while (0)
#endif

// One cell: 4 slices x (unpack, 2 MMAs per token slab, promotion at group ends).
// w0s/w1s: this lane's four words (one per slice) of channels n0+gq and n0+gq+8;
// srow0/srow1: staged scale rows of the same channels.
template <int MT, int SPP, bool ONE, bool PARTIALS, bool FULL>
__device__ __forceinline__ void compute_cell(const DecodeParams &p, const uint32_t (&w0s)[4],
                                             const uint32_t (&w1s)[4], const unsigned char *srow0,
                                             const unsigned char *srow1,
                                             const unsigned char *const (&brow)[MT], int kl,
                                             int kb, int n0, int m0, int gq, int t,
                                             float (&acc)[MT][4]) {
    // FULL: the block has all four slices (always, except possibly the last block of K)
    const int R = FULL ? 4 : p.tail_slices;
    const int magic[4] = {kMagicInt, kMagicInt, kMagicInt, kMagicInt};
    int D[MT][4];   // int32 accumulators of the current group; a group never outlives a cell
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int i = 0; i < 4; ++i) D[mt][i] = kMagicInt;
    float s0s[4 / SPP], s1s[4 / SPP];
    if constexpr (!PARTIALS) {
        if constexpr (SPP == 4) {
            const int gi = (int)(((long long)kb * kBlockK) / p.group);
            s0s[0] = reinterpret_cast<const float *>(srow0)[gi];
            s1s[0] = reinterpret_cast<const float *>(srow1)[gi];
        } else if constexpr (SPP == 2) {   // staged rows are 16-byte aligned: 8-byte loads are fine
            const float2 v0 = reinterpret_cast<const float2 *>(srow0)[kl];
            const float2 v1 = reinterpret_cast<const float2 *>(srow1)[kl];
            s0s[0] = v0.x; s0s[1] = v0.y; s1s[0] = v1.x; s1s[1] = v1.y;
        } else {
            const float4 v0 = reinterpret_cast<const float4 *>(srow0)[kl];
            const float4 v1 = reinterpret_cast<const float4 *>(srow1)[kl];
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
                const uint4 b = *reinterpret_cast<const uint4 *>(brow[mt] + kl * kBlockK + s * kSliceK);
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
                        acc[mt][0] = fmaf(s0, __int_as_float(D[mt][0]) - kMagicFloat, acc[mt][0]);
                        acc[mt][2] = fmaf(s1, __int_as_float(D[mt][2]) - kMagicFloat, acc[mt][2]);
                        if constexpr (!ONE) {
                            acc[mt][1] = fmaf(s0, __int_as_float(D[mt][1]) - kMagicFloat, acc[mt][1]);
                            acc[mt][3] = fmaf(s1, __int_as_float(D[mt][3]) - kMagicFloat, acc[mt][3]);
                        }
                    }
                }
            }
        }
    }
}

// MT: 8-token slabs per CTA; SPP: 64-k slices per scale group (capped at 4);
// TG: tiles the four warps of a CTA work on side by side (K-lanes per tile = 4 / TG);
// RING: cells a lane keeps in flight; ONE: a single token (half of each accumulator
// quad is dead and is not promoted).
//
// With TG == 4 every warp owns whole tiles: it walks p.tiles_per_warp tiles of the
// chunk one after the other (tile = (blockIdx.x * tiles_per_warp + i) * 4 + warp),
// re-using the activations the CTA staged once, and finishes each tile on its own
// (no CTA barrier after the staging).  With TG < 4 the K-lanes of a tile are summed
// through shared memory and tiles_per_warp is 1.
template <int MT, int SPP, int TG, int RING, bool ONE, bool PARTIALS>
__global__ void __launch_bounds__(kDecodeThreads, W2A8_MINB(MT))
w2a8_decode_kernel(const DecodeParams p) {
    constexpr int KS = kDecodeWarps / TG;
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ int is_last;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int gq = lane >> 2, t = lane & 3;
    const int tl = warp % TG, ks = warp / TG;
    const int TL = (KS == 1) ? p.tiles_per_warp : 1;
    const int ntiles = p.N / 16;
    const int tile0 = blockIdx.x * TL * TG;       // first tile of this CTA
    const int chunk = blockIdx.y;
    const int kb_begin = chunk * p.blocks_per_chunk;
    const int kb_end = min(kb_begin + p.blocks_per_chunk, p.blocks);
    const int nb = kb_end - kb_begin;
    const int m0 = blockIdx.z * (8 * MT);
    const int mrows = min(8 * MT, p.M - m0);
    unsigned char *sm_s = smem;                 // [tiles of the CTA * 16][s_stride]
    unsigned char *acts = smem + p.off_a;       // [mrows + 1][act_stride]
    W2A8_TRACE_POINT(0);

    constexpr int SPB = 4 / SPP;                                  // scales per block and channel
    const int sc_begin = (SPP == 4) ? 0 : SPB * kb_begin;
    const int sc_end = (SPP == 4) ? p.G : min(SPB * kb_end, p.G);
    const int tiles_here = min(TG * TL, ntiles - tile0);
    const int rows_here = tiles_here * 16;

    // This warp's cells, flattened over its tiles: cell c = (tile i = c / nbw, block
    // kl = ks + (c % nbw) * KS); tiles beyond N are cut off.
    const int nbw = (nb - ks + KS - 1) / KS;                       // cells per tile for this K-lane
    int my_tiles = 0;
    for (int i = 0; i < TL; ++i)
        if (tile0 + i * TG + tl < ntiles) my_tiles = i + 1;
    const int my_cells = my_tiles * nbw;

    // Lane-private ring of RING cells in shared memory: slot j of this lane holds the two
    // 16-byte units (channels gq and gq+8) of one cell.  Only this lane writes and reads its
    // slots, so cp.async.wait_group alone orders them (no warp barrier).
    unsigned char *ring = smem + p.off_ring + warp * (RING * 2 * 32 * 16) + lane * 16;
    auto post_cell = [&](int slot, int c) {
        const int ti = c / nbw, kl = ks + (c - ti * nbw) * KS;
        const int kb = kb_begin + kl;
        const int n0 = (tile0 + ti * TG + tl) * 16;
        const int R = (kb == p.blocks - 1) ? p.tail_slices : 4;
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            const uint32_t *wp = p.packed + (size_t)(n0 + gq + 8 * r) * p.words_per_row + 16 * kb;
            unsigned char *dst = ring + (slot * 2 + r) * (32 * 16);
            if (R == 4) {
                cp_async16(smem_u32(dst), wp + 4 * t);
            } else {   // trailing block with fewer slices: words t*R .. t*R+R-1
                uint4 v = make_uint4(0u, 0u, 0u, 0u);
                v.x = __ldg(wp + t * R);
                if (R > 1) v.y = __ldg(wp + t * R + 1);
                if (R > 2) v.z = __ldg(wp + t * R + 2);
                *reinterpret_cast<uint4 *>(dst) = v;
            }
        }
    };

    // ---- first group: scales of the CTA's tiles for the whole chunk + cell 0; then one
    //      group per cell up to half the ring (all independent of the previous kernel) ----
    if constexpr (!PARTIALS) {
        const int nsc = sc_end - sc_begin;
        const float *sbase = p.w_scale + (size_t)tile0 * 16 * p.G + sc_begin;
        if (p.s_vec && (nsc % 4 == 0)) {
            const int nu = nsc / 4;
            for (int r = warp; r < rows_here; r += kDecodeWarps)
                for (int j = lane; j < nu; j += 32)
                    cp_async16(smem_u32(sm_s + r * p.s_stride + 16 * j), sbase + (size_t)r * p.G + 4 * j);
        } else {
            for (int r = warp; r < rows_here; r += kDecodeWarps)
                for (int j = lane; j < nsc; j += 32)
                    cp_async4(smem_u32(sm_s + r * p.s_stride + 4 * j), sbase + (size_t)r * p.G + j);
        }
    }
#pragma unroll
    for (int j = 0; j < RING / 2; ++j) {
        if (j < my_cells) post_cell(j, j);
        cp_async_commit();
    }
    W2A8_TRACE_POINT(1);
    pdl_launch_dependents();
    pdl_wait();
    W2A8_TRACE_POINT(2);

    // ---- next group: the activations of this chunk: [mrows + 1][chunk k (+pad)]; the extra
    //      row is zeros and stands in for tokens beyond M ----------------------------------
    {
        const int row_units = nb * (kBlockK / 16);
        const int klen = min(nb * kBlockK, p.K - kb_begin * kBlockK);
        for (int u = threadIdx.x; u < (mrows + 1) * row_units; u += kDecodeThreads) {
            const int r = u / row_units, cu = u % row_units;
            unsigned char *dst = acts + r * p.act_stride + cu * 16;
            if (r < mrows && cu * 16 < klen)
                cp_async16(smem_u32(dst), p.a + (size_t)(m0 + r) * p.K + (size_t)kb_begin * kBlockK + cu * 16);
            else
                *reinterpret_cast<uint4 *>(dst) = make_uint4(0u, 0u, 0u, 0u);
        }
        cp_async_commit();
    }
    // ---- the second half of the ring ----------------------------------------------------------
#pragma unroll
    for (int j = RING / 2; j < RING; ++j) {
        if (j < my_cells) post_cell(j, j);
        cp_async_commit();
    }
    cp_async_wait_group<RING / 2>();   // scales, the first half of the ring and the activations have landed
    __syncthreads();                   // scales and activations are shared by the CTA
    W2A8_TRACE_POINT(3);

    float acc[MT][4];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[mt][i] = 0.f;

    const unsigned char *brow[MT];   // this lane's token row of each slab (or the zero row)
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
        brow[mt] = acts + ((8 * mt + gq < mrows) ? (8 * mt + gq) : mrows) * p.act_stride + t * 16;
    const size_t MN = (size_t)p.M * p.N;

    // One group is committed per iteration (the cell RING ahead, or nothing), so "at most
    // RING - 1 groups pending" always means that the current cell has landed.
    int ti = 0, ci = 0;              // tile of the current cell, cell index inside the tile
    for (int c = 0; c < my_cells; ++c) {
        cp_async_wait_group<RING - 1>();
        const int slot = c & (RING - 1);
        const uint4 wa = *reinterpret_cast<const uint4 *>(ring + (slot * 2 + 0) * (32 * 16));
        const uint4 wb = *reinterpret_cast<const uint4 *>(ring + (slot * 2 + 1) * (32 * 16));
        if (c + RING < my_cells) post_cell(slot, c + RING);
        cp_async_commit();
        const uint32_t w0s[4] = {wa.x, wa.y, wa.z, wa.w};
        const uint32_t w1s[4] = {wb.x, wb.y, wb.z, wb.w};
        const int kl = ks + ci * KS;
        const int n0 = (tile0 + ti * TG + tl) * 16;
        const unsigned char *srow0 = sm_s + ((ti * TG + tl) * 16 + gq) * p.s_stride;   // floats from sc_begin on
        const unsigned char *srow1 = srow0 + 8 * p.s_stride;
        if (kb_begin + kl != p.blocks - 1 || p.tail_slices == 4)
            compute_cell<MT, SPP, ONE, PARTIALS, true>(p, w0s, w1s, srow0, srow1, brow, kl, kb_begin + kl,
                                                       n0, m0, gq, t, acc);
        else
            compute_cell<MT, SPP, ONE, PARTIALS, false>(p, w0s, w1s, srow0, srow1, brow, kl, kb_begin + kl,
                                                        n0, m0, gq, t, acc);
        if (++ci == nbw) {
            // ---- the tile is complete for this warp --------------------------------------------
            if constexpr (KS == 1 && !PARTIALS) {
                // the warp owns the whole tile: lane (gq, t) holds channels n0+gq, n0+gq+8 for
                // tokens 2t, 2t+1 of each slab
#pragma unroll
                for (int mt = 0; mt < MT; ++mt)
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int mm = m0 + 8 * mt + 2 * t + (i & 1);
                        const int nn = n0 + gq + 8 * (i >> 1);
                        if (mm < p.M) {
                            if (p.chunks == 1) p.y[(size_t)mm * p.N + nn] = acc[mt][i] * (p.a_scale[mm] * (1.0f / kCodeGain));
                            else __stcg(p.ws + chunk * MN + (size_t)mm * p.N + nn, acc[mt][i]);
                        }
                        acc[mt][i] = 0.f;
                    }
                if (p.chunks > 1) {
                    // split-K: the last warp to arrive for this tile and slab sums the chunks in order
                    __threadfence();
                    __syncwarp();
                    unsigned *counter = p.counters + (size_t)blockIdx.z * ntiles + (n0 >> 4);
                    unsigned ticket = 0;
                    if (lane == 0) ticket = atomicAdd(counter, 1u);
                    ticket = __shfl_sync(0xFFFFFFFFu, ticket, 0);
                    if (ticket == (unsigned)p.chunks - 1u) {
                        __threadfence();
#pragma unroll
                        for (int mt = 0; mt < MT; ++mt)
#pragma unroll
                            for (int i = 0; i < 4; ++i) {
                                const int mm = m0 + 8 * mt + 2 * t + (i & 1);
                                const int nn = n0 + gq + 8 * (i >> 1);
                                if (mm < p.M) {
                                    float v = 0.f;
                                    for (int ch = 0; ch < p.chunks; ++ch)
                                        v += __ldcg(p.ws + ch * MN + (size_t)mm * p.N + nn);
                                    p.y[(size_t)mm * p.N + nn] = v * (p.a_scale[mm] * (1.0f / kCodeGain));
                                }
                            }
                        if (lane == 0) *counter = 0u;   // leave the workspace reusable
                    }
                }
            }
            ci = 0;
            ++ti;
        }
    }
    cp_async_wait_all();
    W2A8_TRACE_POINT(5);

    if constexpr (!PARTIALS && KS > 1) {
        // ---- sum the K-lanes of each tile in a fixed order -----------------------
        // lane (gq, t) holds channels n0+gq, n0+gq+8 for tokens 2t, 2t+1 of each slab
        float *red = reinterpret_cast<float *>(acts);   // [KS][TG][MT*4][32], reuses the staging area
        __syncthreads();   // everyone is done reading the staged activations
#pragma unroll
        for (int mt = 0; mt < MT; ++mt)
#pragma unroll
            for (int i = 0; i < 4; ++i)
                red[((ks * TG + tl) * (MT * 4) + mt * 4 + i) * 32 + lane] = acc[mt][i];
        __syncthreads();
        // element e of the CTA: (tile etl, slab mt, quad register i, lane el)
        for (int e = threadIdx.x; e < TG * MT * 128; e += kDecodeThreads) {
            const int el = e & 31, ei = (e >> 5) % (MT * 4), etl = e / (MT * 128);
            const int mt = ei >> 2, i = ei & 3;
            float v = 0.f;
#pragma unroll
            for (int k2 = 0; k2 < KS; ++k2) v += red[((k2 * TG + etl) * (MT * 4) + ei) * 32 + el];
            const int mm = m0 + 8 * mt + 2 * (el & 3) + (i & 1);
            const int nn = (tile0 + etl) * 16 + (el >> 2) + 8 * (i >> 1);
            if (mm < p.M && nn < p.N) {
                if (p.chunks == 1) p.y[(size_t)mm * p.N + nn] = v * (p.a_scale[mm] * (1.0f / kCodeGain));
                else __stcg(p.ws + chunk * MN + (size_t)mm * p.N + nn, v);
            }
        }
        W2A8_TRACE_POINT(6);
        if (p.chunks == 1) return;

        // ---- split-K: the last CTA to arrive sums the partial outputs in order ---
        __threadfence();
        __syncthreads();
        unsigned *counter = p.counters + (size_t)blockIdx.z * ntiles + tile0;
        if (threadIdx.x == 0) is_last = (atomicAdd(counter, 1u) == (unsigned)p.chunks - 1u);
        __syncthreads();
        if (!is_last) return;
        __threadfence();
        for (int e = threadIdx.x; e < TG * MT * 128; e += kDecodeThreads) {
            const int el = e & 31, ei = (e >> 5) % (MT * 4), etl = e / (MT * 128);
            const int mt = ei >> 2, i = ei & 3;
            const int mm = m0 + 8 * mt + 2 * (el & 3) + (i & 1);
            const int nn = (tile0 + etl) * 16 + (el >> 2) + 8 * (i >> 1);
            if (mm < p.M && nn < p.N) {
                float v = 0.f;
                for (int ch = 0; ch < p.chunks; ++ch) v += __ldcg(p.ws + ch * MN + (size_t)mm * p.N + nn);
                p.y[(size_t)mm * p.N + nn] = v * (p.a_scale[mm] * (1.0f / kCodeGain));
            }
        }
        if (threadIdx.x == 0) *counter = 0u;   // leave the workspace reusable
        W2A8_TRACE_POINT(7);
    }
}

#ifdef W2A8_TRACE
extern "C" int w2a8_debug_set_trace(void *buffer) {
    unsigned long long *b = reinterpret_cast<unsigned long long *>(buffer);
    return cudaMemcpyToSymbol(g_trace, &b, sizeof(b)) == cudaSuccess ? 0 : W2A8_ERR_CUDA;
}
#endif

// ---- host side -----------------------------------------------------------------
int env_int(const char *name, int dflt);

static inline int decode_mt(int M) { return M > 32 ? 4 : (M + 7) / 8; }
static inline int round_up(int v, int m) { return (v + m - 1) / m * m; }

struct DecodePlan {
    int mt, tg, ring, tl, chunks, blocks_per_chunk, slabs, groups;
    int s_stride, act_stride, off_a, off_ring, s_vec;
    size_t smem;
};

// Shared-memory footprint of a CTA that stages `nb` blocks of K for tg * tl tiles.
static void plan_smem(DecodePlan &pl, int M, int G, int spp, int nb) {
    const int mrows = M < 8 * pl.mt ? M : 8 * pl.mt;
    // scale rows: a stride of 16 mod 32 bytes (64 m + 16) spreads the 8 channels of a
    // warp read over distinct 16-byte bank groups
    const int nsc = spp == 4 ? G : (4 / spp) * nb;
    pl.s_stride = round_up(nsc * 4, 64) + 16;
    pl.act_stride = nb * kBlockK + kActPad;
    pl.off_a = round_up(pl.tg * pl.tl * 16 * pl.s_stride, 128);
    const size_t act = (size_t)(mrows + 1) * pl.act_stride;
    const size_t red = (size_t)kDecodeWarps * pl.mt * 4 * 32 * sizeof(float);
    pl.off_ring = round_up(pl.off_a + (int)(act > red ? act : red), 128);
    pl.smem = pl.off_ring + (size_t)kDecodeWarps * pl.ring * 2 * 32 * 16;
}

// Launch plan.  Few tokens (one 8-token slab): one tile per CTA, its four warps take
// interleaved blocks of K (shortest serial work per warp).  More tokens: two tiles per
// CTA, two K-lanes each, sharing the staged activations.  Optionally (W2A8_TG=4) every
// warp owns whole tiles and walks several of them, so that the activations a CTA stages
// (M x chunk bytes, which rivals the weight stream once M is large) are read from L2
// once per 4 * tl tiles.  K-chunks are added when the staged data would not fit, when
// a warp would otherwise hold more cells than its ring, or when the grid would leave
// most SMs idle.
static DecodePlan decode_plan(int M, int N, int K, const ShapeInfo &si) {
    DecodePlan pl;
    pl.mt = decode_mt(M);
    pl.slabs = (M + 8 * pl.mt - 1) / (8 * pl.mt);
    const int ntiles = N / 16;
    const int forced_tg = env_int("W2A8_TG", 0);
    // measured on B200: whole-tile warps (tg = 4) lose to K-lanes at every decode shape tried --
    // the number of independent warps matters more than the activation traffic -- so they
    // are only taken on request
    pl.tg = (forced_tg == 1 || forced_tg == 2 || forced_tg == 4) ? forced_tg : (pl.mt == 1 ? 1 : 2);
    pl.ring = pl.tg == 4 ? 8 : kRound;
    pl.tl = 1;
    const int ks = kDecodeWarps / pl.tg;
    const int forced = env_int("W2A8_CHUNKS", 0);
    int chunks = 1;
    if (pl.tg == 4) {
        // whole-tile warps: blocks per chunk (= cells per tile) 4, fewer if the grid is small
        int nb = env_int("W2A8_NB", 4);
        if (nb < 1) nb = 1;
        if (nb > si.blocks) nb = si.blocks;
        auto ctas = [&](int nb_) { return (long long)((ntiles + 3) / 4) * ((si.blocks + nb_ - 1) / nb_) * pl.slabs; };
        while (forced <= 0 && nb > 1 && ctas(nb) < 200) nb /= 2;
        chunks = (si.blocks + nb - 1) / nb;
        if (forced > chunks) chunks = forced;
        if (chunks > si.blocks) chunks = si.blocks;
        pl.blocks_per_chunk = (si.blocks + chunks - 1) / chunks;
        pl.chunks = (si.blocks + pl.blocks_per_chunk - 1) / pl.blocks_per_chunk;
        // tiles per warp: aim at about two CTAs per SM, within the shared-memory budget
        int tl = env_int("W2A8_TL", 0);
        if (tl <= 0) tl = (int)(((long long)ntiles * pl.chunks * pl.slabs) / (4 * 296));
        if (tl < 1) tl = 1;
        if (tl > 16) tl = 16;
        for (;; --tl) {
            pl.tl = tl;
            plan_smem(pl, M, si.G, si.spp, pl.blocks_per_chunk);
            if ((int)pl.smem <= kSmemBudget + 16 * 1024 || tl == 1) break;
        }
        pl.groups = (ntiles + 4 * pl.tl - 1) / (4 * pl.tl);
    } else {
        pl.groups = (ntiles + pl.tg - 1) / pl.tg;
        for (;;) {   // smallest chunk count whose staging fits the budget
            const int bpc = (si.blocks + chunks - 1) / chunks;
            plan_smem(pl, M, si.G, si.spp, bpc);
            if ((int)pl.smem <= kSmemBudget || bpc == 1) break;
            ++chunks;
        }
        if (forced > 0) {
            if (forced > chunks) chunks = forced;
        } else {
            // Measured on B200: a warp should hold all its cells in its ring (later cells
            // wait a full memory latency each), and the whole grid should field about 2000
            // warps or more so that enough loads are in flight; beyond that the cross-CTA
            // sum costs more than further splitting gains.
            const int one_round = (si.blocks + pl.ring * ks - 1) / (pl.ring * ks);
            if (one_round > chunks) chunks = one_round;
            const int min_warps = env_int("W2A8_MIN_WARPS", 2000);
            while ((long long)pl.groups * pl.slabs * kDecodeWarps * chunks < min_warps &&
                   (si.blocks / (chunks * 2)) >= ks)
                chunks *= 2;
        }
        if (chunks > si.blocks) chunks = si.blocks;
        pl.blocks_per_chunk = (si.blocks + chunks - 1) / chunks;
        pl.chunks = (si.blocks + pl.blocks_per_chunk - 1) / pl.blocks_per_chunk;
        plan_smem(pl, M, si.G, si.spp, pl.blocks_per_chunk);
    }
    // scale rows can be copied in 16-byte units when row pitch and chunk starts allow
    const int spb = si.spp == 4 ? 0 : 4 / si.spp;
    pl.s_vec = (si.spp != 4) && (si.G % 4 == 0) && ((spb * pl.blocks_per_chunk) % 4 == 0);
    (void)K;
    return pl;
}

constexpr size_t kStatusBytes = 256;   // workspace header: status word

size_t decode_workspace_bytes(int M, int N, int K, const ShapeInfo &si) {
    const DecodePlan pl = decode_plan(M, N, K, si);
    size_t counters = ((size_t)4 * (N / 16) * pl.slabs + 255) / 256 * 256;   // >= any tile grouping
    // with an environment override in force, size for the finest split
    const bool overridden = env_int("W2A8_CHUNKS", 0) > 0 || env_int("W2A8_TG", 0) > 0 ||
                            env_int("W2A8_NB", 0) > 0 || env_int("W2A8_TL", 0) > 0;
    const int chunks = overridden ? si.blocks : pl.chunks;
    size_t part = (size_t)(chunks > 1 ? chunks : 0) * M * N * sizeof(float);
    return kStatusBytes + counters + part;
}

// Bytes at the start of the workspace that must be zero before a launch: the
// status word and the arrival counters.
size_t decode_workspace_header_bytes(int M, int N, int K, const ShapeInfo &si) {
    const DecodePlan pl = decode_plan(M, N, K, si);
    return kStatusBytes + ((size_t)4 * (N / 16) * pl.slabs + 255) / 256 * 256;
}

template <int MT, int SPP, int TG, bool ONE, bool PARTIALS>
static cudaError_t launch_decode_inst(const DecodeParams &p, dim3 grid, size_t smem, cudaStream_t st) {
    constexpr int RING = TG == 4 ? 8 : kRound;
    static bool configured = false;   // one attribute call per instantiation and process
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(w2a8_decode_kernel<MT, SPP, TG, RING, ONE, PARTIALS>,
                                             cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
        if (e != cudaSuccess) return e;
        configured = true;
    }
    return launch_kernel(w2a8_decode_kernel<MT, SPP, TG, RING, ONE, PARTIALS>, grid, dim3(kDecodeThreads),
                         smem, st, pdl_enabled(), p);
}

template <int MT, int SPP, int TG>
static cudaError_t launch_decode_tg(const DecodeParams &p, bool want_partials, dim3 grid, size_t smem,
                                    cudaStream_t st) {
    if (want_partials) return launch_decode_inst<MT, SPP, TG, false, true>(p, grid, smem, st);
    if (MT == 1 && p.M == 1) return launch_decode_inst<1, SPP, TG, true, false>(p, grid, smem, st);
    return launch_decode_inst<MT, SPP, TG, false, false>(p, grid, smem, st);
}

template <int MT, int SPP>
static cudaError_t launch_decode_mt(const DecodeParams &p, const DecodePlan &pl, bool want_partials,
                                    cudaStream_t st) {
    dim3 grid(pl.groups, pl.chunks, pl.slabs);
    switch (pl.tg) {
        case 1: return launch_decode_tg<MT, SPP, 1>(p, want_partials, grid, pl.smem, st);
        case 2: return launch_decode_tg<MT, SPP, 2>(p, want_partials, grid, pl.smem, st);
        default: return launch_decode_tg<MT, SPP, 4>(p, want_partials, grid, pl.smem, st);
    }
}

template <int SPP>
static cudaError_t launch_decode_spp(const DecodeParams &p, const DecodePlan &pl, bool want_partials,
                                     cudaStream_t st) {
    switch (pl.mt) {
        case 1: return launch_decode_mt<1, SPP>(p, pl, want_partials, st);
        case 2: return launch_decode_mt<2, SPP>(p, pl, want_partials, st);
        case 3: return launch_decode_mt<3, SPP>(p, pl, want_partials, st);
        default: return launch_decode_mt<4, SPP>(p, pl, want_partials, st);
    }
}

// Enqueue the decode kernel.  `partials` != nullptr selects the parity export.
int launch_decode(const int8_t *a, const float *a_scale, const uint32_t *packed,
                  const float *w_scale, float *y, int32_t *partials, int M, int N, int K,
                  int group, const ShapeInfo &si, void *workspace, cudaStream_t st) {
    const DecodePlan pl = decode_plan(M, N, K, si);
    DecodeParams p;
    p.a = a; p.a_scale = a_scale; p.packed = packed; p.w_scale = w_scale;
    p.y = y; p.partials = partials;
    p.M = M; p.N = N; p.K = K; p.G = si.G; p.group = group;
    p.blocks = si.blocks; p.tail_slices = si.tail_slices; p.words_per_row = si.words_per_row;
    p.chunks = pl.chunks; p.blocks_per_chunk = pl.blocks_per_chunk; p.tiles_per_warp = pl.tl;
    p.s_stride = pl.s_stride; p.act_stride = pl.act_stride;
    p.off_a = pl.off_a; p.off_ring = pl.off_ring; p.s_vec = pl.s_vec;
    size_t counters = ((size_t)4 * (N / 16) * pl.slabs + 255) / 256 * 256;
    char *base = reinterpret_cast<char *>(workspace);
    p.status = reinterpret_cast<int *>(base);
    p.counters = reinterpret_cast<unsigned *>(base + kStatusBytes);
    p.ws = reinterpret_cast<float *>(base + kStatusBytes + counters);
    if (partials) {
        // several warps add their share of a large group: start from zero
        if (cudaMemsetAsync(partials, 0, (size_t)M * N * si.G * sizeof(int32_t), st) != cudaSuccess)
            return W2A8_ERR_CUDA;
    }
    cudaError_t e = si.spp == 1 ? launch_decode_spp<1>(p, pl, partials != nullptr, st)
                  : si.spp == 2 ? launch_decode_spp<2>(p, pl, partials != nullptr, st)
                                : launch_decode_spp<4>(p, pl, partials != nullptr, st);
    return e == cudaSuccess ? W2A8_OK : W2A8_ERR_CUDA;
}

}  // namespace w2a8
