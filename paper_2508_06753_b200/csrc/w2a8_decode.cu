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
// K-lanes take runs of consecutive blocks of the chunk, at most RING cells each
// (consecutive, so that the scale pieces a warp requests are neighbours).  The
// K-lanes of a tile are summed through shared memory in a fixed order.  Chunks
// (grid.y; used when K has more blocks than the K-lanes can hold, or when the
// grid would leave SMs idle) are summed in chunk order: inside a thread-block
// cluster when there are at most 8 of them (every CTA writes its sums into the
// shared memory of the cluster's first CTA, one cluster barrier, no trip through
// global memory), else through the workspace by the last CTA to arrive.
// grid.z walks 8*MT-token slabs.
//
// Data movement.  Nothing is staged per CTA, and the warps of a CTA do not meet
// before the final sum.  Weights: every lane owns 16-byte landing slots in
// shared memory and fills them with per-thread asynchronous copies (cp.async,
// L1 bypass), two per cell (its two channels); all cells of a warp are
// requested at once, so the whole weight stream of the CTA is in flight from
// the start.  Scales: lanes 0..15 copy the 16 bytes per channel and cell into
// per-warp slots the same way.  Both are frozen data, so they are requested
// before the kernel waits for the previous kernel of the stream; under
// programmatic dependent launch the weight stream of this kernel therefore
// overlaps the tail of the previous one.  Activations (the only input that can
// depend on the previous kernel) are read after that wait, straight from global
// memory through L1: all CTAs of an SM share them there, which keeps the L2
// traffic at one copy per SM instead of one per CTA.
//
// One 128-bit unit per lane and channel holds word t of each of the four 64-k
// slices of a block -- exactly what the four lanes of an MMA quad must supply
// so that every MMA sums k of a single scale group.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "w2a8_cell.cuh"

namespace w2a8 {

constexpr int kDecodeWarps = 4;
constexpr int kDecodeThreads = kDecodeWarps * 32;
// Resident CTAs per SM the compiler must allow.  One slab: 8 (64 registers), which also lets
// every 4-CTA cluster of a split-K launch be resident at once (clusters are placed inside one
// GPC; with 7 per SM the last few clusters of a 1024-CTA grid waited for a second round).
// RELAX instances (one or two slabs, fp32 scales, default grouping) are compiled for 7 CTAs per
// SM instead: 72 registers, no pressure on the compiler for one slab and one wave instead of one
// and a half for a two-slab grid of up to 1036 CTAs.  The launch code picks them for grids that
// fit 7 per SM and do not need the eighth slot (measured: 4096x14336 at M = 4 5.39 -> 5.15 us, at
// M = 16 9.64 -> 8.92 us; 4096x1024 2.33 -> 2.22 us; but 14336x4096 with its 1024-CTA cluster
// grid 6.0 -> 8.3 us, which therefore stays on the 8-per-SM instance).
#ifndef W2A8_MINB
#define W2A8_MINB(MT) ((MT) == 1 ? 8 : 3)
#endif
constexpr int kRelaxedCtasPerSm = 7;
constexpr int kRound = 4;                      // landing slots (cells) per warp


// The same cell for 16-bit activations and no activation quantiser (the alternative kernel of
// Sec. II): the codes become the bf16 values q - 2 (exact), the activations are the caller's
// bf16 values as they are, and the products are summed in fp32 by `mma.sync.m16n8k16`; the
// group scale multiplies the fp32 sum of its group.
// A lane's word of a slice holds code l (k = 16 t + l of the slice) at bits 8 (l mod 4) +
// 2 (l div 4); MMA j of the slice takes l = 4 j .. 4 j + 3, the two bits at offset 2 j of each
// byte.  With the code left where it is, (0x43 - j) << 8 | (q << 2 j) is the bf16 value
// 2^(7 - 2 j) + q for j = 0, 1, 2 (the code sits in the mantissa, one unit of it worth 1), so a
// mask, a byte permute with the exponent byte and one packed subtraction of 2^(7 - 2 j) + 2 give
// the two bf16 weights of a register; j = 3 would reach the exponent bit and is shifted down to
// the j = 0 form.
// brow[mt]: this lane's 32 activation bytes (16 bf16) of slice 0, token row of slab mt.
template <int MT, int SPP, bool ONE, bool FULL>
__device__ __forceinline__ void compute_cell_a16(const DecodeParams &p, const uint32_t (&w0s)[4],
                                                 const uint32_t (&w1s)[4], const unsigned char *sc0,
                                                 const unsigned char *sc1,
                                                 const int8_t *const (&brow)[MT], float (&acc)[MT][4]) {
    const int R = FULL ? 4 : p.tail_slices;
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
    const float zero[4] = {0.f, 0.f, 0.f, 0.f};
    auto weights = [&](uint32_t c, uint32_t expo, float off, uint32_t sel) -> uint32_t {
        const uint32_t u = __byte_perm(c, expo, sel);
        const __nv_bfloat162 v = __hsub2(*reinterpret_cast<const __nv_bfloat162 *>(&u),
                                         __floats2bfloat162_rn(off, off));
        return *reinterpret_cast<const uint32_t *>(&v);
    };
    float D[MT][4];   // fp32 sums of the current group; a group never outlives a cell
#pragma unroll
    for (int s = 0; s < 4; ++s) {
        if (s < R) {
            const bool first = (s % SPP) == 0;
            const bool last = ((s + 1) % SPP) == 0 || s == R - 1;
            uint32_t X[MT][8];
#pragma unroll
            for (int mt = 0; mt < MT; ++mt) {
                const uint4 lo = ld_act16(brow[mt] + s * (2 * kSliceK));
                const uint4 hi = ld_act16(brow[mt] + s * (2 * kSliceK) + 16);
                X[mt][0] = lo.x; X[mt][1] = lo.y; X[mt][2] = lo.z; X[mt][3] = lo.w;
                X[mt][4] = hi.x; X[mt][5] = hi.y; X[mt][6] = hi.z; X[mt][7] = hi.w;
            }
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                // j is a constant after unrolling
                const uint32_t c0 = j < 3 ? (w0s[s] & (0x03030303u << (2 * j))) : ((w0s[s] >> 6) & 0x03030303u);
                const uint32_t c1 = j < 3 ? (w1s[s] & (0x03030303u << (2 * j))) : ((w1s[s] >> 6) & 0x03030303u);
                const uint32_t expo = j == 1 ? 0x42424242u : j == 2 ? 0x41414141u : 0x43434343u;
                const float off = j == 1 ? 34.f : j == 2 ? 10.f : 130.f;
                const uint32_t a0 = weights(c0, expo, off, 0x4140u), a1 = weights(c1, expo, off, 0x4140u);
                const uint32_t a2 = weights(c0, expo, off, 0x4342u), a3 = weights(c1, expo, off, 0x4342u);
#pragma unroll
                for (int mt = 0; mt < MT; ++mt) {
                    if (first && j == 0) mma_bf16_16x8x16(D[mt], a0, a1, a2, a3, X[mt][2 * j], X[mt][2 * j + 1], zero);
                    else                 mma_bf16_16x8x16(D[mt], a0, a1, a2, a3, X[mt][2 * j], X[mt][2 * j + 1], D[mt]);
                }
            }
            if (last) {
                const float s0 = s0s[s / SPP], s1 = s1s[s / SPP];
#pragma unroll
                for (int mt = 0; mt < MT; ++mt) {
                    acc[mt][0] = fmaf(s0, D[mt][0], acc[mt][0]);
                    acc[mt][2] = fmaf(s1, D[mt][2], acc[mt][2]);
                    if constexpr (!ONE) {
                        acc[mt][1] = fmaf(s0, D[mt][1], acc[mt][1]);
                        acc[mt][3] = fmaf(s1, D[mt][3], acc[mt][3]);
                    }
                }
            }
        }
    }
}

// MT: 8-token slabs per CTA; SPP: 64-k slices per scale group (capped at 4);
// TG: tiles the four warps of a CTA work on side by side (K-lanes per tile = 4 / TG);
// RING: cells a warp can hold (the launch plan never gives it more); ONE: a single
// token (half of each accumulator quad is dead and is not promoted).
//
// A warp handles only a handful of cells, so the code around the cells is kept
// short: one weight pointer per lane with cell c at a fixed stride from it, a
// fully unrolled cell loop (slot and operand offsets are immediates), no
// divisions and no 64-bit multiplies per cell.  Warps do not meet before the
// final sum over the K-lanes.
// A16: p.a holds the caller's bf16 activations (no quantiser, no token scale): compute_cell_a16.
template <int MT, int SPP, int TG, int RING, bool ONE, bool PARTIALS, bool H16 = false, bool A16 = false,
          bool RELAX = false>
__global__ void __launch_bounds__(kDecodeThreads, RELAX ? kRelaxedCtasPerSm : W2A8_MINB(MT))
w2a8_decode_kernel(const DecodeParams p) {
    constexpr int KS = kDecodeWarps / TG;
    constexpr int kSlotBytes = 2 * 32 * 16;     // weights of one cell: two channels x 32 lanes x 16 B
    constexpr int kScaleBytes = 16 * 16;        // scales of one cell: 16 channels x 16 B
    constexpr int kWarpBytes = RING * (kSlotBytes + kScaleBytes);
    constexpr int SPB = 4 / SPP;                // scales per block and channel
    constexpr int kActBytes = A16 ? 2 : 1;      // bytes per activation
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ int is_last;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int gq = lane >> 2, t = lane & 3;
    const int tl = warp % TG, ks = warp / TG;
    const int ntiles = p.N / 16;
    const int tile0 = blockIdx.x * TG;            // first tile of this CTA
    const int chunk = blockIdx.y;
    const int kb_begin = chunk * p.blocks_per_chunk;
    const int kb_end = min(kb_begin + p.blocks_per_chunk, p.blocks);
    const int nb = kb_end - kb_begin;
    const int m0 = blockIdx.z * (8 * MT);
    const int mrows = min(8 * MT, p.M - m0);
    // Split-K in a cluster ends with stores into the shared memory of the cluster's first CTA,
    // which may only be touched once that CTA is known to be running: every CTA arrives here and
    // waits just before its first remote store (the wait costs nothing by then).
    if (p.cluster) cluster_arrive_relaxed();

    // This warp's cells: the chunk is cut into KS runs of consecutive blocks, one per K-lane; cell c
    // is block kb0 + c of tile tile0 + tl (at most RING of them).  Consecutive blocks matter for the
    // scales: the 16-byte pieces a warp asks for, cell after cell, are then neighbours in memory
    // (64 bytes per channel), which DRAM serves far better than isolated 16-byte pieces.
    const int n0 = (tile0 + tl) * 16;
    const int cpw = (int)((unsigned)(nb + KS - 1) / KS);          // cells per K-lane
    const int kb0 = kb_begin + ks * cpw;
    const int my_cells = (tile0 + tl < ntiles) ? max(0, min(cpw, nb - ks * cpw)) : 0;
    // only the last block of K can have fewer than four slices; it is the last cell of its K-lane
    const bool tail_cta = (kb_end == p.blocks) && (p.tail_slices != 4);
    const bool tail_mine = tail_cta && my_cells > 0 && ks * cpw + my_cells == nb;
    const int tail_cell = tail_mine ? my_cells - 1 : -1;
    const int full_cells = my_cells - (tail_mine ? 1 : 0);

    // Landing slots of this warp in shared memory.  Weights: slot c of a lane holds its two
    // 16-byte units (channels gq and gq+8) of cell c; only this lane writes and reads them.
    // Scales: 16 bytes per channel and cell, copied by lanes 0..15 (one channel each) and read
    // by the whole warp after a warp barrier.
    unsigned char *wslots = smem + warp * kWarpBytes + lane * 16;
    unsigned char *sslots = smem + warp * kWarpBytes + RING * kSlotBytes;
    const uint32_t wslots_u32 = smem_u32(wslots);
    const uint32_t sslot_u32 = smem_u32(sslots) + (lane & 15) * 16;
    // word 4t of block kb0 in rows n0 + gq and n0 + gq + 8; cell c is 16 words on
    const uint32_t *wrow0 = p.packed + (size_t)(n0 + gq) * p.words_per_row + 16 * kb0 + 4 * t;
    const uint32_t *wrow1 = wrow0 + (size_t)8 * p.words_per_row;
    // first scale of block kb0 in row n0 + (lane & 15)
    const float *srow = nullptr;
    const unsigned short *srow_h = nullptr;          // the same place when the scales are binary16
    if constexpr (!PARTIALS) {
        const size_t first = (size_t)(n0 + (lane & 15)) * p.G + (SPP != 4 ? SPB * kb0 : 0);
        if constexpr (H16) srow_h = reinterpret_cast<const unsigned short *>(p.w_scale) + first;
        else               srow = p.w_scale + first;
    }
    // binary16 scales that cannot be copied as one aligned unit (odd row pitch, or one scale per
    // cell): loaded and stored by the lane itself -- slower, and rare
    auto copy_scales_h = [&](int c, int first, int count) {
        unsigned short *dst = reinterpret_cast<unsigned short *>(sslots + c * kScaleBytes + (lane & 15) * 16);
        for (int i = 0; i < count; ++i) dst[i] = __ldg(srow_h + first + i);
    };
    auto post_cell = [&](int c) {   // c is a constant after unrolling
        cp_async16(wslots_u32 + c * kSlotBytes, wrow0 + c * 16);
        cp_async16(wslots_u32 + c * kSlotBytes + 32 * 16, wrow1 + c * 16);
        if constexpr (!PARTIALS) {
            if (lane < 16) {
                if constexpr (H16) {
                    if constexpr (SPP == 4) {
                        const int kb = kb0 + c;
                        copy_scales_h(c, p.blocks_per_group >= p.blocks ? 0 : kb / p.blocks_per_group, 1);
                    } else if (p.s_vec) {
                        if constexpr (SPP == 1) cp_async8(sslot_u32 + c * kScaleBytes, srow_h + c * SPB);
                        else                    cp_async4(sslot_u32 + c * kScaleBytes, srow_h + c * SPB);
                    } else {
                        copy_scales_h(c, c * SPB, SPB);
                    }
                } else if constexpr (SPP == 4) {
                    const int kb = kb0 + c;
                    const int gi = p.blocks_per_group >= p.blocks ? 0 : kb / p.blocks_per_group;
                    cp_async4(sslot_u32 + c * kScaleBytes, srow + gi);
                } else if (p.s_vec) {
                    if constexpr (SPP == 1) cp_async16(sslot_u32 + c * kScaleBytes, srow + c * SPB);
                    else                    cp_async8(sslot_u32 + c * kScaleBytes, srow + c * SPB);
                } else {
#pragma unroll
                    for (int i = 0; i < SPB; ++i)
                        cp_async4(sslot_u32 + c * kScaleBytes + 4 * i, srow + c * SPB + i);
                }
            }
        }
    };

    // ---- weights and scales of all full cells: none of it depends on the previous kernel of
    //      the stream, so it is requested before the wait for that kernel; one group per cell --
#pragma unroll
    for (int j = 0; j < RING; ++j) {
        if (j < full_cells) post_cell(j);
        cp_async_commit();
        // Let the next kernel of the stream start once the first cell is requested (measured: a
        // little better than at kernel entry or after all requests; the request instructions
        // themselves queue for microseconds while the memory system is busy).
        if (j == 0) pdl_launch_dependents();
    }
    if (tail_mine) {
        // trailing block of K with R < 4 slices: this lane's words are t*R .. t*R+R-1 of the
        // block; it has R (SPP 1), (R+1)/2 (SPP 2) or one scale per channel
        const int R = p.tail_slices;
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            const uint32_t *wp = (r ? wrow1 : wrow0) + tail_cell * 16 - 4 * t + t * R;
            uint4 v = make_uint4(0u, 0u, 0u, 0u);
            v.x = __ldg(wp);
            if (R > 1) v.y = __ldg(wp + 1);
            if (R > 2) v.z = __ldg(wp + 2);
            *reinterpret_cast<uint4 *>(wslots + tail_cell * kSlotBytes + r * (32 * 16)) = v;
        }
        if constexpr (!PARTIALS) {
            if (lane < 16 && H16) {
                if constexpr (SPP == 4) {
                    const int kb = kb0 + tail_cell;
                    copy_scales_h(tail_cell, p.blocks_per_group >= p.blocks ? 0 : kb / p.blocks_per_group, 1);
                } else {
                    copy_scales_h(tail_cell, tail_cell * SPB, (R + SPP - 1) / SPP);
                }
            } else if (lane < 16) {
                float *dst = reinterpret_cast<float *>(sslots + tail_cell * kScaleBytes + lane * 16);
                if constexpr (SPP == 4) {
                    const int kb = kb0 + tail_cell;
                    dst[0] = __ldg(srow + (p.blocks_per_group >= p.blocks ? 0 : kb / p.blocks_per_group));
                } else {
                    const int nsc = (R + SPP - 1) / SPP;
                    for (int i = 0; i < nsc; ++i) dst[i] = __ldg(srow + tail_cell * SPB + i);
                }
            }
        }
    }
    pdl_wait();

    // The token scale of the outputs this thread will store is only needed by the epilogue, at the
    // very end of the critical path of a short launch: fetch it now.  Output element e of the CTA
    // (see `locate` below) belongs to token row_of(e).
    constexpr int kOutPerThread = ONE ? 1 : TG * MT;          // = ceil(kElems / kDecodeThreads)
    float tok_scale[kOutPerThread];
    if constexpr (!PARTIALS && !A16) {
#pragma unroll
        for (int j = 0; j < kOutPerThread; ++j) {
            const int e = threadIdx.x + j * kDecodeThreads;
            const int el = e & 31, ei = (e >> 5) % (MT * 4);
            const int mm = ONE ? 0 : m0 + 8 * (ei >> 2) + 2 * (el & 3) + (ei & 1);
            tok_scale[j] = mm < p.M ? p.a_scale[mm] * (1.0f / kCodeGain) : 0.f;
        }
    }

    float acc[MT][4];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[mt][i] = 0.f;

    // This lane's activation bytes of block kb0: token row of each slab.  Token columns of an
    // MMA are independent, and columns beyond M are never stored, so they may read any row:
    // the last one.  The activations are read through L1, which all CTAs of an SM share.
    const int8_t *brow[MT];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
        brow[mt] = p.a + ((size_t)(m0 + min(8 * mt + gq, mrows - 1)) * p.K + (size_t)kb0 * kBlockK + t * 16) * kActBytes;
    const size_t MN = (size_t)p.M * p.N;
    const unsigned char *sc0 = sslots + gq * 16, *sc1 = sc0 + 8 * 16;

#pragma unroll
    for (int c = 0; c < RING; ++c) {
        if (c < full_cells) {                                 // warp-uniform
            cp_async_wait_pending(RING - 1 - c);
            __syncwarp();                                     // the scales were copied by other lanes
            const uint4 wa = *reinterpret_cast<const uint4 *>(wslots + c * kSlotBytes);
            const uint4 wb = *reinterpret_cast<const uint4 *>(wslots + c * kSlotBytes + 32 * 16);
            const uint32_t w0s[4] = {wa.x, wa.y, wa.z, wa.w};
            const uint32_t w1s[4] = {wb.x, wb.y, wb.z, wb.w};
            const int8_t *bc[MT];
#pragma unroll
            for (int mt = 0; mt < MT; ++mt) bc[mt] = brow[mt] + c * (kBlockK * kActBytes);
            if constexpr (A16)
                compute_cell_a16<MT, SPP, ONE, true>(p, w0s, w1s, sc0 + c * kScaleBytes, sc1 + c * kScaleBytes, bc, acc);
            else
                compute_cell<MT, SPP, ONE, PARTIALS, true, H16>(p, w0s, w1s, sc0 + c * kScaleBytes,
                                                                sc1 + c * kScaleBytes, bc, kb0 + c, n0, m0, gq, t, acc);
        }
    }
    if (tail_mine) {   // the trailing block is this warp's last cell; its words and scales were stored directly
        __syncwarp();
        const uint4 wa = *reinterpret_cast<const uint4 *>(wslots + tail_cell * kSlotBytes);
        const uint4 wb = *reinterpret_cast<const uint4 *>(wslots + tail_cell * kSlotBytes + 32 * 16);
        const uint32_t w0s[4] = {wa.x, wa.y, wa.z, wa.w};
        const uint32_t w1s[4] = {wb.x, wb.y, wb.z, wb.w};
        const int8_t *bc[MT];
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) bc[mt] = brow[mt] + (size_t)tail_cell * (kBlockK * kActBytes);
        if constexpr (A16)
            compute_cell_a16<MT, SPP, ONE, false>(p, w0s, w1s, sc0 + tail_cell * kScaleBytes,
                                                  sc1 + tail_cell * kScaleBytes, bc, acc);
        else
            compute_cell<MT, SPP, ONE, PARTIALS, false, H16>(p, w0s, w1s, sc0 + tail_cell * kScaleBytes,
                                                             sc1 + tail_cell * kScaleBytes, bc, kb0 + tail_cell,
                                                             n0, m0, gq, t, acc);
    }

    if constexpr (!PARTIALS) {
        // ---- sum the K-lanes of each tile in a fixed order -----------------------
        // Lane (gq, t) holds channels n0+gq, n0+gq+8 for tokens 2t, 2t+1 of each slab.  Each
        // warp parks its sums in its own (now idle) weight slots.
        float *red = reinterpret_cast<float *>(smem + warp * kWarpBytes);
        const float *red0 = reinterpret_cast<const float *>(smem);
        constexpr int kWarpFloats = kWarpBytes / 4;
        __syncwarp();      // every lane has read its slots
        if constexpr (ONE) {
            if (t == 0) { red[gq] = acc[0][0]; red[gq + 8] = acc[0][2]; }
        } else {
#pragma unroll
            for (int mt = 0; mt < MT; ++mt)
#pragma unroll
                for (int i = 0; i < 4; ++i) red[(mt * 4 + i) * 32 + lane] = acc[mt][i];
        }
        __syncthreads();

        // Outputs of the CTA as a flat list: element e = (tile etl, slab mt, quad register i,
        // lane el); with one token only channel (e & 15) of tile (e >> 4) for e < 16 * TG.
        constexpr int kElems = ONE ? TG * 16 : TG * MT * 128;
        auto locate = [&](int e, int &mm, int &nn) -> bool {
            if constexpr (ONE) {
                mm = 0;
                nn = (tile0 + (e >> 4)) * 16 + (e & 15);
            } else {
                const int el = e & 31, ei = (e >> 5) % (MT * 4), etl = e / (MT * 128);
                mm = m0 + 8 * (ei >> 2) + 2 * (el & 3) + (ei & 1);
                nn = (tile0 + etl) * 16 + (el >> 2) + 8 * ((ei & 3) >> 1);
            }
            return mm < p.M && nn < p.N;
        };
        auto cta_sum = [&](int e) -> float {
            float v = 0.f;
            if constexpr (ONE) {
#pragma unroll
                for (int k2 = 0; k2 < KS; ++k2) v += red0[(k2 * TG + (e >> 4)) * kWarpFloats + (e & 15)];
            } else {
                const int el = e & 31, ei = (e >> 5) % (MT * 4), etl = e / (MT * 128);
#pragma unroll
                for (int k2 = 0; k2 < KS; ++k2) v += red0[(k2 * TG + etl) * kWarpFloats + ei * 32 + el];
            }
            return v;
        };

        // final value of y[mm][nn]: fp32, or (16-bit instances, on request) rounded to bf16
        auto store_y = [&](int mm, int nn, float v, float scale) {
            if constexpr (!A16) v *= scale;                                // bf16 weights carry no gain
            if constexpr (H16) {
                if (p.y16) {
                    reinterpret_cast<__nv_bfloat16 *>(p.y)[(size_t)mm * p.ldy + nn] = __float2bfloat16_rn(v);
                    return;
                }
            }
            p.y[(size_t)mm * p.ldy + nn] = v;
        };

        if (p.chunks == 1) {
#pragma unroll
            for (int j = 0; j < kOutPerThread; ++j) {
                const int e = threadIdx.x + j * kDecodeThreads;
                int mm, nn;
                if (e < kElems && locate(e, mm, nn)) store_y(mm, nn, cta_sum(e), tok_scale[j]);
            }
        } else if (p.cluster) {
            // ---- split-K inside a thread-block cluster: the chunks of a tile are the CTAs of one
            //      cluster.  Every CTA writes its sums into the receive buffer of rank 0 (remote
            //      shared memory); after one cluster barrier rank 0 adds them chunk by chunk. ----
            const uint32_t recv_u32 = smem_u32(smem + kDecodeWarps * kWarpBytes);
            const float *recv = reinterpret_cast<const float *>(smem + kDecodeWarps * kWarpBytes);
            const uint32_t rank = cluster_ctarank();
            cluster_wait();            // all CTAs of the cluster have started (arrive at kernel entry)
            for (int e = threadIdx.x; e < kElems; e += kDecodeThreads) {
                int mm, nn;
                if (locate(e, mm, nn)) st_cluster_f32(recv_u32 + (rank * kElems + e) * 4, 0, cta_sum(e));
            }
            cluster_sync();
            if (rank != 0) return;
#pragma unroll
            for (int j = 0; j < kOutPerThread; ++j) {
                const int e = threadIdx.x + j * kDecodeThreads;
                int mm, nn;
                if (e < kElems && locate(e, mm, nn)) {
                    float v = 0.f;
                    for (int ch = 0; ch < p.chunks; ++ch) v += recv[ch * kElems + e];
                    store_y(mm, nn, v, tok_scale[j]);
                }
            }
        } else {
            // ---- split-K through the workspace: the last CTA to arrive sums the partial outputs
            //      chunk by chunk ------------------------------------------------------------------
            for (int e = threadIdx.x; e < kElems; e += kDecodeThreads) {
                int mm, nn;
                if (locate(e, mm, nn)) __stcg(p.ws + chunk * MN + (size_t)mm * p.N + nn, cta_sum(e));
            }
            __threadfence();
            __syncthreads();
            unsigned *counter = p.counters + (size_t)blockIdx.z * ntiles + tile0;
            if (threadIdx.x == 0) is_last = (atomicAdd(counter, 1u) == (unsigned)p.chunks - 1u);
            __syncthreads();
            if (!is_last) return;
            __threadfence();
#pragma unroll
            for (int j = 0; j < kOutPerThread; ++j) {
                const int e = threadIdx.x + j * kDecodeThreads;
                int mm, nn;
                if (e < kElems && locate(e, mm, nn)) {
                    float v = 0.f;
                    for (int ch = 0; ch < p.chunks; ++ch) v += __ldcg(p.ws + ch * MN + (size_t)mm * p.N + nn);
                    store_y(mm, nn, v, tok_scale[j]);
                }
            }
            if (threadIdx.x == 0) *counter = 0u;   // leave the workspace reusable
        }
    }
}

// ---- host side -----------------------------------------------------------------
int env_int(const char *name, int dflt);
bool gemv_preferred(int M, int K, int group, int tiles, int count);
int launch_gemv(const int8_t *a, const float *a_scale, const void *x_bf16, int8_t *a_out, float *a_scale_out,
                int count, const uint32_t *const *packed, const float *const *w_scale, float *const *y,
                const int *N, const int *ldy, int M, int K, int group, cudaStream_t st);

struct DecodePlan {
    int mt, tg, ring, chunks, blocks_per_chunk, slabs, groups, s_vec, cluster;
    size_t smem;
};

// Launch plan for slabs of 8 * mt tokens.  One tile per CTA, its four warps take equal
// runs of consecutive blocks of K (shortest serial work per warp).  K-chunks are added when a warp would
// otherwise have more cells than landing slots, or when the grid would leave most SMs idle.
static DecodePlan decode_plan_mt(int M, int N, int K, const ShapeInfo &si, int mt, bool h16 = false) {
    DecodePlan pl;
    pl.mt = mt;
    pl.slabs = (M + 8 * pl.mt - 1) / (8 * pl.mt);
    const int ntiles = N / 16;
    // the 16-bit instances exist for the default tile grouping and slot count only
    const int forced_tg = h16 ? 0 : env_int("W2A8_TG", 0);
    pl.tg = (forced_tg == 1 || forced_tg == 2) ? forced_tg : 1;
    { const int r = h16 ? 0 : env_int("W2A8_RING", 0); pl.ring = (r == 4 || r == 8) ? r : kRound; }
    const int ks = kDecodeWarps / pl.tg;
    const int forced = env_int("W2A8_CHUNKS", 0);
    int chunks = 1;
    pl.groups = (ntiles + pl.tg - 1) / pl.tg;
    // landing slots: 1 KB of weights and 256 B of scales per cell and warp
    pl.smem = (size_t)kDecodeWarps * pl.ring * (2 * 32 * 16 + 16 * 16);
    // a warp holds all its cells at once: at most ring * ks blocks per chunk
    const int one_round = (si.blocks + pl.ring * ks - 1) / (pl.ring * ks);
    if (one_round > chunks) chunks = one_round;
    if (forced > 0) {
        if (forced > chunks) chunks = forced;
    } else {
        // Measured on B200: the whole grid should field about 2000 warps or more so that
        // enough loads are in flight, and it pays to go on splitting (down to one cell per
        // warp) as long as all CTAs are still resident at once (8 per SM for one slab, 4 for
        // wider slabs); beyond that the extra round of CTAs costs more than the split gains.
        const int min_warps = env_int("W2A8_MIN_WARPS", 2000);
        const long long resident = (long long)sm_count() * (mt == 1 ? 8 : 4);
        auto ctas = [&](int c) { return (long long)pl.groups * pl.slabs * c; };
        while ((ctas(chunks) * kDecodeWarps < min_warps || ctas(chunks * 2) <= resident) &&
               (si.blocks / (chunks * 2)) >= ks)
            chunks *= 2;
    }
    if (chunks > si.blocks) chunks = si.blocks;
    pl.blocks_per_chunk = (si.blocks + chunks - 1) / chunks;
    pl.chunks = (si.blocks + pl.blocks_per_chunk - 1) / pl.blocks_per_chunk;
    pl.s_vec = (si.spp == 1 && si.G % 4 == 0) || (si.spp == 2 && si.G % 2 == 0);
    // up to 8 chunks (the portable cluster size) are summed inside a thread-block cluster;
    // rank 0 receives one partial output per chunk and element of the CTA
    pl.cluster = pl.chunks > 1 && pl.chunks <= 8 && env_int("W2A8_CLUSTER", 1) != 0;
    if (pl.cluster) pl.smem += (size_t)pl.chunks * pl.tg * pl.mt * 128 * sizeof(float);
    (void)K;
    return pl;
}

// Tokens per slab.  Up to 8 tokens: one slab.  More: slabs of 8 tokens (the weights are then
// streamed once per slab, the later slabs from L2) as long as the whole grid is resident at
// once (8 CTAs per SM) -- measured faster on the small matrices of a layer (k/v, q/o), whose
// grids are far from filling the GPU with wider slabs; otherwise wide slabs of equal width, up
// to 32 tokens.  W2A8_MT forces a width.
static DecodePlan decode_plan_uncached(int M, int N, int K, const ShapeInfo &si, bool h16) {
    const int forced = env_int("W2A8_MT", 0);
    if (forced >= 1 && forced <= 4) return decode_plan_mt(M, N, K, si, forced, h16);
    // Widest slab: up to 24 tokens one slab; 25..32 tokens two 16-token slabs (measured 10 % faster
    // than one 32-token slab on 4096x14336 and 8192x8192, equal elsewhere); beyond that as few slabs
    // of at most 32 tokens as cover M, all of the same width (48 tokens: 24 + 24, not 32 + 16).
    int widest;
    if (M <= 24) widest = (M + 7) / 8;
    else if (M <= 32) widest = 2;
    else { const int slabs = (M + 31) / 32; widest = ((M + slabs - 1) / slabs + 7) / 8; }
    if (widest == 1) return decode_plan_mt(M, N, K, si, 1, h16);
    const long long kResidentCtas = (long long)sm_count() * 8;
    const DecodePlan narrow = decode_plan_mt(M, N, K, si, 1, h16);
    if ((long long)narrow.groups * narrow.chunks * narrow.slabs <= kResidentCtas) return narrow;
    return decode_plan_mt(M, N, K, si, widest, h16);
}

// The plan depends on the shape and on the W2A8_* switches of the environment.  Every entry
// point asks for it two to four times per call (workspace check, launch), and each evaluation
// reads a dozen environment variables, so the last plan is kept per thread together with a
// fingerprint of the environment block: the addresses of its strings (the C library makes a
// new string whenever a variable is set to a new value, so any change moves the fingerprint).
extern "C" char **environ;
static uint64_t env_fingerprint() {
    uint64_t h = 1469598103934665603ull;
    for (char **e = environ; e && *e; ++e) h = (h ^ (uint64_t)(uintptr_t)*e) * 1099511628211ull;
    return h;
}

static DecodePlan decode_plan(int M, int N, int K, const ShapeInfo &si, bool h16 = false) {
    struct Key { int M, N, K, G, h16, dev; uint64_t env; };
    thread_local Key key = {0, 0, 0, 0, 0, -2, 0};
    thread_local DecodePlan cached;
    const uint64_t env = env_fingerprint();
    const int dev = current_device();    // the plan depends on the SM count of the device
    if (key.M == M && key.N == N && key.K == K && key.G == si.G && key.h16 == (int)h16 && key.dev == dev &&
        key.env == env)
        return cached;
    cached = decode_plan_uncached(M, N, K, si, h16);
    key = {M, N, K, si.G, (int)h16, dev, env};
    return cached;
}

constexpr size_t kStatusBytes = 256;   // workspace header: status word

size_t decode_workspace_bytes(int M, int N, int K, const ShapeInfo &si) {
    const DecodePlan pl = decode_plan(M, N, K, si);
    size_t counters = ((size_t)4 * (N / 16) * pl.slabs + 255) / 256 * 256;   // >= any tile grouping
    // with an environment override in force, size for the finest split
    const bool overridden = env_int("W2A8_CHUNKS", 0) > 0 || env_int("W2A8_TG", 0) > 0 ||
                            env_int("W2A8_RING", 0) > 0 || env_int("W2A8_MT", 0) > 0;
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

template <int MT, int SPP, int TG, int RING, bool ONE, bool PARTIALS>
static cudaError_t launch_decode_ring(const DecodeParams &p, dim3 grid, size_t smem, cudaStream_t st) {
    static PerDeviceFlags configured;   // per kernel instantiation
    if (cudaError_t e = allow_dynamic_smem(w2a8_decode_kernel<MT, SPP, TG, RING, ONE, PARTIALS>, configured, 200 * 1024)) return e;
    return launch_kernel_cluster(w2a8_decode_kernel<MT, SPP, TG, RING, ONE, PARTIALS>, grid,
                                 dim3(kDecodeThreads), smem, st, pdl_enabled(),
                                 p.cluster ? (unsigned)p.chunks : 1u, p);
}

// RELAX instance of the default configuration (see kRelaxedCtasPerSm).
template <int MT, int SPP, bool ONE>
static cudaError_t launch_decode_relaxed(const DecodeParams &p, dim3 grid, size_t smem, cudaStream_t st) {
    static PerDeviceFlags configured;   // per kernel instantiation
    if (cudaError_t e = allow_dynamic_smem(w2a8_decode_kernel<MT, SPP, 1, kRound, ONE, false, false, false, true>, configured, 200 * 1024)) return e;
    return launch_kernel_cluster(w2a8_decode_kernel<MT, SPP, 1, kRound, ONE, false, false, false, true>, grid,
                                 dim3(kDecodeThreads), smem, st, pdl_enabled(),
                                 p.cluster ? (unsigned)p.chunks : 1u, p);
}

// Whether the grid is better served by the 7-per-SM instance: it has to fit 7 per SM at once
// (cluster grids: with room to spare, clusters are placed inside one GPC), and a two-slab grid
// must be too large for the 4 per SM its roomier default instance gets.
static bool prefer_relaxed(int mt, const DecodeParams &p, dim3 grid) {
    if (env_int("W2A8_RELAX", 1) == 0 || mt > 2) return false;
    const long long ctas = (long long)grid.x * grid.y * grid.z;
    const long long sms = sm_count();
    if (p.cluster) return mt == 1 && ctas <= sms * kRelaxedCtasPerSm / 2;
    if (ctas > sms * kRelaxedCtasPerSm) return false;
    return mt == 1 || ctas > sms * 4;
}

template <int MT, int SPP, int TG, bool ONE, bool PARTIALS>
static cudaError_t launch_decode_inst(const DecodeParams &p, int ring, dim3 grid, size_t smem, cudaStream_t st) {
    if constexpr (MT <= 2 && TG == 1 && !PARTIALS) {
        if (ring == kRound && prefer_relaxed(MT, p, grid)) return launch_decode_relaxed<MT, SPP, ONE>(p, grid, smem, st);
    }
    if (ring == 8) return launch_decode_ring<MT, SPP, TG, 8, ONE, PARTIALS>(p, grid, smem, st);
    return launch_decode_ring<MT, SPP, TG, kRound, ONE, PARTIALS>(p, grid, smem, st);
}

// 16-bit instances (binary16 scales, fp32 or bf16 result): default tile grouping and slot count.
template <int MT, int SPP, bool ONE>
static cudaError_t launch_decode_h16(const DecodeParams &p, dim3 grid, size_t smem, cudaStream_t st) {
    static PerDeviceFlags configured;   // per kernel instantiation
    if (cudaError_t e = allow_dynamic_smem(w2a8_decode_kernel<MT, SPP, 1, kRound, ONE, false, true>, configured, 200 * 1024)) return e;
    return launch_kernel_cluster(w2a8_decode_kernel<MT, SPP, 1, kRound, ONE, false, true>, grid,
                                 dim3(kDecodeThreads), smem, st, pdl_enabled(),
                                 p.cluster ? (unsigned)p.chunks : 1u, p);
}

// 16-bit-activation instances (bf16 x, fp32 scales, fp32 result): default grouping and slots.
template <int MT, int SPP, bool ONE>
static cudaError_t launch_decode_a16(const DecodeParams &p, dim3 grid, size_t smem, cudaStream_t st) {
    static PerDeviceFlags configured;   // per kernel instantiation
    if (cudaError_t e = allow_dynamic_smem(w2a8_decode_kernel<MT, SPP, 1, kRound, ONE, false, false, true>, configured, 200 * 1024)) return e;
    return launch_kernel_cluster(w2a8_decode_kernel<MT, SPP, 1, kRound, ONE, false, false, true>, grid,
                                 dim3(kDecodeThreads), smem, st, pdl_enabled(),
                                 p.cluster ? (unsigned)p.chunks : 1u, p);
}

template <int MT, int SPP, int TG>
static cudaError_t launch_decode_tg(const DecodeParams &p, int ring, bool want_partials, dim3 grid, size_t smem,
                                    cudaStream_t st) {
    if (want_partials) return launch_decode_inst<MT, SPP, TG, false, true>(p, ring, grid, smem, st);
    if (MT == 1 && p.M == 1) return launch_decode_inst<1, SPP, TG, true, false>(p, ring, grid, smem, st);
    return launch_decode_inst<MT, SPP, TG, false, false>(p, ring, grid, smem, st);
}

template <int MT, int SPP>
static cudaError_t launch_decode_mt(const DecodeParams &p, const DecodePlan &pl, bool want_partials,
                                    cudaStream_t st) {
    dim3 grid(pl.groups, pl.chunks, pl.slabs);
    if (p.a16) {
        if (MT == 1 && p.M == 1) return launch_decode_a16<1, SPP, true>(p, grid, pl.smem, st);
        return launch_decode_a16<MT, SPP, false>(p, grid, pl.smem, st);
    }
    if (p.h16) {
        if (MT == 1 && p.M == 1) return launch_decode_h16<1, SPP, true>(p, grid, pl.smem, st);
        return launch_decode_h16<MT, SPP, false>(p, grid, pl.smem, st);
    }
    if (pl.tg == 1) return launch_decode_tg<MT, SPP, 1>(p, pl.ring, want_partials, grid, pl.smem, st);
    return launch_decode_tg<MT, SPP, 2>(p, pl.ring, want_partials, grid, pl.smem, st);
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

// Enqueue the decode kernel.  `partials` != nullptr selects the parity export.  h16: w_scale
// points at binary16 values; y16 (with h16 only): y points at bf16 values.  a16: a points at
// bf16 activations and a_scale is not read.
int launch_decode(const int8_t *a, const float *a_scale, const uint32_t *packed,
                  const void *w_scale, void *y, int32_t *partials, int M, int N, int K,
                  int group, const ShapeInfo &si, void *workspace, cudaStream_t st, bool h16, bool y16,
                  bool a16, int ldy) {
    if ((h16 || a16) && partials) return W2A8_ERR_SHAPE;
    if (h16 && a16) return W2A8_ERR_SHAPE;
    // few tokens, whole blocks, fp32 scales, int8 activations, and a problem small enough to be
    // bound by latency: the persistent kernel
    if (!h16 && !a16 && !partials && gemv_preferred(M, K, group, N / 16, 1)) {
        const uint32_t *pk[1] = {packed};
        const float *sc[1] = {reinterpret_cast<const float *>(w_scale)};
        float *yy[1] = {reinterpret_cast<float *>(y)};
        return launch_gemv(a, a_scale, nullptr, nullptr, nullptr, 1, pk, sc, yy, &N, &ldy, M, K, group, st);
    }
    const DecodePlan pl = decode_plan(M, N, K, si, h16 || a16);
    DecodeParams p;
    p.a = a; p.a_scale = a_scale; p.packed = packed; p.w_scale = reinterpret_cast<const float *>(w_scale);
    p.y = reinterpret_cast<float *>(y); p.partials = partials; p.h16 = h16 ? 1 : 0; p.y16 = (h16 && y16) ? 1 : 0;
    p.a16 = a16 ? 1 : 0; p.ldy = ldy;
    p.M = M; p.N = N; p.K = K; p.G = si.G; p.group = group;
    p.blocks = si.blocks; p.tail_slices = si.tail_slices; p.words_per_row = si.words_per_row;
    p.chunks = pl.chunks; p.blocks_per_chunk = pl.blocks_per_chunk;
    p.blocks_per_group = (group + kBlockK - 1) / kBlockK; p.s_vec = pl.s_vec;
    p.cluster = (pl.cluster && partials == nullptr) ? 1 : 0;
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
