// Persistent form of the memory-bound W2A8 kernel for few tokens (decode): one CTA of 16
// warps per SM streams its share of the 16-channel tiles of one or several weight matrices
// that share their activations (q|k|v, gate|up), once.  The inner step is the cell of
// w2a8_cell.cuh (up-convert and int8 multiply-accumulate of Sec. II-C); the K-splitting and
// the quantiser fused into the GEMV are those of Sec. II-D, restated for sm_100a:
//
//  * Work.  The 16 warps are TG tiles side by side x KS K-lanes (TG * KS = 16); a K-lane owns
//    the same run of consecutive 256-k blocks in every tile it works on.  KS depends on K alone
//    and a tile's output is the sum of its K-lanes in lane order, so the bits of y do not depend
//    on which CTA or launch computed the tile: a grouped launch gives the bits of the separate
//    launches.  CTA b owns a contiguous range of tiles and walks it in rounds (as many tiles as
//    the partial buffer holds); a K-lane parks its sums of a tile in shared memory and goes on
//    to its next tile.  Warps never meet inside a round: one CTA barrier per round, after which
//    the K-lanes are added, scaled and stored while the warps are already in the next round
//    (two partial buffers).
//  * Data movement.  Every warp runs its own ring of kGvRing landing slots (1 KB of weights +
//    256 B of scales per cell) filled by per-thread asynchronous copies, and refills a slot as
//    soon as it has consumed it, across tiles and rounds: the stream never drains inside a
//    launch.  The first ring-full is requested before the kernel waits for its predecessor in
//    the stream (weights are frozen data), so under programmatic dependent launch it overlaps
//    that kernel's tail -- and because one CTA takes half of an SM's registers and less than
//    half of its shared memory, the whole next launch is resident and streaming while this one
//    computes.
//  * Activations.  When a K-lane is a single block (K <= 4096) and there are at most 8 tokens,
//    the lane's activation bytes are loaded once and stay in registers for the whole launch
//    (BCACHE).  Otherwise they are read per cell, through L1 from the int8 rows a8_quantize wrote
//    or from a copy staged once per CTA in shared memory with a row pitch that makes the
//    B-fragment loads conflict-free.  The staged copy is either copied from those rows or
//    quantised by the CTA itself from the bf16 input (the fused operator of Sec. II-D; every CTA
//    repeats the abs-max of the few tokens, which costs less than a separate launch and its
//    hand-over).
#include <stdlib.h>

#include "w2a8_cell.cuh"
#include "w2a8_quant.cuh"

namespace w2a8 {

int env_int(const char *name, int dflt);

constexpr int kGvWarps = 16;                      // warps per CTA of the full-SM form (the other has 8, two CTAs per SM)
constexpr int kGvRing = 4;                        // landing slots (cells) per warp (a power of two)
constexpr int kGvMaxMats = 4;                     // weight matrices per launch
constexpr int kGvWSlot = 2 * 32 * 16;             // weights of a cell: two channels x 32 lanes x 16 B
constexpr int kGvSSlot = 16 * 16;                 // scales of a cell: 16 channels x 16 B
constexpr int kGvWarpBytes = kGvRing * (kGvWSlot + kGvSSlot);
constexpr int kGvRingBytes = kGvWarps * kGvWarpBytes;
constexpr int kGvPartBytes = 32 * 1024;           // partial sums of one round (there are two buffers)
constexpr int kGvMaxFuseM = 8;                    // most tokens the kernel quantises itself
constexpr int kGvMaxTokens = 32;                  // most tokens the kernel takes at all
constexpr int kGvMaxSmem = 220 * 1024;            // dynamic shared memory the kernel may ask for
constexpr int kGvMaxSmemHalf = 112 * 1024;        // the same for the 8-warp form (two CTAs per SM)
constexpr int kGvPartBytesHalf = 16 * 1024;       // its partial sums of one round
constexpr int kGvActPad = 64;                     // staged token rows are K + 64 bytes apart

struct GemvMat {
    const uint32_t *packed;
    const float *w_scale;
    float *y;
    int tile_end;         // tiles of this matrix and of all matrices before it
    int ldy;              // elements between consecutive token rows of y
};

struct GemvParams {
    GemvMat mat[kGvMaxMats];
    const int8_t *a;            // int8 activations [M][K] (not fused)
    const float *a_scale;       // their scales [M] (not fused)
    const uint16_t *x;          // bf16 activations [M][K]: the kernel quantises them itself
    int8_t *a_out;              // fused: where the int8 rows are also written (may be null)
    float *a_scale_out;         // fused: where the token scales are also written (may be null)
    int nmats, M, K, G, blocks, words_per_row;
    int tiles, slabs, vtiles;   // vtiles = tiles x slabs of 8 * MT tokens ("virtual tiles")
    int tg, ks_shift;           // tiles side by side; K-lanes per tile = 1 << ks_shift
    int round_tiles;            // virtual tiles per round (a multiple of 4 * tg)
    int per_cta, extra;         // CTA b owns per_cta (+ 1 if b < extra) consecutive virtual tiles
    int blocks_per_group;       // 256-k blocks per scale group (groups of 256 and more)
    int s_vec;                  // the scales of a cell and channel can be copied as one unit
    int act_stride;             // bytes between staged token rows
};

// MT: 8-token slabs per virtual tile; SPP: 64-k slices per scale group (capped at 4); ONE: a single
// token; ASMEM: activations staged in shared memory (copied, or quantised here when p.x is set);
// BCACHE: NB blocks per K-lane and all tokens in one tile (M <= 8 * MT): activation fragments live
// in registers.  W: warps per CTA.  16: one CTA per SM, NB = 1.  8: two CTAs per SM (the same warps
// and registers per SM), NB = 2 -- a launch's CTAs then leave and arrive in units of half an SM, so
// the head of the next launch (under programmatic dependent launch: its first ring-full of weights)
// overlaps the tail of this one instead of waiting for a whole SM.
template <int MT, int SPP, bool ONE, bool ASMEM, bool BCACHE, int W>
__global__ void __launch_bounds__(W * 32, W == 8 ? 2 : 1)
w2a8_gemv_kernel(const __grid_constant__ GemvParams p) {
    constexpr int kThreads = W * 32;
    constexpr int kRingBytes = W * kGvWarpBytes;
    constexpr int NB = (BCACHE && W == 8) ? 2 : 1;      // blocks per K-lane with register-resident activations
    constexpr int SPB = 4 / SPP;                  // scales per block and channel
    constexpr int kRed = ONE ? 16 : MT * 128;     // sums a K-lane parks per tile
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ uint32_t wmax[kGvMaxFuseM][W];
    __shared__ float s_scale[kGvMaxTokens];     // token scales: written here, read by the epilogue
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int gq = lane >> 2, t = lane & 3;
    const int TG = p.tg, KS = 1 << p.ks_shift;
    const int tl = warp % TG, ks = warp / TG;
    // this K-lane's run of blocks in every tile
    const int b0 = (ks * p.blocks) >> p.ks_shift;
    const int n_my = BCACHE ? NB : (((ks + 1) * p.blocks) >> p.ks_shift) - b0;

    unsigned char *wslots = smem + warp * kGvWarpBytes + lane * 16;
    unsigned char *sslots = smem + warp * kGvWarpBytes + kGvRing * kGvWSlot;
    const uint32_t wslots_u32 = smem_u32(wslots);
    const uint32_t sslot_u32 = smem_u32(sslots) + (lane & 15) * 16;
    const int part_floats = p.round_tiles * KS * kRed;
    float *part_all = reinterpret_cast<float *>(smem + kRingBytes);
    unsigned char *act = smem + kRingBytes + 2 * part_floats * 4;

    // this CTA's virtual tiles: v_lo + li, li < nt_cta; this warp takes li = tl, tl + TG, ...
    const int v_lo = (int)blockIdx.x * p.per_cta + min((int)blockIdx.x, p.extra);
    const int nt_cta = p.per_cta + ((int)blockIdx.x < p.extra ? 1 : 0);

    // Virtual tile vt: its matrix and first channel; this lane's 16-byte unit of block b0 in row
    // n0 + gq, the scales of block b0 in row n0 + (lane & 15), the tile's outputs in token row 0,
    // its token slab, and the last tile of its matrix.
    struct Where { const uint32_t *w; const float *s; float *y; int ldy, slab, mat_end; };
    auto locate = [&](int vt, Where &o) {
        const int T = p.slabs == 1 ? vt : vt / p.slabs;
        o.slab = p.slabs == 1 ? 0 : vt - T * p.slabs;
        const uint32_t *packed = p.mat[0].packed;
        const float *w_scale = p.mat[0].w_scale;
        float *y = p.mat[0].y;
        int ldy = p.mat[0].ldy, first = 0, end = p.mat[0].tile_end;
#pragma unroll
        for (int i = 1; i < kGvMaxMats; ++i) {
            if (i < p.nmats && T >= p.mat[i - 1].tile_end) {
                packed = p.mat[i].packed; w_scale = p.mat[i].w_scale; y = p.mat[i].y; ldy = p.mat[i].ldy;
                first = p.mat[i - 1].tile_end; end = p.mat[i].tile_end;
            }
        }
        const int n0 = (T - first) * 16;
        o.w = packed + (size_t)(n0 + gq) * p.words_per_row + 16 * b0 + 4 * t;
        o.s = w_scale + (size_t)(n0 + (lane & 15)) * p.G + (SPP != 4 ? SPB * b0 : 0);
        o.y = y + n0;
        o.ldy = ldy;
        o.mat_end = end;
    };

    // ---- request side: a cursor over this warp's cells, kGvRing cells ahead of the compute --
    int q_li = tl, q_c = 0;
    Where qw;
    if (q_li < nt_cta && n_my > 0) locate(v_lo + q_li, qw);
    else q_li = nt_cta;
    const size_t w_tile_step = (size_t)TG * 16 * p.words_per_row;       // words from a tile to the warp's next
    const size_t s_tile_step = (size_t)TG * 16 * p.G;
    auto request = [&](int slot) {
        const uint32_t wdst = wslots_u32 + slot * kGvWSlot;
        cp_async16(wdst, qw.w + 16 * q_c);
        cp_async16(wdst + 32 * 16, qw.w + (size_t)8 * p.words_per_row + 16 * q_c);
        if (lane < 16) {
            const uint32_t sdst = sslot_u32 + slot * kGvSSlot;
            if constexpr (SPP == 4) {
                const int gi = p.blocks_per_group >= p.blocks ? 0 : (b0 + q_c) / p.blocks_per_group;
                cp_async4(sdst, qw.s + gi);
            } else if (p.s_vec) {
                if constexpr (SPP == 1) cp_async16(sdst, qw.s + q_c * SPB);
                else                    cp_async8(sdst, qw.s + q_c * SPB);
            } else {
#pragma unroll
                for (int i = 0; i < SPB; ++i) cp_async4(sdst + 4 * i, qw.s + q_c * SPB + i);
            }
        }
        if (++q_c == n_my) {
            q_c = 0;
            q_li += TG;
            if (q_li < nt_cta) {
                // the next tile of this warp: TG tiles on in the same matrix, unless a matrix ends
                // in between or the tiles are token slabs of one another
                if (p.slabs == 1 && (p.nmats == 1 || v_lo + q_li < qw.mat_end)) {
                    qw.w += w_tile_step;
                    qw.s += s_tile_step;
                } else {
                    locate(v_lo + q_li, qw);
                }
            }
        }
    };
    // Weights and scales are frozen data: the first ring-full is requested before the wait for
    // the previous kernel of the stream.  One copy group per cell, empty groups past the end.
#pragma unroll
    for (int r = 0; r < kGvRing; ++r) {
        if (q_li < nt_cta) request(r);
        cp_async_commit();
        if (r == 0) pdl_launch_dependents();
    }
    pdl_wait();
    // The token scales are only needed by the epilogue, at the very end of the critical path of a
    // short launch: fetch them now (the first CTA barrier orders them before their use).
    if (!(ASMEM && p.x != nullptr) && threadIdx.x < p.M) s_scale[threadIdx.x] = p.a_scale[threadIdx.x];

    // ---- activations into shared memory (ASMEM) ---------------------------------------
    if constexpr (ASMEM) {
        if (p.x) {
            // Quantise the M <= 8 token rows here (same operations as a8_quantize, same bits).
            const int nvec = p.K >> 3;                    // 16-byte vectors (8 bf16) per row
            uint32_t am[kGvMaxFuseM];
#pragma unroll
            for (int m = 0; m < kGvMaxFuseM; ++m) am[m] = 0u;
            for (int i = threadIdx.x; i < nvec; i += kThreads) {
#pragma unroll
                for (int m = 0; m < kGvMaxFuseM; ++m)
                    if (m < p.M)
                        am[m] = amax8(am[m], ld_act16(reinterpret_cast<const int8_t *>(p.x + (size_t)m * p.K) + 16 * i));
            }
#pragma unroll
            for (int m = 0; m < kGvMaxFuseM; ++m) {
                if (m < p.M) {
                    uint32_t v = am[m];
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) v = max(v, __shfl_xor_sync(0xFFFFFFFFu, v, o));
                    if (lane == 0) wmax[m][warp] = v;
                }
            }
            __syncthreads();
            for (int m = 0; m < p.M; ++m) {
                uint32_t v = wmax[m][lane & (W - 1)];
#pragma unroll
                for (int o = W / 2; o > 0; o >>= 1) v = max(v, __shfl_xor_sync(0xFFFFFFFFu, v, o));
                float inv;
                const float s = quant_scale(v, &inv);
                if (threadIdx.x == 0) {
                    s_scale[m] = s;
                    if (p.a_scale_out && blockIdx.x == 0) p.a_scale_out[m] = s;
                }
                const int8_t *xr = reinterpret_cast<const int8_t *>(p.x + (size_t)m * p.K);
                int round = 0;
                for (int i = threadIdx.x; i < nvec; i += kThreads, ++round) {
                    const uint4 xv = ld_act16(xr + 16 * i);
                    uint2 o;
                    o.x = quant4(xv.x, xv.y, inv);
                    o.y = quant4(xv.z, xv.w, inv);
                    *reinterpret_cast<uint2 *>(act + (size_t)m * p.act_stride + 8 * i) = o;
                    // the int8 rows for the caller: the CTAs share the writing
                    if (p.a_out && (round % (int)gridDim.x) == (int)blockIdx.x)
                        *reinterpret_cast<uint2 *>(p.a_out + (size_t)m * p.K + 8 * i) = o;
                }
            }
        } else {
            const int nvec = p.K >> 4;                    // 16-byte vectors per int8 row
            for (int m = 0; m < p.M; ++m)
                for (int i = threadIdx.x; i < nvec; i += kThreads)
                    *reinterpret_cast<uint4 *>(act + (size_t)m * p.act_stride + 16 * i) =
                        ld_act16(p.a + (size_t)m * p.K + 16 * i);
        }
        __syncthreads();
    }
    const uint32_t act_u32 = smem_u32(act);

    // This lane's activation bytes of block kb, token row `row` (MMA column gq of a slab).  Token
    // columns of an MMA are independent and columns beyond M are never stored: they read the last row.
    auto act_at = [&](int row, int kb) -> const int8_t * {
        if constexpr (ASMEM) return act_ptr(act_u32 + row * p.act_stride + kb * kBlockK + t * 16);
        else                 return p.a + (size_t)row * p.K + kb * kBlockK + t * 16;
    };
    uint4 B[NB][MT][4];
    if constexpr (BCACHE) {
#pragma unroll
        for (int nb = 0; nb < NB; ++nb)
#pragma unroll
            for (int mt = 0; mt < MT; ++mt) {
                const int8_t *src = act_at(min(8 * mt + gq, p.M - 1), b0 + nb);
#pragma unroll
                for (int s = 0; s < 4; ++s)
                    B[nb][mt][s] = ASMEM ? ld_act16_smem(src + s * kSliceK) : ld_act16(src + s * kSliceK);
            }
    }

    // ---- compute side ---------------------------------------------------------------------
    const DecodeParams no_params = {};   // the full-block, no-export cell reads none of it
    int slot = 0, buf = 0;
    for (int rbase = 0; rbase < nt_cta; rbase += p.round_tiles, buf ^= 1) {
        const int nt = min(p.round_tiles, nt_cta - rbase);
        float *part = part_all + buf * part_floats + ks * kRed;
        // park the sums of one tile (local index li in the round) for the final addition
        auto park = [&](int li, float (&acc)[MT][4]) {
            float *dst = part + li * KS * kRed;
            if constexpr (ONE) {
                if (t == 0) { dst[gq] = acc[0][0]; dst[gq + 8] = acc[0][2]; }
            } else {
#pragma unroll
                for (int mt = 0; mt < MT; ++mt)
#pragma unroll
                    for (int i = 0; i < 4; ++i) dst[(mt * 4 + i) * 32 + lane] = acc[mt][i];
            }
        };
        if constexpr (BCACHE) {
            // NB cells per tile; a ring-full of tiles per trip so that the slot offsets are immediates
            // (rounds are multiples of that many tiles per warp, so every round starts at slot 0)
            constexpr int kTrip = kGvRing / NB;
            for (int li = tl; li < nt; li += kTrip * TG) {
#pragma unroll
                for (int u = 0; u < kTrip; ++u) {
                    if (li + u * TG < nt) {                       // warp-uniform
                        float acc[MT][4];
#pragma unroll
                        for (int mt = 0; mt < MT; ++mt)
#pragma unroll
                            for (int i = 0; i < 4; ++i) acc[mt][i] = 0.f;
#pragma unroll
                        for (int nb = 0; nb < NB; ++nb) {
                            const int sl = u * NB + nb;           // a constant after unrolling
                            cp_async_wait_group<kGvRing - 1>();
                            __syncwarp();                         // the scales were copied by other lanes
                            const uint4 wa = *reinterpret_cast<const uint4 *>(wslots + sl * kGvWSlot);
                            const uint4 wb = *reinterpret_cast<const uint4 *>(wslots + sl * kGvWSlot + 32 * 16);
                            const unsigned char *sc0 = sslots + sl * kGvSSlot + gq * 16;
                            compute_cell_breg<MT, SPP, ONE>(wa, wb, sc0, sc0 + 8 * 16, B[nb], acc);
                            __syncwarp();                         // every lane has read the slot
                            if (q_li < nt_cta) request(sl);
                            cp_async_commit();
                        }
                        park(li + u * TG, acc);
                    }
                }
            }
        } else {
            for (int li = tl; li < nt; li += TG) {
                int m0 = 0;
                if (p.slabs != 1) m0 = ((v_lo + rbase + li) % p.slabs) * (8 * MT);
                const int mrows = min(8 * MT, p.M - m0);
                float acc[MT][4];
#pragma unroll
                for (int mt = 0; mt < MT; ++mt)
#pragma unroll
                    for (int i = 0; i < 4; ++i) acc[mt][i] = 0.f;
                const int8_t *brow[MT];
#pragma unroll
                for (int mt = 0; mt < MT; ++mt) brow[mt] = act_at(m0 + min(8 * mt + gq, mrows - 1), b0);
                for (int c = 0; c < n_my; ++c) {
                    cp_async_wait_group<kGvRing - 1>();
                    __syncwarp();
                    const uint4 wa = *reinterpret_cast<const uint4 *>(wslots + slot * kGvWSlot);
                    const uint4 wb = *reinterpret_cast<const uint4 *>(wslots + slot * kGvWSlot + 32 * 16);
                    const uint32_t w0s[4] = {wa.x, wa.y, wa.z, wa.w};
                    const uint32_t w1s[4] = {wb.x, wb.y, wb.z, wb.w};
                    const unsigned char *sc0 = sslots + slot * kGvSSlot + gq * 16;
                    const int8_t *bc[MT];
#pragma unroll
                    for (int mt = 0; mt < MT; ++mt) bc[mt] = brow[mt] + c * kBlockK;
                    compute_cell<MT, SPP, ONE, false, true, false, ASMEM>(no_params, w0s, w1s, sc0, sc0 + 8 * 16, bc,
                                                                          0, 0, 0, gq, t, acc);
                    __syncwarp();
                    if (q_li < nt_cta) request(slot);
                    cp_async_commit();
                    slot = (slot + 1) & (kGvRing - 1);
                }
                park(li, acc);
            }
        }
        __syncthreads();

        // ---- the round's outputs: K-lanes of a tile in lane order, scale, store ----------------
        const float *rpart = part_all + buf * part_floats;
        for (int e = threadIdx.x; e < nt * kRed; e += kThreads) {
            const int li = e / kRed, r = e % kRed;
            Where ow;
            locate(v_lo + rbase + li, ow);
            int mm, nn;
            if constexpr (ONE) {
                mm = 0;
                nn = r;
            } else {
                const int el = r & 31, ei = r >> 5;
                mm = ow.slab * (8 * MT) + 8 * (ei >> 2) + 2 * (el & 3) + (ei & 1);
                nn = (el >> 2) + 8 * ((ei & 3) >> 1);
            }
            if (mm >= p.M) continue;
            // all K-lane sums of the output are fetched first (independent loads), then added in
            // lane order: the order, and with it the bits of y, does not depend on anything else
            const float *src = rpart + li * KS * kRed + r;
            float part[W];
#pragma unroll
            for (int k2 = 0; k2 < W; ++k2) part[k2] = k2 < KS ? src[k2 * kRed] : 0.f;
            float v = 0.f;
#pragma unroll
            for (int k2 = 0; k2 < W; ++k2) v += part[k2];
            ow.y[(size_t)mm * ow.ldy + nn] = v * (s_scale[mm] * (1.0f / kCodeGain));
        }
    }
}

// ---- host side ---------------------------------------------------------------------------
struct GemvPlan {
    int mt, slabs, vtiles, ks_shift, tg, round_tiles, grid, asmem, bcache, act_stride, s_vec;
    int warps;                  // warps per CTA: 16 (one CTA per SM) or 8 (two)
    size_t smem;
};

// Warps per CTA for a problem: the 8-warp form (two CTAs per SM) for up to eight tokens when its
// shared memory fits twice into an SM with the activations staged (so that the fused and the
// unfused call of a shape run the same form).  A function of M and K alone, like the K-lanes: the
// bits of y do not depend on how the matrices of a layer are grouped into launches.
// W2A8_GEMV_WARPS = 8 / 16 overrides (8 only where it fits).
static int gemv_warps(int M, int K) {
    const bool fits = M <= 8 && (size_t)8 * kGvWarpBytes + 2 * (size_t)kGvPartBytesHalf + (size_t)M * (K + kGvActPad) <=
                                    (size_t)kGvMaxSmemHalf;
    const int forced = env_int("W2A8_GEMV_WARPS", 0);
    if (forced == 16) return 16;
    if (forced == 8) return fits ? 8 : 16;
    return fits ? 8 : 16;
}

// Whether this kernel serves the shape at all: whole 256-k blocks only (a ragged last block is
// left to the one-shot streaming kernel), at most kGvMaxTokens tokens.  W2A8_GEMV=0 switches the
// kernel off, and so does any switch that forces a launch plan of the one-shot kernel.
bool gemv_supported(int M, int K, int group) {
    (void)group;
    if (K % kBlockK != 0 || M > kGvMaxTokens) return false;
    if (env_int("W2A8_GEMV", 1) == 0) return false;
    for (const char *name : {"W2A8_CHUNKS", "W2A8_TG", "W2A8_RING", "W2A8_MT", "W2A8_CLUSTER", "W2A8_MIN_WARPS",
                             "W2A8_RELAX"})
        if (getenv(name) && *getenv(name)) return false;
    return true;
}

// Whether the persistent kernel is expected to beat the one-shot streaming kernel (one launch per
// matrix) on `count` matrices of `tiles` 16-channel tiles in all.  Measured on B200 (us per call
// incl. the quantiser launch, back to back over rotating weight copies; one-shot / persistent):
//   Llama-3-8B linears, group 64, M = 1, 4, 8, 16 tokens
//     q|k|v  4096 x (4096+1024+1024):   8.9 / 5.2    9.3 / 5.3    9.9 / 5.8   11.4 / 12.9
//     o      4096 x 4096:               4.7 / 4.7    5.2 / 4.8    5.2 / 5.2    6.1 / 11.4
//     gate   4096 x 14336 (alone):      5.0 / 6.2
//     gate|up 4096 x (14336+14336):    11.7 / 10.9  12.4 / 12.9  13.2 / 13.1  19.2 / 24.6
//     down   14336 x 4096:              7.4 / 8.3    8.2 / 10.0   8.3 / 10.4  14.3 / 12.9
//   Llama-3-70B linears, group 128, M = 1, 8, 32 tokens
//     q|k|v  8192 x (8192+1024+1024):  13.4 / 10.3  14.8 / 12.4  31.9 / 28.8
//     o      8192 x 8192:               8.4 / 9.3    9.3 / 10.3  23.7 / 23.7
//     gate|up 8192 x (28672+28672):    47.2 / 33.0  55.7 / 49.0   140 / 142
//     down   28672 x 8192:             27.8 / 23.2  32.0 / 29.7  80.7 / 64.6
// The one-shot kernel is at its best when the whole problem is one wave of its CTAs (8 per SM, 16
// cells of one 16-channel tile x one 256-k block each); the persistent kernel is ahead on groups
// of matrices that are latency-bound one by one, on problems of more than one such wave, and
// where a K-lane is a single block so that the activation fragments stay in registers (K <= 4096,
// at most 16 tokens) unless the problem is a single matrix near the one-wave size.  (The table was
// taken before the register-resident form existed for 9 .. 16 tokens and before the 8-warp form: with
// that one the persistent side reads 4.75 / 4.2 / 10.1 / 7.7 at one token and 5.2 / 4.5 / 11.4 / 9.8 at
// four for q|k|v / o / gate|up / down, which leaves the choices as they are.)
// W2A8_GEMV=2: whenever it serves the shape; W2A8_GEMV=0: never.
bool gemv_preferred(int M, int K, int group, int tiles, int count) {
    if (!gemv_supported(M, K, group)) return false;
    if (env_int("W2A8_GEMV", 1) == 2) return true;
    const long long blocks = K / kBlockK, cells = (long long)tiles * blocks;
    const long long one_wave = (long long)sm_count() * 8 * 16;          // cells the one-shot kernel holds at once
    if (M <= 8) {
        if (count >= 2 || cells > one_wave) return true;
        return blocks <= 16 && cells <= 8192;
    }
    // two slabs of 8 tokens per tile: ahead with register-resident activations (up to 16 tokens,
    // K <= 4096) and on long rows
    return (M <= 16 && blocks <= 16) || blocks >= 32;
}

// The kernel can quantise the activations itself for this many tokens and this K.
bool gemv_can_fuse(int M, int K, int group) {
    if (!gemv_supported(M, K, group) || M > kGvMaxFuseM) return false;
    if (gemv_warps(M, K) == 8) return true;      // by construction of gemv_warps
    return (size_t)M * (K + kGvActPad) <= (size_t)(kGvMaxSmem - kGvRingBytes - 2 * kGvPartBytes);
}

// The paper exposes the abs-max scales "inside the GEMM or in a kernel of their own" as a knob
// (Sec. II-D) and finds the fused form ahead for GEMV-sized problems only.  Here every CTA repeats
// the abs-max, and under programmatic dependent launch a separate quantiser launch hides behind the
// weight prefetch of the kernel that follows it.  Measured on B200 (us per call, fused / quantiser
// launch + persistent kernel): one token, K = 4096: 5.3 / 4.75 (q|k|v), 4.7 / 4.2 (o), 10.7 / 10.1
// (gate|up); one token, K = 14336: 9.3 / 7.7; four tokens, K = 4096: 8.8 / 5.2; eight: 13.9 / 5.7.  So
// the separate launch is ahead everywhere on the device (the layer pass at one token: 25.9 against
// 28.3 us); what fusing saves is one launch on the host.  The automatic rule therefore fuses only up
// to W2A8_FUSE_MAX_ELEMS values of M * K per CTA (default 0: never; W2A8_FUSE_ON asks for it).
bool gemv_fuse_preferred(int M, int K, int group) {
    if (!gemv_can_fuse(M, K, group)) return false;
    return (long long)M * K <= (long long)env_int("W2A8_FUSE_MAX_ELEMS", 0);
}

static GemvPlan gemv_plan(int M, int K, int tiles, const ShapeInfo &si, bool fused) {
    GemvPlan pl;
    pl.mt = M <= 8 ? 1 : 2;
    pl.slabs = (M + 8 * pl.mt - 1) / (8 * pl.mt);
    pl.warps = gemv_warps(M, K);
    const int ctas_per_sm = 16 / pl.warps;
    // K-lanes per tile with 16 warps: 16 when the row has at least 16 blocks, else 8, else 4 (with 2, 4
    // tiles side by side); half as many with 8 warps.  A function of M and K alone.
    const int ks16 = si.blocks >= 16 ? 16 : si.blocks >= 8 ? 8 : 4;
    const int ks = ks16 / ctas_per_sm;
    pl.ks_shift = ks == 16 ? 4 : ks == 8 ? 3 : ks == 4 ? 2 : 1;
    pl.tg = pl.warps / ks;
    // register-resident activations: a K-lane holds one block (16 warps) or two (8 warps)
    pl.bcache = pl.slabs == 1 && si.blocks == ks16 && env_int("W2A8_GEMV_BCACHE", 1) != 0;
    const int nb = pl.bcache ? ctas_per_sm : 1;
    pl.vtiles = tiles * pl.slabs;
    const int sms = sm_count() * ctas_per_sm;
    pl.grid = pl.vtiles < sms ? pl.vtiles : sms;
    const int ring_bytes = pl.warps * kGvWarpBytes;
    const int part_budget = pl.warps == 8 ? kGvPartBytesHalf : kGvPartBytes;
    const size_t max_smem = pl.warps == 8 ? kGvMaxSmemHalf : kGvMaxSmem;
    // tiles per round: what one partial buffer holds, no more than a CTA has, in units that keep
    // the ring aligned (see the BCACHE loop)
    const int red_floats = (M == 1) ? 16 : pl.mt * 128;
    const int unit = pl.bcache ? (kGvRing / nb) * pl.tg : pl.tg;
    const int per_cta = (pl.vtiles + pl.grid - 1) / pl.grid;
    int fit = part_budget / (ks * red_floats * 4) / unit * unit;
    if (fit < unit) fit = unit;
    const int need = (per_cta + unit - 1) / unit * unit;
    pl.round_tiles = need < fit ? need : fit;
    pl.s_vec = (si.spp == 1 && si.G % 4 == 0) || (si.spp == 2 && si.G % 2 == 0);
    pl.act_stride = K + kGvActPad;
    const size_t act_bytes = (size_t)M * pl.act_stride;
    const size_t part_bytes = (size_t)2 * pl.round_tiles * ks * red_floats * 4;
    // staged activations: always when the kernel quantises; else for two-slab tiles when they fit
    // (their B-fragment loads from L1 touch eight lines each), or on request
    const int forced = env_int("W2A8_GEMV_ASMEM", -1);
    pl.asmem = fused ? 1 : (forced >= 0 ? (forced != 0) : (pl.mt == 2)) &&
                           ring_bytes + part_bytes + act_bytes <= max_smem;
    pl.smem = (size_t)ring_bytes + part_bytes + (pl.asmem ? act_bytes : 0);
    return pl;
}

template <int MT, int SPP, bool ONE, bool ASMEM, bool BCACHE, int W>
static cudaError_t launch_gemv_w(const GemvParams &p, const GemvPlan &pl, cudaStream_t st) {
    static PerDeviceFlags configured;   // per kernel instantiation
    if (cudaError_t e = allow_dynamic_smem(w2a8_gemv_kernel<MT, SPP, ONE, ASMEM, BCACHE, W>, configured,
                                           W == 8 ? kGvMaxSmemHalf : kGvMaxSmem))
        return e;
    return launch_kernel(w2a8_gemv_kernel<MT, SPP, ONE, ASMEM, BCACHE, W>, dim3(pl.grid), dim3(W * 32), pl.smem, st,
                         pdl_enabled(), p);
}

template <int MT, int SPP, bool ONE, bool ASMEM, bool BCACHE>
static cudaError_t launch_gemv_inst(const GemvParams &p, const GemvPlan &pl, cudaStream_t st) {
    if constexpr (MT == 1) {
        if (pl.warps == 8) return launch_gemv_w<MT, SPP, ONE, ASMEM, BCACHE, 8>(p, pl, st);
    }
    return launch_gemv_w<MT, SPP, ONE, ASMEM, BCACHE, 16>(p, pl, st);
}

template <int MT, int SPP, bool ONE>
static cudaError_t launch_gemv_act(const GemvParams &p, const GemvPlan &pl, cudaStream_t st) {
    if (pl.bcache)
        return pl.asmem ? launch_gemv_inst<MT, SPP, ONE, true, true>(p, pl, st)
                        : launch_gemv_inst<MT, SPP, ONE, false, true>(p, pl, st);
    return pl.asmem ? launch_gemv_inst<MT, SPP, ONE, true, false>(p, pl, st)
                    : launch_gemv_inst<MT, SPP, ONE, false, false>(p, pl, st);
}

template <int SPP>
static cudaError_t launch_gemv_spp(const GemvParams &p, const GemvPlan &pl, cudaStream_t st) {
    if (pl.mt == 1 && p.M == 1) return launch_gemv_act<1, SPP, true>(p, pl, st);
    if (pl.mt == 1) return launch_gemv_act<1, SPP, false>(p, pl, st);
    return launch_gemv_act<2, SPP, false>(p, pl, st);
}

// Enqueue one launch over `count` weight matrices (1 .. 4) that share their activations.  Either
// a / a_scale (int8 rows from a8_quantize) or x_bf16 (the kernel quantises; a_out / a_scale_out,
// if not null, receive what a8_quantize would write).  The caller has checked the arguments and
// gemv_supported (and gemv_can_fuse when x_bf16 is given).
int launch_gemv(const int8_t *a, const float *a_scale, const void *x_bf16, int8_t *a_out, float *a_scale_out,
                int count, const uint32_t *const *packed, const float *const *w_scale, float *const *y,
                const int *N, const int *ldy, int M, int K, int group, cudaStream_t st) {
    if (count < 1 || count > kGvMaxMats) return W2A8_ERR_SHAPE;
    ShapeInfo si;
    if (!shape_ok(M, N[0], K, group, &si)) return W2A8_ERR_SHAPE;
    GemvParams p = {};
    int tiles = 0;
    for (int i = 0; i < count; ++i) {
        if (N[i] < 16 || N[i] % 16 != 0) return W2A8_ERR_SHAPE;
        tiles += N[i] / 16;
        p.mat[i].packed = packed[i]; p.mat[i].w_scale = w_scale[i]; p.mat[i].y = y[i];
        p.mat[i].tile_end = tiles; p.mat[i].ldy = ldy[i];
    }
    const GemvPlan pl = gemv_plan(M, K, tiles, si, x_bf16 != nullptr);
    if (x_bf16 && !pl.asmem) return W2A8_ERR_SHAPE;
    p.a = a; p.a_scale = a_scale; p.x = reinterpret_cast<const uint16_t *>(x_bf16);
    p.a_out = a_out; p.a_scale_out = a_scale_out;
    p.nmats = count; p.M = M; p.K = K; p.G = si.G; p.blocks = si.blocks; p.words_per_row = si.words_per_row;
    p.tiles = tiles; p.slabs = pl.slabs; p.vtiles = pl.vtiles; p.tg = pl.tg; p.ks_shift = pl.ks_shift;
    p.round_tiles = pl.round_tiles; p.per_cta = pl.vtiles / pl.grid; p.extra = pl.vtiles % pl.grid;
    p.blocks_per_group = (group + kBlockK - 1) / kBlockK; p.s_vec = pl.s_vec; p.act_stride = pl.act_stride;
    cudaError_t e = si.spp == 1 ? launch_gemv_spp<1>(p, pl, st)
                  : si.spp == 2 ? launch_gemv_spp<2>(p, pl, st)
                                : launch_gemv_spp<4>(p, pl, st);
    return e == cudaSuccess ? W2A8_OK : W2A8_ERR_CUDA;
}

}  // namespace w2a8
