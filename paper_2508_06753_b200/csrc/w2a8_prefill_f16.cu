// Tensor-core kernel for many tokens with 16-bit operands: the "alternative implementation" of
// Sec. II -- the 2-bit codes become 16-bit weights and meet 16-bit activations in a 16-bit x
// 16-bit -> 32-bit matrix instruction, so that no int32 -> float conversion follows -- on the
// 5th-generation tensor cores (tcgen05.mma kind::f16, bf16 operands, fp32 accumulators in tensor
// memory).  The structure is that of the int8 kernel (w2a8_prefill.cu): persistent CTAs walk
// 128-channel x 128-token tiles; unpack warps turn packed words into the K-major, 128-byte-swizzled
// A operand; TMA brings the activations as the B operand; MMA issuers hand accumulator buffers to
// drain warps in units of two scale groups.  What differs:
//   * A stage is 128 k (half a 256-k block of the packed layout): 128 rows x 128 k of bf16 are
//     two [128][128 B] sub-tiles, as are the activations; one MMA covers K = 16.
//   * The unpack writes the bf16 values code - 2 (exact): one mask, one byte permute with an
//     exponent byte and one packed subtraction per two weights (see compute_cell_a16), four warps.
//   * The accumulators are fp32, so the drain is a tensor-memory load and one packed FMA per two
//     values -- no conversion instruction, which is what bounds the int8 kernel at small groups.
// It serves w2a16_gemm (bf16 activations as they are: the sums are fp32 sums of exact products)
// and, with the int8 activations copied out as bf16 values first, w2a8_gemm: every product and
// every partial sum of a group is then an integer below 2^24, so the fp32 group sums are the
// exact int32 sums of the int8 kernel, bit for bit.
#include <cuda_bf16.h>

#include <type_traits>

#include "w2a8_tc.cuh"

namespace w2a8 {

int env_int(const char *name, int dflt);

// Four warpgroups, with the register file re-balanced between them at kernel entry (setmaxnreg):
//   warps 0-3   two MMA issuers, the TMA producer, one spare       (56 registers per thread)
//   warps 4-7   unpack                                             (104)
//   warps 8-15  drain: 64 fp32 accumulators + 64 staged values     (176)
constexpr int kHfFirstUnpackWarp = 4;    // four unpack warps: two teams of two
constexpr int kHfFirstDrainWarp = 8;
constexpr int kHfThreads = 32 * 16;
constexpr int kHfDrainCols = 64;         // token columns per drain warp (two warps share a lane quarter)
constexpr int kHfBM = 128;               // channels per tile (UMMA M)
constexpr int kHfBN = 128;               // tokens per tile (UMMA N)
constexpr int kHfBK = 128;               // k per stage = half a W2P block
constexpr int kHfStages = 3;
constexpr int kHfHalfBytes = 128 * 128;  // one [128 rows][128 B] swizzled sub-tile = 64 k of bf16
constexpr int kHfStageBytes = 4 * kHfHalfBytes;   // A: 2 sub-tiles, B: 2 sub-tiles
constexpr int kHfAccBufs = 4;            // accumulator buffers in tensor memory (groups in flight)
constexpr int kHfTmemCols = kHfAccBufs * kHfBN;
constexpr int kHfUnits = kHfAccBufs / 2; // hand-off unit between MMA and drain: two groups

struct HfParams {
    const uint32_t *packed;
    const float *w_scale;
    const float *a_scale;    // token scales, or null (activations are the caller's bf16 values)
    float *y;
    int32_t *partials;
    int *status;
    int M, N, K, G, group;
    int words_per_row;
    int slices_per_group;    // group / 64
    int ldy;
};

// Give registers back to / take registers from the pool of the CTA (whole warpgroup, converged).
template <int N>
__device__ __forceinline__ void hf_setmaxnreg_dec() { asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N)); }
template <int N>
__device__ __forceinline__ void hf_setmaxnreg_inc() { asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N)); }

// Two exact bf16 weights code - 2 from two bytes of c, where every byte of c holds a code at bit
// offset 2 j: with the exponent byte 0x43 - j in front, the 16 bits are the bf16 value
// 2^(7 - 2 j) + code; subtracting 2^(7 - 2 j) + 2 leaves code - 2.
__device__ __forceinline__ uint32_t hf_weights(uint32_t c, uint32_t expo, float off, uint32_t sel) {
    const uint32_t u = __byte_perm(c, expo, sel);
    const __nv_bfloat162 v = __hsub2(*reinterpret_cast<const __nv_bfloat162 *>(&u), __floats2bfloat162_rn(off, off));
    return *reinterpret_cast<const uint32_t *>(&v);
}

// The 16 codes of a packed word (k = 16 t .. 16 t + 15 of a slice) as 16 bf16 values in k order:
// two 16-byte vectors.
__device__ __forceinline__ void hf_unpack_word(uint32_t w, uint4 &lo, uint4 &hi) {
    uint32_t r[8];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const uint32_t c = j < 3 ? (w & (0x03030303u << (2 * j))) : ((w >> 6) & 0x03030303u);
        const uint32_t expo = j == 1 ? 0x42424242u : j == 2 ? 0x41414141u : 0x43434343u;
        const float off = j == 1 ? 34.f : j == 2 ? 10.f : 130.f;
        r[2 * j] = hf_weights(c, expo, off, 0x4140u);
        r[2 * j + 1] = hf_weights(c, expo, off, 0x4342u);
    }
    lo = make_uint4(r[0], r[1], r[2], r[3]);
    hi = make_uint4(r[4], r[5], r[6], r[7]);
}

template <bool PARTIALS, int DPS>
__global__ void __launch_bounds__(kHfThreads, 1)
w2a16_prefill_kernel(const __grid_constant__ CUtensorMap act_map, const HfParams p) {
    extern __shared__ unsigned char hf_smem_raw[];
    __shared__ __align__(8) unsigned long long bar_full[kHfStages], bar_empty[kHfStages];
    __shared__ __align__(8) unsigned long long bar_acc_full[kHfUnits], bar_acc_empty[kHfAccBufs];
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag_s;
    volatile int *abort_flag = &abort_flag_s;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int nstages = p.K / kHfBK;        // stages per tile
    const int dps = p.slices_per_group;     // 64-k slices between two drains
    const int ngroups = (p.K / 64) / dps;   // scale groups per tile
    const int units_per_tile = (ngroups + 1) / 2;
    const int tiles_m = (p.M + kHfBN - 1) / kHfBN;
    const int ntiles = (p.N / kHfBM) * tiles_m;
    const uint32_t smem_base = (pf_smem_u32(hf_smem_raw) + 1023u) & ~1023u;
    unsigned char *smem_gen = hf_smem_raw + (smem_base - pf_smem_u32(hf_smem_raw));

    if (threadIdx.x == 0) {
        abort_flag_s = 0;
        for (int s = 0; s < kHfStages; ++s) {
            pf_mbar_init(pf_smem_u32(&bar_full[s]), 2 + 1);   // the two unpack warps of a team + the TMA producer
            pf_mbar_init(pf_smem_u32(&bar_empty[s]), 2);                   // one commit per MMA-issuing thread
        }
        for (int b = 0; b < kHfUnits; ++b) pf_mbar_init(pf_smem_u32(&bar_acc_full[b]), 1);
        // buffers are handed back one by one (one arrive per drain warp)
        for (int b = 0; b < kHfAccBufs; ++b) pf_mbar_init(pf_smem_u32(&bar_acc_empty[b]), 8);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        pf_fence_proxy_async();
    }
    if (warp == 1) pf_tmem_alloc(pf_smem_u32(&tmem_base_slot), kHfTmemCols);
    pf_tc_fence_before();
    __syncthreads();
    pf_tc_fence_after();
    const uint32_t tmem_base = tmem_base_slot;

    if (warp < kHfFirstUnpackWarp) {
        hf_setmaxnreg_dec<56>();
        if (warp == 2 && lane == 0) {
            // ===== TMA producer: activations, 128 tokens x 128 k per stage ===================
            int s = 0, round = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < ntiles && ok; tile += gridDim.x) {
                const int m0 = (tile % tiles_m) * kHfBN;
                for (int it = 0; it < nstages; ++it) {
                    if (round > 0 && !pf_wait(pf_smem_u32(&bar_empty[s]), (round - 1) & 1, abort_flag)) {
                        ok = false;
                        break;
                    }
                    const uint32_t bar = pf_smem_u32(&bar_full[s]);
                    const uint32_t dst = smem_base + s * kHfStageBytes + 2 * kHfHalfBytes;
                    pf_mbar_arrive_expect_tx(bar, 2 * kHfHalfBytes);
                    pf_tma_load_2d(dst, &act_map, it * kHfBK, m0, bar);
                    pf_tma_load_2d(dst + kHfHalfBytes, &act_map, it * kHfBK + 64, m0, bar);
                    if (++s == kHfStages) { s = 0; ++round; }
                }
            }
        }
        // ===== MMA issuers: thread w owns the hand-off units of parity w ======================
        // Straight-line code per stage (see the int8 kernel: the issue rate of a lone thread is
        // set by the scalar instructions between two MMAs): specialised on the 64-k slices per
        // group (DPS = 1, 2, or 0 for groups of whole 256-k blocks), K-step offsets as immediates
        // on the low descriptor word.  A stage is two 64-k sub-tiles of four K = 16 steps each.
        if (warp < 2 && lane == 0) {
            const int w = warp;
            const uint64_t a_desc0 = pf_smem_desc(smem_base);
            const uint64_t b_desc0 = pf_smem_desc(smem_base + 2 * kHfHalfBytes);
            const uint32_t a_lo0 = (uint32_t)a_desc0, a_hi = (uint32_t)(a_desc0 >> 32);
            const uint32_t b_lo0 = (uint32_t)b_desc0, b_hi = (uint32_t)(b_desc0 >> 32);
            const uint32_t acc_empty_bar0 = pf_smem_u32(&bar_acc_empty[2 * w]), acc_empty_bar1 = pf_smem_u32(&bar_acc_empty[2 * w + 1]);
            const uint32_t acc_full_bar = pf_smem_u32(&bar_acc_full[w]);
            const uint32_t t0 = tmem_base + 2 * w * kHfBN;
            int s = 0;
            uint32_t so = 0;                // stage offset in 16-byte units
            uint32_t full_parity = 0;
            bool ok = true;
            // K step j of a stage (j = 0..7: sub-tile j / 4, step j % 4 of it) into buffer 2 w + b
            auto step = [&](auto jc, int b, uint32_t accumulate) {
                constexpr int j = decltype(jc)::value;
                constexpr uint32_t koff = (j >> 2) * (kHfHalfBytes >> 4) + (j & 3) * 2;
                const uint64_t ad = ((uint64_t)a_hi << 32) | (a_lo0 + so + koff);
                const uint64_t bd = ((uint64_t)b_hi << 32) | (b_lo0 + so + koff);
                pf_mma_f16(t0 + b * kHfBN, ad, bd, pf_instr_desc_bf16(kHfBM, kHfBN), accumulate);
            };
            auto next_stage = [&]() {
                pf_mma_commit(pf_smem_u32(&bar_empty[s]));
                so += kHfStageBytes >> 4;
                if (++s == kHfStages) { s = 0; so = 0; full_parity ^= 1u; }
            };
            using J0 = std::integral_constant<int, 0>; using J1 = std::integral_constant<int, 1>;
            using J2 = std::integral_constant<int, 2>; using J3 = std::integral_constant<int, 3>;
            using J4 = std::integral_constant<int, 4>; using J5 = std::integral_constant<int, 5>;
            using J6 = std::integral_constant<int, 6>; using J7 = std::integral_constant<int, 7>;
            if constexpr (DPS == 1) {
                // 64-k groups: a stage is one unit (two groups); the threads take alternate stages
                int u = 0;                  // unit (= stage) index across tiles
                for (int tile = blockIdx.x; tile < ntiles && ok; tile += gridDim.x) {
                    for (int it = 0; it < nstages && ok; ++it, ++u) {
                        ok = pf_wait(pf_smem_u32(&bar_full[s]), full_parity, abort_flag);
                        if (!ok) break;
                        if ((u & 1) == w) {
                            // each buffer must have been read out by the drain warps since its last use
                            if (u >= kHfUnits) ok = pf_wait(acc_empty_bar0, (uint32_t)((u >> 1) - 1) & 1u, abort_flag);
                            if (!ok) break;
                            pf_tc_fence_after();
                            step(J0{}, 0, 0u); step(J1{}, 0, 1u); step(J2{}, 0, 1u); step(J3{}, 0, 1u);
                            if (u >= kHfUnits) ok = pf_wait(acc_empty_bar1, (uint32_t)((u >> 1) - 1) & 1u, abort_flag);
                            if (!ok) break;
                            pf_tc_fence_after();
                            step(J4{}, 1, 0u); step(J5{}, 1, 1u); step(J6{}, 1, 1u); step(J7{}, 1, 1u);
                            pf_mma_commit(acc_full_bar);
                        }
                        next_stage();
                    }
                }
            } else {
                // groups of one stage (DPS == 2) or of whole 256-k blocks (two stages each): all
                // eight steps of a stage go to one buffer; unit = two consecutive groups (the
                // last unit of a tile may hold one)
                const int spg = dps >> 1;   // stages per group
                int unit0 = 0;              // units of the tiles before this one
                int uses0 = 0, uses1 = 0;   // groups this thread has put into its first / second buffer
                for (int tile = blockIdx.x; tile < ntiles && ok; tile += gridDim.x, unit0 += units_per_tile) {
                    int group_idx = 0, pos = 0;     // group of this tile, stage inside the group
                    for (int it = 0; it < nstages && ok; ++it) {
                        ok = pf_wait(pf_smem_u32(&bar_full[s]), full_parity, abort_flag);
                        if (!ok) break;
                        const int u = unit0 + (group_idx >> 1);
                        const bool mine = (u & 1) == w;
                        if (mine) {
                            const int b = group_idx & 1;
                            if (pos == 0) {     // a new group: its buffer must have been read out since its last use
                                const int uses = b ? uses1 : uses0;
                                if (uses >= 1) ok = pf_wait(b ? acc_empty_bar1 : acc_empty_bar0, (uint32_t)(uses - 1) & 1u, abort_flag);
                                if (!ok) break;
                                if (b) ++uses1; else ++uses0;
                            }
                            pf_tc_fence_after();
                            step(J0{}, b, (DPS == 2 || pos == 0) ? 0u : 1u);
                            step(J1{}, b, 1u); step(J2{}, b, 1u); step(J3{}, b, 1u);
                            step(J4{}, b, 1u); step(J5{}, b, 1u); step(J6{}, b, 1u); step(J7{}, b, 1u);
                        }
                        if (DPS == 2 || ++pos == spg) {
                            pos = 0;
                            const bool unit_done = (group_idx & 1) == 1 || group_idx == ngroups - 1;
                            if (mine && unit_done) pf_mma_commit(acc_full_bar);
                            ++group_idx;
                        }
                        next_stage();
                    }
                }
            }
        }
    } else if (warp < kHfFirstDrainWarp) {
        hf_setmaxnreg_dec<104>();
        // ===== unpack warps: packed words -> bf16 values, K-major, 128-byte swizzle =========
        // Two teams of two warps; a stage is half a 256-k block, so team j fills every stage of
        // parity j: slices 2 j and 2 j + 1 of each block.  A stage's fixed costs (the wait for the
        // slot, the proxy fence, the arrive) overlap the other team's unpack.  A thread owns eight
        // units of a stage (row r = u / 4, quarter t = u % 4): word t of the stage's two slices.
        constexpr int kUnits = 8;
        const int team = (warp - kHfFirstUnpackWarp) >> 1;
        const int ut = ((warp - kHfFirstUnpackWarp) & 1) * 32 + lane;
        auto request = [&](uint2 (&w)[kUnits], int tile, int blk) {
            const int n0 = (tile / tiles_m) * kHfBM;
#pragma unroll
            for (int i = 0; i < kUnits; ++i) {
                const int u = ut + 64 * i;
                const int r = u >> 2, t = u & 3;
                w[i] = __ldg(reinterpret_cast<const uint2 *>(p.packed + (size_t)(n0 + r) * p.words_per_row +
                                                             16 * blk + 4 * t + 2 * team));
            }
        };
        const int nblocks = nstages >> 1;
        int tile = blockIdx.x, blk = 0;
        int s = team, round = 0;                    // slot and use count of the slot for this team's stage
        uint2 w_nxt[kUnits];
        if (tile < ntiles) request(w_nxt, tile, 0);
        while (tile < ntiles) {
            uint2 w_cur[kUnits];
#pragma unroll
            for (int i = 0; i < kUnits; ++i) w_cur[i] = w_nxt[i];
            // next block's words in flight (possibly the first block of the next tile)
            int tile_nxt = tile, blk_nxt = blk + 1;
            if (blk_nxt == nblocks) { blk_nxt = 0; tile_nxt += gridDim.x; }
            if (tile_nxt < ntiles) request(w_nxt, tile_nxt, blk_nxt);
            if (round > 0 && !pf_wait(pf_smem_u32(&bar_empty[s]), (round - 1) & 1, abort_flag)) break;
            unsigned char *a_stage = smem_gen + s * kHfStageBytes;
#pragma unroll
            for (int i = 0; i < kUnits; ++i) {
                const int u = ut + 64 * i;
                const int r = u >> 2, t = u & 3;
                const uint32_t ws[2] = {w_cur[i].x, w_cur[i].y};
#pragma unroll
                for (int sl = 0; sl < 2; ++sl) {    // slice sl of the stage: k = 64 sl + 16 t .. + 15
                    uint4 lo, hi;
                    hf_unpack_word(ws[sl], lo, hi);
                    unsigned char *row = a_stage + sl * kHfHalfBytes + r * 128;
                    *reinterpret_cast<uint4 *>(row + (((2 * t) ^ (r & 7)) << 4)) = lo;
                    *reinterpret_cast<uint4 *>(row + (((2 * t + 1) ^ (r & 7)) << 4)) = hi;
                }
            }
            pf_fence_proxy_async();     // make the generic-proxy stores visible to the tensor core
            __syncwarp();
            if (lane == 0) pf_mbar_arrive(pf_smem_u32(&bar_full[s]));
            tile = tile_nxt; blk = blk_nxt;
            s += 2;
            if (s >= kHfStages) { s -= kHfStages; ++round; }
        }
    } else {
        hf_setmaxnreg_inc<176>();
        // ===== drain warps: TMEM -> registers, fp32 accumulate with the group scale ======
        const int q4 = warp & 3;                    // TMEM lane quarter this warp may access
        const int col0 = ((warp - kHfFirstDrainWarp) >> 2) * kHfDrainCols;
        const int ch = q4 * 32 + lane;
        const uint32_t tlane = tmem_base + ((uint32_t)(q4 * 32) << 16) + col0;
        bool ok = true;
        int unit0 = 0;
        for (int tile = blockIdx.x; tile < ntiles && ok; tile += gridDim.x, unit0 += units_per_tile) {
            const int n = (tile / tiles_m) * kHfBM + ch;
            const int m0 = (tile % tiles_m) * kHfBN;
            float acc[kHfDrainCols];
#pragma unroll
            for (int j = 0; j < kHfDrainCols; ++j) acc[j] = 0.f;
            const float *sc_row = PARTIALS ? nullptr : p.w_scale + (size_t)n * p.G;
            uint32_t sc_nxt[8] = {0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u};
            auto refill = [&](int g0) {
                if constexpr (!PARTIALS) {
#pragma unroll
                    for (int u = 0; u < 8; ++u)
                        if (g0 + u < ngroups) sc_nxt[u] = __float_as_uint(__ldg(sc_row + g0 + u));
                }
            };
            refill(0);
            int v0[32], v1[32];                         // first / second half of the current group (fp32 bit patterns)
            ok = pf_wait_warp(pf_smem_u32(&bar_acc_full[unit0 & 1]), (unit0 >> 1) & 1, abort_flag);
            if (ok) { pf_tc_fence_after(); pf_tmem_ld32(tlane + (2 * (unit0 & 1)) * kHfBN, v0); }
            for (int g0 = 0; g0 < ngroups && ok; g0 += 8) {
                float sc_cur[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) sc_cur[u] = __uint_as_float(sc_nxt[u]);
                refill(g0 + 8);
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    const int gi = g0 + u;
                    if (gi >= ngroups || !ok) break;
                    const int unit = unit0 + (gi >> 1);
                    const int buf = 2 * (unit & 1) + (gi & 1);
                    const float sc = sc_cur[u];
                    pf_tmem_ld_wait();                     // first half of group gi is in v0
                    pf_tmem_ld32(tlane + buf * kHfBN + 32, v1);
                    if (PARTIALS) {
#pragma unroll
                        for (int j = 0; j < 32; ++j) {
                            const int m = m0 + col0 + j;
                            if (m < p.M) p.partials[((size_t)m * p.N + n) * p.G + gi] = __float2int_rn(__int_as_float(v0[j]));
                        }
                    } else {
#pragma unroll
                        for (int j = 0; j < 32; j += 2)
                            pf_fma2(acc[j], acc[j + 1], __int_as_float(v0[j]), __int_as_float(v0[j + 1]), sc);
                    }
                    pf_tmem_ld_wait();                     // second half is in v1
                    {   // this warp's share of the buffer has been read: hand it back
                        pf_tc_fence_before();
                        __syncwarp();
                        if (lane == 0) pf_mbar_arrive(pf_smem_u32(&bar_acc_empty[buf]));
                    }
                    if (gi + 1 < ngroups) {                // request the first half of the next group
                        const int nunit = unit0 + ((gi + 1) >> 1);
                        if (((gi + 1) & 1) == 0) {
                            ok = pf_wait(pf_smem_u32(&bar_acc_full[nunit & 1]), (nunit >> 1) & 1, abort_flag);
                            if (!ok) break;
                            pf_tc_fence_after();
                        }
                        pf_tmem_ld32(tlane + (2 * (nunit & 1) + ((gi + 1) & 1)) * kHfBN, v0);
                    }
                    if (PARTIALS) {
#pragma unroll
                        for (int j = 0; j < 32; ++j) {
                            const int m = m0 + col0 + 32 + j;
                            if (m < p.M) p.partials[((size_t)m * p.N + n) * p.G + gi] = __float2int_rn(__int_as_float(v1[j]));
                        }
                    } else {
#pragma unroll
                        for (int j = 0; j < 32; j += 2)
                            pf_fma2(acc[32 + j], acc[32 + j + 1], __int_as_float(v1[j]), __int_as_float(v1[j + 1]), sc);
                    }
                }
            }
            pf_tmem_ld_wait();
            if (!PARTIALS && ok) {
#pragma unroll
                for (int j = 0; j < kHfDrainCols; ++j) {
                    const int m = m0 + col0 + j;
                    if (m < p.M) p.y[(size_t)m * p.ldy + n] = p.a_scale ? acc[j] * __ldg(p.a_scale + m) : acc[j];
                }
            }
        }
    }

    // ---- wind down ---------------------------------------------------------------------
    pf_tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0 && abort_flag_s) atomicExch(p.status, W2A8_ERR_TIMEOUT);
    if (warp == 1) {
        pf_tc_fence_after();
        pf_tmem_dealloc(tmem_base, kHfTmemCols);
    }
}

// int8 activations as bf16 values (exact): the copy the 16-bit kernel reads when it serves w2a8_gemm
__global__ void __launch_bounds__(256)
a8_to_bf16_kernel(const int8_t *__restrict__ a, __nv_bfloat16 *__restrict__ out, size_t n16) {
    pdl_launch_dependents();
    pdl_wait();
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n16; i += (size_t)gridDim.x * blockDim.x) {
        const uint4 v = *reinterpret_cast<const uint4 *>(a + 16 * i);
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
        uint32_t o[8];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const int b0 = (int)(int8_t)(w[q] & 0xFF), b1 = (int)(int8_t)((w[q] >> 8) & 0xFF);
            const int b2 = (int)(int8_t)((w[q] >> 16) & 0xFF), b3 = (int)(int8_t)(w[q] >> 24);
            const __nv_bfloat162 lo = __floats2bfloat162_rn((float)b0, (float)b1);
            const __nv_bfloat162 hi = __floats2bfloat162_rn((float)b2, (float)b3);
            o[2 * q] = *reinterpret_cast<const uint32_t *>(&lo);
            o[2 * q + 1] = *reinterpret_cast<const uint32_t *>(&hi);
        }
        uint4 *dst = reinterpret_cast<uint4 *>(out + 16 * i);
        dst[0] = make_uint4(o[0], o[1], o[2], o[3]);
        dst[1] = make_uint4(o[4], o[5], o[6], o[7]);
    }
}

// ---- host side -----------------------------------------------------------------------
// Shapes the 16-bit tensor-core kernel tiles: as the int8 kernel, with whole 128-k stages.  fp32
// group sums of exact integer products are exact as long as they stay below 2^24: 254 * group for
// int8 activations (group <= 65536); for bf16 activations no such bound is needed.
bool prefill_f16_supported(int M, int N, int K, int group) {
    if (M < 64) return false;
    if (N % kHfBM != 0 || K % 256 != 0) return false;
    return group == 64 || group == 128 || group % 256 == 0;
}

// Bytes of scratch the int8 entry needs for the bf16 copy of its activations.
size_t prefill_f16_scratch_bytes(int M, int K) { return ((size_t)M * K * 2 + 255) / 256 * 256; }

// Enqueue the 16-bit tensor-core kernel.  x_bf16: [M][K] bf16 activations (device); a_scale: token
// scales or null.  `partials` != nullptr selects the export of the (integer-valued) group sums.
int launch_prefill_f16(const void *x_bf16, const float *a_scale, const uint32_t *packed, const float *w_scale,
                       float *y, int32_t *partials, int M, int N, int K, int group, int *status, cudaStream_t st,
                       int ldy) {
    EncodeTiledFn encode = encode_tiled_fn();
    if (!encode) return W2A8_ERR_CUDA;
    CUtensorMap map;
    const cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)M};
    const cuuint64_t strides[1] = {(cuuint64_t)K * 2};             // bytes between tokens
    const cuuint32_t box[2] = {64u, (cuuint32_t)kHfBN};            // 64 k (128 bytes) x 128 tokens
    const cuuint32_t estr[2] = {1u, 1u};
    if (encode(&map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(x_bf16), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return W2A8_ERR_CUDA;
    HfParams p;
    p.packed = packed; p.w_scale = w_scale; p.a_scale = a_scale; p.y = y; p.partials = partials;
    p.status = status; p.ldy = ldy;
    p.M = M; p.N = N; p.K = K; p.G = K / group; p.group = group;
    p.words_per_row = K / 16;
    p.slices_per_group = group / 64;
    const size_t smem = (size_t)kHfStages * kHfStageBytes + 1024;
    const long long tiles = (long long)(N / kHfBM) * ((M + kHfBN - 1) / kHfBN);
    const int sms = sm_count();
    dim3 grid((unsigned)(tiles < sms ? tiles : sms));
    static PerDeviceFlags configured[6];
    auto launch = [&](auto kernel, int slot) -> bool {
        if (allow_dynamic_smem(kernel, configured[slot], (int)smem) != cudaSuccess) return false;
        kernel<<<grid, kHfThreads, smem, st>>>(map, p);
        return true;
    };
    // the MMA-issuing code is specialised on the 64-k slices per scale group: 1, 2, or whole blocks (0)
    auto launch_dps = [&](auto partials_c, int slot0) -> bool {
        constexpr bool P = decltype(partials_c)::value;
        if (group == 64) return launch(w2a16_prefill_kernel<P, 1>, slot0);
        if (group == 128) return launch(w2a16_prefill_kernel<P, 2>, slot0 + 1);
        return launch(w2a16_prefill_kernel<P, 0>, slot0 + 2);
    };
    const bool launched = partials ? launch_dps(std::true_type{}, 3) : launch_dps(std::false_type{}, 0);
    if (!launched) return W2A8_ERR_CUDA;
    return cudaGetLastError() == cudaSuccess ? W2A8_OK : W2A8_ERR_CUDA;
}

// int8 activations -> bf16 copy in `scratch` (M * K * 2 bytes), on the stream.
int launch_a8_to_bf16(const int8_t *a, void *scratch, int M, int K, cudaStream_t st) {
    const size_t n16 = (size_t)M * K / 16;
    const unsigned grid = (unsigned)((n16 + 255) / 256 < (size_t)sm_count() * 8 ? (n16 + 255) / 256 : (size_t)sm_count() * 8);
    cudaError_t e = launch_kernel(a8_to_bf16_kernel, dim3(grid ? grid : 1), dim3(256), 0, st, pdl_enabled(), a,
                                  reinterpret_cast<__nv_bfloat16 *>(scratch), n16);
    return e == cudaSuccess ? W2A8_OK : W2A8_ERR_CUDA;
}

}  // namespace w2a8
