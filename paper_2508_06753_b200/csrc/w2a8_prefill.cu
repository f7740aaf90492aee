// Compute-bound W2A8 kernel for many tokens (prefill): 5th-generation tensor
// cores (tcgen05.mma kind::i8) with accumulators in tensor memory.  It is the
// sm_100a counterpart of the paper's fused GEMM for the compute-bound case
// (Sec. II-D: tiles of the output, low-bit weights fed to the matrix unit,
// int32 -> float dequantisation in registers), with the 2-bit -> int8
// up-convert of Sec. II-C done into shared memory because the tensor core has
// no 2-bit operand type.
//
// Persistent CTAs (12 warps, one CTA per SM) walk 128-channel x 128-token tiles of y.
//   A operand (UMMA M = 128): weights.  Two "unpack" warps read the packed words
//     of 128 channels x one 256-k block, expand them to int8 lanes (value
//     64 * (code - 2): one shift + one LOP3 per four weights) and store them
//     K-major with the 128-byte swizzle the tensor core expects.
//   B operand (UMMA N = 128): int8 activations, 128 tokens x 256 k, brought by TMA
//     (issued by one lane of an unpack warp) with the same swizzle.
//   D: int32 in tensor memory, lane = channel, column = token.  Because a lane is
//     a channel, a drain thread needs one weight scale per group, not one per value.
// Per 64-k group (or whatever the scale group is) an MMA thread issues K = 32 steps
// into one of four accumulator buffers (all 512 TMEM columns).  MMA and drain hand
// buffers over in units of two consecutive groups (a barrier round trip costs as much
// as the MMAs of a 64-k group); two threads share the issuing, one unit slot each, in
// straight-line code per stage (the kernel is specialised on the slices per group).
// Eight "drain" warps (two per TMEM lane quarter, 64 token columns each) read finished
// buffers with tcgen05.ld, software-pipelined in 32-column halves, convert to fp32 and
// accumulate scale * value in registers with packed fp32 FMAs.  Stage slots and units
// are numbered across tiles, so the producers run ahead into the next tile while the
// drain warps store y.  Every wait on an mbarrier is bounded; a wait that gives up
// sets the status word of the workspace and the CTA winds down.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include <type_traits>

#include "w2a8_tc.cuh"

namespace w2a8 {
// Of every eight drained values, how many are turned into floats by the integer-add route (the rest
// by the conversion instruction): the two routes load different pipes -- the conversion instruction
// issues at a quarter of the rate of an integer add, the add route takes one more issue slot per two
// values -- and a mix beats either alone (4096 -> 14336, 2048 tokens, group 64: all conversions
// 693 TOPS, all adds 702, half and half 760, two of eight by adds 772).
constexpr int kPfMagicOfEight = 2;

// Two warp layouts (template parameter UW = unpack warps):
//   UW = 2: 12 warps -- 2 MMA issuers, 2 unpack warps (lane 0 of the first also issues the TMA
//           loads), 8 drain warps; every thread has the same 168 registers.
//   UW = 4: 16 warps in four warpgroups whose registers are re-balanced at entry (setmaxnreg):
//           warps 0-3 two MMA issuers, the TMA producer, one spare (56 registers per thread);
//           warps 4-7 unpack (104); warps 8-15 drain (176).
__host__ __device__ constexpr int pf_threads(int uw) { return uw == 4 ? 512 : 384; }
__host__ __device__ constexpr int pf_first_unpack(int uw) { return uw == 4 ? 4 : 2; }
__host__ __device__ constexpr int pf_first_drain(int uw) { return uw == 4 ? 8 : 4; }
constexpr int kPfDrainCols = 64;         // token columns per drain warp (two warps share a lane quarter)
constexpr int kPfBM = 128;               // channels per tile (UMMA M)
constexpr int kPfBN = 128;               // tokens per tile (UMMA N)
constexpr int kPfBK = 256;               // k per stage = one W2P block
constexpr int kPfStages = 3;
constexpr int kPfHalfBytes = 128 * 128;  // one [128 rows][128 B] swizzled sub-tile
constexpr int kPfStageBytes = 4 * kPfHalfBytes;   // A: 2 halves, B: 2 halves
constexpr int kPfAccBufs = 4;             // accumulator buffers in tensor memory (groups in flight)
constexpr int kPfTmemCols = kPfAccBufs * kPfBN;   // 512 columns: all of tensor memory
constexpr int kPfUnits = kPfAccBufs / 2;  // hand-off unit between MMA and drain: two groups (two buffers)

struct PrefillParams {
    const uint32_t *packed;
    const float *w_scale;
    const float *a_scale;
    float *y;
    int32_t *partials;
    int *status;
    int M, N, K, G, group;
    int words_per_row;
    int slices_per_group;    // group / 64
    int y16;                 // 16-bit instance only: y holds bf16 instead of fp32
    int ldy;                 // elements between consecutive token rows of y (>= N)
    int ks_shift;            // log2 of the K splits S: work item = tile * S + split; each split walks K / S
    float *split_out;        // S > 1: [S][M][N] fp32 partial outputs (summed in split order by a second kernel)
};

// H16: w_scale points at IEEE binary16 values; the result is fp32 or, with p.y16, bf16.
template <int N>
__device__ __forceinline__ void pf_setmaxnreg_dec() { asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N)); }
template <int N>
__device__ __forceinline__ void pf_setmaxnreg_inc() { asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N)); }

// SPLIT: work items are (tile, K split) pairs; without it the split count is the constant 1 (the
// general form costs 15 % on the unsplit problem: 596 against 702 TOPS at 2048 tokens, group 64).
template <bool PARTIALS, bool H16, int DPS, int UW, bool SPLIT>
__global__ void __launch_bounds__(pf_threads(UW), 1)
w2a8_prefill_kernel(const __grid_constant__ CUtensorMap act_map, const PrefillParams p) {
    extern __shared__ unsigned char pf_smem_raw[];
    __shared__ __align__(8) unsigned long long bar_full[kPfStages], bar_empty[kPfStages];
    __shared__ __align__(8) unsigned long long bar_acc_full[kPfUnits], bar_acc_empty[kPfAccBufs];
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag_s;
    volatile int *abort_flag = &abort_flag_s;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int ks_shift = SPLIT ? p.ks_shift : 0;
    const int nsplit = 1 << ks_shift;       // K splits: a work item is one tile over K / nsplit
    const int nstages = (p.K / kPfBK) >> ks_shift;        // stages per work item
    const int dps = p.slices_per_group;     // 64-k slices between two drains
    const int ngroups = ((p.K / 64) >> ks_shift) / dps;   // scale groups per work item
    const int units_per_tile = (ngroups + 1) / 2;
    // Persistent CTA: tiles blockIdx.x, blockIdx.x + gridDim.x, ...; consecutive tiles share the
    // channel tile and differ in the token tile, so neighbouring CTAs re-use weights from L2.
    // Stage slots and accumulator units are numbered across tiles (the pipeline does not drain
    // between tiles: producers run ahead into the next tile while the drain warps store y).
    const int tiles_m = (p.M + kPfBN - 1) / kPfBN;
    const int ntiles = ((p.N / kPfBM) * tiles_m) << ks_shift;   // work items; `tile` below is a work-item index
    auto item_n0 = [&](int item) { return ((item >> ks_shift) / tiles_m) * kPfBM; };     // first channel
    auto item_m0 = [&](int item) { return ((item >> ks_shift) % tiles_m) * kPfBN; };     // first token
    auto item_stage0 = [&](int item) { return (item & (nsplit - 1)) * nstages; };          // first 256-k block
    // stage buffers, 1024-byte aligned (swizzle atom = 8 rows x 128 B)
    const uint32_t smem_base = (pf_smem_u32(pf_smem_raw) + 1023u) & ~1023u;

    if (threadIdx.x == 0) {
        abort_flag_s = 0;
        for (int s = 0; s < kPfStages; ++s) {
            // one arrive per unpack warp + the TMA producer's arrive with its transaction bytes
            pf_mbar_init(pf_smem_u32(&bar_full[s]), 2 + 1);   // the two unpack warps of a team + the TMA producer
            pf_mbar_init(pf_smem_u32(&bar_empty[s]), 2);      // one tcgen05.commit per MMA-issuing thread
        }
        for (int b = 0; b < kPfUnits; ++b) pf_mbar_init(pf_smem_u32(&bar_acc_full[b]), 1);   // tcgen05.commit
        // buffers are handed back one by one (one arrive per drain warp): the MMAs of a unit's
        // first group start while the drain warps are still reading its second buffer
        for (int b = 0; b < kPfAccBufs; ++b) pf_mbar_init(pf_smem_u32(&bar_acc_empty[b]), 8);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        pf_fence_proxy_async();
    }
    if (warp == 1) pf_tmem_alloc(pf_smem_u32(&tmem_base_slot), kPfTmemCols);
    pf_tc_fence_before();
    __syncthreads();
    pf_tc_fence_after();
    const uint32_t tmem_base = tmem_base_slot;

    constexpr int kFirstUnpack = pf_first_unpack(UW), kFirstDrain = pf_first_drain(UW);
    if (warp < kFirstUnpack) {
        if constexpr (UW == 4) {
            pf_setmaxnreg_dec<56>();
            if (warp == 2 && lane == 0) {
                // ===== TMA producer: activations, 128 tokens x 256 k per stage ===============
                int s = 0, round = 0;
                for (int tile = blockIdx.x; tile < ntiles; tile += gridDim.x) {
                    const int m0 = item_m0(tile), k0 = item_stage0(tile) * kPfBK;
                    bool ok = true;
                    for (int it = 0; it < nstages; ++it) {
                        if (round > 0 && !pf_wait(pf_smem_u32(&bar_empty[s]), (round - 1) & 1, abort_flag)) {
                            ok = false;
                            break;
                        }
                        const uint32_t bar = pf_smem_u32(&bar_full[s]);
                        const uint32_t dst = smem_base + s * kPfStageBytes + 2 * kPfHalfBytes;
                        pf_mbar_arrive_expect_tx(bar, 2 * kPfHalfBytes);
                        pf_tma_load_2d(dst, &act_map, k0 + it * kPfBK, m0, bar);
                        pf_tma_load_2d(dst + kPfHalfBytes, &act_map, k0 + it * kPfBK + 128, m0, bar);
                        if (++s == kPfStages) { s = 0; ++round; }
                    }
                    if (!ok) break;
                }
            }
        }
        // ===== MMA issuers (one thread in each of warps 0 and 1) =========================
        // The hand-off unit between MMA and drain is two consecutive scale groups (two
        // accumulator buffers, one barrier pair); thread w owns the units of parity w.
        // A lone thread runs a dependent instruction every several cycles, so the cost of
        // issuing is the number of scalar instructions between two MMAs: with loop-carried
        // bookkeeping and 64-bit descriptor arithmetic one thread issued an MMA every ~200
        // cycles (measured with producers and drain switched off: 1.3-1.5 POPS for the pair),
        // three times the 64 cycles the MMA takes.  Written as straight-line code per stage --
        // the kernel is specialised on the slices per group (DPS = 1, 2, or 0 for groups of
        // whole stages), K-step offsets are immediates added to the low descriptor word --
        // the same pair issues at the tensor pipe's rate (3.2-3.3 POPS in that test).
        if (warp < 2 && lane == 0) {
            const int w = warp;             // this thread's unit slot: accumulator buffers 2 w and 2 w + 1
            const uint64_t a_desc0 = pf_smem_desc(smem_base);
            const uint64_t b_desc0 = pf_smem_desc(smem_base + 2 * kPfHalfBytes);
            // Only the low word of a descriptor (start address / 16) changes from step to step
            const uint32_t a_lo0 = (uint32_t)a_desc0, a_hi = (uint32_t)(a_desc0 >> 32);
            const uint32_t b_lo0 = (uint32_t)b_desc0, b_hi = (uint32_t)(b_desc0 >> 32);
            const uint32_t acc_empty_bar0 = pf_smem_u32(&bar_acc_empty[2 * w]), acc_empty_bar1 = pf_smem_u32(&bar_acc_empty[2 * w + 1]);
            const uint32_t acc_full_bar = pf_smem_u32(&bar_acc_full[w]);
            const uint32_t t0 = tmem_base + 2 * w * kPfBN;
            int s = 0;
            uint32_t so = 0;                // stage offset in 16-byte units
            uint32_t full_parity = 0;
            bool ok = true;
            // K step j of a stage (j = 0..7: 64-k slice j / 2, half j % 2 of it) into buffer 2 w + b
            auto step = [&](auto jc, int b, uint32_t accumulate) {
                constexpr int j = decltype(jc)::value;
                constexpr uint32_t koff = ((j >> 2) & 1) * (kPfHalfBytes >> 4) + (j & 3) * 2;
                const uint64_t ad = ((uint64_t)a_hi << 32) | (a_lo0 + so + koff);
                const uint64_t bd = ((uint64_t)b_hi << 32) | (b_lo0 + so + koff);
                pf_mma_i8(t0 + b * kPfBN, ad, bd, pf_instr_desc(kPfBM, kPfBN), accumulate);
            };
            auto next_stage = [&]() {
                pf_mma_commit(pf_smem_u32(&bar_empty[s]));   // stage can be refilled once these MMAs are done
                so += kPfStageBytes >> 4;
                if (++s == kPfStages) { s = 0; so = 0; full_parity ^= 1u; }
            };
            using J0 = std::integral_constant<int, 0>; using J1 = std::integral_constant<int, 1>;
            using J2 = std::integral_constant<int, 2>; using J3 = std::integral_constant<int, 3>;
            using J4 = std::integral_constant<int, 4>; using J5 = std::integral_constant<int, 5>;
            using J6 = std::integral_constant<int, 6>; using J7 = std::integral_constant<int, 7>;
            if constexpr (DPS == 1) {
                // 64-k groups: a stage holds two units; ngroups is a multiple of four, so every
                // tile starts on an even unit and thread w always takes slices 2 w and 2 w + 1.
                int c = 0;                  // units this thread has issued so far
                for (int tile = blockIdx.x; tile < ntiles && ok; tile += gridDim.x) {
                    for (int it = 0; it < nstages && ok; ++it, ++c) {
                        ok = pf_wait(pf_smem_u32(&bar_full[s]), full_parity, abort_flag);
                        if (!ok) break;
                        // each buffer must have been read out by the drain warps since its last use
                        if (c >= 1) ok = pf_wait(acc_empty_bar0, (uint32_t)(c - 1) & 1u, abort_flag);
                        if (!ok) break;
                        pf_tc_fence_after();
                        if (w == 0) { step(J0{}, 0, 0u); step(J1{}, 0, 1u); }
                        else        { step(J4{}, 0, 0u); step(J5{}, 0, 1u); }
                        if (c >= 1) ok = pf_wait(acc_empty_bar1, (uint32_t)(c - 1) & 1u, abort_flag);
                        if (!ok) break;
                        pf_tc_fence_after();
                        if (w == 0) { step(J2{}, 1, 0u); step(J3{}, 1, 1u); }
                        else        { step(J6{}, 1, 0u); step(J7{}, 1, 1u); }
                        pf_mma_commit(acc_full_bar);
                        next_stage();
                    }
                }
            } else if constexpr (DPS == 2) {
                // 128-k groups: a stage is one unit; the two threads take alternate stages
                int u = 0;                  // unit (= stage) index across tiles
                for (int tile = blockIdx.x; tile < ntiles && ok; tile += gridDim.x) {
                    for (int it = 0; it < nstages && ok; ++it, ++u) {
                        ok = pf_wait(pf_smem_u32(&bar_full[s]), full_parity, abort_flag);
                        if (!ok) break;
                        if ((u & 1) == w) {
                            if (u >= kPfUnits) ok = pf_wait(acc_empty_bar0, (uint32_t)((u >> 1) - 1) & 1u, abort_flag);
                            if (!ok) break;
                            pf_tc_fence_after();
                            step(J0{}, 0, 0u); step(J1{}, 0, 1u); step(J2{}, 0, 1u); step(J3{}, 0, 1u);
                            if (u >= kPfUnits) ok = pf_wait(acc_empty_bar1, (uint32_t)((u >> 1) - 1) & 1u, abort_flag);
                            if (!ok) break;
                            pf_tc_fence_after();
                            step(J4{}, 1, 0u); step(J5{}, 1, 1u); step(J6{}, 1, 1u); step(J7{}, 1, 1u);
                            pf_mma_commit(acc_full_bar);
                        }
                        next_stage();
                    }
                }
            } else {
                // groups of whole stages (a multiple of 256 k): all eight steps of a stage go to
                // one buffer; unit = two consecutive groups (the last unit of a tile may hold one)
                const int spg = dps >> 2;   // stages per group
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
                            step(J0{}, b, pos == 0 ? 0u : 1u);
                            step(J1{}, b, 1u); step(J2{}, b, 1u); step(J3{}, b, 1u);
                            step(J4{}, b, 1u); step(J5{}, b, 1u); step(J6{}, b, 1u); step(J7{}, b, 1u);
                        }
                        if (++pos == spg) {
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
    } else if (warp < kFirstDrain) {
        if constexpr (UW == 4) pf_setmaxnreg_dec<104>();
        // ===== unpack warps: packed words -> int8 lanes, K-major, 128-byte swizzle =====
        // Teams of two warps; team j fills stages j, j + kTeams, ... (numbered across tiles).  With
        // two teams a stage's fixed costs -- the wait for the slot, the proxy fence, the arrive --
        // overlap the other team's unpack instead of adding to every stage.
        constexpr int kTeams = UW / 2;
        constexpr int kUnits = 8;                   // 16-byte units per thread and stage
        const int team = (warp - kFirstUnpack) >> 1;
        const int ut = ((warp - kFirstUnpack) & 1) * 32 + lane;
        // Unit u: 16 bytes of packed words (word t = u % 4 of the four slices) of one row.  The eight
        // lanes whose 16-byte stores share a shared-memory wavefront take rows that differ by four:
        // under the 128-byte swizzle (chunk ^= row % 8) their two groups of four chunks are then the
        // two halves of a 128-byte row, one store per bank (consecutive rows would share a half).
        auto unit_row = [](int u) { return (u >> 5) * 8 + ((u >> 2) & 1) * 4 + ((u >> 3) & 3); };
        auto request = [&](uint4 (&w)[kUnits], int tile, int it) {
            const int n0 = item_n0(tile), blk = item_stage0(tile) + it;
#pragma unroll
            for (int i = 0; i < kUnits; ++i) {
                const int u = ut + 64 * i;
                const int r = unit_row(u), t = u & 3;
                w[i] = __ldg(reinterpret_cast<const uint4 *>(p.packed + (size_t)(n0 + r) * p.words_per_row +
                                                             16 * blk + 4 * t));
            }
        };
        auto advance = [&](int &tile, int &it) {    // the next stage in the order the CTA walks them
            if (++it == nstages) { it = 0; tile += gridDim.x; }
        };
        int tile = blockIdx.x, it = 0;
        for (int j = 0; j < team; ++j) advance(tile, it);
        int s = team, round = 0;                    // slot and use count of the slot for this team's stage
        uint4 w_nxt[kUnits];
        if (tile < ntiles) request(w_nxt, tile, it);
        while (tile < ntiles) {
            uint4 w[kUnits];
#pragma unroll
            for (int i = 0; i < kUnits; ++i) w[i] = w_nxt[i];
            // the words of this team's next stage in flight (possibly in the next tile)
            int tile_nxt = tile, it_nxt = it;
#pragma unroll
            for (int j = 0; j < kTeams; ++j) advance(tile_nxt, it_nxt);
            if (tile_nxt < ntiles) request(w_nxt, tile_nxt, it_nxt);
            if (round > 0 && !pf_wait(pf_smem_u32(&bar_empty[s]), (round - 1) & 1, abort_flag)) break;
            if (UW == 2 && warp == kFirstUnpack && lane == 0) {
                // this lane is also the TMA producer: activations, 128 tokens x 256 k per stage
                const int m0 = item_m0(tile), k = (item_stage0(tile) + it) * kPfBK;
                const uint32_t bar = pf_smem_u32(&bar_full[s]);
                const uint32_t dst = smem_base + s * kPfStageBytes + 2 * kPfHalfBytes;
                pf_mbar_arrive_expect_tx(bar, 2 * kPfHalfBytes);
                pf_tma_load_2d(dst, &act_map, k, m0, bar);
                pf_tma_load_2d(dst + kPfHalfBytes, &act_map, k + 128, m0, bar);
            }
            const uint32_t a_stage = smem_base + s * kPfStageBytes;      // shared-space address
#pragma unroll
            for (int i = 0; i < kUnits; ++i) {
                const int u = ut + 64 * i;
                const int r = unit_row(u), t = u & 3;
                const uint32_t ws[4] = {w[i].x, w[i].y, w[i].z, w[i].w};
#pragma unroll
                for (int sl = 0; sl < 4; ++sl) {    // slice sl: k = 64 sl + 16 t .. + 15 of this block
                    const int chunk = (4 * (sl & 1) + t) ^ (r & 7);
                    pf_st_shared_v4(a_stage + (sl >> 1) * kPfHalfBytes + r * 128 + chunk * 16,
                                    lane_codes(ws[sl], 0), lane_codes(ws[sl], 1), lane_codes(ws[sl], 2), lane_codes(ws[sl], 3));
                }
            }
            pf_fence_proxy_async();     // make the generic-proxy stores visible to the tensor core
            __syncwarp();
            if (lane == 0) pf_mbar_arrive(pf_smem_u32(&bar_full[s]));
            tile = tile_nxt; it = it_nxt;
            s += kTeams;
            if (s >= kPfStages) { s -= kPfStages; ++round; }
        }
    } else {
        // ===== drain warps: TMEM -> registers, fp32 accumulate with the group scale ======
        const int q4 = warp & 3;                    // TMEM lane quarter this warp may access
        if constexpr (UW == 4) pf_setmaxnreg_inc<176>();
        const int col0 = ((warp - kFirstDrain) >> 2) * kPfDrainCols;   // first token column of this warp
        const int ch = q4 * 32 + lane;              // channel inside the tile = TMEM lane
        const uint32_t tlane = tmem_base + ((uint32_t)(q4 * 32) << 16) + col0;
        bool ok = true;
        int unit0 = 0;                              // units of the tiles before this one
        for (int tile = blockIdx.x; tile < ntiles && ok; tile += gridDim.x, unit0 += units_per_tile) {
            const int n = item_n0(tile) + ch;
            const int m0 = item_m0(tile);
            const int split = tile & (nsplit - 1);
            const int gbase = split * ngroups;          // first scale group of this work item
            float acc[kPfDrainCols];
#pragma unroll
            for (int j = 0; j < kPfDrainCols; ++j) acc[j] = 0.f;
            // Scales are fetched eight groups ahead (a drain takes a few hundred cycles, a
            // global load several hundred): a ring of eight, refilled once per eight groups.
            const float *sc_row = PARTIALS ? nullptr : p.w_scale + (size_t)n * p.G + gbase;
            const unsigned short *sc_row_h = reinterpret_cast<const unsigned short *>(p.w_scale) + (size_t)n * p.G + gbase;
            // The ring holds what the loads return, untouched: any instruction that reads a
            // loaded register makes the warp wait for that load.  fp32: eight values.  binary16:
            // eight values widened when they are taken out -- fetched as one 16-byte load when the
            // row pitch allows (G % 8 == 0: registers 0..3 hold two scales each), else as eight
            // 16-bit loads into 32-bit registers.
            const bool vec8 = H16 && (p.G % 8 == 0) && (gbase % 8 == 0);
            uint32_t sc_nxt[8] = {0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u};
            auto refill = [&](int g0) {
                if constexpr (PARTIALS) {
                    return;
                } else if constexpr (H16) {
                    if (vec8) {
                        if (g0 < ngroups) {
                            const uint4 v = __ldg(reinterpret_cast<const uint4 *>(sc_row_h + g0));
                            sc_nxt[0] = v.x; sc_nxt[1] = v.y; sc_nxt[2] = v.z; sc_nxt[3] = v.w;
                        }
                    } else {
#pragma unroll
                        for (int u = 0; u < 8; ++u)
                            if (g0 + u < ngroups)
                                asm volatile("ld.global.nc.u16 %0, [%1];" : "=r"(sc_nxt[u]) : "l"(sc_row_h + g0 + u));
                    }
                } else {
#pragma unroll
                    for (int u = 0; u < 8; ++u)
                        if (g0 + u < ngroups) sc_nxt[u] = __float_as_uint(__ldg(sc_row + g0 + u));
                }
            };
            auto take = [&](int u) -> float {          // u is a constant after unrolling
                if constexpr (H16) {
                    // one conversion that names the half of the register it reads
                    const __half2 pair = *reinterpret_cast<const __half2 *>(&sc_nxt[u >> 1]);
                    const __half2 lone = *reinterpret_cast<const __half2 *>(&sc_nxt[u]);
                    if (vec8) return (u & 1) ? __high2float(pair) : __low2float(pair);
                    return __low2float(lone);
                } else {
                    return __uint_as_float(sc_nxt[u]);
                }
            };
            refill(0);
            // Software pipeline over 32-column halves: while one half is converted and
            // accumulated, the next half (possibly of the next group) is on its way from TMEM.
            int v0[32], v1[32];                         // first / second half of the current group
            ok = pf_wait_warp(pf_smem_u32(&bar_acc_full[unit0 & 1]), (unit0 >> 1) & 1, abort_flag);
            if (ok) { pf_tc_fence_after(); pf_tmem_ld32(tlane + (2 * (unit0 & 1)) * kPfBN, v0); }
            for (int g0 = 0; g0 < ngroups && ok; g0 += 8) {
                float sc_cur[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    sc_cur[u] = take(u);
                }
                refill(g0 + 8);
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    const int gi = g0 + u;
                    if (gi >= ngroups || !ok) break;
                    const int unit = unit0 + (gi >> 1);            // group gi lives in buffer 2 (unit % 2) + gi % 2
                    const int buf = 2 * (unit & 1) + (gi & 1);
                    const float sc = sc_cur[u];
                    pf_tmem_ld_wait();                     // first half of group gi is in v0
                    pf_tmem_ld32(tlane + buf * kPfBN + 32, v1);
                    if (PARTIALS) {
#pragma unroll
                        for (int j = 0; j < 32; ++j) {
                            const int m = m0 + col0 + j;
                            if (m < p.M) p.partials[((size_t)m * p.N + n) * p.G + gi] = v0[j] >> 6;
                        }
                    } else {
#pragma unroll
                        for (int j = 0; j < 32; j += 2) {
                            if ((j & 7) < kPfMagicOfEight) pf_cvt_fma2<DPS == 1 || DPS == 2>(acc[j], acc[j + 1], v0[j], v0[j + 1], sc);
                            else                  pf_cvt_fma2<false>(acc[j], acc[j + 1], v0[j], v0[j + 1], sc);
                        }
                    }
                    pf_tmem_ld_wait();                     // second half is in v1
                    {
                        // all of this warp's share of the buffer has been read: hand it back
                        pf_tc_fence_before();
                        __syncwarp();
                        if (lane == 0) pf_mbar_arrive(pf_smem_u32(&bar_acc_empty[buf]));
                    }
                    if (gi + 1 < ngroups) {                // request the first half of the next group
                        const int nunit = unit0 + ((gi + 1) >> 1);
                        if (((gi + 1) & 1) == 0) {         // it opens a new unit: wait for its MMAs
                            ok = pf_wait(pf_smem_u32(&bar_acc_full[nunit & 1]), (nunit >> 1) & 1, abort_flag);   // all lanes poll: no broadcast step
                            if (!ok) break;
                            pf_tc_fence_after();
                        }
                        pf_tmem_ld32(tlane + (2 * (nunit & 1) + ((gi + 1) & 1)) * kPfBN, v0);
                    }
                    if (PARTIALS) {
#pragma unroll
                        for (int j = 0; j < 32; ++j) {
                            const int m = m0 + col0 + 32 + j;
                            if (m < p.M) p.partials[((size_t)m * p.N + n) * p.G + gi] = v1[j] >> 6;
                        }
                    } else {
#pragma unroll
                        for (int j = 0; j < 32; j += 2)
                            if ((j & 7) < kPfMagicOfEight) pf_cvt_fma2<DPS == 1 || DPS == 2>(acc[32 + j], acc[32 + j + 1], v1[j], v1[j + 1], sc);
                            else                  pf_cvt_fma2<false>(acc[32 + j], acc[32 + j + 1], v1[j], v1[j + 1], sc);
                    }
                }
            }
            pf_tmem_ld_wait();
            if (!PARTIALS && ok) {
#pragma unroll
                for (int j = 0; j < kPfDrainCols; ++j) {
                    const int m = m0 + col0 + j;
                    if (m < p.M) {
                        const float v = acc[j] * (__ldg(p.a_scale + m) * (1.0f / kCodeGain));
                        if (SPLIT)        p.split_out[((size_t)split * p.M + m) * p.N + n] = v;
                        else if (H16 && p.y16) reinterpret_cast<__nv_bfloat16 *>(p.y)[(size_t)m * p.ldy + n] = __float2bfloat16_rn(v);
                        else              p.y[(size_t)m * p.ldy + n] = v;
                    }
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
        pf_tmem_dealloc(tmem_base, kPfTmemCols);
    }
}

// Sum of the K-split partial outputs in split order (fixed order: the result does not depend on
// which CTA finished first).  One thread per four consecutive channels.
__global__ void pf_splitk_reduce_kernel(const float *__restrict__ split_out, void *__restrict__ y, int M, int N,
                                        int nsplit, int ldy, int y16) {
    const size_t quads = (size_t)M * (N / 4);
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < quads; i += (size_t)gridDim.x * blockDim.x) {
        const int m = (int)(i / (N / 4)), n = (int)(i % (N / 4)) * 4;
        float4 acc = __ldcs(reinterpret_cast<const float4 *>(split_out + (size_t)m * N + n));
        for (int sidx = 1; sidx < nsplit; ++sidx) {
            const float4 v = __ldcs(reinterpret_cast<const float4 *>(split_out + ((size_t)sidx * M + m) * N + n));
            acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
        }
        if (y16) {
            __nv_bfloat16 *out = reinterpret_cast<__nv_bfloat16 *>(y) + (size_t)m * ldy + n;
            out[0] = __float2bfloat16_rn(acc.x); out[1] = __float2bfloat16_rn(acc.y);
            out[2] = __float2bfloat16_rn(acc.z); out[3] = __float2bfloat16_rn(acc.w);
        } else {
            *reinterpret_cast<float4 *>(reinterpret_cast<float *>(y) + (size_t)m * ldy + n) = acc;
        }
    }
}

// ---- host side -----------------------------------------------------------------------
int env_int(const char *name, int dflt);

// Unpack warps (warp layout) by scale group; W2A8_PF_UNPACK_WARPS = 2 or 4 overrides.
int prefill_unpack_warps(int group) {
    const int forced = env_int("W2A8_PF_UNPACK_WARPS", 0);
    if (forced == 2 || forced == 4) return forced;
    // Measured on B200 (4096 -> 14336, 2048 tokens, POPS with 2 / 4 unpack warps): group 64: 717 / 637;
    // 128: 946 / 1006; 256: 1105 / 1328; K: 1130 / 1455.  With 64-k groups the drain warps are the
    // bottleneck and two more warps competing for their issue slots cost more than a faster unpack
    // gains; from 128 up the unpack is.
    return group >= 128 ? 4 : 2;
}
bool prefill_supported(int M, int N, int K, int group) {
    if (M < 64) return false;
    if (N % kPfBM != 0 || K % kPfBK != 0) return false;
    if (!(group == 64 || group == 128 || group % 256 == 0)) return false;   // group == K implies K % 256 == 0 here
    if ((long long)64 * 254 * group >= (1ll << 31)) return false;           // int32 accumulator range
    return true;
}

// Cost of one round of tiles (one 128 x 128 tile per SM) in seconds per unit of K, by scale group:
// the drain runs once per group, so larger groups are cheaper.  From the kernel's measured rates on
// B200 at 4096 -> 14336, 2048 tokens (12 rounds): group 64: 717 TOPS = 6.8 ns per k and round (the
// rule keeps the 7 ns it was fitted with), 128: 1021 = 4.8, 256: 1356 = 3.6, K: 1657 = 2.9.
static double prefill_round_seconds_per_k(int group) {
    return group <= 64 ? 7.0e-9 : group <= 128 ? 4.8e-9 : group <= 256 ? 3.6e-9 : 3.0e-9;
}
constexpr double kStreamSecondsPerMac = 8.0e-15;    // streaming kernel, per token x weight
// a round of 128 x 256 tiles of the one-scale-per-channel kernel (2114 TOPS at 4096 -> 14336, 2048 tokens: 6 rounds)
constexpr double kWideRoundSecondsPerK = 4.63e-9;

static double split_plan(int M, int N, int K, int tile_tokens, double round_seconds_per_k, int *channels);
bool prefill_uses_wide(int M, int N, int K, int group);

constexpr size_t kPfSplitOffset = 256;              // byte offset of the K-split partial outputs in the workspace

// Estimated time of the tensor-core path with the work of every tile split `nsplit` ways along K:
// rounds of one work item per SM, each K / nsplit long, plus (split only) the launch of the summing
// kernel and its traffic.
static double prefill_seconds(int M, int N, int K, int group, int nsplit) {
    const long long items = (long long)(N / kPfBM) * ((M + kPfBN - 1) / kPfBN) * nsplit;
    const long long sms = sm_count();
    const long long rounds = (items + sms - 1) / sms;
    double t = (double)rounds * (K / nsplit) * prefill_round_seconds_per_k(group);
    if (nsplit > 1) t += 2.0e-6 + (double)(nsplit + 1) * M * N * 4.0 / 3.0e12;
    return t;
}

// K splits for a shape the kernel supports: 1, 2, 4 or 8.  A problem with few output tiles leaves
// most SMs idle (one CTA per 128 x 128 tile walking all of K); splitting K puts more of them to work
// at the price of fp32 partial outputs in the workspace and a second, small kernel that adds them in
// split order.  Every split is a whole number of 256-k blocks and of scale groups, at least two blocks.
// W2A8_PF_KSPLIT = 1, 2, 4, 8 forces a count (if it divides the shape).
int prefill_ksplit(int M, int N, int K, int group) {
    auto valid = [&](int sp) {
        if (sp == 1) return true;
        const int ks = K / sp;
        return K % sp == 0 && ks % kPfBK == 0 && ks % group == 0 && ks >= 2 * kPfBK;
    };
    const int forced = env_int("W2A8_PF_KSPLIT", 0);
    if (forced == 1 || forced == 2 || forced == 4 || forced == 8) return valid(forced) ? forced : 1;
    int best = 1;
    double best_t = prefill_seconds(M, N, K, group, 1);
    for (int sp = 2; sp <= 8; sp *= 2) {
        if (!valid(sp)) continue;
        const double t = prefill_seconds(M, N, K, group, sp);
        if (t < best_t * 0.95) { best_t = t; best = sp; }      // a split has to pay by 5 % or more
    }
    return best;
}

// Bytes the kernel needs in the workspace (behind the status word) for a shape: the K-split partial outputs.
size_t prefill_workspace_bytes(int M, int N, int K, int group) {
    const int sp = prefill_ksplit(M, N, K, group);
    return sp > 1 ? kPfSplitOffset + (size_t)sp * M * N * sizeof(float) : 0;
}

// Whether the tensor-core kernel is expected to beat the streaming kernel on a shape it supports.
// At group 64 without a K split the two cost models cross at M * N of about 0.95 million per round of
// tiles (measured: 14336x4096 at M = 128: 94 us against 66 us streaming; at M = 256: 97 against 127;
// 4096x4096 at M = 64: 31 against 11); the same margin (the tensor-core estimate has to be 8 % below
// the streaming one) is kept with a split.  `can_split` = false: the caller's kernel has no K split.
bool prefill_preferred(int M, int N, int K, int group, bool can_split) {
    const int sp = can_split ? prefill_ksplit(M, N, K, group) : 1;
    double t_tc = prefill_seconds(M, N, K, group, sp);
    if (can_split && prefill_uses_wide(M, N, K, group)) {
        int c;
        const double t_wide = split_plan(M, N, K, 256, kWideRoundSecondsPerK, &c);
        if (t_wide < t_tc) t_tc = t_wide;
    }
    const double t_stream = kStreamSecondsPerMac * (double)M * (double)N * (double)K;
    return t_tc * (950000.0 / 875000.0) < t_stream;
}

bool prefill_wide_supported(int M, int N, int K, int group);
int launch_prefill_wide(const int8_t *a, const float *a_scale, const uint32_t *packed, const void *w_scale,
                        void *y, int M, int N, int K, int *status, cudaStream_t st, bool h16, bool y16, int ldy);

// Best way to give the first channel tiles to a tensor-core kernel with tiles of `tile_tokens` tokens and
// the last few (at most eight) to the streaming kernel: tiles are handed out in rounds of one tile per SM
// (148 on B200), and a last round with a handful of tiles costs as much as a full one (4096x14336 at
// M = 512: 448 tiles = 3 rounds + 4 tiles).  Returns the estimated seconds; *channels = a multiple of 128.
static double split_plan(int M, int N, int K, int tile_tokens, double round_seconds_per_k, int *channels) {
    const int ct = N / kPfBM, tiles_m = (M + tile_tokens - 1) / tile_tokens;
    const long long sms = sm_count();
    const double round_s = round_seconds_per_k * K;
    double best = 1e30;
    int best_ct = ct;
    for (int c = ct; c >= 1 && c >= ct - 8; --c) {
        const long long rounds = ((long long)c * tiles_m + sms - 1) / sms;
        double t = (double)rounds * round_s;
        if (c < ct) t += 2.0e-6 + kStreamSecondsPerMac * (double)M * (double)(ct - c) * kPfBM * (double)K;
        if (t < best * 0.97) { best = t; best_ct = c; }      // a split has to pay by 3 % or more
    }
    *channels = best_ct * kPfBM;
    return best;
}

// One scale per channel and many tokens: whether the 256-token-tile kernel takes the shape (its round of
// tiles costs more per k, but there are half as many tiles).  W2A8_PF_WIDE = 0 never, 2 whenever supported.
bool prefill_uses_wide(int M, int N, int K, int group) {
    if (!prefill_wide_supported(M, N, K, group)) return false;
    if (env_int("W2A8_PF_WIDE", 1) == 2) return true;
    if (prefill_ksplit(M, N, K, group) > 1) return false;
    int c128, c256;
    return split_plan(M, N, K, 256, kWideRoundSecondsPerK, &c256) <
           split_plan(M, N, K, kPfBN, prefill_round_seconds_per_k(group), &c128);
}

// How many of the N channels the tensor-core kernel should take when the rest may go to the
// streaming kernel (see split_plan).  Returns a multiple of 128 in (0, N].
int prefill_channel_split(int M, int N, int K, int group) {
    if (prefill_ksplit(M, N, K, group) > 1 && !prefill_uses_wide(M, N, K, group)) return N;   // few tiles: K is split instead
    int channels;
    if (prefill_uses_wide(M, N, K, group)) split_plan(M, N, K, 256, kWideRoundSecondsPerK, &channels);
    else                                   split_plan(M, N, K, kPfBN, prefill_round_seconds_per_k(group), &channels);
    return channels;
}

// Enqueue the prefill kernel.  `partials` != nullptr selects the parity export.
int launch_prefill(const int8_t *a, const float *a_scale, const uint32_t *packed, const void *w_scale,
                   void *y, int32_t *partials, int M, int N, int K, int group, int *status,
                   cudaStream_t st, bool h16, bool y16, int ldy) {
    if (h16 && partials) return W2A8_ERR_SHAPE;
    // one scale per channel and enough tokens: the 256-token-tile kernel
    if (!partials && ldy >= N && prefill_uses_wide(M, ldy, K, group) &&
        (N == ldy || N == prefill_channel_split(M, ldy, K, group)))
        return launch_prefill_wide(a, a_scale, packed, w_scale, y, M, N, K, status, st, h16, y16, ldy);
    EncodeTiledFn encode = encode_tiled_fn();
    if (!encode) return W2A8_ERR_CUDA;
    CUtensorMap map;
    const cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)M};
    const cuuint64_t strides[1] = {(cuuint64_t)K};                 // bytes between tokens
    const cuuint32_t box[2] = {128u, (cuuint32_t)kPfBN};          // 128 k x 128 tokens
    const cuuint32_t estr[2] = {1u, 1u};
    if (encode(&map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<int8_t *>(a), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return W2A8_ERR_CUDA;
    PrefillParams p;
    p.packed = packed; p.w_scale = reinterpret_cast<const float *>(w_scale); p.a_scale = a_scale;
    p.y = reinterpret_cast<float *>(y); p.partials = partials; p.y16 = (h16 && y16) ? 1 : 0;
    p.ldy = ldy;
    p.status = status;
    p.M = M; p.N = N; p.K = K; p.G = K / group; p.group = group;
    p.words_per_row = K / 16;
    p.slices_per_group = group / 64;
    // K split: only for the whole matrix (the caller gives no channel remainder to the streaming
    // kernel then) and never for the parity export
    const int nsplit = (partials || ldy != N) ? 1 : prefill_ksplit(M, N, K, group);
    p.ks_shift = nsplit == 8 ? 3 : nsplit == 4 ? 2 : nsplit == 2 ? 1 : 0;
    p.split_out = nsplit > 1 ? reinterpret_cast<float *>(reinterpret_cast<char *>(status) + kPfSplitOffset) : nullptr;
    const size_t smem = (size_t)kPfStages * kPfStageBytes + 1024;
    const long long tiles = (long long)(N / kPfBM) * ((M + kPfBN - 1) / kPfBN) * nsplit;
    const int sms = sm_count();
    dim3 grid((unsigned)(tiles < sms ? tiles : sms));   // persistent CTAs, one per SM
    static PerDeviceFlags configured[21];
    auto launch = [&](auto kernel, int slot, int threads) -> bool {
        if (allow_dynamic_smem(kernel, configured[slot], (int)smem) != cudaSuccess) return false;
        kernel<<<grid, threads, smem, st>>>(map, p);
        return true;
    };
    // The MMA-issuing code is specialised on the 64-k slices per scale group: 1, 2, or whole stages
    // (0); the warp layout on the number of unpack warps (the parity export keeps the 12-warp one).
    // A K split runs on the group's default layout only.
    const int uw = nsplit > 1 ? (group >= 128 ? 4 : 2) : prefill_unpack_warps(group);
    auto launch_dps = [&](auto partials_c, auto h16_c, auto uw_c, int slot0) -> bool {
        constexpr bool P = decltype(partials_c)::value, H = decltype(h16_c)::value;
        constexpr int U = decltype(uw_c)::value;
        if (group == 64) return launch(w2a8_prefill_kernel<P, H, 1, U, false>, slot0, pf_threads(U));
        if (group == 128) return launch(w2a8_prefill_kernel<P, H, 2, U, false>, slot0 + 1, pf_threads(U));
        return launch(w2a8_prefill_kernel<P, H, 0, U, false>, slot0 + 2, pf_threads(U));
    };
    auto launch_split = [&](auto h16_c, int slot0) -> bool {
        constexpr bool H = decltype(h16_c)::value;
        if (group == 64) return launch(w2a8_prefill_kernel<false, H, 1, 2, true>, slot0, pf_threads(2));
        if (group == 128) return launch(w2a8_prefill_kernel<false, H, 2, 4, true>, slot0 + 1, pf_threads(4));
        return launch(w2a8_prefill_kernel<false, H, 0, 4, true>, slot0 + 2, pf_threads(4));
    };
    using U2 = std::integral_constant<int, 2>;
    using U4 = std::integral_constant<int, 4>;
    const bool launched =
        partials     ? launch_dps(std::true_type{}, std::false_type{}, U2{}, 3)
        : nsplit > 1 ? (h16 ? launch_split(std::true_type{}, 18) : launch_split(std::false_type{}, 15))
        : h16        ? (uw == 4 ? launch_dps(std::false_type{}, std::true_type{}, U4{}, 12)
                                : launch_dps(std::false_type{}, std::true_type{}, U2{}, 6))
                     : (uw == 4 ? launch_dps(std::false_type{}, std::false_type{}, U4{}, 9)
                                : launch_dps(std::false_type{}, std::false_type{}, U2{}, 0));
    if (!launched) return W2A8_ERR_CUDA;
    if (nsplit > 1) {
        const size_t quads = (size_t)M * (N / 4);
        const unsigned blocks = (unsigned)((quads + 255) / 256 < (size_t)(8 * sms) ? (quads + 255) / 256 : (size_t)(8 * sms));
        pf_splitk_reduce_kernel<<<blocks, 256, 0, st>>>(p.split_out, y, M, N, nsplit, ldy, p.y16);
    }
    return cudaGetLastError() == cudaSuccess ? W2A8_OK : W2A8_ERR_CUDA;
}

}  // namespace w2a8
