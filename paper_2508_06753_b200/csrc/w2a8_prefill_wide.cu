// Tensor-core W2A8 kernel for one scale per output channel (group = K) and many tokens: the int8
// kernel of w2a8_prefill.cu with 256-token tiles.  With no per-group drain the producers bound that
// kernel (two unpack teams need about twice the time of the MMAs of a 128-token tile); a tile of
// 128 channels x 256 tokens feeds every unpacked weight stage to twice the MACs (tcgen05.mma with
// N = 256) and halves the shared-memory operand reads per MAC (Sec. II-D: larger tiles of the output
// per work-group where the data allow it; Sec. II-C: the 2-bit -> int8 up-convert in shared memory).
// The accumulators of such a tile (128 x 256 int32) fill half of tensor memory, so two tiles are in
// flight and a tile's only drain is its epilogue -- which is why this form needs group = K: with
// finer groups the fp32 running sums of a 128 x 256 tile would not fit the register file.
//
//   16 warps in four warpgroups, registers re-balanced at entry (setmaxnreg):
//     warps 0-3   two MMA issuers (half of every stage's K steps each), the TMA producer, a spare (56)
//     warps 4-7   unpack: two teams of two warps on alternate 128-k stages (104)
//     warps 8-15  epilogue: two warps per TMEM lane quarter, 128 token columns each (176)
//   A stage is 128 k: weights 128 rows x 128 B (int8 lanes 64 * (code - 2), 128-byte swizzle) + activations
//   256 rows x 128 B by one TMA box; four stages of 48 KB.  Every wait is bounded; a wait that gives up
//   sets the status word of the workspace and the CTA winds down.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "w2a8_tc.cuh"

namespace w2a8 {

constexpr int kWdThreads = 32 * 16;
constexpr int kWdFirstUnpack = 4, kWdFirstDrain = 8;
constexpr int kWdBM = 128;                // channels per tile (UMMA M)
constexpr int kWdBN = 256;                // tokens per tile (UMMA N)
constexpr int kWdBK = 128;                // k per stage: half a 256-k block of the packed layout
constexpr int kWdStages = 4;
constexpr int kWdABytes = 128 * 128;      // weights of a stage: [128 rows][128 B], swizzled
constexpr int kWdBBytes = 256 * 128;      // activations of a stage: [256 rows][128 B], swizzled
constexpr int kWdStageBytes = kWdABytes + kWdBBytes;
constexpr int kWdTmemCols = 2 * kWdBN;    // two accumulator buffers: all of tensor memory

struct WideParams {
    const uint32_t *packed;
    const void *w_scale;     // one scale per channel: fp32, or binary16 (H16)
    const float *a_scale;
    void *y;                 // fp32, or bf16 (H16 with y16)
    int *status;
    int M, N, K;
    int words_per_row;
    int y16;
    int ldy;
};

template <int N>
__device__ __forceinline__ void wd_setmaxnreg_dec() { asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N)); }
template <int N>
__device__ __forceinline__ void wd_setmaxnreg_inc() { asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N)); }

template <bool H16>
__global__ void __launch_bounds__(kWdThreads, 1)
w2a8_prefill_wide_kernel(const __grid_constant__ CUtensorMap act_map, const WideParams p) {
    extern __shared__ unsigned char wd_smem_raw[];
    __shared__ __align__(8) unsigned long long bar_full[kWdStages], bar_empty[kWdStages];
    __shared__ __align__(8) unsigned long long bar_acc_full[2], bar_acc_empty[2], bar_first;
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag_s;
    volatile int *abort_flag = &abort_flag_s;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int nstages = p.K / kWdBK;        // stages per tile (even: K is a multiple of 256)
    const int tiles_m = (p.M + kWdBN - 1) / kWdBN;
    const int ntiles = (p.N / kWdBM) * tiles_m;
    // Persistent CTA: tiles blockIdx.x, blockIdx.x + gridDim.x, ...; consecutive tiles share the channel tile
    const uint32_t smem_base = (pf_smem_u32(wd_smem_raw) + 1023u) & ~1023u;

    if (threadIdx.x == 0) {
        abort_flag_s = 0;
        for (int s = 0; s < kWdStages; ++s) {
            pf_mbar_init(pf_smem_u32(&bar_full[s]), 2 + 1);   // the two unpack warps of a team + the TMA producer
            pf_mbar_init(pf_smem_u32(&bar_empty[s]), 2);      // one tcgen05.commit per MMA-issuing thread
        }
        for (int b = 0; b < 2; ++b) {
            pf_mbar_init(pf_smem_u32(&bar_acc_full[b]), 2);   // tcgen05.commit of both issuers after a tile's last stage
            pf_mbar_init(pf_smem_u32(&bar_acc_empty[b]), 8);  // one arrive per epilogue warp
        }
        pf_mbar_init(pf_smem_u32(&bar_first), 1);             // tcgen05.commit after a tile's first stage
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        pf_fence_proxy_async();
    }
    if (warp == 1) pf_tmem_alloc(pf_smem_u32(&tmem_base_slot), kWdTmemCols);
    pf_tc_fence_before();
    __syncthreads();
    pf_tc_fence_after();
    const uint32_t tmem_base = tmem_base_slot;

    if (warp < kWdFirstUnpack) {
        wd_setmaxnreg_dec<56>();
        if (warp == 2 && lane == 0) {
            // ===== TMA producer: activations, 256 tokens x 128 k per stage ===================
            int s = 0, round = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < ntiles && ok; tile += gridDim.x) {
                const int m0 = (tile % tiles_m) * kWdBN;
                for (int it = 0; it < nstages; ++it) {
                    if (round > 0 && !pf_wait(pf_smem_u32(&bar_empty[s]), (round - 1) & 1, abort_flag)) {
                        ok = false;
                        break;
                    }
                    const uint32_t bar = pf_smem_u32(&bar_full[s]);
                    pf_mbar_arrive_expect_tx(bar, kWdBBytes);
                    pf_tma_load_2d(smem_base + s * kWdStageBytes + kWdABytes, &act_map, it * kWdBK, m0, bar);
                    if (++s == kWdStages) { s = 0; ++round; }
                }
            }
        }
        // ===== MMA issuers: both threads issue into the tile's accumulator buffer ==================
        // A lone thread needs a wait (a few hundred cycles even on a complete barrier) plus ~100
        // cycles per MMA for every stage, more than the 512 cycles the stage's MMAs take; so thread 0
        // issues K steps 0 and 1 of a stage and thread 1 steps 2 and 3.  Integer accumulation does not
        // depend on the order, except that the tile's first MMA (which overwrites the buffer) has to
        // come first: thread 0 issues all of stage 0 and commits `bar_first`; thread 1 waits for it
        // before its first MMA of the tile.  Straight-line issue: descriptors = 32-bit base + immediates.
        if (warp < 2 && lane == 0) {
            const int w = warp;
            const uint64_t a_desc0 = pf_smem_desc(smem_base);
            const uint64_t b_desc0 = pf_smem_desc(smem_base + kWdABytes);
            const uint32_t a_lo0 = (uint32_t)a_desc0, a_hi = (uint32_t)(a_desc0 >> 32);
            const uint32_t b_lo0 = (uint32_t)b_desc0, b_hi = (uint32_t)(b_desc0 >> 32);
            constexpr uint32_t idesc = pf_instr_desc(kWdBM, kWdBN);
            int s = 0;
            uint32_t so = 0;                // stage offset in 16-byte units
            uint32_t full_parity = 0;
            bool ok = true;
            int seq = 0;                    // tiles of this CTA so far
            for (int tile = blockIdx.x; tile < ntiles && ok; tile += gridDim.x, ++seq) {
                const int buf = seq & 1;
                const uint32_t d_tmem = tmem_base + buf * kWdBN;
                for (int it = 0; it < nstages && ok; ++it) {
                    ok = pf_wait(pf_smem_u32(&bar_full[s]), full_parity, abort_flag);
                    if (!ok) break;
                    const uint64_t ad = ((uint64_t)a_hi << 32) | (a_lo0 + so);
                    const uint64_t bd = ((uint64_t)b_hi << 32) | (b_lo0 + so);
                    if (it == 0) {
                        if (w == 0) {
                            if (seq >= 2) {     // the epilogue warps must have read out this buffer's last tile
                                ok = pf_wait(pf_smem_u32(&bar_acc_empty[buf]), (uint32_t)((seq >> 1) - 1) & 1u, abort_flag);
                                if (!ok) break;
                            }
                            pf_tc_fence_after();
                            pf_mma_i8(d_tmem, ad, bd, idesc, 0u);
                            pf_mma_i8(d_tmem, ad + 2, bd + 2, idesc, 1u);
                            pf_mma_i8(d_tmem, ad + 4, bd + 4, idesc, 1u);
                            pf_mma_i8(d_tmem, ad + 6, bd + 6, idesc, 1u);
                            pf_mma_commit(pf_smem_u32(&bar_first));
                        }
                    } else {
                        if (it == 1 && w == 1) {
                            ok = pf_wait(pf_smem_u32(&bar_first), (uint32_t)seq & 1u, abort_flag);
                            if (!ok) break;
                        }
                        pf_tc_fence_after();
                        pf_mma_i8(d_tmem, ad + 4 * w, bd + 4 * w, idesc, 1u);
                        pf_mma_i8(d_tmem, ad + 4 * w + 2, bd + 4 * w + 2, idesc, 1u);
                        if (it == nstages - 1) pf_mma_commit(pf_smem_u32(&bar_acc_full[buf]));
                    }
                    pf_mma_commit(pf_smem_u32(&bar_empty[s]));   // stage can be refilled once these MMAs are done
                    so += kWdStageBytes >> 4;
                    if (++s == kWdStages) { s = 0; so = 0; full_parity ^= 1u; }
                }
            }
        }
    } else if (warp < kWdFirstDrain) {
        wd_setmaxnreg_dec<104>();
        // ===== unpack warps: packed words -> int8 lanes, K-major, 128-byte swizzle =====
        // Two teams of two warps; a stage is half a 256-k block, so team j fills every stage of parity
        // j: slices 2 j and 2 j + 1 of each block.  A thread owns eight units of a stage (a row and a
        // quarter t of it): word t of the stage's two slices.  Rows are dealt so that the eight lanes of
        // a shared-memory wavefront cover all eight 16-byte chunk positions of the swizzled row.
        constexpr int kUnits = 8;
        const int team = (warp - kWdFirstUnpack) >> 1;
        const int ut = ((warp - kWdFirstUnpack) & 1) * 32 + lane;
        auto unit_row = [](int u) { return (u >> 5) * 8 + ((u >> 2) & 1) * 4 + ((u >> 3) & 3); };
        auto request = [&](uint2 (&wv)[kUnits], int tile, int blk) {
            const int n0 = (tile / tiles_m) * kWdBM;
#pragma unroll
            for (int i = 0; i < kUnits; ++i) {
                const int u = ut + 64 * i;
                const int r = unit_row(u), t = u & 3;
                wv[i] = __ldg(reinterpret_cast<const uint2 *>(p.packed + (size_t)(n0 + r) * p.words_per_row +
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
            int tile_nxt = tile, blk_nxt = blk + 1;
            if (blk_nxt == nblocks) { blk_nxt = 0; tile_nxt += gridDim.x; }
            if (tile_nxt < ntiles) request(w_nxt, tile_nxt, blk_nxt);
            if (round > 0 && !pf_wait(pf_smem_u32(&bar_empty[s]), (round - 1) & 1, abort_flag)) break;
            const uint32_t a_stage = smem_base + s * kWdStageBytes;
#pragma unroll
            for (int i = 0; i < kUnits; ++i) {
                const int u = ut + 64 * i;
                const int r = unit_row(u), t = u & 3;
                const uint32_t ws[2] = {w_cur[i].x, w_cur[i].y};
#pragma unroll
                for (int sl = 0; sl < 2; ++sl) {    // slice sl of the stage: k = 64 sl + 16 t .. + 15
                    const int chunk = (4 * sl + t) ^ (r & 7);
                    pf_st_shared_v4(a_stage + r * 128 + chunk * 16, lane_codes(ws[sl], 0), lane_codes(ws[sl], 1),
                                    lane_codes(ws[sl], 2), lane_codes(ws[sl], 3));
                }
            }
            pf_fence_proxy_async();     // make the generic-proxy stores visible to the tensor core
            __syncwarp();
            if (lane == 0) pf_mbar_arrive(pf_smem_u32(&bar_full[s]));
            tile = tile_nxt; blk = blk_nxt;
            s += 2;
            if (s >= kWdStages) { s -= kWdStages; ++round; }
        }
    } else {
        wd_setmaxnreg_inc<176>();
        // ===== epilogue warps: TMEM -> registers -> y, one scale per channel ================
        const int q4 = warp & 3;                    // TMEM lane quarter this warp may access
        const int col0 = ((warp - kWdFirstDrain) >> 2) * 128;     // first token column of this warp
        const int ch = q4 * 32 + lane;              // channel inside the tile = TMEM lane
        bool ok = true;
        int seq = 0;
        for (int tile = blockIdx.x; tile < ntiles && ok; tile += gridDim.x, ++seq) {
            const int n = (tile / tiles_m) * kWdBM + ch;
            const int m0 = (tile % tiles_m) * kWdBN;
            const int buf = seq & 1;
            float sc;
            if constexpr (H16) sc = __half2float(reinterpret_cast<const __half *>(p.w_scale)[n]);
            else               sc = __ldg(reinterpret_cast<const float *>(p.w_scale) + n);
            ok = pf_wait(pf_smem_u32(&bar_acc_full[buf]), (uint32_t)(seq >> 1) & 1u, abort_flag);   // all lanes poll
            if (!ok) break;
            pf_tc_fence_after();
            const uint32_t taddr = tmem_base + ((uint32_t)(q4 * 32) << 16) + buf * kWdBN + col0;
            int v0[32], v1[32];
            auto store32 = [&](const int (&v)[32], int c) {
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    const int m = m0 + col0 + 32 * c + j;
                    if (m < p.M) {
                        // same order of operations as the 128-token kernel: (sum * w scale) * (token scale / 64)
                        const float val = ((float)v[j] * sc) * (__ldg(p.a_scale + m) * (1.0f / kCodeGain));
                        if (H16 && p.y16) reinterpret_cast<__nv_bfloat16 *>(p.y)[(size_t)m * p.ldy + n] = __float2bfloat16_rn(val);
                        else              reinterpret_cast<float *>(p.y)[(size_t)m * p.ldy + n] = val;
                    }
                }
            };
            pf_tmem_ld32(taddr, v0);
            pf_tmem_ld_wait();
            pf_tmem_ld32(taddr + 32, v1);
            store32(v0, 0);
            pf_tmem_ld_wait();
            pf_tmem_ld32(taddr + 64, v0);
            store32(v1, 1);
            pf_tmem_ld_wait();
            pf_tmem_ld32(taddr + 96, v1);
            store32(v0, 2);
            pf_tmem_ld_wait();
            // this warp's share of the buffer has been read: hand it back before the last stores
            pf_tc_fence_before();
            __syncwarp();
            if (lane == 0) pf_mbar_arrive(pf_smem_u32(&bar_acc_empty[buf]));
            store32(v1, 3);
        }
    }

    // ---- wind down ---------------------------------------------------------------------
    pf_tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0 && abort_flag_s) atomicExch(p.status, W2A8_ERR_TIMEOUT);
    if (warp == 1) {
        pf_tc_fence_after();
        pf_tmem_dealloc(tmem_base, kWdTmemCols);
    }
}

// ---- host side -----------------------------------------------------------------------
int env_int(const char *name, int dflt);

bool prefill_wide_supported(int M, int N, int K, int group) {
    if (group != K) return false;
    if (M < 129) return false;                        // a 256-token tile would be more than half empty
    if (N % kWdBM != 0 || K % 256 != 0) return false;
    if ((long long)64 * 254 * K >= (1ll << 31)) return false;   // int32 accumulator range
    return env_int("W2A8_PF_WIDE", 1) != 0;
}

// Enqueue the 256-token-tile kernel on the first N channels of a matrix whose y rows are ldy apart.
int launch_prefill_wide(const int8_t *a, const float *a_scale, const uint32_t *packed, const void *w_scale,
                        void *y, int M, int N, int K, int *status, cudaStream_t st, bool h16, bool y16, int ldy) {
    EncodeTiledFn encode = encode_tiled_fn();
    if (!encode) return W2A8_ERR_CUDA;
    CUtensorMap map;
    const cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)M};
    const cuuint64_t strides[1] = {(cuuint64_t)K};                 // bytes between tokens
    const cuuint32_t box[2] = {128u, (cuuint32_t)kWdBN};          // 128 k x 256 tokens
    const cuuint32_t estr[2] = {1u, 1u};
    if (encode(&map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<int8_t *>(a), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return W2A8_ERR_CUDA;
    WideParams p;
    p.packed = packed; p.w_scale = w_scale; p.a_scale = a_scale; p.y = y; p.status = status;
    p.M = M; p.N = N; p.K = K; p.words_per_row = K / 16; p.y16 = (h16 && y16) ? 1 : 0; p.ldy = ldy;
    const size_t smem = (size_t)kWdStages * kWdStageBytes + 1024;
    const long long tiles = (long long)(N / kWdBM) * ((M + kWdBN - 1) / kWdBN);
    const int sms = sm_count();
    dim3 grid((unsigned)(tiles < sms ? tiles : sms));   // persistent CTAs, one per SM
    static PerDeviceFlags configured[2];
    if (h16) {
        if (allow_dynamic_smem(w2a8_prefill_wide_kernel<true>, configured[1], (int)smem) != cudaSuccess) return W2A8_ERR_CUDA;
        w2a8_prefill_wide_kernel<true><<<grid, kWdThreads, smem, st>>>(map, p);
    } else {
        if (allow_dynamic_smem(w2a8_prefill_wide_kernel<false>, configured[0], (int)smem) != cudaSuccess) return W2A8_ERR_CUDA;
        w2a8_prefill_wide_kernel<false><<<grid, kWdThreads, smem, st>>>(map, p);
    }
    return cudaGetLastError() == cudaSuccess ? W2A8_OK : W2A8_ERR_CUDA;
}

}  // namespace w2a8
