// C ABI of the W2A8 library, the off-line weight packer and the per-token
// activation quantiser.  Declarations and contracts: include/w2a8.h.
#include <math.h>
#include <stdlib.h>

#include "w2a8_common.cuh"
#include "w2a8_quant.cuh"

namespace w2a8 {

int launch_decode(const int8_t *a, const float *a_scale, const uint32_t *packed,
                  const void *w_scale, void *y, int32_t *partials, int M, int N, int K,
                  int group, const ShapeInfo &si, void *workspace, cudaStream_t st, bool h16, bool y16,
                  bool a16, int ldy);
size_t decode_workspace_bytes(int M, int N, int K, const ShapeInfo &si);
size_t decode_workspace_header_bytes(int M, int N, int K, const ShapeInfo &si);

bool gemv_supported(int M, int K, int group);
bool gemv_preferred(int M, int K, int group, int tiles, int count);
bool gemv_can_fuse(int M, int K, int group);
bool gemv_fuse_preferred(int M, int K, int group);
int launch_gemv(const int8_t *a, const float *a_scale, const void *x_bf16, int8_t *a_out, float *a_scale_out,
                int count, const uint32_t *const *packed, const float *const *w_scale, float *const *y,
                const int *N, const int *ldy, int M, int K, int group, cudaStream_t st);

bool prefill_supported(int M, int N, int K, int group);
bool prefill_preferred(int M, int N, int K, int group, bool can_split);
size_t prefill_workspace_bytes(int M, int N, int K, int group);
int prefill_ksplit(int M, int N, int K, int group);
bool prefill_uses_wide(int M, int N, int K, int group);
int launch_prefill(const int8_t *a, const float *a_scale, const uint32_t *packed, const void *w_scale,
                   void *y, int32_t *partials, int M, int N, int K, int group, int *status,
                   cudaStream_t st, bool h16, bool y16, int ldy);
int prefill_channel_split(int M, int N, int K, int group);
bool prefill_f16_supported(int M, int N, int K, int group);
size_t prefill_f16_scratch_bytes(int M, int K);
int launch_prefill_f16(const void *x_bf16, const float *a_scale, const uint32_t *packed, const float *w_scale,
                       float *y, int32_t *partials, int M, int N, int K, int group, int *status, cudaStream_t st,
                       int ldy);
int launch_a8_to_bf16(const int8_t *a, void *scratch, int M, int K, cudaStream_t st);

int env_int(const char *name, int dflt) {
    const char *v = getenv(name);
    return (v && *v) ? atoi(v) : dflt;
}

bool pdl_enabled() {
    static const bool on = env_int("W2A8_PDL", 1) != 0;
    return on;
}

int current_device() {
    int dev = -1;
    return cudaGetDevice(&dev) == cudaSuccess ? dev : -1;
}

namespace {
struct DeviceInfo {
    std::atomic<int> known{0};   // 0 = not looked up yet
    int status = 0, sms = 0;
};
DeviceInfo g_devices[kMaxDevices];

// Architecture check and SM count of the current device, looked up once per device.
const DeviceInfo *device_info() {
    const int dev = current_device();
    if (dev < 0 || dev >= kMaxDevices) return nullptr;
    DeviceInfo &d = g_devices[dev];
    if (!d.known.load(std::memory_order_acquire)) {
        int major = 0, sms = 0;
        if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
            return nullptr;
        // racing threads write the same values
        d.status = (major == 10) ? W2A8_OK : W2A8_ERR_ARCH;
        d.sms = sms > 0 ? sms : 1;
        d.known.store(1, std::memory_order_release);
    }
    return &d;
}
}  // namespace

int check_device() {
    const DeviceInfo *d = device_info();
    return d ? d->status : W2A8_ERR_CUDA;
}

int sm_count() {
    const DeviceInfo *d = device_info();
    return d ? d->sms : 148;
}

// ---- w2_pack ---------------------------------------------------------------------
// One thread builds one 32-bit word from 16 consecutive codes of a row.
__global__ void __launch_bounds__(256)
w2_pack_kernel(const uint8_t *__restrict__ codes, uint32_t *__restrict__ packed, int N, int K,
               int blocks, int tail_slices) {
    const int wpr = K / kWordK;
    const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (size_t)N * wpr) return;
    const int n = (int)(idx / wpr), wi = (int)(idx % wpr);
    const int b = wi / 16, r = wi % 16;
    const int R = (b == blocks - 1) ? tail_slices : 4;
    const int t = r / R, s = r % R;
    const int k0 = kBlockK * b + kSliceK * s + kWordK * t;
    const uint4 v = *reinterpret_cast<const uint4 *>(codes + (size_t)n * K + k0);
    // byte lane bb of v.{x,y,z,w} is code l = 4 j + bb (j = 0..3 for x..w);
    // it goes to bits [8 bb + 2 j, 8 bb + 2 j + 1]
    const uint32_t m = 0x03030303u;
    packed[idx] = (v.x & m) | ((v.y & m) << 2) | ((v.z & m) << 4) | ((v.w & m) << 6);
}

// ---- a8_quantize -----------------------------------------------------------------
// One CTA per token.  Abs-max over the row (bf16 magnitudes order like their bit
// patterns), then x * (1 / (amax / 127)), round to nearest even, clamp, store 8
// int8 per 16-byte vector.  Rows of up to kQuantRegThreads * 4 vectors (K <= 16384)
// stay in registers between the two steps; longer rows are re-read from L1/L2.
constexpr int kQuantThreads = 256;
constexpr int kQuantRegThreads = 512;

__global__ void __launch_bounds__(kQuantThreads)
a8_quantize_kernel(const uint16_t *__restrict__ x, int M, int K, int8_t *__restrict__ a,
                   float *__restrict__ a_scale) {
    pdl_launch_dependents();
    pdl_wait();   // x may come from the previous kernel of the stream
    const int m = blockIdx.x;
    const uint4 *xr = reinterpret_cast<const uint4 *>(x + (size_t)m * K);
    const int nvec = K / 8;
    uint32_t amax_bits = 0;
    for (int i = threadIdx.x; i < nvec; i += kQuantThreads) {
        const uint4 v = xr[i];
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            amax_bits = max(amax_bits, w[j] & 0x7FFFu);
            amax_bits = max(amax_bits, (w[j] >> 16) & 0x7FFFu);
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) amax_bits = max(amax_bits, __shfl_xor_sync(0xFFFFFFFFu, amax_bits, o));
    __shared__ uint32_t wmax[kQuantThreads / 32];
    if ((threadIdx.x & 31) == 0) wmax[threadIdx.x >> 5] = amax_bits;
    __syncthreads();
    amax_bits = 0;
#pragma unroll
    for (int w = 0; w < kQuantThreads / 32; ++w) amax_bits = max(amax_bits, wmax[w]);

    const float amax = bf16_bits_to_float(amax_bits);
    const float s = __fdiv_rn(amax, 127.0f);
    float inv = __fdiv_rn(1.0f, s);
    const bool dead = !(amax > 0.0f) || !(fabsf(inv) <= 3.402823466e38f);
    if (dead) inv = 0.0f;
    if (threadIdx.x == 0) a_scale[m] = dead ? 0.0f : s;

    uint2 *ar = reinterpret_cast<uint2 *>(a + (size_t)m * K);
    for (int i = threadIdx.x; i < nvec; i += kQuantThreads) {
        const uint4 v = xr[i];
        uint2 o;
        o.x = quant4(v.x, v.y, inv);
        o.y = quant4(v.z, v.w, inv);
        ar[i] = o;
    }
}

// VPT 16-byte vectors per thread, all loaded before the reduction starts.
template <int VPT>
__global__ void __launch_bounds__(kQuantRegThreads)
a8_quantize_reg_kernel(const uint16_t *__restrict__ x, int M, int K, int8_t *__restrict__ a,
                       float *__restrict__ a_scale) {
    pdl_launch_dependents();
    pdl_wait();
    const int m = blockIdx.x;
    const uint4 *xr = reinterpret_cast<const uint4 *>(x + (size_t)m * K);
    const int nvec = K / 8;
    uint4 v[VPT];
#pragma unroll
    for (int j = 0; j < VPT; ++j) {
        const int i = threadIdx.x + j * kQuantRegThreads;
        v[j] = i < nvec ? xr[i] : make_uint4(0u, 0u, 0u, 0u);
    }
    uint32_t amax_bits = 0;
#pragma unroll
    for (int j = 0; j < VPT; ++j) {
        const uint32_t w[4] = {v[j].x, v[j].y, v[j].z, v[j].w};
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            amax_bits = max(amax_bits, w[q] & 0x7FFFu);
            amax_bits = max(amax_bits, (w[q] >> 16) & 0x7FFFu);
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) amax_bits = max(amax_bits, __shfl_xor_sync(0xFFFFFFFFu, amax_bits, o));
    __shared__ uint32_t wmax[kQuantRegThreads / 32];
    if ((threadIdx.x & 31) == 0) wmax[threadIdx.x >> 5] = amax_bits;
    __syncthreads();
    amax_bits = wmax[threadIdx.x & (kQuantRegThreads / 32 - 1)];
#pragma unroll
    for (int o = kQuantRegThreads / 64; o > 0; o >>= 1)
        amax_bits = max(amax_bits, __shfl_xor_sync(0xFFFFFFFFu, amax_bits, o));

    float inv;
    const float s = quant_scale(amax_bits, &inv);
    if (threadIdx.x == 0) a_scale[m] = s;
    uint2 *ar = reinterpret_cast<uint2 *>(a + (size_t)m * K);
#pragma unroll
    for (int j = 0; j < VPT; ++j) {
        const int i = threadIdx.x + j * kQuantRegThreads;
        if (i < nvec) {
            uint2 o;
            o.x = quant4(v[j].x, v[j].y, inv);
            o.y = quant4(v[j].z, v[j].w, inv);
            ar[i] = o;
        }
    }
}


// ---- read-bandwidth probe ----------------------------------------------------------
// Plain 128-bit loads of a buffer, summed so that nothing can be dropped: what this device
// delivers to a kernel that only reads, measured with the library's own launch path.
__global__ void __launch_bounds__(512)
w2a8_read_probe_kernel(const uint4 *__restrict__ src, size_t nvec, unsigned *__restrict__ out) {
    unsigned acc = 0;
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    // four independent loads in flight per thread and trip
    for (; i + 3 * stride < nvec; i += 4 * stride) {
        const uint4 v0 = __ldcs(src + i), v1 = __ldcs(src + i + stride);
        const uint4 v2 = __ldcs(src + i + 2 * stride), v3 = __ldcs(src + i + 3 * stride);
        acc += (v0.x ^ v0.y ^ v0.z ^ v0.w) + (v1.x ^ v1.y ^ v1.z ^ v1.w) + (v2.x ^ v2.y ^ v2.z ^ v2.w) +
               (v3.x ^ v3.y ^ v3.z ^ v3.w);
    }
    for (; i < nvec; i += stride) {
        const uint4 v = __ldcs(src + i);
        acc += v.x ^ v.y ^ v.z ^ v.w;
    }
    if (acc == 0x9E3779B9u) atomicAdd(out, acc);     // practically never: keeps the loads alive
}

}  // namespace w2a8

// ====================================================================== C ABI ==
using namespace w2a8;

extern "C" {

int w2a8_version(void) { return 100; }

const char *w2a8_status_string(int status) {
    switch (status) {
        case W2A8_OK: return "ok";
        case W2A8_ERR_NULL: return "null pointer argument";
        case W2A8_ERR_SHAPE: return "unsupported shape (need K % 64 == 0, N % 16 == 0, M >= 1, "
                                    "group in {64, 128, multiple of 256, K} dividing K)";
        case W2A8_ERR_ALIGN: return "pointer not 16-byte aligned";
        case W2A8_ERR_WORKSPACE: return "workspace missing or too small";
        case W2A8_ERR_CUDA: return "CUDA runtime or launch error";
        case W2A8_ERR_ARCH: return "device is not sm_100";
        case W2A8_ERR_TIMEOUT: return "a bounded device-side wait gave up";
        default: return "unknown status";
    }
}

size_t w2_packed_bytes(int N, int K) {
    if (!shape_ok(1, N, K, 64, nullptr)) return 0;
    return (size_t)N * K / 4;
}

int w2_pack(const uint8_t *codes, int N, int K, uint32_t *packed, void *stream) {
    if (!codes || !packed) return W2A8_ERR_NULL;
    ShapeInfo si;
    if (!shape_ok(1, N, K, 64, &si)) return W2A8_ERR_SHAPE;
    if (!aligned16(codes) || !aligned16(packed)) return W2A8_ERR_ALIGN;
    if (int st = check_device()) return st;
    const size_t words = (size_t)N * si.words_per_row;
    const unsigned grid = (unsigned)((words + 255) / 256);
    cudaError_t e = launch_kernel(w2_pack_kernel, dim3(grid), dim3(256), 0, (cudaStream_t)stream,
                                  false, codes, packed, N, K, si.blocks, si.tail_slices);
    return e == cudaSuccess ? W2A8_OK : W2A8_ERR_CUDA;
}

int a8_quantize(const void *x_bf16, int M, int K, int8_t *a, float *a_scale, void *stream) {
    if (!x_bf16 || !a || !a_scale) return W2A8_ERR_NULL;
    if (M < 1 || K < 64 || K % 64 != 0) return W2A8_ERR_SHAPE;
    if (!aligned16(x_bf16) || !aligned16(a) || (reinterpret_cast<uintptr_t>(a_scale) & 3u))
        return W2A8_ERR_ALIGN;
    if (int st = check_device()) return st;
    const uint16_t *x = reinterpret_cast<const uint16_t *>(x_bf16);
    cudaStream_t st = (cudaStream_t)stream;
    const int vpt = (K / 8 + kQuantRegThreads - 1) / kQuantRegThreads;
    cudaError_t e;
    if (vpt <= 1)
        e = launch_kernel(a8_quantize_reg_kernel<1>, dim3(M), dim3(kQuantRegThreads), 0, st,
                          pdl_enabled(), x, M, K, a, a_scale);
    else if (vpt <= 2)
        e = launch_kernel(a8_quantize_reg_kernel<2>, dim3(M), dim3(kQuantRegThreads), 0, st,
                          pdl_enabled(), x, M, K, a, a_scale);
    else if (vpt <= 4)
        e = launch_kernel(a8_quantize_reg_kernel<4>, dim3(M), dim3(kQuantRegThreads), 0, st,
                          pdl_enabled(), x, M, K, a, a_scale);
    else
        e = launch_kernel(a8_quantize_kernel, dim3(M), dim3(kQuantThreads), 0, st,
                          pdl_enabled(), x, M, K, a, a_scale);
    return e == cudaSuccess ? W2A8_OK : W2A8_ERR_CUDA;
}

static bool takes_tensor_core_kernel(int M, int N, int K, int group);
static bool takes_tensor_core_kernel_ex(int M, int N, int K, int group, bool can_split);
static int tensor_core_channels(int M, int N, int K, int group);

static bool tensor_core_kind_is_16(int M, int N, int K, int group);

// Workspace of the kernels themselves (status word, split-K counters and partial outputs).
static size_t kernel_workspace_bytes(int M, int N, int K, int group) {
    ShapeInfo si;
    if (!shape_ok(M, N, K, group, &si)) return 0;
    size_t need = decode_workspace_bytes(M, N, K, si);
    if (takes_tensor_core_kernel(M, N, K, group)) {
        // partial outputs of a K split of the int8 tensor-core kernel
        const size_t split = prefill_workspace_bytes(M, N, K, group);
        if (split > need) need = split;
        // the last channel tiles may be given to the streaming kernel, with a plan of its own
        const int n_tc = tensor_core_channels(M, N, K, group);
        ShapeInfo rest;
        if (n_tc < N && shape_ok(M, N - n_tc, K, group, &rest)) {
            const size_t r = decode_workspace_bytes(M, N - n_tc, K, rest);
            if (r > need) need = r;
        }
    }
    return (need + 255) / 256 * 256;
}

size_t w2a8_workspace_bytes(int M, int N, int K, int group) {
    size_t need = kernel_workspace_bytes(M, N, K, group);
    if (need == 0) return 0;
    // the 16-bit tensor-core kernel reads the int8 activations from a bf16 copy kept behind that
    if (takes_tensor_core_kernel(M, N, K, group) && tensor_core_kind_is_16(M, N, K, group))
        need += prefill_f16_scratch_bytes(M, K);
    return need;
}

int w2a8_workspace_init(void *workspace, size_t workspace_bytes, void *stream) {
    if (!workspace) return W2A8_ERR_NULL;
    if (cudaMemsetAsync(workspace, 0, workspace_bytes, (cudaStream_t)stream) != cudaSuccess)
        return W2A8_ERR_CUDA;
    return W2A8_OK;
}

int w2a8_workspace_status(const void *workspace, void *stream) {
    if (!workspace) return W2A8_ERR_NULL;
    int status = 0;
    if (cudaMemcpyAsync(&status, workspace, sizeof(int), cudaMemcpyDeviceToHost,
                        (cudaStream_t)stream) != cudaSuccess)
        return W2A8_ERR_CUDA;
    if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return W2A8_ERR_CUDA;
    return status;
}

// W2A8_PREFILL: 0 = never the tensor-core kernel, 2 = whenever it supports the shape, else
// (default) when it supports the shape and is expected to be the faster one.
static bool takes_tensor_core_kernel_ex(int M, int N, int K, int group, bool can_split) {
    if (!prefill_supported(M, N, K, group)) return false;
    const int mode = env_int("W2A8_PREFILL", 1);
    if (mode == 0) return false;
    if (mode == 2) return true;
    return prefill_preferred(M, N, K, group, can_split);
}
// int8 activations: the int8 kernel can split K for problems with few output tiles, the 16-bit one cannot
static bool takes_tensor_core_kernel(int M, int N, int K, int group) {
    return takes_tensor_core_kernel_ex(M, N, K, group, !tensor_core_kind_is_16(M, N, K, group));
}

// Channels the tensor-core kernel takes (the rest, if any, goes to the streaming kernel in a
// second launch): all of them with W2A8_PREFILL=2 or W2A8_PF_SPLIT=0.
static int tensor_core_channels(int M, int N, int K, int group) {
    if (env_int("W2A8_PREFILL", 1) == 2 || env_int("W2A8_PF_SPLIT", 1) == 0) return N;
    return prefill_channel_split(M, N, K, group);
}

int w2a8_read_probe(const void *buffer, size_t bytes, unsigned *sink, void *stream) {
    if (!buffer || !sink) return W2A8_ERR_NULL;
    if (!aligned16(buffer) || bytes < 16) return W2A8_ERR_ALIGN;
    if (int st = check_device()) return st;
    const int ctas = sm_count() * 4;
    cudaError_t e = launch_kernel(w2a8_read_probe_kernel, dim3(ctas), dim3(512), 0, (cudaStream_t)stream, false,
                                  reinterpret_cast<const uint4 *>(buffer), bytes / 16, sink);
    return e == cudaSuccess ? W2A8_OK : W2A8_ERR_CUDA;
}

// Which tensor-core kernel serves the int8 entries for a shape the tensor-core path takes: the int8
// kernel (kind::i8, int32 accumulators, conversion in the drain) or the 16-bit one (kind::f16 on a
// bf16 copy of the activations, fp32 accumulators holding the same exact integers).
// W2A8_TC_KIND=8 / 16 forces one.
static bool tensor_core_kind_is_16(int M, int N, int K, int group) {
    if (!prefill_f16_supported(M, N, K, group)) return false;
    if ((long long)254 * group >= (1ll << 24)) return false;      // fp32 must hold the group sums exactly
    const int forced = env_int("W2A8_TC_KIND", 0);
    if (forced == 8) return false;
    if (forced == 16) return true;
    return false;
}

int w2a8_tensor_core_kind(int M, int N, int K, int group) {
    ShapeInfo si;
    if (!shape_ok(M, N, K, group, &si)) return W2A8_ERR_SHAPE;
    if (!takes_tensor_core_kernel(M, N, K, group)) return 0;
    return tensor_core_kind_is_16(M, N, K, group) ? 16 : 8;
}

int w2a8_kernel_for(int M, int N, int K, int group) {
    ShapeInfo si;
    if (!shape_ok(M, N, K, group, &si)) return W2A8_ERR_SHAPE;
    return takes_tensor_core_kernel(M, N, K, group) ? 1 : 0;
}

int w2a8_tensor_core_channels(int M, int N, int K, int group) {
    ShapeInfo si;
    if (!shape_ok(M, N, K, group, &si)) return W2A8_ERR_SHAPE;
    return takes_tensor_core_kernel(M, N, K, group) ? tensor_core_channels(M, N, K, group) : 0;
}

int w2a8_tensor_core_ksplit(int M, int N, int K, int group) {
    ShapeInfo si;
    if (!shape_ok(M, N, K, group, &si)) return W2A8_ERR_SHAPE;
    if (!takes_tensor_core_kernel(M, N, K, group)) return 0;
    if (tensor_core_kind_is_16(M, N, K, group)) return 1;
    return prefill_ksplit(M, N, K, group);
}

int w2a8_tensor_core_tile_tokens(int M, int N, int K, int group) {
    ShapeInfo si;
    if (!shape_ok(M, N, K, group, &si)) return W2A8_ERR_SHAPE;
    if (!takes_tensor_core_kernel(M, N, K, group)) return 0;
    if (tensor_core_kind_is_16(M, N, K, group)) return 128;
    return prefill_uses_wide(M, N, K, group) ? 256 : 128;
}

}  // extern "C"

namespace w2a8 {
// Bytes at the start of a workspace that have to be zero when a GEMM call starts (status word and
// split-K arrival counters of whichever kernels serve the shape).  The kernels leave them zero.
size_t gemm_header_bytes(int M, int N, int K, int group) {
    ShapeInfo si;
    if (!shape_ok(M, N, K, group, &si)) return 0;
    size_t need = decode_workspace_header_bytes(M, N, K, si);
    if (takes_tensor_core_kernel(M, N, K, group)) {
        const int n_tc = tensor_core_channels(M, N, K, group);
        ShapeInfo rest;
        if (n_tc < N && shape_ok(M, N - n_tc, K, group, &rest)) {
            const size_t r = decode_workspace_header_bytes(M, N - n_tc, K, rest);
            if (r > need) need = r;
        }
    }
    return need;
}

// Pick the kernel(s) for a checked problem and enqueue them.  Many tokens: tensor-core path
// (tcgen05); few tokens, shapes it does not tile, or too few output tiles to fill the GPU:
// streaming path.  h16: w_scale holds binary16 values; y16 (with h16): y holds bf16 values;
// a16: a holds bf16 activations.
int gemm_dispatch(const int8_t *a, const float *a_scale, const uint32_t *packed, const void *w_scale,
                  void *y, int32_t *partials, int M, int N, int K, int group, const ShapeInfo &si,
                  void *workspace, void *stream, bool h16, bool y16, bool a16) {
    const bool takes = a16 ? takes_tensor_core_kernel_ex(M, N, K, group, false) : takes_tensor_core_kernel(M, N, K, group);
    const bool tc16 = !h16 && takes && prefill_f16_supported(M, N, K, group) &&
                      (a16 || tensor_core_kind_is_16(M, N, K, group));
    if (tc16 || (!a16 && takes)) {
        // The tensor-core kernel takes the first n_tc channels; when a last round of a few tiles
        // would cost a whole round, the remaining channel tiles go to the streaming kernel in a
        // second launch (rows of the packed matrix and of the scales are independent; both kernels
        // write their own columns of y).  The parity export is never split.
        const int n_tc = partials ? N : tensor_core_channels(M, N, K, group);
        int st;
        if (tc16) {
            // 16-bit operands: the caller's bf16 activations as they are (a16), or a bf16 copy of
            // the int8 activations kept behind the kernels' own workspace
            const void *x = a;
            if (!a16) {
                void *copy = reinterpret_cast<char *>(workspace) + kernel_workspace_bytes(M, N, K, group);
                if (int e = launch_a8_to_bf16(a, copy, M, K, (cudaStream_t)stream)) return e;
                x = copy;
            }
            st = launch_prefill_f16(x, a16 ? nullptr : a_scale, packed, reinterpret_cast<const float *>(w_scale),
                                    reinterpret_cast<float *>(y), partials, M, n_tc, K, group,
                                    reinterpret_cast<int *>(workspace), (cudaStream_t)stream, N);
        } else {
            st = launch_prefill(a, a_scale, packed, w_scale, y, partials, M, n_tc, K, group,
                                reinterpret_cast<int *>(workspace), (cudaStream_t)stream, h16, y16, N);
        }
        ShapeInfo rest;
        if (st != W2A8_OK || n_tc >= N || !shape_ok(M, N - n_tc, K, group, &rest)) return st;
        const size_t scale_bytes = h16 ? 2 : 4, y_bytes = (h16 && y16) ? 2 : 4;
        return launch_decode(a, a_scale, packed + (size_t)n_tc * si.words_per_row,
                             reinterpret_cast<const char *>(w_scale) + (size_t)n_tc * si.G * scale_bytes,
                             reinterpret_cast<char *>(y) + (size_t)n_tc * y_bytes, nullptr, M, N - n_tc, K,
                             group, rest, workspace, (cudaStream_t)stream, h16, y16, a16, N);
    }
    return launch_decode(a, a_scale, packed, w_scale, y, partials, M, N, K, group, si, workspace,
                         (cudaStream_t)stream, h16, y16, a16, N);
}
}  // namespace w2a8

extern "C" {

static int gemm_common(const int8_t *a, const float *a_scale, const uint32_t *packed,
                       const void *w_scale, void *y, int32_t *partials, int M, int N, int K,
                       int group, void *workspace, size_t workspace_bytes, void *stream,
                       bool h16 = false, bool y16 = false, bool a16 = false) {
    ShapeInfo si;
    if (!shape_ok(M, N, K, group, &si)) return W2A8_ERR_SHAPE;
    if (!aligned16(a) || !aligned16(packed) || (y && !aligned16(y)) ||
        (w_scale && !aligned16(w_scale)) || (partials && !aligned16(partials)) ||
        (a_scale && (reinterpret_cast<uintptr_t>(a_scale) & 3u)))
        return W2A8_ERR_ALIGN;
    const size_t need = w2a8_workspace_bytes(M, N, K, group);
    if (!workspace || workspace_bytes < need || !aligned16(workspace)) return W2A8_ERR_WORKSPACE;
    if (int st = check_device()) return st;
    return gemm_dispatch(a, a_scale, packed, w_scale, y, partials, M, N, K, group, si, workspace, stream,
                         h16, y16, a16);
}

int w2a16_gemm(const void *x_bf16, const uint32_t *packed, const float *w_scale, float *y, int M, int N,
               int K, int group, void *workspace, size_t workspace_bytes, void *stream) {
    if (!x_bf16 || !packed || !w_scale || !y) return W2A8_ERR_NULL;
    return gemm_common(reinterpret_cast<const int8_t *>(x_bf16), nullptr, packed, w_scale, y, nullptr, M, N, K,
                       group, workspace, workspace_bytes, stream, false, false, true);
}

int w2a8_gemm_h16(const int8_t *a, const float *a_scale, const uint32_t *packed,
                  const uint16_t *w_scale_h, void *y, int y_is_bf16, int M, int N, int K, int group,
                  void *workspace, size_t workspace_bytes, void *stream) {
    if (!a || !a_scale || !packed || !w_scale_h || !y) return W2A8_ERR_NULL;
    return gemm_common(a, a_scale, packed, w_scale_h, y, nullptr, M, N, K, group, workspace,
                       workspace_bytes, stream, true, y_is_bf16 != 0);
}

int w2a8_gemm(const int8_t *a, const float *a_scale, const uint32_t *packed, const float *w_scale,
              float *y, int M, int N, int K, int group, void *workspace, size_t workspace_bytes,
              void *stream) {
    if (!a || !a_scale || !packed || !w_scale || !y) return W2A8_ERR_NULL;
    return gemm_common(a, a_scale, packed, w_scale, y, nullptr, M, N, K, group, workspace,
                       workspace_bytes, stream);
}

int w2a8_gemm_partials(const int8_t *a, const uint32_t *packed, int32_t *partials, int M, int N,
                       int K, int group, void *workspace, size_t workspace_bytes, void *stream) {
    if (!a || !packed || !partials) return W2A8_ERR_NULL;
    return gemm_common(a, nullptr, packed, nullptr, nullptr, partials, M, N, K, group, workspace,
                       workspace_bytes, stream);
}

static inline size_t up256(size_t v) { return (v + 255) / 256 * 256; }

// ---- matrices that share their activations --------------------------------------------------
constexpr int kMaxGroup = 4;

// bit 0: the group runs as one launch of the persistent kernel; bit 1: that launch quantises the
// activations itself.  fuse: W2A8_FUSE_AUTO / _OFF / _ON.  Negative: error.
static int grouped_plan(int count, const int *N, int M, int K, int group, int fuse, bool have_x) {
    if (count < 1 || count > kMaxGroup || !N) return W2A8_ERR_SHAPE;
    int tiles = 0;
    for (int i = 0; i < count; ++i) {
        if (!shape_ok(M, N[i], K, group, nullptr)) return W2A8_ERR_SHAPE;
        tiles += N[i] / 16;
    }
    int plan = 0;
    if (have_x && fuse != W2A8_FUSE_OFF && gemv_can_fuse(M, K, group) &&
        (fuse == W2A8_FUSE_ON || gemv_fuse_preferred(M, K, group)))
        plan = 3;
    else if (gemv_preferred(M, K, group, tiles, count))
        plan = 1;
    return plan;
}

size_t w2a8_grouped_workspace_bytes(int count, const int *N, int M, int K, int group) {
    if (count < 1 || count > kMaxGroup || !N) return 0;
    size_t need = 0;
    for (int i = 0; i < count; ++i) {
        const size_t b = w2a8_workspace_bytes(M, N[i], K, group);
        if (b == 0) return 0;
        if (b > need) need = b;
    }
    return need;
}

int w2a8_grouped_plan(int count, const int *N, int M, int K, int group, int fuse) {
    return grouped_plan(count, N, M, K, group, fuse, true);
}

static int grouped_common(const void *x_bf16, const int8_t *a_in, const float *a_scale_in, int8_t *a, float *a_scale,
                          int count, const uint32_t *const *packed, const float *const *w_scale, float *const *y,
                          const int *N, int M, int K, int group, int fuse, void *workspace, size_t workspace_bytes,
                          void *stream) {
    if (!packed || !w_scale || !y || !N) return W2A8_ERR_NULL;
    const int plan = grouped_plan(count, N, M, K, group, fuse, x_bf16 != nullptr);
    if (plan < 0) return plan;
    for (int i = 0; i < count; ++i) {
        if (!packed[i] || !w_scale[i] || !y[i]) return W2A8_ERR_NULL;
        if (!aligned16(packed[i]) || !aligned16(w_scale[i]) || !aligned16(y[i])) return W2A8_ERR_ALIGN;
    }
    if (x_bf16 && !aligned16(x_bf16)) return W2A8_ERR_ALIGN;
    if ((a && !aligned16(a)) || (a_in && !aligned16(a_in))) return W2A8_ERR_ALIGN;
    if ((a_scale && (reinterpret_cast<uintptr_t>(a_scale) & 3u)) ||
        (a_scale_in && (reinterpret_cast<uintptr_t>(a_scale_in) & 3u)))
        return W2A8_ERR_ALIGN;
    const size_t need = w2a8_grouped_workspace_bytes(count, N, M, K, group);
    if (!workspace || workspace_bytes < need || !aligned16(workspace)) return W2A8_ERR_WORKSPACE;
    if (int st = check_device()) return st;
    if (plan == 3)          // one launch: quantise and multiply
        return launch_gemv(nullptr, nullptr, x_bf16, a, a_scale, count, packed, w_scale, y, N, N, M, K, group,
                           (cudaStream_t)stream);
    if (x_bf16) {
        if (!a || !a_scale) return W2A8_ERR_NULL;    // the quantiser needs somewhere to write
        if (int st = a8_quantize(x_bf16, M, K, a, a_scale, stream)) return st;
        a_in = a;
        a_scale_in = a_scale;
    }
    if (plan == 1)          // one launch over all matrices
        return launch_gemv(a_in, a_scale_in, nullptr, nullptr, nullptr, count, packed, w_scale, y, N, N, M, K, group,
                           (cudaStream_t)stream);
    for (int i = 0; i < count; ++i)     // one launch per matrix (same stream, so one workspace serves all)
        if (int st = w2a8_gemm(a_in, a_scale_in, packed[i], w_scale[i], y[i], M, N[i], K, group, workspace,
                               workspace_bytes, stream))
            return st;
    return W2A8_OK;
}

int w2a8_gemm_grouped(const int8_t *a, const float *a_scale, int count, const uint32_t *const *packed,
                      const float *const *w_scale, float *const *y, const int *N, int M, int K, int group,
                      void *workspace, size_t workspace_bytes, void *stream) {
    if (!a || !a_scale) return W2A8_ERR_NULL;
    return grouped_common(nullptr, a, a_scale, nullptr, nullptr, count, packed, w_scale, y, N, M, K, group,
                          W2A8_FUSE_OFF, workspace, workspace_bytes, stream);
}

int w2a8_linear_grouped(const void *x_bf16, int8_t *a, float *a_scale, int count, const uint32_t *const *packed,
                        const float *const *w_scale, float *const *y, const int *N, int M, int K, int group,
                        int fuse, void *workspace, size_t workspace_bytes, void *stream) {
    if (!x_bf16) return W2A8_ERR_NULL;
    if (fuse != W2A8_FUSE_AUTO && fuse != W2A8_FUSE_OFF && fuse != W2A8_FUSE_ON) return W2A8_ERR_SHAPE;
    return grouped_common(x_bf16, nullptr, nullptr, a, a_scale, count, packed, w_scale, y, N, M, K, group, fuse,
                          workspace, workspace_bytes, stream);
}

int w2a8_linear(const void *x_bf16, int8_t *a, float *a_scale, const uint32_t *packed,
                const float *w_scale, float *y, int M, int N, int K, int group, void *workspace,
                size_t workspace_bytes, void *stream) {
    if (!x_bf16 || !a || !a_scale || !packed || !w_scale || !y) return W2A8_ERR_NULL;
    return w2a8_linear_grouped(x_bf16, a, a_scale, 1, &packed, &w_scale, &y, &N, M, K, group, W2A8_FUSE_AUTO,
                               workspace, workspace_bytes, stream);
}

size_t w2a8_linear_host_workspace_bytes(int M, int N, int K, int group) {
    const size_t g = w2a8_workspace_bytes(M, N, K, group);
    if (g == 0) return 0;
    return up256(g) + up256((size_t)M * K * 2) + up256((size_t)M * K) + up256((size_t)M * 4) +
           up256((size_t)M * N * 4);
}

constexpr int kDecodeMaxZeroCopyTokens = 32;

// Device-side address of a page-locked, mapped host allocation; nullptr for pageable memory
// (or anything else the device cannot address directly).
static void *mapped_device_pointer(const void *host) {
    cudaPointerAttributes attr;
    if (cudaPointerGetAttributes(&attr, host) != cudaSuccess) {
        cudaGetLastError();   // pageable memory is reported as an error by older drivers
        return nullptr;
    }
    if (attr.type != cudaMemoryTypeHost || attr.devicePointer == nullptr) return nullptr;
    return attr.devicePointer;
}

int w2a8_linear_host(const void *x_host, int M, int K, const uint32_t *packed,
                     const float *w_scale, int N, int group, float *y_host, void *workspace,
                     size_t workspace_bytes, void *stream) {
    if (!x_host || !packed || !w_scale || !y_host) return W2A8_ERR_NULL;
    const size_t need = w2a8_linear_host_workspace_bytes(M, N, K, group);
    if (need == 0) return W2A8_ERR_SHAPE;
    if (!workspace || workspace_bytes < need || !aligned16(workspace)) return W2A8_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    char *p = reinterpret_cast<char *>(workspace);
    const size_t gemm_ws = w2a8_workspace_bytes(M, N, K, group);
    void *ws = p;                     p += up256(gemm_ws);
    void *x_dev = p;                  p += up256((size_t)M * K * 2);
    int8_t *a = (int8_t *)p;          p += up256((size_t)M * K);
    float *a_scale = (float *)p;      p += up256((size_t)M * 4);
    float *y_dev = (float *)p;
    // Few tokens: the transfers are a few KB, and a copy-engine operation costs more in launch
    // latency than it moves.  If both host buffers are page-locked and mapped (so the device can
    // address them), the quantiser reads x over the bus itself and the GEMM stores y straight to
    // the host buffer.  Otherwise, and for many tokens, staged copies.
    static const int zero_copy_max = env_int("W2A8_ZEROCOPY_MAX", kDecodeMaxZeroCopyTokens);
    const void *x_map = (M <= zero_copy_max) ? mapped_device_pointer(x_host) : nullptr;
    void *y_map = (M <= zero_copy_max) ? mapped_device_pointer(y_host) : nullptr;
    if (x_map && y_map && aligned16(x_map) && aligned16(y_map)) {
        if (int s = a8_quantize(x_map, M, K, a, a_scale, stream)) return s;
        return w2a8_gemm(a, a_scale, packed, w_scale, reinterpret_cast<float *>(y_map), M, N, K, group, ws,
                         gemm_ws, stream);
    }
    if (cudaMemcpyAsync(x_dev, x_host, (size_t)M * K * 2, cudaMemcpyHostToDevice, st) != cudaSuccess)
        return W2A8_ERR_CUDA;
    if (int s = a8_quantize(x_dev, M, K, a, a_scale, stream)) return s;
    if (int s = w2a8_gemm(a, a_scale, packed, w_scale, y_dev, M, N, K, group, ws, gemm_ws, stream))
        return s;
    if (cudaMemcpyAsync(y_host, y_dev, (size_t)M * N * 4, cudaMemcpyDeviceToHost, st) != cudaSuccess)
        return W2A8_ERR_CUDA;
    return W2A8_OK;
}

size_t w2a8_linear_grouped_host_workspace_bytes(int count, const int *N, int M, int K, int group) {
    const size_t g = w2a8_grouped_workspace_bytes(count, N, M, K, group);
    if (g == 0) return 0;
    size_t need = up256(g) + up256((size_t)M * K * 2) + up256((size_t)M * K) + up256((size_t)M * 4);
    for (int i = 0; i < count; ++i) need += up256((size_t)M * N[i] * 4);
    return need;
}

int w2a8_linear_grouped_host(const void *x_host, int M, int K, int count, const uint32_t *const *packed,
                             const float *const *w_scale, const int *N, int group, float *const *y_host,
                             void *workspace, size_t workspace_bytes, void *stream) {
    if (!x_host || !packed || !w_scale || !N || !y_host) return W2A8_ERR_NULL;
    const size_t need = w2a8_linear_grouped_host_workspace_bytes(count, N, M, K, group);
    if (need == 0) return W2A8_ERR_SHAPE;
    if (!workspace || workspace_bytes < need || !aligned16(workspace)) return W2A8_ERR_WORKSPACE;
    for (int i = 0; i < count; ++i)
        if (!y_host[i]) return W2A8_ERR_NULL;
    cudaStream_t st = (cudaStream_t)stream;
    char *p = reinterpret_cast<char *>(workspace);
    const size_t gemm_ws = w2a8_grouped_workspace_bytes(count, N, M, K, group);
    void *ws = p;                     p += up256(gemm_ws);
    void *x_dev = p;                  p += up256((size_t)M * K * 2);
    int8_t *a = (int8_t *)p;          p += up256((size_t)M * K);
    float *a_scale = (float *)p;      p += up256((size_t)M * 4);
    float *y_dev[kMaxGroup];
    for (int i = 0; i < count; ++i) { y_dev[i] = (float *)p; p += up256((size_t)M * N[i] * 4); }
    // As in w2a8_linear_host: with few tokens and page-locked, mapped buffers the quantiser reads x
    // over the bus itself -- once for the whole group -- and the GEMMs store straight to the host
    // buffers; otherwise staged copies.  The quantiser always runs as a launch of its own here:
    // inside the GEMM launch every CTA would fetch x over the bus.
    static const int zero_copy_max = env_int("W2A8_ZEROCOPY_MAX", kDecodeMaxZeroCopyTokens);
    const void *x_map = (M <= zero_copy_max) ? mapped_device_pointer(x_host) : nullptr;
    float *y_map[kMaxGroup];
    bool direct = x_map != nullptr && aligned16(x_map);
    for (int i = 0; i < count && direct; ++i) {
        y_map[i] = reinterpret_cast<float *>(mapped_device_pointer(y_host[i]));
        direct = y_map[i] != nullptr && aligned16(y_map[i]);
    }
    if (direct) {
        if (int s = a8_quantize(x_map, M, K, a, a_scale, stream)) return s;
        return w2a8_gemm_grouped(a, a_scale, count, packed, w_scale, y_map, N, M, K, group, ws, gemm_ws, stream);
    }
    if (cudaMemcpyAsync(x_dev, x_host, (size_t)M * K * 2, cudaMemcpyHostToDevice, st) != cudaSuccess)
        return W2A8_ERR_CUDA;
    if (int s = a8_quantize(x_dev, M, K, a, a_scale, stream)) return s;
    if (int s = w2a8_gemm_grouped(a, a_scale, count, packed, w_scale, y_dev, N, M, K, group, ws, gemm_ws, stream))
        return s;
    for (int i = 0; i < count; ++i)
        if (cudaMemcpyAsync(y_host[i], y_dev[i], (size_t)M * N[i] * 4, cudaMemcpyDeviceToHost, st) != cudaSuccess)
            return W2A8_ERR_CUDA;
    return W2A8_OK;
}

}  // extern "C"
