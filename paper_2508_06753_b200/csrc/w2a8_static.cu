// w2a8_gemm_static: w2a8_gemm for callers that cannot hand over a
// workspace.  Its scratch (status word, split-K arrival counters, split-K
// partial outputs) lives in a fixed array that is part of the library image, so
// the call allocates nothing.  Contract and limits: include/w2a8.h.
#include <mutex>

#include "w2a8_common.cuh"

namespace w2a8 {
int gemm_dispatch(const int8_t *a, const float *a_scale, const uint32_t *packed, const void *w_scale,
                  void *y, int32_t *partials, int M, int N, int K, int group, const ShapeInfo &si,
                  void *workspace, void *stream, bool h16, bool y16, bool a16);
size_t gemm_header_bytes(int M, int N, int K, int group);
}  // namespace w2a8

// The scratch itself.  Every GPU that loads the library carries these bytes
// until the process exits.  In host code this name is only a handle for the
// runtime (it is not a device address): the address the kernels use is looked
// up per device below.
static __device__ __align__(256) unsigned char g_static_scratch[W2A8_STATIC_SCRATCH_BYTES];

namespace {
void *g_scratch_ptr[w2a8::kMaxDevices] = {};
std::mutex g_scratch_mutex;

// Device address of the scratch array on the current device; looked up once
// per device, with that device current.
int static_scratch(void **out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= w2a8::kMaxDevices) return W2A8_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_scratch_mutex);
    if (!g_scratch_ptr[dev]) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) return W2A8_ERR_CUDA;
        g_scratch_ptr[dev] = p;
    }
    *out = g_scratch_ptr[dev];
    return W2A8_OK;
}
}  // namespace

extern "C" int w2a8_gemm_static(const int8_t *a, const float *a_scale, const uint32_t *packed,
                                const float *w_scale, float *y, int M, int N, int K, int group,
                                void *stream) {
    using namespace w2a8;
    if (!a || !a_scale || !packed || !w_scale || !y) return W2A8_ERR_NULL;
    ShapeInfo si;
    if (!shape_ok(M, N, K, group, &si)) return W2A8_ERR_SHAPE;
    if (!aligned16(a) || !aligned16(packed) || !aligned16(y) || !aligned16(w_scale) ||
        (reinterpret_cast<uintptr_t>(a_scale) & 3u))
        return W2A8_ERR_ALIGN;
    // the problem's scratch must fit the fixed array: refuse, never truncate
    if (w2a8_workspace_bytes(M, N, K, group) > (size_t)W2A8_STATIC_SCRATCH_BYTES) return W2A8_ERR_WORKSPACE;
    if (int st = check_device()) return st;
    void *scratch = nullptr;
    if (int st = static_scratch(&scratch)) return st;
    // The array keeps whatever the previous call left.  The status word and the
    // arrival counters must start at zero; the partial outputs are fully written
    // before they are read, so they need no clearing.
    if (cudaMemsetAsync(scratch, 0, gemm_header_bytes(M, N, K, group), (cudaStream_t)stream) != cudaSuccess)
        return W2A8_ERR_CUDA;
    // same kernel choice and launch configuration as w2a8_gemm
    return gemm_dispatch(a, a_scale, packed, w_scale, y, nullptr, M, N, K, group, si, scratch, stream,
                         false, false, false);
}
