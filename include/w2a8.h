/*
 * w2a8.h -- C ABI of the B200 (sm_100a) W2A8 library: 2-bit weights x int8
 * activations -> int32 per-group sums -> fp32 outputs.
 *
 * Naming (GEMM convention, not the paper's): M = tokens, N = output channels,
 * K = contraction length, group = number of consecutive k that share one fp32
 * weight scale.  (The paper calls the weights A [its M x K], the activations
 * B [its N x K] and the result C.)
 *
 * General rules for every entry point
 *   - Returns a w2a8_status (0 = OK, negative = error).  Never throws, never
 *     exits, never allocates or frees device memory.
 *   - Unless a parameter says HOST, every pointer is a DEVICE pointer owned by
 *     the caller, 16-byte aligned, valid until the enqueued work has run.
 *     Nothing is retained after the call returns.
 *   - `stream` is a cudaStream_t passed as void* (NULL = default stream).  All
 *     work is enqueued on it; the calls do not synchronise.
 *   - Argument errors are detected on the host before anything is launched.
 *     Launch failures are reported as W2A8_ERR_CUDA.
 *   - Kernels are launched with programmatic dependent launch: they may start
 *     while the previous kernel of the stream drains, but touch nothing except
 *     the frozen weights and scales until that kernel has completed.  Set the
 *     environment variable W2A8_PDL=0 to launch them plainly.
 *
 * Shape rules: K % 64 == 0, N % 16 == 0, M >= 1, K % group == 0 and group is
 * 64, 128, a multiple of 256, or K itself (one scale per output channel).
 */
#ifndef W2A8_H_
#define W2A8_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    W2A8_OK = 0,
    W2A8_ERR_NULL = -1,      /* a required pointer is NULL */
    W2A8_ERR_SHAPE = -2,     /* M, N, K or group violates the shape rules */
    W2A8_ERR_ALIGN = -3,     /* a pointer is not 16-byte aligned */
    W2A8_ERR_WORKSPACE = -4, /* workspace missing or too small */
    W2A8_ERR_CUDA = -5,      /* a CUDA runtime call or launch failed */
    W2A8_ERR_ARCH = -6,      /* the current device is not sm_100 */
    W2A8_ERR_TIMEOUT = -7    /* a bounded device-side wait gave up (see w2a8_workspace_status) */
} w2a8_status;

/* Library version: major * 10000 + minor * 100 + patch. */
int w2a8_version(void);

/* Static, human-readable text for a status code. */
const char *w2a8_status_string(int status);

/*
 * Size in bytes of the packed form of an N x K code matrix: N * K / 4
 * (16 two-bit codes per 32-bit word; Sec. II-B: a 256-bit load carries 128
 * codes).  Returns 0 for shapes that violate the shape rules.
 */
size_t w2_packed_bytes(int N, int K);

/*
 * w2_pack -- re-lay frozen 2-bit codes into the streaming format, once, ahead
 * of time (Sec. II-B / II-C: weights are frozen at inference, so they are
 * packed off-line into a layout from which one shift+mask yields int8 lanes in
 * dot-product order).
 *   codes  [N][K] uint8, row-major, one code per byte; only the low two bits
 *          are used (value = code - 2, i.e. {0,1,2,3} -> {-2,-1,0,1}).
 *   packed [N][K/16] uint32, fully overwritten.  Layout ("W2P"):
 *          a row is cut into blocks of up to four 64-k slices; inside block b
 *          with R slices (R = 4 except possibly the last), the word holding
 *          k = 256 b + 64 s + 16 t + l (s < R, t < 4, l < 16) is word
 *          16 b + t R + s of the row, and code l sits at bit
 *          8 (l mod 4) + 2 (l div 4) of that word.
 */
int w2_pack(const uint8_t *codes, int N, int K, uint32_t *packed, void *stream);

/*
 * a8_quantize -- per-token symmetric abs-max quantisation of bf16 activations
 * to int8 (Sec. II-D: multiply by the inverse of the scale, convert to int8;
 * the scale comes from the abs-max of the quantisation granule, here one
 * token).  For token m, all in fp32 with round-to-nearest-even operations:
 *   amax = max_k |x[m][k]|, a_scale[m] = amax / 127, inv = 1 / a_scale[m],
 *   a[m][k] = clamp(rne(x[m][k] * inv), -127, 127).
 * A row with amax == 0, or with a non-finite inv, gives a[m][:] = 0 and
 * a_scale[m] = 0.  NaN / Inf inputs are outside the contract.
 *   x_bf16  [M][K] bf16 bit patterns, row-major
 *   a       [M][K] int8, fully overwritten
 *   a_scale [M] fp32, fully overwritten (4-byte alignment suffices)
 */
int a8_quantize(const void *x_bf16, int M, int K, int8_t *a, float *a_scale, void *stream);

/*
 * Workspace size in bytes that w2a8_gemm / w2a8_gemm_partials need for this
 * problem (status word, split-K arrival counters and partial outputs; the
 * larger of what the kernels that may serve the shape need).  Returns 0 for
 * shapes that violate the shape rules.  The workspace must be zero-filled once
 * (w2a8_workspace_init) before its first use; the kernels leave it reusable.
 * One workspace serves any sequence of calls on one stream as long as it is at
 * least as large as each call needs; calls that may overlap on the device
 * (different streams) need separate workspaces.
 */
size_t w2a8_workspace_bytes(int M, int N, int K, int group);

/* Zero-fill a workspace (asynchronous, on `stream`). */
int w2a8_workspace_init(void *workspace, size_t workspace_bytes, void *stream);

/*
 * Read back the device status word kept at the start of a workspace.  Every
 * wait inside the kernels (on an asynchronous-copy barrier) is bounded; a wait
 * that gives up records W2A8_ERR_TIMEOUT here and the kernel returns without
 * producing valid outputs instead of hanging.  Synchronises `stream`.  Returns
 * the recorded status (W2A8_OK if none), or W2A8_ERR_CUDA / W2A8_ERR_NULL.
 */
int w2a8_workspace_status(const void *workspace, void *stream);

/*
 * w2a8_gemm -- y[m][n] = a_scale[m] * sum_gi w_scale[n][gi] * P[m][n][gi] with
 * P[m][n][gi] = sum_{k in group gi} a[m][k] * (code[n][k] - 2), the int32
 * sums being exact (Sec. II-C microkernel: int2 weights up-converted to int8,
 * int8 multiply-accumulate into int32; Sec. II-D: int32 -> float times the
 * product of activation and weight scales; K-splitting for small shapes).
 * fp32 summation order is unspecified but fixed for a given problem shape:
 * repeated calls give bitwise-equal outputs.
 *   a       [M][K] int8 (from a8_quantize)         a_scale [M] fp32
 *   packed  [N][K/16] uint32 (from w2_pack)        w_scale [N][K/group] fp32
 *   y       [M][N] fp32, row-major, fully overwritten
 *   workspace / workspace_bytes: see w2a8_workspace_bytes.
 * M >= 64 with N % 128 == 0 and K % 256 == 0 takes the tensor-core kernel
 * (tcgen05, 128 x 128 output tiles) when there are enough output tiles for it
 * to be the faster one (M * N above about 0.95 million per round of 148
 * tiles); everything else takes a memory-bound streaming kernel (weights
 * read once per slab of up to 32 tokens): the one-shot kernel when the problem
 * is about one wave of its CTAs, the persistent one (at most 32 tokens,
 * K % 256 == 0) for small matrices with K <= 4096 and for problems of more
 * than one wave.  w2a8_kernel_for reports tensor-core or streaming.
 * A problem given to the tensor-core kernel may leave its last (at most
 * eight) 128-channel tiles to the streaming kernel, as a second launch on the
 * same stream (w2a8_tensor_core_channels); the result does not depend on it
 * beyond fp32 summation order.
 */
int w2a8_gemm(const int8_t *a, const float *a_scale, const uint32_t *packed,
              const float *w_scale, float *y, int M, int N, int K, int group,
              void *workspace, size_t workspace_bytes, void *stream);

/*
 * w2a8_gemm with the storage recipe of the paper's end-to-end ternary section
 * (groups of 128 along K, weight scales kept in 16 bits): the weight scales
 * are IEEE binary16 bit patterns -- the 16-bit type the direct-conversion
 * listing of Sec. II names for its scale -- and the result is fp32 or bf16.
 *
 *   w_scale_h  device, [N][K/group] binary16, row-major, 16-byte aligned
 *   y          device, [M][N], 16-byte aligned: fp32 when y_is_bf16 == 0,
 *              else bf16
 * Everything else (a, a_scale, packed, shapes, group, workspace -- sized by
 * w2a8_workspace_bytes --, stream, dispatch by M, error codes, asynchronous
 * completion) is as for w2a8_gemm; any group w2a8_gemm takes is accepted.
 *
 * The value computed is that of w2a8_gemm called with every scale widened
 * (exactly) to fp32; with y_is_bf16 that fp32 value is rounded once to bf16,
 * to nearest, ties to even.  Scale bytes per weight drop from 32/group bit to
 * 16/group bit, result bytes from 4 to 2 per element.
 */
int w2a8_gemm_h16(const int8_t* a, const float* a_scale, const uint32_t* packed,
                  const uint16_t* w_scale_h, void* y, int y_is_bf16, int M, int N, int K, int group,
                  void* workspace, size_t workspace_bytes, void* stream);

/*
 * The alternative kernel of Sec. II ("Alternative implementation"): the 2-bit
 * weights are turned into 16-bit values and multiplied with 16-bit
 * activations, so the activations are not quantised and no dequantisation
 * follows:
 *
 *   y[m][n] = sum_gi w_scale[n][gi] * sum_{k in group gi} x[m][k] * (q[n][k] - 2)
 *
 *   x_bf16   device, [M][K] bf16, row-major, 16-byte aligned
 *   packed, w_scale, y (fp32 [M][N]), shapes, group, workspace (sized by
 *   w2a8_workspace_bytes), stream, error codes, asynchronous completion:
 *   as for w2a8_gemm.  No a8_quantize call is needed before it.
 *
 * Arithmetic: the codes become the bf16 values q - 2 (exact), every product
 * with a bf16 activation is exact in fp32, and the products of one scale group
 * are summed in fp32 by the tensor core (`mma.sync` bf16, fp32 accumulate; the
 * order inside the instruction is the hardware's); each group sum is then
 * multiplied by its fp32 scale and added in fp32.  Where the paper folds the
 * scale into the 16-bit weight (exact only for ternary codes and a 16-bit
 * scale), this build applies it to the group sum, which is exact for all four
 * code values and keeps fp32 scales.  The result differs from the exact sum by
 * fp32 summation error only (of the order sqrt(K) * 2^-24 relative to the
 * magnitude of the terms).  Few tokens take the streaming kernel (`mma.sync`
 * bf16); shapes the tensor-core path takes (see w2a8_gemm) run on the 16-bit
 * tensor-core kernel: tcgen05 kind::f16 with bf16 operands and fp32 accumulators
 * in tensor memory, the group scale applied when an accumulator is drained.
 */
int w2a16_gemm(const void* x_bf16, const uint32_t* packed, const float* w_scale, float* y,
               int M, int N, int K, int group, void* workspace, size_t workspace_bytes, void* stream);

/*
 * Which kernel w2a8_gemm / w2a8_gemm_h16 / w2a8_linear use for a shape:
 * 0 = streaming kernel, 1 = tensor-core kernel, W2A8_ERR_SHAPE for a shape
 * that is not accepted.  Host only, launches nothing.  (The paper picks its
 * kernel variant per shape with an auto-tuner, Sec. II; here the rule is fixed
 * and measured.)
 */
int w2a8_kernel_for(int M, int N, int K, int group);

/*
 * Which tensor-core kernel serves w2a8_gemm / w2a8_gemm_partials for a shape the
 * tensor-core path takes: 8 = the int8 kernel (tcgen05 kind::i8, int32
 * accumulators), 16 = the 16-bit kernel (kind::f16 on a bf16 copy of the int8
 * activations made by a small kernel in front; every product and partial sum is
 * an integer below 2^24, so the fp32 accumulators hold the same exact group sums
 * and no int32 -> float conversion is needed), 0 = the shape goes to a streaming
 * kernel.  W2A8_TC_KIND=8 / 16 in the environment forces one.  Host only.
 */
int w2a8_tensor_core_kind(int M, int N, int K, int group);

/*
 * How many of the N output channels the tensor-core kernel computes for this
 * shape: 0 when the streaming kernel takes the whole problem, N when the
 * tensor-core kernel does, and a multiple of 128 in between when the last
 * channel tiles are given to the streaming kernel in a second launch (the
 * tensor-core kernel works in rounds of one 128 x 128 tile per SM, and a last
 * round with a handful of tiles costs as much as a full one).  Host only.
 * W2A8_ERR_SHAPE for a shape that is not accepted.
 */
int w2a8_tensor_core_channels(int M, int N, int K, int group);

/*
 * How many ways the tensor-core kernel splits K for this shape: 0 when the
 * streaming kernel takes the problem, else 1, 2, 4 or 8.  A problem with few
 * 128 x 128 output tiles would leave most SMs idle; with a split every tile
 * becomes that many work items (each a whole number of 256-k blocks and of
 * scale groups), whose fp32 partial outputs go to the workspace and are added
 * in split order by a second, small kernel on the same stream -- so the result
 * does not depend on timing, and differs from the unsplit sum only by the order
 * of fp32 additions (Sec. II-D: splitting along K to put all cores to work).
 * w2a8_workspace_bytes covers the partial outputs.  W2A8_PF_KSPLIT = 1, 2, 4, 8
 * forces a count where it divides the shape.  Host only.  W2A8_ERR_SHAPE for a
 * shape that is not accepted.
 */
int w2a8_tensor_core_ksplit(int M, int N, int K, int group);

/*
 * Token rows per output tile of the tensor-core kernel that serves this shape:
 * 0 when the streaming kernel takes the problem, else 128, or 256 for the
 * kernel with 128-channel x 256-token tiles.  That one needs one scale per
 * channel (group == K): a tile's accumulators then stay in tensor memory until
 * its epilogue, every unpacked weight stage feeds twice the MACs (Sec. II-D:
 * larger output tiles per work-group; Sec. II-C: the up-convert in shared
 * memory), and the result is bit-equal to the 128-token kernel's.  It is taken
 * when the cost model expects it to be faster (many tokens, enough tiles);
 * W2A8_PF_WIDE = 0 never, 2 whenever the shape allows.  Host only.
 * W2A8_ERR_SHAPE for a shape that is not accepted.
 */
int w2a8_tensor_core_tile_tokens(int M, int N, int K, int group);

/*
 * w2a8_gemm_partials -- parity/debug export of the exact int32 per-group sums
 * P[m][n][gi] computed by the same inner-product code as w2a8_gemm.
 *   partials [M][N][K/group] int32, fully overwritten.
 */
int w2a8_gemm_partials(const int8_t *a, const uint32_t *packed, int32_t *partials,
                       int M, int N, int K, int group,
                       void *workspace, size_t workspace_bytes, void *stream);

/*
 * w2a8_gemm_grouped -- w2a8_gemm for `count` (1 .. 4) weight matrices that
 * share their activations (q|k|v of an attention block, gate|up of an MLP):
 * y[i] = W2A8(a; packed[i], w_scale[i]) for every i.  All matrices have the
 * same K and group; N[i] may differ.  The matrices stay where they are in
 * memory (no concatenated copy).  This is the K-splitting / launch-amortising
 * side of Sec. II-D: small GEMV shapes are bound by launch and fork-join cost,
 * so several of them are walked by one persistent launch (one CTA per SM, tiles
 * of all matrices dealt to the CTAs) when that is expected to be faster than
 * one launch per matrix, and otherwise run as `count` w2a8_gemm launches.
 *   a, a_scale                     as for w2a8_gemm (DEVICE)
 *   packed, w_scale, y, N          HOST arrays of `count` entries; the entries of
 *                                  the first three are DEVICE pointers as for w2a8_gemm
 *   workspace                      w2a8_grouped_workspace_bytes(count, N, M, K, group)
 * Each y[i] holds, bit for bit, what w2a8_gemm computes for matrix i with the
 * same kernel choice; with either kernel it is within the tolerance of
 * w2a8_gemm's contract and repeated calls give equal bits.
 */
int w2a8_gemm_grouped(const int8_t *a, const float *a_scale, int count, const uint32_t *const *packed,
                      const float *const *w_scale, float *const *y, const int *N, int M, int K, int group,
                      void *workspace, size_t workspace_bytes, void *stream);

/* Workspace bytes for the grouped entry points (0 for arguments they reject). */
size_t w2a8_grouped_workspace_bytes(int count, const int *N, int M, int K, int group);

/*
 * w2a8_linear_grouped -- bf16 activations in, scaled outputs of `count`
 * matrices out: the fused operator of Sec. II-D ("abs-max scales inside the
 * GEMM or in a kernel of their own", exposed there as a tuning knob and found
 * ahead for GEMV-sized problems only).  `fuse` is that knob:
 *   W2A8_FUSE_OFF   a8_quantize as a launch of its own, then w2a8_gemm_grouped
 *   W2A8_FUSE_ON    one launch: every CTA of the persistent kernel computes the
 *                   token scales and the int8 rows itself (same operations as
 *                   a8_quantize, same bits) into its shared memory.  Possible for
 *                   at most 8 tokens, K % 256 == 0 and rows that fit shared
 *                   memory; where it is not possible this behaves like _OFF.
 *   W2A8_FUSE_AUTO  _OFF, unless W2A8_FUSE_MAX_ELEMS in the environment allows
 *                   fusing up to that many values of M * K per CTA (default 0):
 *                   on B200 the separate quantiser launch hides behind the weight
 *                   prefetch of the launch that follows it, so it is the faster
 *                   form on the device for every token count (measured: 0.5 us per
 *                   call at one token, several us from four tokens on); fusing
 *                   saves one launch on the host
 *   x_bf16     [M][K] bf16 bit patterns, DEVICE
 *   a, a_scale DEVICE buffers that receive what a8_quantize would write; they may
 *              be NULL when the call fuses (then nothing is written), and must
 *              not be NULL otherwise (W2A8_ERR_NULL)
 *   the rest as for w2a8_gemm_grouped.
 * w2a8_grouped_plan reports what a call will do: bit 0 = one launch of the
 * persistent kernel for the whole group, bit 1 = that launch also quantises.
 * a and a_scale are bitwise those of a8_quantize; every y is bitwise that of
 * w2a8_gemm_grouped when that call takes the persistent kernel too, and differs
 * from it by fp32 summation order only otherwise.
 */
#define W2A8_FUSE_AUTO (-1)
#define W2A8_FUSE_OFF 0
#define W2A8_FUSE_ON 1
int w2a8_linear_grouped(const void *x_bf16, int8_t *a, float *a_scale, int count, const uint32_t *const *packed,
                        const float *const *w_scale, float *const *y, const int *N, int M, int K, int group,
                        int fuse, void *workspace, size_t workspace_bytes, void *stream);
int w2a8_grouped_plan(int count, const int *N, int M, int K, int group, int fuse);

/*
 * w2a8_linear -- w2a8_linear_grouped for one matrix with W2A8_FUSE_AUTO:
 * y = W2A8(x) for bf16 activations in device memory.
 *   x_bf16  [M][K] bf16 bit patterns, DEVICE
 *   a, a_scale   caller-provided DEVICE buffers ([M][K] int8, [M] fp32) that
 *           receive exactly what a8_quantize would write; they stay valid, so
 *           later w2a8_gemm calls on other weight matrices can reuse them
 *   the rest as for w2a8_gemm (same workspace size).
 * a and a_scale are bitwise what a8_quantize produces.  y is bitwise what
 * w2a8_gemm produces when both calls are served by the same kernel; when this
 * call fuses and w2a8_gemm would take the one-shot kernel for the matrix, the
 * two differ by fp32 summation order only (both within w2a8_gemm's tolerance,
 * both repeatable bit for bit).
 */
int w2a8_linear(const void *x_bf16, int8_t *a, float *a_scale, const uint32_t *packed,
                const float *w_scale, float *y, int M, int N, int K, int group,
                void *workspace, size_t workspace_bytes, void *stream);

/*
 * Workspace size for w2a8_linear_host: staging for x, a, a_scale and y plus
 * the GEMM workspace.  Zero-fill once with w2a8_workspace_init.
 */
size_t w2a8_linear_host_workspace_bytes(int M, int N, int K, int group);

/*
 * w2a8_linear_host -- the whole path for callers whose activations live in
 * HOST memory: copy x to the device, a8_quantize, w2a8_gemm, copy y back
 * (the fused "bf16 in, scaled output" use of Sec. II-D, with weights resident).
 *   x_host [M][K] bf16 bit patterns, HOST (pinned memory makes the copies
 *          asynchronous);  y_host [M][N] fp32, HOST, fully overwritten once the
 *          stream has run.  packed, w_scale, workspace: DEVICE.
 * With up to 32 tokens and both host buffers page-locked and mapped (16-byte
 * aligned), no copy is enqueued at all: the kernels read x and write y in host
 * memory directly over the bus, which at these sizes (a few KB) is faster than
 * two copy-engine operations.  Results are identical either way.
 * The call itself does not synchronise; synchronise the stream before reading
 * y_host.
 */
int w2a8_linear_host(const void *x_host, int M, int K, const uint32_t *packed,
                     const float *w_scale, int N, int group, float *y_host,
                     void *workspace, size_t workspace_bytes, void *stream);

/*
 * w2a8_linear_grouped_host -- w2a8_linear_host for `count` (1 .. 4) matrices
 * that share their activations: x is brought to the device and quantised once,
 * then the group runs as in w2a8_gemm_grouped and every y_host[i] ([M][N[i]]
 * fp32, HOST) receives its result.  packed, w_scale, N, y_host are HOST arrays of
 * `count` entries; the entries of packed and w_scale are DEVICE pointers, those of
 * y_host HOST pointers.  Zero-copy rule, workspace initialisation and
 * asynchronous completion as for w2a8_linear_host; workspace size from
 * w2a8_linear_grouped_host_workspace_bytes.
 */
size_t w2a8_linear_grouped_host_workspace_bytes(int count, const int *N, int M, int K, int group);
int w2a8_linear_grouped_host(const void *x_host, int M, int K, int count, const uint32_t *const *packed,
                             const float *const *w_scale, const int *N, int group, float *const *y_host,
                             void *workspace, size_t workspace_bytes, void *stream);

/*
 * w2a8_read_probe -- measurement aid, not part of the method (the paper's
 * counterpart is the bandwidth roofline of Sec. II-E, which needs the machine's
 * attainable read bandwidth): one kernel that reads `bytes` bytes of `buffer`
 * (DEVICE, 16-byte aligned) with plain 128-bit loads on `stream` and does
 * nothing else.  Timed by the caller over a buffer larger than L2, it gives the
 * read-only ceiling a streaming kernel on this device can be compared with.
 * `sink` is a DEVICE word the kernel may add to (it practically never does).
 */
int w2a8_read_probe(const void *buffer, size_t bytes, unsigned *sink, void *stream);

/*
 * w2a8_gemm_static -- w2a8_gemm without a workspace argument.  (The paper has no
 * counterpart; this entry exists for integration reasons only.)
 *
 * Who needs it: callers that are not in a position to allocate device memory
 * and have no workspace to pass -- for instance a serving runtime that handed
 * the whole GPU to its own memory pool at start-up, a custom-operator slot that
 * only receives input and output pointers, or a latency-critical loop in which
 * an allocation (and the implicit synchronisation it can bring) is forbidden.
 * For them the scratch of the kernel (status word, split-K arrival counters and
 * split-K partial outputs) is a fixed array of W2A8_STATIC_SCRATCH_BYTES bytes
 * inside the library image.  Every GPU that loads the library holds that array
 * until the process exits.  The call performs no cudaMalloc / cudaFree and calls
 * no allocating library routine.
 *
 * Arguments and result: exactly those of w2a8_gemm (same kernel, same launch
 * configuration, same bits in y).  Problems whose scratch need
 * (w2a8_workspace_bytes) exceeds W2A8_STATIC_SCRATCH_BYTES are refused with
 * W2A8_ERR_WORKSPACE; nothing is launched.
 *
 * First use on a device: the first call made while a given device is current
 * looks up the device address of the array (a host-side query, no allocation).
 * Make that first call outside any stream capture.
 *
 * Sharing: all calls on a device use the same array, which keeps the contents
 * the previous call left; each call clears the part that must start at zero
 * (on `stream`, before the kernel).  Two calls that can overlap on the device
 * (different streams, or different host threads on different streams) race on
 * it and give undefined results: keep such calls on one stream, or use
 * w2a8_gemm with separate workspaces.
 */
#define W2A8_STATIC_SCRATCH_BYTES (8u << 20)
int w2a8_gemm_static(const int8_t *a, const float *a_scale, const uint32_t *packed,
                     const float *w_scale, float *y, int M, int N, int K, int group, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* W2A8_H_ */
