/*
 * lce.h -- C ABI of the B200 (sm_100a) binarized 2-D convolution library.
 *
 * The operations are the ones the Larq Compute Engine paper defines in its
 * Section 3.2 "Operator implementations": LceQuantize (sign + bit-pack),
 * LceBConv2d (im2col over packed words, XOR+POPCOUNT binary GEMM, fused output
 * transform), LceBMaxPool2d (bitwise AND) and LceDequantize.
 *
 * Common rules
 *   - Unless a function says "host", every data pointer is a DEVICE pointer owned
 *     by the caller; the library never frees or keeps it.  Buffers of one call
 *     must not overlap.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).
 *     Device-pointer entry points only enqueue work on it: they never synchronise,
 *     never allocate and are safe to capture in a CUDA graph.
 *   - Every function returns an lce_status.  Argument errors are detected on the
 *     host before anything is launched; nothing is printed and nothing throws.
 *   - Bit convention (Section 3.2, LceQuantize): a 0 bit stands for +1.0, a 1 bit
 *     for -1.0.  Channel c of a pixel lives in word c/32, bit c%32 (least
 *     significant bit = lowest channel).  The channel axis is padded up to a
 *     multiple of 32 and pad bits are always 0, in activations, weights and
 *     bit-packed outputs alike.
 *   - Layouts are NHWC with the channel axis packed: activations
 *     uint32 [batch][h][w][ceil(c/32)], weights uint32 [out_c][kh][kw][ceil(in_c/32)].
 */
#ifndef LCE_B200_H_
#define LCE_B200_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    LCE_OK = 0,
    LCE_ERR_INVALID_ARG = 1,    /* null pointer, non-positive extent, bad enum, empty output */
    LCE_ERR_UNSUPPORTED = 2,    /* valid request that no kernel here implements */
    LCE_ERR_ALIGNMENT = 3,      /* a pointer is not aligned to its element size (4 bytes; packed weights: 256) */
    LCE_ERR_CUDA = 4,           /* the CUDA runtime reported an error at launch / copy */
    LCE_ERR_DEVICE_TIMEOUT = 5, /* a bounded device-side wait of an earlier kernel on this device gave up:
                                   that kernel's output is incomplete; see lce_device_status */
    LCE_ERR_WORKSPACE = 6       /* caller's workspace is too small */
} lce_status;

/* Section 3.2, LceBConv2d: padded locations hold zero words (= +1.0, "one-padding");
 * zero-padding is supported through a correction of the accumulator. */
typedef enum { LCE_PAD_VALID = 0, LCE_PAD_SAME_ONE = 1, LCE_PAD_SAME_ZERO = 2 } lce_padding;

/* Section 3.2, LceBConv2d: full-precision output or bit-packed output; INT32 exposes
 * the raw accumulator (used by tests). */
typedef enum { LCE_OUT_FLOAT32 = 0, LCE_OUT_BITPACKED = 1, LCE_OUT_INT32 = 2 } lce_out_type;

/* Fused activation of the float output transform (Section 3.2; Section 5: ReLU before
 * batch-norm in QuickNet).  Applied to the accumulator before multiplier and bias. */
typedef enum { LCE_ACT_NONE = 0, LCE_ACT_RELU = 1 } lce_activation;

/* Which kernel lce_bconv2d uses; every kernel gives the same, exact result.
 *   TILED  the XOR/POPC kernels on the integer pipes (1x1, 3x3, 5x5 filters, equal strides 1 or 2; a
 *          one-word kernel when kh*kw*in_c <= 32);
 *   TENSOR the tensor-core formulation: bits expanded to +-1 (0 for padding) as 4-bit e2m1 values,
 *          tcgen05 kind::mxf4 with unit block scales, fp32 accumulators in TMEM (exact: every sum is an
 *          integer below 2^24).  Filters of up to 64 taps, equal strides of 1 or 2, in_c <= 1024, every
 *          padding mode and output type.  Needs weights packed by lce_bconv2d_pack_weights;
 *   DIRECT one thread per output, any shape (fallback, not tuned);
 *   AUTO   TENSOR when the weights are packed and the layer is large enough to pay for that kernel's
 *          start-up (at least 2^28 binary MACs, 2^29 when the filter does not fit in shared memory, 2^31
 *          for 3x3 or smaller filters on at most 32 input channels), otherwise TILED where it covers the
 *          shape, otherwise DIRECT.  lce_bconv2d_plan tells which.
 * Forcing a kernel on a shape (or on plain weights) it does not cover returns LCE_ERR_UNSUPPORTED. */
typedef enum { LCE_KERNEL_AUTO = 0, LCE_KERNEL_DIRECT = 1, LCE_KERNEL_TILED = 2, LCE_KERNEL_TENSOR = 3 } lce_kernel;

const char *lce_version(void);
const char *lce_status_string(lce_status status);

/* LceQuantize (Section 3.2): out bit = (x < 0), so +0.0, -0.0 and NaN give a 0 bit.
 *   x   fp32  [rows][channels]            (rows = batch*h*w of an NHWC tensor)
 *   out uint32[rows][ceil(channels/32)]
 * rows == 0 is a no-op.  Binary weights are packed with the same call on the
 * [out_c*kh*kw][in_c] view of an OHWI float tensor (Section 3.1, weight compression). */
lce_status lce_bitpack(const float *x, uint32_t *out, int64_t rows, int32_t channels, void *stream);

/* LceDequantize (Section 3.2, footnote to LceQuantize): packed bits -> +1.0f / -1.0f.
 *   in  uint32[rows][ceil(channels/32)]   out fp32 [rows][channels] */
lce_status lce_unpack(const uint32_t *in, float *out, int64_t rows, int32_t channels, void *stream);

/* LceBConv2d (Section 3.2).  in_c is the TRUE channel count: K = kernel_h*kernel_w*in_c. */
typedef struct {
    int32_t batch, in_h, in_w, in_c;
    int32_t out_c, kernel_h, kernel_w, stride_h, stride_w;
    int32_t padding;    /* lce_padding; SAME follows TensorFlow: out = ceil(in/stride),
                           total pad max((out-1)*stride+k-in, 0), floor(half) before */
    int32_t out_type;   /* lce_out_type */
    int32_t activation; /* lce_activation; FLOAT32 output only */
    int32_t kernel;     /* lce_kernel */
    int32_t weights_packed; /* 0: `weights` is the plain word tensor [out_c][kh][kw][ceil(in_c/32)];
                               1: `weights` is the buffer lce_bconv2d_pack_weights wrote for this
                                  same descriptor (geometry fields must match) */
} lce_bconv2d_desc;

/* Output extent of the convolution; LCE_ERR_INVALID_ARG if the descriptor is malformed or
 * the output would be empty. */
lce_status lce_bconv2d_out_shape(const lce_bconv2d_desc *desc, int32_t *out_h, int32_t *out_w);

/* acc[n][oh][ow][o] = sum over (ky,kx,c) of a(n, oh*s-pt+ky, ow*s-pl+kx, c) * w[o][ky][kx][c]
 *                   = K - 2*popcount(a XOR w) over the packed words (Section 2; Section 3.2),
 * with out-of-image taps +1 (SAME_ONE) or 0 (SAME_ZERO), then the output transform:
 *   FLOAT32   out fp32  [batch][oh][ow][out_c]           = fmaf((float)act(acc), multiplier[o], bias[o])
 *             (one rounding); multiplier, bias fp32[out_c] required, thresholds ignored.
 *   BITPACKED out uint32[batch][oh][ow][ceil(out_c/32)]  bit o = (acc < thresholds[o]);
 *             thresholds int32[out_c] required; activation must be LCE_ACT_NONE (the converter
 *             folds it into the thresholds, Section 3.1); multiplier, bias ignored.
 *   INT32     out int32 [batch][oh][ow][out_c]           = acc.
 *   input   uint32[batch][in_h][in_w][ceil(in_c/32)]     weights uint32[out_c][kh][kw][ceil(in_c/32)]
 * With desc->weights_packed == 1, `weights` is instead the buffer written by
 * lce_bconv2d_pack_weights (the fast path: nothing is derived from the weights per call).
 * Pad bits of input and weights must be 0.  The float / int32 fast paths want `output` 16-byte
 * aligned (out_c a multiple of 4); a buffer that is only 4-byte aligned is served by the direct kernel
 * under AUTO.  The weights and per-channel arrays are constants of the model: the kernels read them
 * before they wait for the stream's previous kernel where that kernel lets its dependents start early
 * (programmatic dependent launch; this library's convolution kernels do), so they must not be the
 * output of such a kernel that may still be running.  What lce_bconv2d_pack_weights, a copy or an
 * ordinary kernel wrote earlier on the stream is complete before this call's kernel is scheduled.
 * Errors: INVALID_ARG
 * (null/extent/enum/missing per-channel array), ALIGNMENT, UNSUPPORTED (a forced kernel does not cover
 * the shape), CUDA, DEVICE_TIMEOUT (see lce_device_status; nothing is launched). */
lce_status lce_bconv2d(const lce_bconv2d_desc *desc, const uint32_t *input, const uint32_t *weights,
                       const float *multiplier, const float *bias, const int32_t *thresholds,
                       void *output, void *stream);

/* LceBConv2d with its float-output neighbours fused into the output transform (Section 3.2: fused
 * operations run on the accumulators before they are written; Section 5.3: a shortcut is float
 * output -> Add -> LceQuantize).  desc->out_type must be LCE_OUT_FLOAT32.  Per output value:
 *   y = fmaf((float)act(acc), multiplier[o], bias[o]);  if residual: y = y + residual[...] (fp32);
 *   if out_float:  out_float[...] = y;   if out_packed: bit o of the pixel's word = (y < 0).
 *   residual   fp32 [batch][oh][ow][out_c] or NULL       out_float fp32 same shape, or NULL
 *   out_packed uint32 [batch][oh][ow][ceil(out_c/32)] or NULL   (at least one output required)
 * The results are bit-identical to lce_bconv2d -> lce_add_f32 -> lce_bitpack run one after the
 * other.  Only shapes the tiled kernels cover (3x3 and 5x5 with equal strides of 1 or 2, 1x1) are accepted; others return
 * LCE_ERR_UNSUPPORTED. */
lce_status lce_bconv2d_fused(const lce_bconv2d_desc *desc, const uint32_t *input, const uint32_t *weights,
                             const float *multiplier, const float *bias, const float *residual,
                             float *out_float, uint32_t *out_packed, void *stream);

/* LceQuantize fused into LceBConv2d's loader (Section 3.2: a binarized convolution whose input is a
 * full-precision tensor is preceded by LceQuantize; Section 5.3 counts that op's share of the run
 * time).  `input` is the fp32 activation tensor [batch][in_h][in_w][in_c] (device); the kernel
 * takes the sign bit of each value (negative -> bit 1, as lce_bitpack does) while it stages the
 * rows, so the packed tensor never exists in memory.  Everything else is lce_bconv2d, and the
 * result is bit-identical to lce_bitpack followed by lce_bconv2d.  Covers the shapes of the tiled
 * KxK kernel (3x3 and 5x5 filters, equal strides of 1 or 2); anything else, and desc->kernel set to
 * DIRECT or TENSOR, returns LCE_ERR_UNSUPPORTED (call lce_bitpack, then lce_bconv2d).
 * Cost: the sign loads are synchronous and every channel block and halo row repeats them, so on
 * this GPU the call is slower than lce_bitpack + lce_bconv2d for every measured shape; what it
 * saves is the packed tensor's memory. */
lce_status lce_bconv2d_f32(const lce_bconv2d_desc *desc, const float *input, const uint32_t *weights,
                           const float *multiplier, const float *bias, const int32_t *thresholds,
                           void *output, void *stream);

/* Which kernel lce_bconv2d would launch for this descriptor, and with what shape: host arithmetic
 * only, nothing is launched and no GPU is needed (without one the plan is made for 148 SMs).  The
 * paper's engine picks its kernel and tiling per layer when the model is loaded (Section 3.1); this
 * is that choice made visible.  Fields that do not apply to the chosen kernel are 0.
 *   kernel              LCE_KERNEL_DIRECT, LCE_KERNEL_TILED or LCE_KERNEL_TENSOR (the one-word patch
 *                       kernel for very few input channels reports LCE_KERNEL_TILED with patch = 1).
 *                       For LCE_KERNEL_TENSOR: tile_pixels = grid positions per tile, ctas, shared_bytes,
 *                       weights_resident = 1 when every tap of a channel block stays in shared memory
 *                       (fetched once per CTA; weight_stages = taps), 0 when they stream past once per
 *                       tile (weight_stages = stages of the ring, each a group of consecutive taps)
 *   pointwise           1 for the 1x1 tiled kernel
 *   warps_per_cta, pixels_per_thread, tile_pixels, shared_bytes      the variant of the tiled kernel
 *   ctas                CTAs of the launch; ctas_half_block of them work on the last, at most
 *                       32-channel block with the 8-pixel x 4-group lane mapping
 *   pixels_per_cta      flat output pixels each CTA of a full channel block owns (KxK kernel);
 *                       pixels_per_cta_half_block the same for the half block
 * Output buffers are assumed 16-byte aligned.  Errors: INVALID_ARG; UNSUPPORTED when desc->kernel
 * forces a kernel that does not cover the shape. */
typedef struct lce_bconv2d_plan_info {
    int32_t kernel, patch, pointwise;
    int32_t warps_per_cta, pixels_per_thread, tile_pixels;
    int32_t ctas, ctas_half_block, pixels_per_cta, pixels_per_cta_half_block;
    int64_t shared_bytes;
    int32_t weight_stages, weights_resident;
} lce_bconv2d_plan_info;
lce_status lce_bconv2d_plan(const lce_bconv2d_desc *desc, lce_bconv2d_plan_info *plan);

/* A convolution bound to its buffers: checked once, launched many times (Section 3.1: the paper's
 * engine prepares every operator when the model is loaded and only runs it per inference).
 * lce_bconv2d_plan_create takes the arguments of lce_bconv2d, makes all of its host-side checks,
 * including that a kernel covers the shape, and on LCE_OK stores a handle in *plan; nothing is
 * launched.  lce_plan_run launches the convolution on `stream` exactly as lce_bconv2d would (asynchronous,
 * no allocation, capturable in a CUDA graph); it may be called any number of times, from one host
 * thread at a time.  The handle is a small host object owned by the library until lce_plan_destroy
 * (NULL is ignored); it holds the descriptor and the pointers, never the buffers, which stay the
 * caller's and must outlive the runs.  Errors: those of lce_bconv2d; INVALID_ARG for a NULL plan. */
typedef struct lce_plan lce_plan;
lce_status lce_bconv2d_plan_create(const lce_bconv2d_desc *desc, const uint32_t *input, const uint32_t *weights,
                                   const float *multiplier, const float *bias, const int32_t *thresholds,
                                   void *output, lce_plan **plan);
lce_status lce_plan_run(const lce_plan *plan, void *stream);
void lce_plan_destroy(lce_plan *plan);

/* Load-time weight packing (Section 3.2: the paper's BGEMM also re-arranges the weights ahead of
 * time for its access pattern; Section 3.1: weights are converted once, when the model is built).  Rewrites
 * the plain packed weights into the operand layout the tiled kernel copies straight into shared
 * memory, so that none of that work is repeated per call.  The packed buffer also keeps a copy of
 * the plain words, and, where the tensor-core kernel covers the geometry, that kernel's operand image
 * (every weight bit expanded to a 4-bit +-1, pad channels 0).  It is valid for every padding mode, output
 * type and activation of the same geometry (batch, sizes, channels, kernel, stride).  The first call in a
 * process also sets up a few bytes of pinned host memory for the device-timeout flag: make it outside
 * any stream capture.
 *   weights uint32[out_c][kh][kw][ceil(in_c/32)] (device)  ->  packed: device buffer of
 *   lce_bconv2d_packed_weights_bytes(desc) bytes, 256-byte aligned, owned by the caller.
 * lce_bconv2d_packed_weights_bytes returns 0 for a malformed descriptor. */
size_t lce_bconv2d_packed_weights_bytes(const lce_bconv2d_desc *desc);
lce_status lce_bconv2d_pack_weights(const lce_bconv2d_desc *desc, const uint32_t *weights, void *packed,
                                    void *stream);

/* Host-buffer form of lce_bconv2d, for callers whose tensors live in host memory: every data
 * pointer is a HOST pointer (pinned memory makes the copies asynchronous); `workspace` is a
 * DEVICE buffer of at least lce_bconv2d_host_workspace_bytes(desc) bytes that the call uses
 * for the device copies of input, weights, per-channel arrays and output.  Copies in, runs
 * the same kernel as lce_bconv2d (weights_packed must be 0), copies the output back, all on `stream`, and returns after
 * synchronising that stream.  LCE_ERR_WORKSPACE if workspace_bytes is too small. */
size_t lce_bconv2d_host_workspace_bytes(const lce_bconv2d_desc *desc);
lce_status lce_bconv2d_host(const lce_bconv2d_desc *desc, const uint32_t *input, const uint32_t *weights,
                            const float *multiplier, const float *bias, const int32_t *thresholds,
                            void *output, void *workspace, size_t workspace_bytes, void *stream);

/* lce_bconv2d_host without the final synchronisation: the copies and the kernel are only enqueued on
 * `stream`.  Host buffers must be pinned for the copies to be asynchronous, and all buffers
 * (`output` and `workspace` included) belong to the call until the caller has synchronised `stream`;
 * calls on different streams with different workspaces overlap (one layer's copy back with the next
 * layer's copies in and kernel). */
lce_status lce_bconv2d_host_async(const lce_bconv2d_desc *desc, const uint32_t *input, const uint32_t *weights,
                                  const float *multiplier, const float *bias, const int32_t *thresholds,
                                  void *output, void *workspace, size_t workspace_bytes, void *stream);

/* (No counterpart in the paper.)  lce_bconv2d_host for callers that cannot allocate device memory:
 * a process whose allocator is off limits (a real-time loop, a sandboxed plug-in that only ever
 * sees host tensors) has no way to produce the `workspace` argument above.  This form keeps the
 * staging area inside the library, in one fixed device array of
 * lce_bconv2d_host_noalloc_max_bytes() = 8 MiB per GPU, and calls no cudaMalloc, cudaFree or any
 * other allocating routine.  Arguments and result are those of lce_bconv2d_host without the
 * workspace; a call whose lce_bconv2d_host_workspace_bytes(desc) exceeds the array returns
 * LCE_ERR_WORKSPACE and does nothing.
 *   - The first call on each device looks up the array's device address (with that device
 *     current).  The call synchronises `stream` before it returns, so it cannot be part of a stream
 *     capture anyway.
 *   - All calls on a device share the one array, which still holds the previous call's data:
 *     nothing needs clearing (every region is rewritten before it is read), but two calls that
 *     overlap on the GPU (different streams, different threads) would overwrite each other.
 *     Serialise them. */
size_t lce_bconv2d_host_noalloc_max_bytes(void);
lce_status lce_bconv2d_host_noalloc(const lce_bconv2d_desc *desc, const uint32_t *input, const uint32_t *weights,
                                    const float *multiplier, const float *bias, const int32_t *thresholds,
                                    void *output, void *stream);

/* LceBMaxPool2d (Section 3.2): max-pool of +-1 values on packed words = bitwise AND of the
 * window's words.  padding is LCE_PAD_VALID or LCE_PAD_SAME_ONE (TensorFlow SAME; taps outside
 * the image are skipped).
 *   in uint32[batch][in_h][in_w][ceil(channels/32)] -> out uint32[batch][oh][ow][ceil(channels/32)] */
lce_status lce_bmaxpool(const uint32_t *in, uint32_t *out, int32_t batch, int32_t in_h, int32_t in_w,
                        int32_t channels, int32_t pool_h, int32_t pool_w, int32_t stride_h,
                        int32_t stride_w, int32_t padding, void *stream);

/* fp32 residual add out = a + b (one rounding), the shortcut pattern of Section 5.3
 * (float output -> Add -> LceQuantize).  n == 0 is a no-op; out may equal a or b. */
lce_status lce_add_f32(const float *a, const float *b, float *out, int64_t n, void *stream);

/* Status of the bounded device-side waits.  The tensor-core kernel's warps meet through mbarriers
 * (operands ready, MMAs complete, accumulator read out); every such wait is limited to 0.2 s, after
 * which the kernel stops working, waits (bounded) for its copies and MMAs in flight, frees its tensor
 * memory and returns, leaving its output incomplete.  It records that in a device word and in a word
 * of mapped host memory; from then on lce_bconv2d, lce_bconv2d_fused and lce_plan_run on that device
 * return LCE_ERR_DEVICE_TIMEOUT without launching, until lce_device_status_reset.
 *   lce_device_status        *status (HOST pointer) = 0 if no wait has given up on the current device
 *                            since load or the last reset, 1 otherwise.  Synchronous (reads the device word).
 *   lce_device_status_reset  clears both words for the current device.  Synchronous.
 *   lce_device_wait_probe    self-test of that machinery: launches one tiny kernel on `stream` whose
 *                            wait (limit_ns, 1 .. 10^9) is on a barrier nobody arrives at, so it runs out,
 *                            is reported like a real one, and the kernel returns normally.  Touches no
 *                            tensor; follow it with lce_device_status_reset. */
lce_status lce_device_status(int32_t *status);
lce_status lce_device_status_reset(void);
lce_status lce_device_wait_probe(uint64_t limit_ns, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* LCE_B200_H_ */
