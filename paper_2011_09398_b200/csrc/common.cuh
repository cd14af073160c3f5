// Shared host-side helpers of the library: geometry of an LceBConv2d call and launch checks.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "lce.h"

namespace lce {

// TensorFlow VALID / SAME extents (paper Section 3.2: LCE extends TFLite, "same" padding).
struct Axis {
    int32_t out;         // output extent
    int32_t pad_before;  // padding in front of element 0
};

inline Axis axis_geometry(int32_t in, int32_t k, int32_t stride, int32_t padding)
{
    Axis a{0, 0};
    if (padding == LCE_PAD_VALID) {
        a.out = in >= k ? (in - k) / stride + 1 : 0;
        return a;
    }
    a.out = (in + stride - 1) / stride;
    int32_t total = (a.out - 1) * stride + k - in;
    if (total < 0) total = 0;
    a.pad_before = total / 2;
    return a;
}

struct ConvGeom {
    int32_t N, H, W, Cin, Cw, Cout, Cow, KH, KW, sh, sw, OH, OW, pt, pl;
    int32_t padding, out_type, activation;
    int64_t M;  // N*OH*OW output pixels
};

inline lce_status make_geom(const lce_bconv2d_desc *d, ConvGeom *g)
{
    if (!d) return LCE_ERR_INVALID_ARG;
    if (d->batch <= 0 || d->in_h <= 0 || d->in_w <= 0 || d->in_c <= 0 || d->out_c <= 0 ||
        d->kernel_h <= 0 || d->kernel_w <= 0 || d->stride_h <= 0 || d->stride_w <= 0)
        return LCE_ERR_INVALID_ARG;
    if (d->padding < LCE_PAD_VALID || d->padding > LCE_PAD_SAME_ZERO) return LCE_ERR_INVALID_ARG;
    if (d->out_type < LCE_OUT_FLOAT32 || d->out_type > LCE_OUT_INT32) return LCE_ERR_INVALID_ARG;
    if (d->activation < LCE_ACT_NONE || d->activation > LCE_ACT_RELU) return LCE_ERR_INVALID_ARG;
    if (d->kernel < LCE_KERNEL_AUTO || d->kernel > LCE_KERNEL_TENSOR) return LCE_ERR_INVALID_ARG;
    if (d->weights_packed != 0 && d->weights_packed != 1) return LCE_ERR_INVALID_ARG;
    Axis ah = axis_geometry(d->in_h, d->kernel_h, d->stride_h, d->padding);
    Axis aw = axis_geometry(d->in_w, d->kernel_w, d->stride_w, d->padding);
    if (ah.out <= 0 || aw.out <= 0) return LCE_ERR_INVALID_ARG;
    g->N = d->batch; g->H = d->in_h; g->W = d->in_w; g->Cin = d->in_c; g->Cw = (d->in_c + 31) / 32;
    g->Cout = d->out_c; g->Cow = (d->out_c + 31) / 32;
    g->KH = d->kernel_h; g->KW = d->kernel_w; g->sh = d->stride_h; g->sw = d->stride_w;
    g->OH = ah.out; g->OW = aw.out; g->pt = ah.pad_before; g->pl = aw.pad_before;
    g->padding = d->padding; g->out_type = d->out_type; g->activation = d->activation;
    g->M = (int64_t)g->N * g->OH * g->OW;
    // the index arithmetic of the kernels is 32-bit on words: keep every tensor below 2^31 words
    int64_t in_words = (int64_t)g->N * g->H * g->W * g->Cw;
    int64_t out_elems = g->M * g->Cout;
    int64_t w_words = (int64_t)g->Cout * g->KH * g->KW * g->Cw;
    if (in_words >= (1ll << 31) || out_elems >= (1ll << 31) || w_words >= (1ll << 31))
        return LCE_ERR_UNSUPPORTED;
    return LCE_OK;
}

inline bool aligned(const void *p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

inline lce_status launch_status()
{
    return cudaGetLastError() == cudaSuccess ? LCE_OK : LCE_ERR_CUDA;
}

// The opt-in to more than 48 KB of dynamic shared memory is a driver call; it is made once per kernel,
// device and size (a larger request later raises it), not on every launch.  One instance per kernel.
struct SmemOptIn {
    static constexpr int kDevices = 64;
    std::atomic<size_t> granted[kDevices];
    SmemOptIn() { for (auto &g : granted) g.store(0, std::memory_order_relaxed); }
    template <typename Kernel>
    bool ensure(Kernel kernel, size_t smem_bytes)
    {
        if (smem_bytes <= 48 * 1024) return true;
        int dev = -1;
        if (cudaGetDevice(&dev) != cudaSuccess) return false;
        const bool tracked = dev >= 0 && dev < kDevices;
        if (tracked && granted[dev].load(std::memory_order_acquire) >= smem_bytes) return true;
        if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes) != cudaSuccess) return false;
        if (tracked) {  // concurrent callers may both set the attribute; the recorded size only grows
            size_t seen = granted[dev].load(std::memory_order_relaxed);
            while (seen < smem_bytes && !granted[dev].compare_exchange_weak(seen, smem_bytes, std::memory_order_release)) {}
        }
        return true;
    }
};

// Kernel entry points implemented in the other translation units.
lce_status launch_bconv_direct(const ConvGeom &g, const uint32_t *in, const uint32_t *w, const float *mult,
                               const float *bias, const int32_t *thr, void *out, cudaStream_t s);
// Returns LCE_ERR_UNSUPPORTED without launching when the tiled kernel does not cover the shape.
// w_image: the tiled part of a packed-weights buffer, or nullptr to derive operands from `w`.
// residual / out_packed: fused shortcut add and fused LceQuantize of a float output (both optional;
// with out_packed given, `out` may be null).
lce_status launch_bconv_tiled(const ConvGeom &g, const uint32_t *in, const uint32_t *w, const uint32_t *w_image,
                              const float *mult, const float *bias, const int32_t *thr, void *out, cudaStream_t s,
                              const float *residual = nullptr, uint32_t *out_packed = nullptr,
                              const float *in_f32 = nullptr);
// One-word-patch kernel for tiny channel counts (KH*KW*Cin <= 32); plain weights only.
bool patch_covers(const ConvGeom &g);
lce_status launch_bconv_patch(const ConvGeom &g, const uint32_t *in, const uint32_t *w, const float *mult,
                              const float *bias, const int32_t *thr, void *out, cudaStream_t s);
// Tensor-core kernel (tcgen05 kind::mxf4 on e2m1 operands): any filter of up to 64 taps, equal strides
// of 1 or 2, every padding mode; needs the weight image that launch_pack_weights_tensor writes at load
// time (w_image; null -> LCE_ERR_UNSUPPORTED).  residual / out_packed as for the tiled kernel (float
// output, out_c a multiple of 32).
bool tensor_covers(const ConvGeom &g);
size_t tensor_weight_image_bytes(const ConvGeom &g);
lce_status launch_pack_weights_tensor(const ConvGeom &g, const uint32_t *w, void *image, cudaStream_t s);
lce_status launch_bconv_tensor(const ConvGeom &g, const uint32_t *in, const void *w_image, const float *mult,
                               const float *bias, const int32_t *thr, void *out, cudaStream_t s,
                               const float *residual = nullptr, uint32_t *out_packed = nullptr);
struct TensorPlanInfo {
    int32_t tile_positions, ctas, weight_stages, weights_resident;
    int64_t shared_bytes;
};
lce_status tensor_plan_info(const ConvGeom &g, TensorPlanInfo *info);
// Bounded device-side waits: status word, its reset, the host-visible flag (no synchronisation), and a
// tiny kernel whose wait is meant to run out (nobody arrives at its barrier).
lce_status tensor_device_status(int *status);
lce_status tensor_device_status_reset();
bool tensor_timeout_flagged();
lce_status tensor_wait_probe(uint64_t limit_ns, cudaStream_t s);
// Bytes of the tiled kernel's weight image for this geometry (0 if the kernel does not cover it).
// Launch plan of the tiled kernels for a geometry (no buffers involved), for lce_bconv2d_plan.
struct TiledPlanInfo {
    int32_t pointwise, warps_per_cta, pixels_per_thread, tile_pixels, ctas, ctas_half_block, pixels_per_cta,
        pixels_per_cta_half_block;
    int64_t shared_bytes;
};
lce_status tiled_plan_info(const ConvGeom &g, TiledPlanInfo *info);
size_t tiled_weight_image_bytes(const ConvGeom &g);
lce_status launch_pack_weights_tiled(const ConvGeom &g, const uint32_t *w, uint32_t *image, cudaStream_t s);

}  // namespace lce
