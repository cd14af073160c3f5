// C ABI front: version/status strings, shape query and the LceBConv2d dispatch (device- and
// host-buffer forms).  All argument checks happen here, before anything is launched.
#include "common.cuh"

#include <new>

namespace lce {
namespace {

lce_status check_conv_args(const lce_bconv2d_desc *desc, ConvGeom *g, const void *input, const void *weights,
                           const void *multiplier, const void *bias, const void *thresholds, const void *output)
{
    lce_status st = make_geom(desc, g);
    if (st != LCE_OK) return st;
    if (!input || !weights || !output) return LCE_ERR_INVALID_ARG;
    if (g->out_type == LCE_OUT_FLOAT32 && (!multiplier || !bias)) return LCE_ERR_INVALID_ARG;
    if (g->out_type == LCE_OUT_BITPACKED) {
        if (!thresholds) return LCE_ERR_INVALID_ARG;
        if (g->activation != LCE_ACT_NONE) return LCE_ERR_INVALID_ARG;
    }
    return LCE_OK;
}

size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

size_t plain_weight_bytes(const ConvGeom &g) { return round_up((size_t)g.Cout * g.KH * g.KW * g.Cw * 4, 256); }

lce_status dispatch(const lce_bconv2d_desc *desc, const ConvGeom &g, const uint32_t *input, const uint32_t *weights,
                    const float *multiplier, const float *bias, const int32_t *thresholds, void *output,
                    cudaStream_t s)
{
    // a packed-weights buffer = [plain words, rounded up to 256 bytes][tiled image]
    const uint32_t *image = nullptr;
    if (desc->weights_packed) {
        if (!aligned(weights, 256)) return LCE_ERR_ALIGNMENT;
        if (tiled_weight_image_bytes(g) > 0)
            image = reinterpret_cast<const uint32_t *>(reinterpret_cast<const char *>(weights) + plain_weight_bytes(g));
    }
    if (desc->kernel == LCE_KERNEL_DIRECT)
        return launch_bconv_direct(g, input, weights, multiplier, bias, thresholds, output, s);
    if (desc->kernel == LCE_KERNEL_TENSOR)
        return launch_bconv_tensor(g, input, weights, multiplier, bias, thresholds, output, s);
    if (patch_covers(g)) return launch_bconv_patch(g, input, weights, multiplier, bias, thresholds, output, s);
    lce_status st = launch_bconv_tiled(g, input, weights, image, multiplier, bias, thresholds, output, s);
    if (st == LCE_ERR_UNSUPPORTED && desc->kernel == LCE_KERNEL_AUTO)
        st = launch_bconv_direct(g, input, weights, multiplier, bias, thresholds, output, s);
    return st;
}

struct HostLayout {
    size_t in, w, mult, bias, thr, out, total;
    size_t in_bytes, w_bytes, ch_bytes, out_bytes;
};

HostLayout host_layout(const ConvGeom &g)
{
    HostLayout L{};
    L.in_bytes = (size_t)g.N * g.H * g.W * g.Cw * 4;
    L.w_bytes = (size_t)g.Cout * g.KH * g.KW * g.Cw * 4;
    L.ch_bytes = (size_t)g.Cout * 4;
    L.out_bytes = (size_t)g.M * (g.out_type == LCE_OUT_BITPACKED ? g.Cow : g.Cout) * 4;
    size_t off = 0;
    L.in = off;   off += round_up(L.in_bytes, 256);
    L.w = off;    off += round_up(L.w_bytes, 256);
    L.mult = off; off += round_up(L.ch_bytes, 256);
    L.bias = off; off += round_up(L.ch_bytes, 256);
    L.thr = off;  off += round_up(L.ch_bytes, 256);
    L.out = off;  off += round_up(L.out_bytes, 256);
    L.total = off;
    return L;
}

}  // namespace
}  // namespace lce

extern "C" const char *lce_version(void) { return "lce-b200 0.1 (sm_100a)"; }

extern "C" const char *lce_status_string(lce_status status)
{
    switch (status) {
        case LCE_OK: return "ok";
        case LCE_ERR_INVALID_ARG: return "invalid argument";
        case LCE_ERR_UNSUPPORTED: return "unsupported";
        case LCE_ERR_ALIGNMENT: return "misaligned pointer";
        case LCE_ERR_CUDA: return "CUDA error";
        case LCE_ERR_DEVICE_TIMEOUT: return "device-side wait timed out";
        case LCE_ERR_WORKSPACE: return "workspace too small";
    }
    return "unknown status";
}

extern "C" lce_status lce_device_status(int32_t *status)
{
    if (!status) return LCE_ERR_INVALID_ARG;
    int v = 0;
    lce_status st = lce::tensor_device_status(&v);
    if (st != LCE_OK) return st;
    *status = v;
    return LCE_OK;
}

extern "C" lce_status lce_bconv2d_out_shape(const lce_bconv2d_desc *desc, int32_t *out_h, int32_t *out_w)
{
    lce::ConvGeom g;
    lce_status st = lce::make_geom(desc, &g);
    if (st != LCE_OK) return st;
    if (!out_h || !out_w) return LCE_ERR_INVALID_ARG;
    *out_h = g.OH;
    *out_w = g.OW;
    return LCE_OK;
}

extern "C" lce_status lce_bconv2d_plan(const lce_bconv2d_desc *desc, lce_bconv2d_plan_info *plan)
{
    using namespace lce;
    ConvGeom g;
    lce_status st = make_geom(desc, &g);
    if (st != LCE_OK) return st;
    if (!plan) return LCE_ERR_INVALID_ARG;
    *plan = lce_bconv2d_plan_info{};
    // the same order of preference as dispatch()
    if (desc->kernel == LCE_KERNEL_DIRECT) { plan->kernel = LCE_KERNEL_DIRECT; return LCE_OK; }
    if (desc->kernel == LCE_KERNEL_TENSOR) {
        if (!tensor_covers(g)) return LCE_ERR_UNSUPPORTED;
        plan->kernel = LCE_KERNEL_TENSOR;
        return LCE_OK;
    }
    if (patch_covers(g)) { plan->kernel = LCE_KERNEL_TILED; plan->patch = 1; return LCE_OK; }
    TiledPlanInfo info{};
    st = tiled_plan_info(g, &info);
    if (st == LCE_ERR_UNSUPPORTED && desc->kernel == LCE_KERNEL_AUTO) { plan->kernel = LCE_KERNEL_DIRECT; return LCE_OK; }
    if (st != LCE_OK) return st;
    plan->kernel = LCE_KERNEL_TILED;
    plan->pointwise = info.pointwise;
    plan->warps_per_cta = info.warps_per_cta;
    plan->pixels_per_thread = info.pixels_per_thread;
    plan->tile_pixels = info.tile_pixels;
    plan->ctas = info.ctas;
    plan->ctas_half_block = info.ctas_half_block;
    plan->pixels_per_cta = info.pixels_per_cta;
    plan->pixels_per_cta_half_block = info.pixels_per_cta_half_block;
    plan->shared_bytes = info.shared_bytes;
    return LCE_OK;
}

extern "C" lce_status lce_bconv2d(const lce_bconv2d_desc *desc, const uint32_t *input, const uint32_t *weights,
                                  const float *multiplier, const float *bias, const int32_t *thresholds,
                                  void *output, void *stream)
{
    using namespace lce;
    ConvGeom g;
    lce_status st = check_conv_args(desc, &g, input, weights, multiplier, bias, thresholds, output);
    if (st != LCE_OK) return st;
    if (!aligned(input, 4) || !aligned(weights, 4) || !aligned(output, 4) ||
        (multiplier && !aligned(multiplier, 4)) || (bias && !aligned(bias, 4)) ||
        (thresholds && !aligned(thresholds, 4)))
        return LCE_ERR_ALIGNMENT;
    return dispatch(desc, g, input, weights, multiplier, bias, thresholds, output, static_cast<cudaStream_t>(stream));
}

// ---- plan objects: the checks of lce_bconv2d once, the launch many times ---------------------------
struct lce_plan {
    lce_bconv2d_desc desc;
    lce::ConvGeom geom;
    const uint32_t *input, *weights;
    const float *multiplier, *bias;
    const int32_t *thresholds;
    void *output;
};

extern "C" lce_status lce_bconv2d_plan_create(const lce_bconv2d_desc *desc, const uint32_t *input, const uint32_t *weights,
                                              const float *multiplier, const float *bias, const int32_t *thresholds,
                                              void *output, lce_plan **plan)
{
    using namespace lce;
    if (!plan) return LCE_ERR_INVALID_ARG;
    *plan = nullptr;
    ConvGeom g;
    lce_status st = check_conv_args(desc, &g, input, weights, multiplier, bias, thresholds, output);
    if (st != LCE_OK) return st;
    if (!aligned(input, 4) || !aligned(weights, 4) || !aligned(output, 4) ||
        (multiplier && !aligned(multiplier, 4)) || (bias && !aligned(bias, 4)) ||
        (thresholds && !aligned(thresholds, 4)))
        return LCE_ERR_ALIGNMENT;
    lce_bconv2d_plan_info info;
    st = lce_bconv2d_plan(desc, &info);  // is there a kernel for this shape (and for a forced kernel choice)?
    if (st != LCE_OK) return st;
    lce_plan *h = new (std::nothrow) lce_plan;
    if (!h) return LCE_ERR_CUDA;
    h->desc = *desc;
    h->geom = g;
    h->input = input; h->weights = weights; h->multiplier = multiplier; h->bias = bias; h->thresholds = thresholds;
    h->output = output;
    *plan = h;
    return LCE_OK;
}

extern "C" lce_status lce_plan_run(const lce_plan *plan, void *stream)
{
    if (!plan) return LCE_ERR_INVALID_ARG;
    return lce::dispatch(&plan->desc, plan->geom, plan->input, plan->weights, plan->multiplier, plan->bias, plan->thresholds,
                         plan->output, static_cast<cudaStream_t>(stream));
}

extern "C" void lce_plan_destroy(lce_plan *plan) { delete plan; }

extern "C" lce_status lce_bconv2d_fused(const lce_bconv2d_desc *desc, const uint32_t *input, const uint32_t *weights,
                                        const float *multiplier, const float *bias, const float *residual,
                                        float *out_float, uint32_t *out_packed, void *stream)
{
    using namespace lce;
    ConvGeom g;
    lce_status st = make_geom(desc, &g);
    if (st != LCE_OK) return st;
    if (g.out_type != LCE_OUT_FLOAT32) return LCE_ERR_INVALID_ARG;
    if (!input || !weights || !multiplier || !bias || (!out_float && !out_packed)) return LCE_ERR_INVALID_ARG;
    if (!aligned(input, 4) || !aligned(weights, 4) || !aligned(multiplier, 4) || !aligned(bias, 4) ||
        !aligned(residual, 4) || !aligned(out_float, 4) || !aligned(out_packed, 4))
        return LCE_ERR_ALIGNMENT;
    const uint32_t *image = nullptr;
    if (desc->weights_packed) {
        if (!aligned(weights, 256)) return LCE_ERR_ALIGNMENT;
        if (tiled_weight_image_bytes(g) > 0)
            image = reinterpret_cast<const uint32_t *>(reinterpret_cast<const char *>(weights) + plain_weight_bytes(g));
    }
    if (desc->kernel == LCE_KERNEL_DIRECT || patch_covers(g)) return LCE_ERR_UNSUPPORTED;
    return launch_bconv_tiled(g, input, weights, image, multiplier, bias, nullptr, out_float,
                              static_cast<cudaStream_t>(stream), residual, out_packed);
}

extern "C" lce_status lce_bconv2d_f32(const lce_bconv2d_desc *desc, const float *input, const uint32_t *weights,
                                      const float *multiplier, const float *bias, const int32_t *thresholds,
                                      void *output, void *stream)
{
    using namespace lce;
    ConvGeom g;
    lce_status st = check_conv_args(desc, &g, input, weights, multiplier, bias, thresholds, output);
    if (st != LCE_OK) return st;
    if (!aligned(input, 4) || !aligned(weights, 4) || !aligned(output, 4) ||
        (multiplier && !aligned(multiplier, 4)) || (bias && !aligned(bias, 4)) ||
        (thresholds && !aligned(thresholds, 4)))
        return LCE_ERR_ALIGNMENT;
    const uint32_t *image = nullptr;
    if (desc->weights_packed) {
        if (!aligned(weights, 256)) return LCE_ERR_ALIGNMENT;
        if (tiled_weight_image_bytes(g) > 0)
            image = reinterpret_cast<const uint32_t *>(reinterpret_cast<const char *>(weights) + plain_weight_bytes(g));
    }
    if (desc->kernel == LCE_KERNEL_DIRECT || desc->kernel == LCE_KERNEL_TENSOR) return LCE_ERR_UNSUPPORTED;
    return launch_bconv_tiled(g, nullptr, weights, image, multiplier, bias, thresholds, output,
                              static_cast<cudaStream_t>(stream), nullptr, nullptr, input);
}

extern "C" size_t lce_bconv2d_packed_weights_bytes(const lce_bconv2d_desc *desc)
{
    lce::ConvGeom g;
    if (lce::make_geom(desc, &g) != LCE_OK) return 0;
    return lce::plain_weight_bytes(g) + lce::tiled_weight_image_bytes(g);
}

extern "C" lce_status lce_bconv2d_pack_weights(const lce_bconv2d_desc *desc, const uint32_t *weights, void *packed,
                                               void *stream)
{
    using namespace lce;
    ConvGeom g;
    lce_status st = make_geom(desc, &g);
    if (st != LCE_OK) return st;
    if (!weights || !packed) return LCE_ERR_INVALID_ARG;
    if (!aligned(weights, 4) || !aligned(packed, 256)) return LCE_ERR_ALIGNMENT;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const size_t plain = (size_t)g.Cout * g.KH * g.KW * g.Cw * 4;
    if (cudaMemcpyAsync(packed, weights, plain, cudaMemcpyDeviceToDevice, s) != cudaSuccess) return LCE_ERR_CUDA;
    if (tiled_weight_image_bytes(g) == 0) return LCE_OK;
    return launch_pack_weights_tiled(g, weights, reinterpret_cast<uint32_t *>(static_cast<char *>(packed) + plain_weight_bytes(g)), s);
}

extern "C" size_t lce_bconv2d_host_workspace_bytes(const lce_bconv2d_desc *desc)
{
    lce::ConvGeom g;
    if (lce::make_geom(desc, &g) != LCE_OK) return 0;
    return lce::host_layout(g).total;
}

namespace lce {
namespace {
lce_status host_conv(const lce_bconv2d_desc *desc, const uint32_t *input, const uint32_t *weights, const float *multiplier,
                     const float *bias, const int32_t *thresholds, void *output, void *workspace, size_t workspace_bytes,
                     void *stream, bool synchronise)
{
    ConvGeom g;
    lce_status st = check_conv_args(desc, &g, input, weights, multiplier, bias, thresholds, output);
    if (st != LCE_OK) return st;
    if (!workspace || desc->weights_packed) return LCE_ERR_INVALID_ARG;
    if (!aligned(workspace, 256)) return LCE_ERR_ALIGNMENT;
    const HostLayout L = host_layout(g);
    if (workspace_bytes < L.total) return LCE_ERR_WORKSPACE;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    char *ws = static_cast<char *>(workspace);
    bool ok = cudaMemcpyAsync(ws + L.in, input, L.in_bytes, cudaMemcpyHostToDevice, s) == cudaSuccess;
    ok = ok && cudaMemcpyAsync(ws + L.w, weights, L.w_bytes, cudaMemcpyHostToDevice, s) == cudaSuccess;
    if (multiplier) ok = ok && cudaMemcpyAsync(ws + L.mult, multiplier, L.ch_bytes, cudaMemcpyHostToDevice, s) == cudaSuccess;
    if (bias) ok = ok && cudaMemcpyAsync(ws + L.bias, bias, L.ch_bytes, cudaMemcpyHostToDevice, s) == cudaSuccess;
    if (thresholds) ok = ok && cudaMemcpyAsync(ws + L.thr, thresholds, L.ch_bytes, cudaMemcpyHostToDevice, s) == cudaSuccess;
    if (!ok) return LCE_ERR_CUDA;
    st = dispatch(desc, g, reinterpret_cast<const uint32_t *>(ws + L.in), reinterpret_cast<const uint32_t *>(ws + L.w),
                  multiplier ? reinterpret_cast<const float *>(ws + L.mult) : nullptr,
                  bias ? reinterpret_cast<const float *>(ws + L.bias) : nullptr,
                  thresholds ? reinterpret_cast<const int32_t *>(ws + L.thr) : nullptr, ws + L.out, s);
    if (st != LCE_OK) return st;
    if (cudaMemcpyAsync(output, ws + L.out, L.out_bytes, cudaMemcpyDeviceToHost, s) != cudaSuccess) return LCE_ERR_CUDA;
    if (synchronise && cudaStreamSynchronize(s) != cudaSuccess) return LCE_ERR_CUDA;
    return LCE_OK;
}
}  // namespace
}  // namespace lce

extern "C" lce_status lce_bconv2d_host(const lce_bconv2d_desc *desc, const uint32_t *input, const uint32_t *weights,
                                       const float *multiplier, const float *bias, const int32_t *thresholds,
                                       void *output, void *workspace, size_t workspace_bytes, void *stream)
{
    return lce::host_conv(desc, input, weights, multiplier, bias, thresholds, output, workspace, workspace_bytes, stream, true);
}

extern "C" lce_status lce_bconv2d_host_async(const lce_bconv2d_desc *desc, const uint32_t *input, const uint32_t *weights,
                                             const float *multiplier, const float *bias, const int32_t *thresholds,
                                             void *output, void *workspace, size_t workspace_bytes, void *stream)
{
    return lce::host_conv(desc, input, weights, multiplier, bias, thresholds, output, workspace, workspace_bytes, stream, false);
}

// ---- host-buffer convolution that allocates nothing ---------------------------------------------
// Some callers cannot give lce_bconv2d_host the device workspace it asks for, because they are not
// in a position to call cudaMalloc at all: code running inside a memory-capped or allocator-less
// host process, a real-time loop that must not take the allocator's locks, a plug-in that is only
// handed host tensors.  For them the staging area lives inside the library itself, as a
// file-scope device array that every GPU loading the library carries until the process exits.

#define LCE_STATIC_WORKSPACE_BYTES (8u << 20)

static __device__ __align__(256) unsigned char g_static_workspace[LCE_STATIC_WORKSPACE_BYTES];

namespace lce {
namespace {

constexpr int kMaxDevices = 64;
void *g_static_workspace_addr[kMaxDevices];  // device address of g_static_workspace, per device; 0 = not looked up yet

}  // namespace
}  // namespace lce

extern "C" size_t lce_bconv2d_host_noalloc_max_bytes(void) { return LCE_STATIC_WORKSPACE_BYTES; }

extern "C" lce_status lce_bconv2d_host_noalloc(const lce_bconv2d_desc *desc, const uint32_t *input,
                                               const uint32_t *weights, const float *multiplier, const float *bias,
                                               const int32_t *thresholds, void *output, void *stream)
{
    using namespace lce;
    ConvGeom g;
    lce_status st = check_conv_args(desc, &g, input, weights, multiplier, bias, thresholds, output);
    if (st != LCE_OK) return st;
    if (desc->weights_packed) return LCE_ERR_INVALID_ARG;
    const HostLayout L = host_layout(g);
    if (L.total > LCE_STATIC_WORKSPACE_BYTES) return LCE_ERR_WORKSPACE;  // this call does not fit the built-in array

    // In host code the array's name is only a stand-in for the symbol, not a device address: ask the
    // runtime for the address once per device, with that device current.
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return LCE_ERR_CUDA;
    if (g_static_workspace_addr[dev] == nullptr) {
        void *addr = nullptr;
        if (cudaGetSymbolAddress(&addr, g_static_workspace) != cudaSuccess || addr == nullptr) return LCE_ERR_CUDA;
        g_static_workspace_addr[dev] = addr;
    }
    char *ws = static_cast<char *>(g_static_workspace_addr[dev]);

    // Nothing in the array has to start at zero: every region is written in full (by the copies in,
    // or by the kernel) before anything reads it.
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    bool ok = cudaMemcpyAsync(ws + L.in, input, L.in_bytes, cudaMemcpyHostToDevice, s) == cudaSuccess;
    ok = ok && cudaMemcpyAsync(ws + L.w, weights, L.w_bytes, cudaMemcpyHostToDevice, s) == cudaSuccess;
    if (multiplier) ok = ok && cudaMemcpyAsync(ws + L.mult, multiplier, L.ch_bytes, cudaMemcpyHostToDevice, s) == cudaSuccess;
    if (bias) ok = ok && cudaMemcpyAsync(ws + L.bias, bias, L.ch_bytes, cudaMemcpyHostToDevice, s) == cudaSuccess;
    if (thresholds) ok = ok && cudaMemcpyAsync(ws + L.thr, thresholds, L.ch_bytes, cudaMemcpyHostToDevice, s) == cudaSuccess;
    if (!ok) return LCE_ERR_CUDA;
    st = dispatch(desc, g, reinterpret_cast<const uint32_t *>(ws + L.in), reinterpret_cast<const uint32_t *>(ws + L.w),
                  multiplier ? reinterpret_cast<const float *>(ws + L.mult) : nullptr,
                  bias ? reinterpret_cast<const float *>(ws + L.bias) : nullptr,
                  thresholds ? reinterpret_cast<const int32_t *>(ws + L.thr) : nullptr, ws + L.out, s);
    if (st != LCE_OK) return st;
    if (cudaMemcpyAsync(output, ws + L.out, L.out_bytes, cudaMemcpyDeviceToHost, s) != cudaSuccess) return LCE_ERR_CUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) return LCE_ERR_CUDA;
    return LCE_OK;
}
