// C ABI front: version/status strings, shape query and the LceBConv2d dispatch (device- and
// host-buffer forms).  All argument checks happen here, before anything is launched.
#include "common.cuh"

#include <atomic>
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

// A packed-weights buffer = [plain words][operand image of the tiled XOR/POPC kernel][operand image of
// the tensor-core kernel], each part rounded up to 256 bytes; a part a kernel does not cover is empty.
struct WeightViews {
    const uint32_t *plain;
    const uint32_t *tiled;
    const void *tensor;
};

lce_status weight_views(const lce_bconv2d_desc *desc, const ConvGeom &g, const uint32_t *weights, WeightViews *v)
{
    v->plain = weights;
    v->tiled = nullptr;
    v->tensor = nullptr;
    if (!desc->weights_packed) return LCE_OK;
    if (!aligned(weights, 256)) return LCE_ERR_ALIGNMENT;
    const char *base = reinterpret_cast<const char *>(weights);
    size_t off = plain_weight_bytes(g);
    const size_t tiled = tiled_weight_image_bytes(g), tensor = tensor_weight_image_bytes(g);
    if (tiled > 0) v->tiled = reinterpret_cast<const uint32_t *>(base + off);
    off += round_up(tiled, 256);
    if (tensor > 0) v->tensor = base + off;
    return LCE_OK;
}

// The tiled kernels write float / int32 rows with 128-bit accesses when the channel count allows it,
// and then need 16-byte aligned buffers.
bool tiled_accepts(const ConvGeom &g, const void *out, const void *residual)
{
    return !((g.Cout & 3) == 0 && g.out_type != LCE_OUT_BITPACKED && (!aligned(out, 16) || !aligned(residual, 16)));
}

// AUTO takes the tensor-core kernel when the weights were packed at load time (its operand image exists)
// and the layer is large enough to pay for that kernel's start-up, by what was measured on the paper's
// layer sweep (batch 1 and 64) and the ImageNet-shaped bodies: from 2^28 binary MACs when all taps of a channel
// block stay in shared memory, from 2^29 when they have to stream past once per tile; 3x3 and smaller filters
// on at most 32 input channels (half of every 64-deep MMA is padding) only from 2^31, where the two kernels
// draw level (the 112x112x32 stride-2 layer of an ImageNet stem, 2^34 MACs, is twice as fast on the tensor cores).
bool tensor_preferred(const ConvGeom &g)
{
    if (patch_covers(g)) return false;
    TensorPlanInfo t{};
    if (tensor_plan_info(g, &t) != LCE_OK) return false;
    const double macs = (double)g.M * g.Cout * g.KH * g.KW * g.Cin;
    if (g.Cin <= 32 && g.KH * g.KW <= 9) return macs >= 2147483648.0;
    return macs >= (t.weights_resident ? 268435456.0 : 536870912.0);
}

enum KernelPick { PICK_NONE = 0, PICK_DIRECT, PICK_PATCH, PICK_TILED, PICK_TENSOR };

// One place decides which kernel a call gets; lce_bconv2d_plan shows the same decision.
KernelPick pick_kernel(const lce_bconv2d_desc *desc, const ConvGeom &g, bool have_tensor_image, bool tiled_buffers_ok)
{
    TiledPlanInfo info{};
    switch (desc->kernel) {
        case LCE_KERNEL_DIRECT: return PICK_DIRECT;
        case LCE_KERNEL_TENSOR: return have_tensor_image && tensor_covers(g) ? PICK_TENSOR : PICK_NONE;
        case LCE_KERNEL_TILED:
            if (patch_covers(g)) return PICK_PATCH;
            return tiled_buffers_ok && tiled_plan_info(g, &info) == LCE_OK ? PICK_TILED : PICK_NONE;
        default: break;
    }
    if (have_tensor_image && tensor_preferred(g) && tensor_covers(g)) return PICK_TENSOR;
    if (patch_covers(g)) return PICK_PATCH;
    if (tiled_buffers_ok && tiled_plan_info(g, &info) == LCE_OK) return PICK_TILED;
    return PICK_DIRECT;
}

lce_status dispatch(const lce_bconv2d_desc *desc, const ConvGeom &g, const uint32_t *input, const uint32_t *weights,
                    const float *multiplier, const float *bias, const int32_t *thresholds, void *output,
                    cudaStream_t s)
{
    if (tensor_timeout_flagged()) return LCE_ERR_DEVICE_TIMEOUT;  // an earlier kernel on this device gave up a wait
    WeightViews v;
    lce_status st = weight_views(desc, g, weights, &v);
    if (st != LCE_OK) return st;
    switch (pick_kernel(desc, g, v.tensor != nullptr, tiled_accepts(g, output, nullptr))) {
        case PICK_DIRECT: return launch_bconv_direct(g, input, v.plain, multiplier, bias, thresholds, output, s);
        case PICK_PATCH: return launch_bconv_patch(g, input, v.plain, multiplier, bias, thresholds, output, s);
        case PICK_TILED: return launch_bconv_tiled(g, input, v.plain, v.tiled, multiplier, bias, thresholds, output, s);
        case PICK_TENSOR: return launch_bconv_tensor(g, input, v.tensor, multiplier, bias, thresholds, output, s);
        default: return LCE_ERR_UNSUPPORTED;
    }
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

extern "C" lce_status lce_device_status_reset(void) { return lce::tensor_device_status_reset(); }

extern "C" lce_status lce_device_wait_probe(uint64_t limit_ns, void *stream)
{
    if (limit_ns == 0 || limit_ns > 1000000000ull) return LCE_ERR_INVALID_ARG;  // at most a second
    return lce::tensor_wait_probe(limit_ns, static_cast<cudaStream_t>(stream));
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
    // the decision dispatch() makes, for 16-byte aligned buffers
    const bool have_tensor_image = desc->weights_packed && tensor_weight_image_bytes(g) > 0;
    switch (pick_kernel(desc, g, have_tensor_image, true)) {
        case PICK_DIRECT: plan->kernel = LCE_KERNEL_DIRECT; return LCE_OK;
        case PICK_PATCH: plan->kernel = LCE_KERNEL_TILED; plan->patch = 1; return LCE_OK;
        case PICK_TENSOR: {
            TensorPlanInfo t{};
            st = tensor_plan_info(g, &t);
            if (st != LCE_OK) return st;
            plan->kernel = LCE_KERNEL_TENSOR;
            plan->tile_pixels = t.tile_positions;
            plan->ctas = t.ctas;
            plan->weight_stages = t.weight_stages;
            plan->weights_resident = t.weights_resident;
            plan->shared_bytes = t.shared_bytes;
            return LCE_OK;
        }
        case PICK_TILED: break;
        default: return LCE_ERR_UNSUPPORTED;
    }
    TiledPlanInfo info{};
    st = tiled_plan_info(g, &info);
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
    // is there a kernel for this shape, these buffers and a forced kernel choice?  (A float / int32 output
    // that is only 4-byte aligned rules the tiled kernel out: AUTO then records the direct kernel, a
    // forced LCE_KERNEL_TILED fails here rather than at every run.)
    WeightViews v;
    st = weight_views(desc, g, weights, &v);
    if (st != LCE_OK) return st;
    if (pick_kernel(desc, g, v.tensor != nullptr, tiled_accepts(g, output, nullptr)) == PICK_NONE) return LCE_ERR_UNSUPPORTED;
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
    if (tensor_timeout_flagged()) return LCE_ERR_DEVICE_TIMEOUT;
    WeightViews v;
    st = weight_views(desc, g, weights, &v);
    if (st != LCE_OK) return st;
    if (desc->kernel == LCE_KERNEL_DIRECT || patch_covers(g)) return LCE_ERR_UNSUPPORTED;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // the tensor-core kernel fuses the same neighbours when whole 32-channel words and 16-byte rows allow it
    const bool tensor_ok = v.tensor && tensor_covers(g) && (g.Cout & 31) == 0 && aligned(out_float, 16) && aligned(residual, 16);
    if (desc->kernel == LCE_KERNEL_TENSOR && !tensor_ok) return LCE_ERR_UNSUPPORTED;
    if (tensor_ok && (desc->kernel == LCE_KERNEL_TENSOR || (desc->kernel == LCE_KERNEL_AUTO && tensor_preferred(g))))
        return launch_bconv_tensor(g, input, v.tensor, multiplier, bias, nullptr, out_float, s, residual, out_packed);
    return launch_bconv_tiled(g, input, v.plain, v.tiled, multiplier, bias, nullptr, out_float, s, residual, out_packed);
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
    WeightViews v;
    st = weight_views(desc, g, weights, &v);
    if (st != LCE_OK) return st;
    if (desc->kernel == LCE_KERNEL_DIRECT || desc->kernel == LCE_KERNEL_TENSOR) return LCE_ERR_UNSUPPORTED;
    return launch_bconv_tiled(g, nullptr, v.plain, v.tiled, multiplier, bias, thresholds, output,
                              static_cast<cudaStream_t>(stream), nullptr, nullptr, input);
}

extern "C" size_t lce_bconv2d_packed_weights_bytes(const lce_bconv2d_desc *desc)
{
    lce::ConvGeom g;
    if (lce::make_geom(desc, &g) != LCE_OK) return 0;
    return lce::plain_weight_bytes(g) + lce::round_up(lce::tiled_weight_image_bytes(g), 256) + lce::tensor_weight_image_bytes(g);
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
    size_t off = plain_weight_bytes(g);
    const size_t tiled = tiled_weight_image_bytes(g), tensor = tensor_weight_image_bytes(g);
    if (tiled > 0) {
        st = launch_pack_weights_tiled(g, weights, reinterpret_cast<uint32_t *>(static_cast<char *>(packed) + off), s);
        if (st != LCE_OK) return st;
    }
    off += round_up(tiled, 256);
    if (tensor > 0) return launch_pack_weights_tensor(g, weights, static_cast<char *>(packed) + off, s);
    return LCE_OK;
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
std::atomic<void *> g_static_workspace_addr[kMaxDevices];  // device address of g_static_workspace, per device; null = not looked up yet

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
    if (host_layout(g).total > LCE_STATIC_WORKSPACE_BYTES) return LCE_ERR_WORKSPACE;  // this call does not fit the built-in array

    // In host code the array's name is only a stand-in for the symbol, not a device address: ask the
    // runtime for the address once per device, with that device current.  (Two threads making the
    // first call together both look it up and store the same value.)
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return LCE_ERR_CUDA;
    void *addr = g_static_workspace_addr[dev].load(std::memory_order_acquire);
    if (addr == nullptr) {
        if (cudaGetSymbolAddress(&addr, g_static_workspace) != cudaSuccess || addr == nullptr) return LCE_ERR_CUDA;
        g_static_workspace_addr[dev].store(addr, std::memory_order_release);
    }
    // Nothing in the array has to start at zero: every region is written in full (by the copies in,
    // or by the kernel) before anything reads it.  From here on this is lce_bconv2d_host on that array.
    return host_conv(desc, input, weights, multiplier, bias, thresholds, output, addr, LCE_STATIC_WORKSPACE_BYTES, stream, true);
}
