"""ctypes binding of include/lce.h.  Argument marshalling only."""
from __future__ import annotations

import ctypes
from pathlib import Path
from typing import Optional, Tuple

import torch

_LIB_PATH = Path(__file__).resolve().parent / "liblce_b200.so"

PAD_VALID, PAD_SAME_ONE, PAD_SAME_ZERO = 0, 1, 2
OUT_FLOAT32, OUT_BITPACKED, OUT_INT32 = 0, 1, 2
ACT_NONE, ACT_RELU = 0, 1
KERNEL_AUTO, KERNEL_DIRECT, KERNEL_TILED, KERNEL_TENSOR = 0, 1, 2, 3


class LceError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {lce_status_string(status)} (lce_status {status})")


class BConv2dDesc(ctypes.Structure):
    """Mirror of lce_bconv2d_desc."""
    _fields_ = [(n, ctypes.c_int32) for n in (
        "batch", "in_h", "in_w", "in_c", "out_c", "kernel_h", "kernel_w", "stride_h", "stride_w",
        "padding", "out_type", "activation", "kernel", "weights_packed")]


_lib = None


def library() -> ctypes.CDLL:
    """Loads liblce_b200.so (built by paper_2011_09398_b200.build); raises if it is missing."""
    global _lib
    if _lib is None:
        if not _LIB_PATH.exists():
            raise ImportError(f"{_LIB_PATH} is missing: run `python -m paper_2011_09398_b200.build` "
                              "(there is no fallback path)")
        lib = ctypes.CDLL(str(_LIB_PATH))
        vp, i32, i64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64
        lib.lce_version.restype = ctypes.c_char_p
        lib.lce_status_string.restype = ctypes.c_char_p
        lib.lce_status_string.argtypes = [ctypes.c_int]
        lib.lce_bitpack.argtypes = [vp, vp, i64, i32, vp]
        lib.lce_unpack.argtypes = [vp, vp, i64, i32, vp]
        lib.lce_bconv2d_out_shape.argtypes = [ctypes.POINTER(BConv2dDesc), ctypes.POINTER(i32), ctypes.POINTER(i32)]
        lib.lce_bconv2d.argtypes = [ctypes.POINTER(BConv2dDesc), vp, vp, vp, vp, vp, vp, vp]
        lib.lce_bconv2d_f32.argtypes = [ctypes.POINTER(BConv2dDesc), vp, vp, vp, vp, vp, vp, vp]
        lib.lce_bconv2d_f32.restype = ctypes.c_int
        lib.lce_bconv2d_fused.argtypes = [ctypes.POINTER(BConv2dDesc), vp, vp, vp, vp, vp, vp, vp, vp]
        lib.lce_bconv2d_fused.restype = ctypes.c_int
        lib.lce_bconv2d_packed_weights_bytes.restype = ctypes.c_size_t
        lib.lce_bconv2d_packed_weights_bytes.argtypes = [ctypes.POINTER(BConv2dDesc)]
        lib.lce_bconv2d_pack_weights.argtypes = [ctypes.POINTER(BConv2dDesc), vp, vp, vp]
        lib.lce_bconv2d_host_workspace_bytes.restype = ctypes.c_size_t
        lib.lce_bconv2d_host_workspace_bytes.argtypes = [ctypes.POINTER(BConv2dDesc)]
        lib.lce_bconv2d_host.argtypes = [ctypes.POINTER(BConv2dDesc), vp, vp, vp, vp, vp, vp, vp, ctypes.c_size_t, vp]
        lib.lce_bconv2d_host_async.argtypes = [ctypes.POINTER(BConv2dDesc), vp, vp, vp, vp, vp, vp, vp, ctypes.c_size_t, vp]
        lib.lce_bconv2d_host_async.restype = ctypes.c_int
        lib.lce_bconv2d_host_noalloc_max_bytes.restype = ctypes.c_size_t
        lib.lce_bconv2d_host_noalloc_max_bytes.argtypes = []
        lib.lce_bconv2d_host_noalloc.argtypes = [ctypes.POINTER(BConv2dDesc), vp, vp, vp, vp, vp, vp, vp]
        lib.lce_bconv2d_host_noalloc.restype = ctypes.c_int
        lib.lce_bconv2d_plan_create.argtypes = [ctypes.POINTER(BConv2dDesc), vp, vp, vp, vp, vp, vp, ctypes.POINTER(vp)]
        lib.lce_bconv2d_plan_create.restype = ctypes.c_int
        lib.lce_plan_run.argtypes = [vp, vp]
        lib.lce_plan_run.restype = ctypes.c_int
        lib.lce_plan_destroy.argtypes = [vp]
        lib.lce_plan_destroy.restype = None
        lib.lce_bmaxpool.argtypes = [vp, vp] + [i32] * 9 + [vp]
        lib.lce_add_f32.argtypes = [vp, vp, vp, i64, vp]
        for name in ("lce_bitpack", "lce_unpack", "lce_bconv2d_out_shape", "lce_bconv2d", "lce_bconv2d_host",
                     "lce_bconv2d_pack_weights",
                     "lce_bmaxpool", "lce_add_f32"):
            getattr(lib, name).restype = ctypes.c_int
        _lib = lib
    return _lib


def lce_version() -> str:
    return library().lce_version().decode()


def lce_status_string(status: int) -> str:
    return library().lce_status_string(int(status)).decode()


def _check(status: int, where: str) -> None:
    if status != 0:
        raise LceError(status, where)


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _dev(t: torch.Tensor, dtype, name: str) -> int:
    if not t.is_cuda:
        raise ValueError(f"{name} must be a CUDA tensor (there is no CPU path)")
    if t.dtype != dtype or not t.is_contiguous():
        raise ValueError(f"{name} must be contiguous {dtype}")
    return t.data_ptr()


def _words(c: int) -> int:
    return (c + 31) // 32


def make_desc(batch, in_h, in_w, in_c, out_c, kernel=(3, 3), stride=(1, 1), padding=PAD_SAME_ONE,
              out_type=OUT_FLOAT32, activation=ACT_NONE, kernel_choice=KERNEL_AUTO, weights_packed=0) -> BConv2dDesc:
    return BConv2dDesc(batch, in_h, in_w, in_c, out_c, kernel[0], kernel[1], stride[0], stride[1],
                       padding, out_type, activation, kernel_choice, weights_packed)


def lce_bconv2d_out_shape(desc: BConv2dDesc) -> Tuple[int, int]:
    oh, ow = ctypes.c_int32(), ctypes.c_int32()
    _check(library().lce_bconv2d_out_shape(ctypes.byref(desc), ctypes.byref(oh), ctypes.byref(ow)), "lce_bconv2d_out_shape")
    return oh.value, ow.value


def lce_bitpack(x: torch.Tensor, out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """LceQuantize: fp32 [..., C] -> int32-typed words [..., ceil(C/32)] (bit pattern of uint32)."""
    C = x.shape[-1]
    rows = x.numel() // C if C else 0
    if out is None:
        out = torch.empty(x.shape[:-1] + (_words(C),), dtype=torch.int32, device=x.device)
    _check(library().lce_bitpack(_dev(x, torch.float32, "x"), _dev(out, torch.int32, "out"), rows, C, _stream()), "lce_bitpack")
    return out


def lce_unpack(words: torch.Tensor, channels: int, out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """LceDequantize: words [..., ceil(C/32)] -> fp32 [..., C] of +-1.0."""
    rows = words.numel() // _words(channels)
    if out is None:
        out = torch.empty(words.shape[:-1] + (channels,), dtype=torch.float32, device=words.device)
    _check(library().lce_unpack(_dev(words, torch.int32, "words"), _dev(out, torch.float32, "out"), rows, channels, _stream()), "lce_unpack")
    return out


def pack_weights(w_ohwi: torch.Tensor) -> torch.Tensor:
    """Binary weight compression: fp32/int8 +-1 weights [Cout,KH,KW,Cin] -> words [Cout,KH,KW,ceil(Cin/32)]
    by the same LceQuantize kernel (a load-time step)."""
    return lce_bitpack(w_ohwi.to(torch.float32).contiguous())


def lce_bconv2d(desc: BConv2dDesc, input: torch.Tensor, weights: torch.Tensor,
                multiplier: Optional[torch.Tensor] = None, bias: Optional[torch.Tensor] = None,
                thresholds: Optional[torch.Tensor] = None, out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """LceBConv2d on packed words; allocates `out` with torch when not given."""
    oh, ow = lce_bconv2d_out_shape(desc)
    if out is None:
        if desc.out_type == OUT_FLOAT32:
            out = torch.empty((desc.batch, oh, ow, desc.out_c), dtype=torch.float32, device=input.device)
        elif desc.out_type == OUT_BITPACKED:
            out = torch.empty((desc.batch, oh, ow, _words(desc.out_c)), dtype=torch.int32, device=input.device)
        else:
            out = torch.empty((desc.batch, oh, ow, desc.out_c), dtype=torch.int32, device=input.device)
    expect_in = desc.batch * desc.in_h * desc.in_w * _words(desc.in_c)
    expect_w = desc.out_c * desc.kernel_h * desc.kernel_w * _words(desc.in_c)
    if desc.weights_packed:
        expect_w = lce_bconv2d_packed_weights_bytes(desc) // 4
    if input.numel() != expect_in or weights.numel() != expect_w:
        raise ValueError("input / weights size does not match the descriptor")
    out_dtype = torch.float32 if desc.out_type == OUT_FLOAT32 else torch.int32
    _check(library().lce_bconv2d(
        ctypes.byref(desc), _dev(input, torch.int32, "input"), _dev(weights, torch.int32, "weights"),
        _dev(multiplier, torch.float32, "multiplier") if multiplier is not None else None,
        _dev(bias, torch.float32, "bias") if bias is not None else None,
        _dev(thresholds, torch.int32, "thresholds") if thresholds is not None else None,
        _dev(out, out_dtype, "out"), _stream()), "lce_bconv2d")
    return out


def lce_bconv2d_f32(desc: BConv2dDesc, input: torch.Tensor, weights: torch.Tensor,
                    multiplier: Optional[torch.Tensor] = None, bias: Optional[torch.Tensor] = None,
                    thresholds: Optional[torch.Tensor] = None, out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """LceQuantize + LceBConv2d in one kernel: `input` is the fp32 tensor [batch][in_h][in_w][in_c]."""
    oh, ow = lce_bconv2d_out_shape(desc)
    if out is None:
        last = _words(desc.out_c) if desc.out_type == OUT_BITPACKED else desc.out_c
        out = torch.empty((desc.batch, oh, ow, last), dtype=torch.float32 if desc.out_type == OUT_FLOAT32 else torch.int32,
                          device=input.device)
    expect_w = desc.out_c * desc.kernel_h * desc.kernel_w * _words(desc.in_c)
    if desc.weights_packed:
        expect_w = lce_bconv2d_packed_weights_bytes(desc) // 4
    if input.numel() != desc.batch * desc.in_h * desc.in_w * desc.in_c or weights.numel() != expect_w:
        raise ValueError("input / weights size does not match the descriptor")
    out_dtype = torch.float32 if desc.out_type == OUT_FLOAT32 else torch.int32
    _check(library().lce_bconv2d_f32(
        ctypes.byref(desc), _dev(input, torch.float32, "input"), _dev(weights, torch.int32, "weights"),
        _dev(multiplier, torch.float32, "multiplier") if multiplier is not None else None,
        _dev(bias, torch.float32, "bias") if bias is not None else None,
        _dev(thresholds, torch.int32, "thresholds") if thresholds is not None else None,
        _dev(out, out_dtype, "out"), _stream()), "lce_bconv2d_f32")
    return out


class BConv2dPlanInfo(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in ("kernel", "patch", "pointwise", "warps_per_cta", "pixels_per_thread", "tile_pixels",
                                               "ctas", "ctas_half_block", "pixels_per_cta", "pixels_per_cta_half_block")] + \
               [("shared_bytes", ctypes.c_int64), ("weight_stages", ctypes.c_int32), ("weights_resident", ctypes.c_int32)]


def lce_bconv2d_plan(desc: BConv2dDesc) -> dict:
    """The kernel and launch shape lce_bconv2d would use for `desc` (host arithmetic only)."""
    info = BConv2dPlanInfo()
    fn = library().lce_bconv2d_plan
    fn.argtypes = [ctypes.POINTER(BConv2dDesc), ctypes.POINTER(BConv2dPlanInfo)]
    fn.restype = ctypes.c_int
    _check(fn(ctypes.byref(desc), ctypes.byref(info)), "lce_bconv2d_plan")
    return {n: getattr(info, n) for n, _ in BConv2dPlanInfo._fields_}


class BConv2dPlan:
    """Handle of lce_bconv2d_plan_create; keeps the bound tensors alive.  `out` is the output tensor."""

    def __init__(self, handle: int, tensors, out: torch.Tensor):
        self.handle, self._tensors, self.out = handle, tensors, out


def lce_bconv2d_plan_create(desc: BConv2dDesc, input: torch.Tensor, weights: torch.Tensor,
                            multiplier: Optional[torch.Tensor] = None, bias: Optional[torch.Tensor] = None,
                            thresholds: Optional[torch.Tensor] = None, out: Optional[torch.Tensor] = None) -> BConv2dPlan:
    """lce_bconv2d bound to its buffers: all checks now, launches later with lce_plan_run."""
    oh, ow = lce_bconv2d_out_shape(desc)
    out_dtype = torch.float32 if desc.out_type == OUT_FLOAT32 else torch.int32
    if out is None:
        last = _words(desc.out_c) if desc.out_type == OUT_BITPACKED else desc.out_c
        out = torch.empty((desc.batch, oh, ow, last), dtype=out_dtype, device=input.device)
    handle = ctypes.c_void_p()
    _check(library().lce_bconv2d_plan_create(
        ctypes.byref(desc), _dev(input, torch.int32, "input"), _dev(weights, torch.int32, "weights"),
        _dev(multiplier, torch.float32, "multiplier") if multiplier is not None else None,
        _dev(bias, torch.float32, "bias") if bias is not None else None,
        _dev(thresholds, torch.int32, "thresholds") if thresholds is not None else None,
        _dev(out, out_dtype, "out"), ctypes.byref(handle)), "lce_bconv2d_plan_create")
    return BConv2dPlan(handle.value, (input, weights, multiplier, bias, thresholds), out)


def lce_plan_run(plan: BConv2dPlan) -> torch.Tensor:
    """Launches the planned convolution on torch's current stream; returns the plan's output tensor."""
    _check(library().lce_plan_run(plan.handle, _stream()), "lce_plan_run")
    return plan.out


def lce_plan_destroy(plan: BConv2dPlan) -> None:
    library().lce_plan_destroy(plan.handle)
    plan.handle = None


def lce_bconv2d_fused(desc: BConv2dDesc, input, weights, multiplier, bias, residual=None, out_float=None,
                      out_packed=None) -> None:
    """LceBConv2d (float output) with the shortcut add and/or the next LceQuantize fused in; the
    caller supplies whichever of out_float / out_packed it wants."""
    opt = lambda t, dt, n: _dev(t, dt, n) if t is not None else None
    _check(library().lce_bconv2d_fused(
        ctypes.byref(desc), _dev(input, torch.int32, "input"), _dev(weights, torch.int32, "weights"),
        _dev(multiplier, torch.float32, "multiplier"), _dev(bias, torch.float32, "bias"),
        opt(residual, torch.float32, "residual"), opt(out_float, torch.float32, "out_float"),
        opt(out_packed, torch.int32, "out_packed"), _stream()), "lce_bconv2d_fused")


def lce_bconv2d_packed_weights_bytes(desc: BConv2dDesc) -> int:
    return int(library().lce_bconv2d_packed_weights_bytes(ctypes.byref(desc)))


def lce_bconv2d_pack_weights(desc: BConv2dDesc, weights: torch.Tensor, out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Load-time weight packing; returns the packed buffer (int32 words) to pass as `weights`
    together with a descriptor whose weights_packed is 1."""
    nbytes = lce_bconv2d_packed_weights_bytes(desc)
    if out is None:
        out = torch.empty(nbytes // 4, dtype=torch.int32, device=weights.device)
    _check(library().lce_bconv2d_pack_weights(ctypes.byref(desc), _dev(weights, torch.int32, "weights"),
                                              _dev(out, torch.int32, "packed"), _stream()), "lce_bconv2d_pack_weights")
    return out


def lce_bconv2d_host_workspace_bytes(desc: BConv2dDesc) -> int:
    return int(library().lce_bconv2d_host_workspace_bytes(ctypes.byref(desc)))


def _host(t: Optional[torch.Tensor], dtype, name: str):
    if t is None:
        return None
    if t.is_cuda or t.dtype != dtype or not t.is_contiguous():
        raise ValueError(f"{name} must be a contiguous host {dtype} tensor")
    return t.data_ptr()


def lce_bconv2d_host(desc: BConv2dDesc, input, weights, multiplier, bias, thresholds, out, workspace: torch.Tensor) -> None:
    """Host-buffer form: all tensors on the host (pinned for asynchronous copies) except `workspace`
    (a CUDA uint8 tensor of at least lce_bconv2d_host_workspace_bytes(desc))."""
    out_dtype = torch.float32 if desc.out_type == OUT_FLOAT32 else torch.int32
    _check(library().lce_bconv2d_host(
        ctypes.byref(desc), _host(input, torch.int32, "input"), _host(weights, torch.int32, "weights"),
        _host(multiplier, torch.float32, "multiplier"), _host(bias, torch.float32, "bias"),
        _host(thresholds, torch.int32, "thresholds"), _host(out, out_dtype, "out"),
        _dev(workspace, torch.uint8, "workspace"), workspace.numel(), _stream()), "lce_bconv2d_host")


def lce_bconv2d_host_async(desc: BConv2dDesc, input, weights, multiplier, bias, thresholds, out, workspace: torch.Tensor) -> None:
    """lce_bconv2d_host that only enqueues its copies and kernel on the current stream; the caller
    synchronises the stream before touching `out` (or reusing `workspace`)."""
    out_dtype = torch.float32 if desc.out_type == OUT_FLOAT32 else torch.int32
    _check(library().lce_bconv2d_host_async(
        ctypes.byref(desc), _host(input, torch.int32, "input"), _host(weights, torch.int32, "weights"),
        _host(multiplier, torch.float32, "multiplier"), _host(bias, torch.float32, "bias"),
        _host(thresholds, torch.int32, "thresholds"), _host(out, out_dtype, "out"),
        _dev(workspace, torch.uint8, "workspace"), workspace.numel(), _stream()), "lce_bconv2d_host_async")


def lce_bconv2d_host_noalloc_max_bytes() -> int:
    return int(library().lce_bconv2d_host_noalloc_max_bytes())


def lce_bconv2d_host_noalloc(desc: BConv2dDesc, input, weights, multiplier, bias, thresholds, out) -> None:
    """lce_bconv2d_host without the workspace argument: for callers that cannot allocate device
    memory.  Every tensor is a host tensor; the staging area is a fixed array inside the library
    (shared by all calls on the device, so do not overlap calls)."""
    out_dtype = torch.float32 if desc.out_type == OUT_FLOAT32 else torch.int32
    _check(library().lce_bconv2d_host_noalloc(
        ctypes.byref(desc), _host(input, torch.int32, "input"), _host(weights, torch.int32, "weights"),
        _host(multiplier, torch.float32, "multiplier"), _host(bias, torch.float32, "bias"),
        _host(thresholds, torch.int32, "thresholds"), _host(out, out_dtype, "out"), _stream()), "lce_bconv2d_host_noalloc")


def lce_bmaxpool(words: torch.Tensor, channels: int, pool=(2, 2), stride=(2, 2), padding=PAD_VALID,
                 out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """LceBMaxPool2d on packed words [N,H,W,ceil(C/32)]."""
    N, H, W, Cw = words.shape
    if Cw != _words(channels):
        raise ValueError("last dimension does not match channels")

    def osz(size, k, s):
        if padding == PAD_VALID:
            return (size - k) // s + 1 if size >= k else 0
        return -(-size // s)

    if out is None:
        out = torch.empty((N, osz(H, pool[0], stride[0]), osz(W, pool[1], stride[1]), Cw), dtype=torch.int32, device=words.device)
    _check(library().lce_bmaxpool(_dev(words, torch.int32, "words"), _dev(out, torch.int32, "out"), N, H, W, channels,
                                  pool[0], pool[1], stride[0], stride[1], padding, _stream()), "lce_bmaxpool")
    return out


def lce_add_f32(a: torch.Tensor, b: torch.Tensor, out: Optional[torch.Tensor] = None) -> torch.Tensor:
    if out is None:
        out = torch.empty_like(a)
    if a.numel() != b.numel() or a.numel() != out.numel():
        raise ValueError("size mismatch")
    _check(library().lce_add_f32(_dev(a, torch.float32, "a"), _dev(b, torch.float32, "b"), _dev(out, torch.float32, "out"),
                                 a.numel(), _stream()), "lce_add_f32")
    return out


def lce_device_status() -> int:
    """0 unless a bounded device-side wait has given up on the current device."""
    v = ctypes.c_int32()
    lib = library()
    lib.lce_device_status.argtypes = [ctypes.POINTER(ctypes.c_int32)]
    lib.lce_device_status.restype = ctypes.c_int
    _check(lib.lce_device_status(ctypes.byref(v)), "lce_device_status")
    return v.value


def lce_device_status_reset() -> None:
    """Clears the status of the bounded device-side waits for the current device."""
    lib = library()
    lib.lce_device_status_reset.argtypes = []
    lib.lce_device_status_reset.restype = ctypes.c_int
    _check(lib.lce_device_status_reset(), "lce_device_status_reset")


def lce_device_wait_probe(limit_ns: int) -> None:
    """Launches the tiny kernel whose bounded wait is meant to run out (see lce.h); asynchronous."""
    lib = library()
    lib.lce_device_wait_probe.argtypes = [ctypes.c_uint64, ctypes.c_void_p]
    lib.lce_device_wait_probe.restype = ctypes.c_int
    _check(lib.lce_device_wait_probe(int(limit_ns), _stream()), "lce_device_wait_probe")
