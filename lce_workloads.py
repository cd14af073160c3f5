"""Seeded synthetic inputs and layer lists for the Bconv2D workloads.

This module serves both the CPU oracle's tests and the CUDA path's tests and
benchmark, and therefore holds none of the method's arithmetic: it draws random
tensors and names shapes, nothing else.  (Binarizing, packing, convolving and
thresholding all live on either side of the parity comparison, never here.)

Recipe (stand-in for the ImageNet-shaped ResNet-18 / QuickNet layers the paper
benchmarks in its Section 4): ``numpy.random.default_rng(SEED0 + 100*config +
tensor_index)``; activations fp32 ~ N(0,1); weights uniform over {-1,+1};
multiplier ~ U(0.5,1.5); bias ~ N(0, sigma=0.1); thresholds
rint(sqrt(K) * N(0,1)) as int32 with K = KH*KW*Cin.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import List, Optional

import numpy as np

SEED0 = 201109398000

PAD_VALID, PAD_SAME_ONE, PAD_SAME_ZERO = 0, 1, 2
OUT_FLOAT32, OUT_BITPACKED, OUT_INT32 = 0, 1, 2


@dataclass(frozen=True)
class ConvSpec:
    """Shape of one LceBConv2d call (paper Section 3.2)."""
    name: str
    batch: int
    in_h: int
    in_w: int
    in_c: int
    out_c: int
    kernel: int = 3
    stride: int = 1
    padding: int = PAD_SAME_ONE
    out_type: int = OUT_BITPACKED

    @property
    def out_h(self) -> int:
        return _out(self.in_h, self.kernel, self.stride, self.padding)

    @property
    def out_w(self) -> int:
        return _out(self.in_w, self.kernel, self.stride, self.padding)

    @property
    def K(self) -> int:
        return self.kernel * self.kernel * self.in_c

    @property
    def in_words(self) -> int:
        return (self.in_c + 31) // 32

    @property
    def binary_macs(self) -> int:
        """True binary multiply-accumulates: N*OH*OW*Cout*KH*KW*Cin."""
        return self.batch * self.out_h * self.out_w * self.out_c * self.K

    @property
    def word_ops(self) -> int:
        """32-bit XOR+POPC+accumulate slots: N*OH*OW*Cout*KH*KW*ceil(Cin/32)."""
        return self.batch * self.out_h * self.out_w * self.out_c * self.kernel * self.kernel * self.in_words

    @property
    def algorithmic_bytes(self) -> int:
        """Packed input once + packed weights once + output."""
        inp = 4 * self.batch * self.in_h * self.in_w * self.in_words
        wts = 4 * self.out_c * self.kernel * self.kernel * self.in_words
        pix = self.batch * self.out_h * self.out_w
        out = pix * 4 * ((self.out_c + 31) // 32) if self.out_type == OUT_BITPACKED else pix * 4 * self.out_c
        return inp + wts + out


def _out(size: int, k: int, s: int, padding: int) -> int:
    # shape bookkeeping only (TensorFlow VALID / SAME output extents)
    if padding == PAD_VALID:
        return (size - k) // s + 1 if size >= k else 0
    return -(-size // s)


def _rng(config: int, tensor_index: int) -> np.random.Generator:
    return np.random.default_rng(SEED0 + 100 * config + tensor_index)


def activations(config: int, tensor_index: int, shape) -> np.ndarray:
    return _rng(config, tensor_index).standard_normal(shape, dtype=np.float32)


def weights_pm1(config: int, tensor_index: int, spec: ConvSpec) -> np.ndarray:
    """int8 [Cout,KH,KW,Cin], uniform over {-1,+1}."""
    r = _rng(config, tensor_index)
    shape = (spec.out_c, spec.kernel, spec.kernel, spec.in_c)
    return (2 * r.integers(0, 2, size=shape, dtype=np.int8) - 1).astype(np.int8)


def multiplier(config: int, tensor_index: int, out_c: int) -> np.ndarray:
    return _rng(config, tensor_index).uniform(0.5, 1.5, size=out_c).astype(np.float32)


def bias(config: int, tensor_index: int, out_c: int) -> np.ndarray:
    return (0.1 * _rng(config, tensor_index).standard_normal(out_c)).astype(np.float32)


def thresholds(config: int, tensor_index: int, spec: ConvSpec) -> np.ndarray:
    z = _rng(config, tensor_index).standard_normal(spec.out_c)
    return np.rint(np.sqrt(float(spec.K)) * z).astype(np.int32)


@dataclass
class ConvTensors:
    spec: ConvSpec
    w_pm1: np.ndarray
    multiplier: Optional[np.ndarray] = None
    bias: Optional[np.ndarray] = None
    thresholds: Optional[np.ndarray] = None


def conv_tensors(config: int, first_index: int, spec: ConvSpec) -> ConvTensors:
    """Draw one layer's parameters: weights, multiplier, bias, thresholds (indices first..first+3)."""
    return ConvTensors(
        spec=spec,
        w_pm1=weights_pm1(config, first_index, spec),
        multiplier=multiplier(config, first_index + 1, spec.out_c),
        bias=bias(config, first_index + 2, spec.out_c),
        thresholds=thresholds(config, first_index + 3, spec),
    )


# --- the five workloads ----------------------------------------------------

def config1_spec() -> ConvSpec:
    """Single conv: batch 1, 14x14x64 -> 64, 3x3, one-padding, float output."""
    return ConvSpec("c1_14x14x64", 1, 14, 14, 64, 64, 3, 1, PAD_SAME_ONE, OUT_FLOAT32)


def config2_specs(batch: int = 64) -> List[ConvSpec]:
    """ResNet-18-shaped 3x3 layers, each with float and with bit-packed output."""
    out = []
    for h, c in ((56, 64), (28, 128), (14, 256), (7, 512)):
        for ot, tag in ((OUT_FLOAT32, "f32"), (OUT_BITPACKED, "bit")):
            out.append(ConvSpec(f"c2_{h}x{h}x{c}_{tag}", batch, h, h, c, c, 3, 1, PAD_SAME_ONE, ot))
    return out


def config3_specs(batch: int = 64) -> List[ConvSpec]:
    """Strided / transition layers, bit-packed outputs."""
    return [
        ConvSpec("c3_56x56x64_s2_128", batch, 56, 56, 64, 128, 3, 2, PAD_SAME_ONE, OUT_BITPACKED),
        ConvSpec("c3_28x28x256_s2_256", batch, 28, 28, 256, 256, 3, 2, PAD_SAME_ONE, OUT_BITPACKED),
        ConvSpec("c3_14x14x256_1x1_512", batch, 14, 14, 256, 512, 1, 1, PAD_SAME_ONE, OUT_BITPACKED),
    ]


def sweep_specs(batch: int = 1) -> List[ConvSpec]:
    """The paper's convolution sweep (Section 5.1): square inputs of 8..64 pixels, Cin = Cout from 32
    to 256, 3x3 and 5x5 filters, stride 1, same padding; float outputs as in a full-precision-output
    benchmark of one layer.  The paper runs it one image at a time; batch scales it for a GPU."""
    specs = []
    for kernel in (3, 5):
        for size in (8, 16, 32, 64):
            for ch in (32, 64, 96, 128, 160, 256):
                specs.append(ConvSpec(f"sweep_{size}x{size}x{ch}_k{kernel}", batch, size, size, ch, ch, kernel, 1,
                                      PAD_SAME_ONE, OUT_FLOAT32))
    return specs


@dataclass(frozen=True)
class Step:
    """One kernel call of a chain. kind: bitpack | bconv | bconv_fused | add | bmaxpool.
    src/src2/dst name buffers of the chain; conv is the layer spec for the conv kinds.
    bconv_fused: float-output conv whose result (+ the residual src2, if named) goes to the float
    buffer dst (if named) and, sign-packed, to dst2 (if named)."""
    kind: str
    src: str
    dst: str
    src2: str = ""
    conv: Optional[ConvSpec] = None
    shape: tuple = ()      # (N,H,W,C) of src for bitpack / add / bmaxpool
    tensor_index: int = -1  # first RNG index of the conv's parameters
    dst2: str = ""


def config4_steps(batch: int = 128, size: int = 56, widths=(64, 128, 256, 512)) -> List[Step]:
    """Residual block stack: per stage  A=bitpack(X); B=bconv3x3(A)->bits;
    F=bconv3x3(B)->float; Y=F+X; between stages P=bitpack(Y); Q=bmaxpool2x2(P);
    X'=bconv1x1(Q; C->2C)->float.  The last Y is the output."""
    steps: List[Step] = []
    idx = 1  # tensor 0 is the input activation
    h = size
    for s, c in enumerate(widths):
        x, a, b, f, y = f"X{s}", f"A{s}", f"B{s}", f"F{s}", f"Y{s}"
        steps.append(Step("bitpack", x, a, shape=(batch, h, h, c)))
        steps.append(Step("bconv", a, b, conv=ConvSpec(f"c4_s{s}_conv1", batch, h, h, c, c, 3, 1, PAD_SAME_ONE, OUT_BITPACKED), tensor_index=idx)); idx += 4
        steps.append(Step("bconv", b, f, conv=ConvSpec(f"c4_s{s}_conv2", batch, h, h, c, c, 3, 1, PAD_SAME_ONE, OUT_FLOAT32), tensor_index=idx)); idx += 4
        steps.append(Step("add", f, y, src2=x, shape=(batch, h, h, c)))
        if s + 1 < len(widths):
            p, q = f"P{s}", f"Q{s}"
            steps.append(Step("bitpack", y, p, shape=(batch, h, h, c)))
            steps.append(Step("bmaxpool", p, q, shape=(batch, h, h, c)))
            h2 = h // 2
            steps.append(Step("bconv", q, f"X{s+1}", conv=ConvSpec(f"c4_s{s}_trans", batch, h2, h2, c, widths[s + 1], 1, 1, PAD_SAME_ONE, OUT_FLOAT32), tensor_index=idx)); idx += 4
            h = h2
    return steps


def config4_fused_steps(batch: int = 128, size: int = 56, widths=(64, 128, 256, 512)) -> List[Step]:
    """config4_steps with every add and every re-quantize folded into the conv before it: same
    tensors, same parameters (tensor indices), 15 launches instead of 25.  Buffers that only fed a
    fused step (F, and Y except the last) are never written."""
    steps: List[Step] = []
    idx = 1
    h = size
    steps.append(Step("bitpack", "X0", "A0", shape=(batch, h, h, widths[0])))
    for s, c in enumerate(widths):
        last = s + 1 == len(widths)
        steps.append(Step("bconv", f"A{s}", f"B{s}", conv=ConvSpec(f"c4_s{s}_conv1", batch, h, h, c, c, 3, 1, PAD_SAME_ONE, OUT_BITPACKED), tensor_index=idx)); idx += 4
        steps.append(Step("bconv_fused", f"B{s}", f"Y{s}" if last else "", src2=f"X{s}", dst2="" if last else f"P{s}",
                          conv=ConvSpec(f"c4_s{s}_conv2", batch, h, h, c, c, 3, 1, PAD_SAME_ONE, OUT_FLOAT32), tensor_index=idx)); idx += 4
        if not last:
            steps.append(Step("bmaxpool", f"P{s}", f"Q{s}", shape=(batch, h, h, c)))
            h2 = h // 2
            steps.append(Step("bconv_fused", f"Q{s}", f"X{s+1}", dst2=f"A{s+1}",
                              conv=ConvSpec(f"c4_s{s}_trans", batch, h2, h2, c, widths[s + 1], 1, 1, PAD_SAME_ONE, OUT_FLOAT32), tensor_index=idx)); idx += 4
            h = h2
    return steps


def config5_steps(batch: int = 256, size: int = 224, in_c: int = 3, stem_c: int = 32,
                  widths=(64, 128, 256, 512), per_stage: int = 4) -> List[Step]:
    """ImageNet-shaped body: bitpack(input) then 3x3 one-padded convs: a stride-2
    stem to stem_c, then per width one stride-2 conv followed by per_stage-1
    stride-1 convs; every conv writes bit-packed output except the last (float)."""
    steps: List[Step] = [Step("bitpack", "X", "T0", shape=(batch, size, size, in_c))]
    convs = []
    h, c = size, in_c
    convs.append((h, c, stem_c, 2)); h, c = -(-h // 2), stem_c
    for wdt in widths:
        convs.append((h, c, wdt, 2)); h, c = -(-h // 2), wdt
        for _ in range(per_stage - 1):
            convs.append((h, c, wdt, 1))
    idx = 1
    for i, (hh, ci, co, st) in enumerate(convs):
        last = i == len(convs) - 1
        spec = ConvSpec(f"c5_L{i+1}", batch, hh, hh, ci, co, 3, st, PAD_SAME_ONE, OUT_FLOAT32 if last else OUT_BITPACKED)
        steps.append(Step("bconv", f"T{i}", f"T{i+1}", conv=spec, tensor_index=idx)); idx += 4
    return steps


def with_batch(spec: ConvSpec, batch: int) -> ConvSpec:
    return replace(spec, batch=batch)
