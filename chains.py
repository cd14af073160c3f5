"""Runs a list of hot-path steps (LceQuantize, LceBConv2d, add, LceBMaxPool2d) as consecutive
C-ABI calls on one stream (harness for the tests and bench.py, next to the workload lists it
runs).  Argument marshalling only: buffers are torch CUDA tensors, weights are packed once at
construction (load time), every step is one library call."""
from __future__ import annotations

from typing import Dict, List

import numpy as np
import torch

import lce_workloads as wl
import paper_2011_09398_b200 as lce


class Chain:
    def __init__(self, steps: List[wl.Step], config: int, device: str = "cuda:0", keep_all: bool = True):
        self.steps, self.config, self.device = steps, config, torch.device(device)
        self.buffers: Dict[str, torch.Tensor] = {}
        self.calls = []
        self.params = {}  # step index -> ConvTensors (host side, for the tests)
        dev = self.device
        for i, st in enumerate(steps):
            if st.kind == "bitpack":
                N, H, W, C = st.shape
                self._ensure(st.src, (N, H, W, C), torch.float32)
                self._ensure(st.dst, (N, H, W, (C + 31) // 32), torch.int32)
            elif st.kind == "add":
                for name in (st.src, st.src2, st.dst):
                    self._ensure(name, st.shape, torch.float32)
            elif st.kind == "bmaxpool":
                N, H, W, C = st.shape
                self._ensure(st.src, (N, H, W, (C + 31) // 32), torch.int32)
                self._ensure(st.dst, (N, H // 2, W // 2, (C + 31) // 32), torch.int32)
            elif st.kind in ("bconv", "bconv_fused"):
                s = st.conv
                t = wl.conv_tensors(config, st.tensor_index, s)
                self.params[i] = t
                desc = lce.make_desc(s.batch, s.in_h, s.in_w, s.in_c, s.out_c, (s.kernel, s.kernel), (s.stride, s.stride),
                                     s.padding, s.out_type, lce.ACT_NONE, lce.KERNEL_AUTO, 1)
                plain = lce.pack_weights(torch.from_numpy(t.w_pm1).to(dev))
                packed = lce.lce_bconv2d_pack_weights(desc, plain)
                self._ensure(st.src, (s.batch, s.in_h, s.in_w, s.in_words), torch.int32)
                if st.kind == "bconv_fused":
                    fshape = (s.batch, s.out_h, s.out_w, s.out_c)
                    for name in (st.dst, st.src2):
                        if name:
                            self._ensure(name, fshape, torch.float32)
                    if st.dst2:
                        self._ensure(st.dst2, (s.batch, s.out_h, s.out_w, (s.out_c + 31) // 32), torch.int32)
                    extra = (torch.from_numpy(t.multiplier).to(dev), torch.from_numpy(t.bias).to(dev), None)
                elif s.out_type == wl.OUT_FLOAT32:
                    self._ensure(st.dst, (s.batch, s.out_h, s.out_w, s.out_c), torch.float32)
                    extra = (torch.from_numpy(t.multiplier).to(dev), torch.from_numpy(t.bias).to(dev), None)
                else:
                    self._ensure(st.dst, (s.batch, s.out_h, s.out_w, (s.out_c + 31) // 32), torch.int32)
                    extra = (None, None, torch.from_numpy(t.thresholds).to(dev))
                self.calls.append((i, desc, packed, extra))
            else:
                raise ValueError(st.kind)
        self._conv = {i: (d, w, e) for i, d, w, e in self.calls}

    def _ensure(self, name, shape, dtype):
        if name not in self.buffers:
            self.buffers[name] = torch.empty(shape, dtype=dtype, device=self.device)
        else:
            b = self.buffers[name]
            if tuple(b.shape) != tuple(shape) or b.dtype != dtype:
                raise ValueError(f"buffer {name}: {tuple(b.shape)} {b.dtype} vs {tuple(shape)} {dtype}")

    def set_input(self, name: str, x: np.ndarray) -> None:
        self.buffers[name].copy_(torch.from_numpy(x))

    def run(self, only=None) -> None:
        """Enqueues every step (or just step `only`) on the current stream; no synchronisation."""
        B = self.buffers
        for i, st in enumerate(self.steps):
            if only is not None and i != only:
                continue
            if st.kind == "bitpack":
                lce.lce_bitpack(B[st.src], B[st.dst])
            elif st.kind == "add":
                lce.lce_add_f32(B[st.src], B[st.src2], B[st.dst])
            elif st.kind == "bmaxpool":
                lce.lce_bmaxpool(B[st.src], st.shape[3], (2, 2), (2, 2), lce.PAD_VALID, B[st.dst])
            elif st.kind == "bconv_fused":
                desc, w, (mult, bias, _) = self._conv[i]
                lce.lce_bconv2d_fused(desc, B[st.src], w, mult, bias, B[st.src2] if st.src2 else None,
                                      B[st.dst] if st.dst else None, B[st.dst2] if st.dst2 else None)
            else:
                desc, w, (mult, bias, thr) = self._conv[i]
                lce.lce_bconv2d(desc, B[st.src], w, mult, bias, thr, B[st.dst])

    @property
    def launches(self) -> int:
        return len(self.steps)
