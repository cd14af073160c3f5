"""The chains of configs 4 and 5 evaluated with the CPU oracle, step by step (test helper)."""
import numpy as np

import lce_workloads as wl
import oracle


def run_chain_oracle(steps, config, inputs):
    """inputs: {buffer name: numpy array}.  Returns every buffer: packed tensors as uint32 words,
    float tensors as float32."""
    B = dict(inputs)
    for st in steps:
        if st.kind == "bitpack":
            B[st.dst] = oracle.bitpack(B[st.src])
        elif st.kind == "add":
            B[st.dst] = oracle.add_f32(B[st.src], B[st.src2])
        elif st.kind == "bmaxpool":
            B[st.dst] = oracle.bmaxpool(B[st.src], st.shape[3], (2, 2), (2, 2), oracle.PAD_VALID)
        elif st.kind == "bconv_fused":
            s = st.conv
            t = wl.conv_tensors(config, st.tensor_index, s)
            acc = oracle.bconv2d_acc(oracle.unpack_pm1(B[st.src], s.in_c), t.w_pm1, (s.stride, s.stride), s.padding)
            y = oracle.transform_float(acc, t.multiplier, t.bias)
            if st.src2:
                y = oracle.add_f32(y, B[st.src2])
            if st.dst:
                B[st.dst] = y
            if st.dst2:
                B[st.dst2] = oracle.bitpack(y)
        elif st.kind == "bconv":
            s = st.conv
            t = wl.conv_tensors(config, st.tensor_index, s)
            a = oracle.unpack_pm1(B[st.src], s.in_c)
            acc = oracle.bconv2d_acc(a, t.w_pm1, (s.stride, s.stride), s.padding)
            if s.out_type == wl.OUT_FLOAT32:
                B[st.dst] = oracle.transform_float(acc, t.multiplier, t.bias)
            else:
                B[st.dst] = oracle.transform_bits(acc, t.thresholds)
    return B
