"""Helpers shared by the GPU parity tests: moving numpy arrays to the device and calling the
C-ABI library through the binding.  Comparison logic stays in the tests."""
import numpy as np
import torch

import paper_2011_09398_b200 as lce

DEV = "cuda:0"


def to_dev_words(words: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(words).view(np.int32)).to(DEV)


def to_dev(a: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a)).to(DEV)


def words_to_host(t: torch.Tensor) -> np.ndarray:
    return t.cpu().numpy().view(np.uint32)


def guarded(shape, dtype, fill):
    """A device buffer with 64 guard elements on each side; returns (whole, view)."""
    n = int(np.prod(shape))
    whole = torch.full((n + 128,), fill, dtype=dtype, device=DEV)
    return whole, whole[64:64 + n].view(shape)


def guards_intact(whole, fill) -> bool:
    return bool((whole[:64] == fill).all().item() and (whole[-64:] == fill).all().item())


def run_bconv(a_words, w_words, spec_kwargs, mult=None, bias=None, thr=None, kernel_choice=lce.KERNEL_AUTO,
              packed=False):
    """a_words/w_words: numpy uint32. Returns the numpy output (uint32 words / int32 / float32),
    after checking the guard words around the output buffer."""
    N, H, W, _ = a_words.shape
    Cout, KH, KW, _ = w_words.shape
    desc = lce.make_desc(N, H, W, spec_kwargs["in_c"], Cout, (KH, KW), spec_kwargs.get("stride", (1, 1)),
                         spec_kwargs.get("padding", lce.PAD_SAME_ONE), spec_kwargs["out_type"],
                         spec_kwargs.get("activation", lce.ACT_NONE), kernel_choice, 1 if packed else 0)
    oh, ow = lce.lce_bconv2d_out_shape(desc)
    ot = spec_kwargs["out_type"]
    if ot == lce.OUT_FLOAT32:
        whole, out = guarded((N, oh, ow, Cout), torch.float32, 12345.0)
        fill = 12345.0
    else:
        last = (Cout + 31) // 32 if ot == lce.OUT_BITPACKED else Cout
        whole, out = guarded((N, oh, ow, last), torch.int32, 0x5A5A5A5A)
        fill = 0x5A5A5A5A
    w_dev = to_dev_words(w_words)
    if packed:
        w_dev = lce.lce_bconv2d_pack_weights(desc, w_dev)
    lce.lce_bconv2d(desc, to_dev_words(a_words), w_dev,
                    to_dev(mult) if mult is not None else None, to_dev(bias) if bias is not None else None,
                    to_dev(thr) if thr is not None else None, out)
    torch.cuda.synchronize()
    assert guards_intact(whole, fill), "kernel wrote outside its output buffer"
    res = out.cpu().numpy()
    return res.view(np.uint32) if ot == lce.OUT_BITPACKED else res
