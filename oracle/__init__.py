"""CPU oracle for the Bconv2D path -- TEST INFRASTRUCTURE, not the product.

A thin numpy/ctypes front for ``oracle.c`` (plain nested loops in +-1 integer
arithmetic; see that file's header for the conventions and the readings of
the paper's Section 3.2 it takes).  Only ``tests/``, the smoke check and the
benchmark's cpu-baseline leg may import this package; it imports nothing from
the CUDA package and the CUDA package never imports it.

"parity unpinned": the bit order inside a packed word (LSB = lowest channel).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "oracle.c"
_LIB = _HERE / "liboracle.so"

PAD_VALID, PAD_SAME_ONE, PAD_SAME_ZERO = 0, 1, 2
ACT_NONE, ACT_RELU = 0, 1


def build(force: bool = False) -> Path:
    """Compile oracle.c into liboracle.so with gcc (rebuilt when the source is newer)."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _LIB.with_suffix(f".so.tmp{os.getpid()}")
        subprocess.run(
            ["gcc", "-O2", "-fopenmp", "-ffp-contract=off", "-shared", "-fPIC",
             "-o", str(tmp), str(_SRC), "-lm"],
            check=True,
        )
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(str(build()))
        i32, i64, p = ctypes.c_int32, ctypes.c_int64, ctypes.c_void_p
        lib.oracle_out_size.restype = i32
        lib.oracle_out_size.argtypes = [i32] * 4
        lib.oracle_pad_before.restype = i32
        lib.oracle_pad_before.argtypes = [i32] * 4
        lib.oracle_sign.argtypes = [p, p, i64]
        lib.oracle_bitpack.argtypes = [p, i64, i32, p]
        lib.oracle_bitpack_pm1.argtypes = [p, i64, i32, p]
        lib.oracle_unpack_pm1.argtypes = [p, i64, i32, p]
        lib.oracle_unpack_f32.argtypes = [p, i64, i32, p]
        lib.oracle_bconv2d_acc.restype = ctypes.c_int
        lib.oracle_bconv2d_acc.argtypes = [p, p] + [i32] * 10 + [p]
        lib.oracle_bconv2d_acc_at.restype = ctypes.c_int
        lib.oracle_bconv2d_acc_at.argtypes = [p, p] + [i32] * 10 + [p, i64, p]
        lib.oracle_transform_float.argtypes = [p, i64, i32, p, p, i32, p]
        lib.oracle_transform_bits.argtypes = [p, i64, i32, p, p]
        lib.oracle_maxpool_pm1.restype = ctypes.c_int
        lib.oracle_maxpool_pm1.argtypes = [p] + [i32] * 9 + [p]
        lib.oracle_add_f32.argtypes = [p, p, p, i64]
        _lib = lib
    return _lib


def _c(a: np.ndarray, dtype) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=dtype)


def _ptr(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def words_for(channels: int) -> int:
    return (channels + 31) // 32


def out_size(in_size: int, k: int, stride: int, padding: int) -> int:
    return int(_load().oracle_out_size(in_size, k, stride, padding))


def pad_before(in_size: int, k: int, stride: int, padding: int) -> int:
    return int(_load().oracle_pad_before(in_size, k, stride, padding))


def sign(x: np.ndarray) -> np.ndarray:
    """-1 where x < 0, +1 elsewhere, as int8 (same shape)."""
    x = _c(x, np.float32)
    s = np.empty(x.shape, np.int8)
    _load().oracle_sign(_ptr(x), _ptr(s), x.size)
    return s


def bitpack(x: np.ndarray) -> np.ndarray:
    """LceQuantize: fp32 [..., C] -> uint32 [..., ceil(C/32)]."""
    x = _c(x, np.float32)
    C = x.shape[-1]
    rows = x.size // C if C else 0
    out = np.empty(x.shape[:-1] + (words_for(C),), np.uint32)
    _load().oracle_bitpack(_ptr(x), rows, C, _ptr(out))
    return out


def bitpack_pm1(s: np.ndarray) -> np.ndarray:
    """Pack +-1 int8 values [..., C] (bit 1 <=> -1) -> uint32 [..., ceil(C/32)]."""
    s = _c(s, np.int8)
    C = s.shape[-1]
    rows = s.size // C if C else 0
    out = np.empty(s.shape[:-1] + (words_for(C),), np.uint32)
    _load().oracle_bitpack_pm1(_ptr(s), rows, C, _ptr(out))
    return out


def unpack_pm1(words: np.ndarray, channels: int) -> np.ndarray:
    """uint32 [..., ceil(C/32)] -> int8 [..., C] in {-1, +1}."""
    words = _c(words, np.uint32)
    assert words.shape[-1] == words_for(channels)
    rows = words.size // words.shape[-1]
    s = np.empty(words.shape[:-1] + (channels,), np.int8)
    _load().oracle_unpack_pm1(_ptr(words), rows, channels, _ptr(s))
    return s


def unpack_f32(words: np.ndarray, channels: int) -> np.ndarray:
    """LceDequantize: uint32 [..., ceil(C/32)] -> fp32 [..., C] in {-1.0, +1.0}."""
    words = _c(words, np.uint32)
    assert words.shape[-1] == words_for(channels)
    rows = words.size // words.shape[-1]
    out = np.empty(words.shape[:-1] + (channels,), np.float32)
    _load().oracle_unpack_f32(_ptr(words), rows, channels, _ptr(out))
    return out


def bconv2d_acc(a: np.ndarray, w: np.ndarray, stride=(1, 1), padding: int = PAD_SAME_ONE) -> np.ndarray:
    """Accumulator of LceBConv2d by the definition.

    a: int8 [N,H,W,Cin] in {-1,+1}; w: int8 [Cout,KH,KW,Cin] in {-1,+1}
    -> int32 [N,OH,OW,Cout].
    """
    a, w = _c(a, np.int8), _c(w, np.int8)
    N, H, W, Cin = a.shape
    Cout, KH, KW, Cin2 = w.shape
    assert Cin == Cin2
    sh, sw = stride
    OH, OW = out_size(H, KH, sh, padding), out_size(W, KW, sw, padding)
    acc = np.empty((N, max(OH, 0), max(OW, 0), Cout), np.int32)
    if acc.size == 0:
        return acc
    rc = _load().oracle_bconv2d_acc(_ptr(a), _ptr(w), N, H, W, Cin, Cout, KH, KW, sh, sw, padding, _ptr(acc))
    assert rc == 0
    return acc


def bconv2d_acc_at(a, w, idx, stride=(1, 1), padding: int = PAD_SAME_ONE) -> np.ndarray:
    """The same definition at sampled output coordinates idx[count,4] = (n, oh, ow, o)."""
    a, w = _c(a, np.int8), _c(w, np.int8)
    idx = _c(idx, np.int32).reshape(-1, 4)
    N, H, W, Cin = a.shape
    Cout, KH, KW, _ = w.shape
    sh, sw = stride
    acc = np.empty((idx.shape[0],), np.int32)
    rc = _load().oracle_bconv2d_acc_at(_ptr(a), _ptr(w), N, H, W, Cin, Cout, KH, KW, sh, sw, padding,
                                       _ptr(idx), idx.shape[0], _ptr(acc))
    assert rc == 0, "sample index out of range"
    return acc


def transform_float(acc: np.ndarray, multiplier, bias, activation: int = ACT_NONE) -> np.ndarray:
    """y = fmaf(float(act(acc)), multiplier[c], bias[c]) (one rounding)."""
    acc = _c(acc, np.int32)
    Cout = acc.shape[-1]
    m, b = _c(multiplier, np.float32), _c(bias, np.float32)
    assert m.shape == (Cout,) and b.shape == (Cout,)
    out = np.empty(acc.shape, np.float32)
    _load().oracle_transform_float(_ptr(acc), acc.size // Cout, Cout, _ptr(m), _ptr(b), activation, _ptr(out))
    return out


def transform_bits(acc: np.ndarray, threshold) -> np.ndarray:
    """bit[c] = (acc < threshold[c]) packed 32 output channels per word."""
    acc = _c(acc, np.int32)
    Cout = acc.shape[-1]
    t = _c(threshold, np.int32)
    assert t.shape == (Cout,)
    out = np.empty(acc.shape[:-1] + (words_for(Cout),), np.uint32)
    _load().oracle_transform_bits(_ptr(acc), acc.size // Cout, Cout, _ptr(t), _ptr(out))
    return out


def bconv2d(a_pm1, w_pm1, stride=(1, 1), padding=PAD_SAME_ONE, out_type="int32",
            multiplier=None, bias=None, threshold=None, activation=ACT_NONE) -> np.ndarray:
    """LceBConv2d = accumulator followed by the output transform named by out_type."""
    acc = bconv2d_acc(a_pm1, w_pm1, stride, padding)
    if out_type == "int32":
        return acc
    if out_type == "float32":
        return transform_float(acc, multiplier, bias, activation)
    if out_type == "bitpacked":
        return transform_bits(acc, threshold)
    raise ValueError(out_type)


def maxpool_pm1(s: np.ndarray, pool=(2, 2), stride=(2, 2), padding: int = PAD_VALID) -> np.ndarray:
    """Max-pool of +-1 int8 values [N,H,W,C]; out-of-image taps are skipped."""
    s = _c(s, np.int8)
    N, H, W, C = s.shape
    OH, OW = out_size(H, pool[0], stride[0], padding), out_size(W, pool[1], stride[1], padding)
    out = np.empty((N, max(OH, 0), max(OW, 0), C), np.int8)
    if out.size == 0:
        return out
    rc = _load().oracle_maxpool_pm1(_ptr(s), N, H, W, C, pool[0], pool[1], stride[0], stride[1], padding, _ptr(out))
    assert rc == 0
    return out


def bmaxpool(words: np.ndarray, channels: int, pool=(2, 2), stride=(2, 2), padding: int = PAD_VALID) -> np.ndarray:
    """LceBMaxPool2d by its meaning: unpack to +-1, max over the window, re-pack."""
    return bitpack_pm1(maxpool_pm1(unpack_pm1(words, channels), pool, stride, padding))


def add_f32(a: np.ndarray, b: np.ndarray) -> np.ndarray:
    a, b = _c(a, np.float32), _c(b, np.float32)
    assert a.shape == b.shape
    out = np.empty(a.shape, np.float32)
    _load().oracle_add_f32(_ptr(a), _ptr(b), _ptr(out), a.size)
    return out
