"""Seeded synthetic inputs shared by the tests, the bench and the oracle's callers.

Holds input generation only (random tensors, token ids, tree shapes, workload
configurations); none of the verification method's arithmetic lives here.
The generator itself is ``gen.c`` (integer hashing + one fp32 multiply), built
on first use with the host C compiler.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libsynth.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile gen.c into libsynth.so next to it (no-op when up to date)."""
    src = os.path.join(_HERE, "gen.c")
    if (not force and os.path.exists(_LIB_PATH)
            and os.path.getmtime(_LIB_PATH) >= os.path.getmtime(src)):
        return _LIB_PATH
    tmp = _LIB_PATH + f".{os.getpid()}.tmp"
    subprocess.check_call(["gcc", "-O3", "-fopenmp", "-shared", "-fPIC", "-o", tmp, src])
    os.replace(tmp, _LIB_PATH)
    return _LIB_PATH


def _load():
    global _lib
    with _lock:
        if _lib is None:
            lib = ctypes.CDLL(build())
            u64, sz, f32 = ctypes.c_uint64, ctypes.c_size_t, ctypes.c_float
            vp = ctypes.c_void_p
            lib.synth_key.restype = u64
            lib.synth_key.argtypes = [u64, u64]
            lib.synth_normal_f32.argtypes = [u64, u64, sz, f32, vp]
            lib.synth_normal_bf16.argtypes = [u64, u64, sz, f32, vp]
            lib.synth_index_i32.argtypes = [u64, u64, sz, u64, vp]
            lib.synth_unit_f32.argtypes = [u64, u64, sz, vp]
            for f in (lib.synth_normal_f32, lib.synth_normal_bf16, lib.synth_index_i32,
                      lib.synth_unit_f32):
                f.restype = None
            _lib = lib
    return _lib


def key(seed: int, tensor: int) -> int:
    return int(_load().synth_key(seed & (2**64 - 1), tensor & (2**64 - 1)))


def _scale(sigma: float) -> np.float32:
    # sigma / 65536 is an exact power-of-two scaling of the fp32 value of sigma
    return np.float32(np.float32(sigma) * np.float32(1.0 / 65536.0))


def normal_f32(seed: int, tensor: int, shape, sigma: float, first: int = 0) -> np.ndarray:
    """fp32 array of N(0, sigma^2)-like values (Irwin-Hall(12), clipped at 6 sigma)."""
    out = np.empty(shape, dtype=np.float32)
    _load().synth_normal_f32(key(seed, tensor), first, out.size, float(_scale(sigma)),
                             out.ctypes.data)
    return out


def normal_bf16(seed: int, tensor: int, shape, sigma: float, first: int = 0) -> np.ndarray:
    """Same values rounded to bf16, returned as raw uint16 words."""
    out = np.empty(shape, dtype=np.uint16)
    _load().synth_normal_bf16(key(seed, tensor), first, out.size, float(_scale(sigma)),
                              out.ctypes.data)
    return out


def index_i32(seed: int, tensor: int, shape, modulus: int, first: int = 0) -> np.ndarray:
    out = np.empty(shape, dtype=np.int32)
    _load().synth_index_i32(key(seed, tensor), first, out.size, int(modulus), out.ctypes.data)
    return out


def unit_f32(seed: int, tensor: int, shape, first: int = 0) -> np.ndarray:
    out = np.empty(shape, dtype=np.float32)
    _load().synth_unit_f32(key(seed, tensor), first, out.size, out.ctypes.data)
    return out


def bf16_to_f32(words: np.ndarray) -> np.ndarray:
    """Widen raw bf16 words to fp32 (exact)."""
    return (words.astype(np.uint32) << np.uint32(16)).view(np.float32)


def f32_to_bf16(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (nearest even), returned as raw uint16 words."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    u = u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    return (u >> np.uint32(16)).astype(np.uint16)
