"""Seeded synthetic inputs (weight blobs, prompts) and the named workload shapes.

Nothing in here performs any of the decoder's arithmetic; it only draws numbers.  The CPU
oracle and the CUDA library are both handed the arrays produced here.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass, replace

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libppd_inputs.so")
_lib = None


@dataclass(frozen=True)
class ModelShape:
    """Decoder-only transformer shape (RMSNorm, RoPE, SwiGLU, multi-head attention)."""
    name: str
    n_layers: int
    d_model: int
    n_heads: int
    head_dim: int
    d_ffn: int
    vocab: int
    rms_eps: float = 1e-5
    rope_theta: float = 10000.0

    def with_layers(self, n_layers: int) -> "ModelShape":
        return replace(self, n_layers=n_layers, name=f"{self.name}-d{n_layers}")

    @property
    def layer_params(self) -> int:
        D, F = self.d_model, self.d_ffn
        return 4 * D * D + 3 * F * D + 2 * D

    @property
    def head_params(self) -> int:
        return self.vocab * self.d_model

    @property
    def blob_elems(self) -> int:
        D, V = self.d_model, self.vocab
        return V * D + self.n_layers * self.layer_params + D + V * D


TINY = ModelShape("tiny", n_layers=4, d_model=256, n_heads=4, head_dim=64, d_ffn=688, vocab=4096)
LLAMA_7B = ModelShape("7b", n_layers=32, d_model=4096, n_heads=32, head_dim=128, d_ffn=11008, vocab=32000)
LLAMA_13B = ModelShape("13b", n_layers=40, d_model=5120, n_heads=40, head_dim=128, d_ffn=13824, vocab=32000)
SHAPES = {s.name: s for s in (TINY, LLAMA_7B, LLAMA_13B)}


@dataclass(frozen=True)
class Workload:
    """One synthetic decode workload: model shape, prompt length P, tokens to generate L, (k, l)."""
    name: str
    shape: ModelShape
    n_prompt: int
    n_gen: int
    k: int
    early_layer: int
    seed: int = 0


WORKLOADS = {
    "tiny": Workload("tiny", TINY, 16, 32, 3, 2),
    "7b": Workload("7b", LLAMA_7B, 512, 256, 3, 16),
    "7b-long": Workload("7b-long", LLAMA_7B, 8192, 128, 3, 16),
    "13b": Workload("13b", LLAMA_13B, 1024, 256, 3, 20),
}


def build(force: bool = False) -> str:
    """Compile the generator with gcc (OpenMP).  Returns the library path."""
    src = os.path.join(_HERE, "gen.c")
    if force or not os.path.exists(_LIB_PATH) or os.path.getmtime(_LIB_PATH) < os.path.getmtime(src):
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-o", _LIB_PATH, src, "-lm"])
    return _LIB_PATH


class _Shape(ctypes.Structure):
    _fields_ = [("n_layers", ctypes.c_int32), ("d_model", ctypes.c_int32),
                ("d_ffn", ctypes.c_int32), ("vocab", ctypes.c_int32)]


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB_PATH)
        lib.ppd_inputs_blob_elems.restype = ctypes.c_size_t
        lib.ppd_inputs_blob_elems.argtypes = [ctypes.POINTER(_Shape)]
        lib.ppd_inputs_gen_weights.restype = ctypes.c_int
        lib.ppd_inputs_gen_weights.argtypes = [ctypes.POINTER(_Shape), ctypes.c_uint64, ctypes.c_double,
                                               ctypes.c_double, ctypes.c_void_p]
        lib.ppd_inputs_gen_prompt.restype = ctypes.c_int
        lib.ppd_inputs_gen_prompt.argtypes = [ctypes.c_int32, ctypes.c_uint64, ctypes.c_int32, ctypes.c_void_p]
        _lib = lib
    return _lib


def gen_weights(shape: ModelShape, seed: int = 0, sigma: float = 0.02, resid_scale: float = 0.1) -> np.ndarray:
    """bf16 weight blob as a uint16 array, in the documented tensor order."""
    lib = _load()
    cs = _Shape(shape.n_layers, shape.d_model, shape.d_ffn, shape.vocab)
    n = lib.ppd_inputs_blob_elems(ctypes.byref(cs))
    assert n == shape.blob_elems
    out = np.empty(n, dtype=np.uint16)
    rc = lib.ppd_inputs_gen_weights(ctypes.byref(cs), seed, sigma, resid_scale, out.ctypes.data)
    if rc != 0:
        raise ValueError("bad model shape")
    return out


def gen_prompt(vocab: int, n: int, seed: int = 1) -> np.ndarray:
    """n uniform-random token ids in [0, vocab), int32.  By convention seed = weight seed + 1."""
    lib = _load()
    out = np.empty(n, dtype=np.int32)
    rc = lib.ppd_inputs_gen_prompt(vocab, seed, n, out.ctypes.data)
    if rc != 0:
        raise ValueError("bad prompt request")
    return out


def blob_views(shape: ModelShape, blob: np.ndarray) -> dict:
    """Named uint16 views into a blob (no copies): 'E', 'g_final', 'W_H', and per layer
    'g1.i', 'Wq.i', 'Wk.i', 'Wv.i', 'Wo.i', 'g2.i', 'Wg.i', 'Wu.i', 'Wd.i'."""
    D, F, V = shape.d_model, shape.d_ffn, shape.vocab
    out, off = {}, 0

    def take(name, rows, cols=None):
        nonlocal off
        n = rows * (cols or 1)
        v = blob[off:off + n]
        out[name] = v.reshape(rows, cols) if cols else v
        off += n

    take("E", V, D)
    for i in range(shape.n_layers):
        take(f"g1.{i}", D)
        for nm in ("Wq", "Wk", "Wv", "Wo"):
            take(f"{nm}.{i}", D, D)
        take(f"g2.{i}", D)
        take(f"Wg.{i}", F, D)
        take(f"Wu.{i}", F, D)
        take(f"Wd.{i}", D, F)
    take("g_final", D)
    take("W_H", V, D)
    assert off == blob.size
    return out


def bf16_to_f32(a: np.ndarray) -> np.ndarray:
    """Widen a uint16 bf16 array to float32 (exact)."""
    return (a.astype(np.uint32) << 16).view(np.float32)
