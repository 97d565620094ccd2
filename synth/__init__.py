"""Seeded synthetic inputs (weights, per-sublayer scales, prompts) for the decoder.

Data only: this package contains none of the decoder's, the cosine rule's or
ADMG's arithmetic.  The CPU oracle and the CUDA library both receive what it
produces as plain buffers, so that they can be compared on identical inputs
without sharing any code.

The recipe stands in for the trained Llama-2 / CodeLlama weights and the
CNN/DM, XSum and HumanEval prompts of the paper's experiments (Section 4),
none of which are available offline:

* every matrix is bf16(N(0, 0.02^2)); the output projections ``wo`` and ``wd``
  of sublayer j (order attn_1, mlp_1, attn_2, ...) are multiplied by a factor
  drawn from U[0.05, 1] before rounding, so that per-sublayer cosine
  similarities spread out;
* RMSNorm gains are bf16(1 + 0.02 z) so that a forgotten gain is detectable;
* embedding and LM head are untied, N(0, 0.02^2);
* prompts are uniform random token ids.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass, field

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "gen.cpp")
_LIB = os.path.join(_HERE, "libsynth.so")


def build(force: bool = False) -> str:
    """Compile the generator into ``libsynth.so`` next to its source."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(
            ["g++", "-O2", "-fopenmp", "-shared", "-fPIC", "-std=c++17", "-o", _LIB, _SRC]
        )
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        lib.synth_normal_bf16.argtypes = [ctypes.c_void_p, ctypes.c_size_t, ctypes.c_uint64, ctypes.c_uint64,
                                          ctypes.c_double, ctypes.c_double, ctypes.c_double]
        lib.synth_normal_bf16.restype = None
        lib.synth_uniform_f64.argtypes = [ctypes.c_void_p, ctypes.c_size_t, ctypes.c_uint64, ctypes.c_uint64,
                                          ctypes.c_double, ctypes.c_double]
        lib.synth_uniform_f64.restype = None
        lib.synth_uniform_i32.argtypes = [ctypes.c_void_p, ctypes.c_size_t, ctypes.c_uint64, ctypes.c_uint64,
                                          ctypes.c_int32]
        lib.synth_uniform_i32.restype = None
        _lib = lib
    return _lib


@dataclass(frozen=True)
class DecoderShape:
    """Dimensions of a Llama-style dense decoder."""
    n_layers: int
    d_model: int
    n_heads: int
    head_dim: int
    d_ffn: int
    vocab: int
    n_kv_heads: int = 0  # 0 = same as n_heads (MHA)

    @property
    def kv_heads(self) -> int:
        return self.n_kv_heads or self.n_heads

    @property
    def kv_dim(self) -> int:
        return self.kv_heads * self.head_dim


# The decoder shapes of the benchmark configurations.
TINY = DecoderShape(n_layers=4, d_model=256, n_heads=4, head_dim=64, d_ffn=688, vocab=1024)
LLAMA_7B = DecoderShape(n_layers=32, d_model=4096, n_heads=32, head_dim=128, d_ffn=11008, vocab=32000)
LLAMA_13B = DecoderShape(n_layers=40, d_model=5120, n_heads=40, head_dim=128, d_ffn=13824, vocab=32000)

# stream identifiers (tensor_id argument of the generator)
_T_EMBED, _T_LM_HEAD, _T_FINAL_NORM, _T_SCALES, _T_PROMPT = 1, 2, 3, 4, 5
_T_VECTOR_BASE = 1 << 32  # free-standing test vectors / matrices, one stream per caller-chosen id
_T_LAYER0, _T_LAYER_STRIDE = 16, 16
_ATTN_NORM, _WQ, _WK, _WV, _WO, _MLP_NORM, _WG, _WU, _WD = range(9)


def normal_bf16(shape, seed: int, tensor_id: int, std: float = 0.02, mean: float = 0.0,
                scale: float = 1.0) -> np.ndarray:
    """bf16 bit patterns (uint16) of (mean + std*z)*scale with z ~ N(0,1)."""
    out = np.empty(shape, dtype=np.uint16)
    _load().synth_normal_bf16(out.ctypes.data, out.size, seed, tensor_id, mean, std, scale)
    return out


def uniform_f64(n: int, seed: int, tensor_id: int, lo: float, hi: float) -> np.ndarray:
    out = np.empty(n, dtype=np.float64)
    _load().synth_uniform_f64(out.ctypes.data, n, seed, tensor_id, lo, hi)
    return out


def make_prompt(vocab: int, n: int, seed: int = 1) -> np.ndarray:
    """n uniform random token ids in [0, vocab)."""
    out = np.empty(n, dtype=np.int32)
    _load().synth_uniform_i32(out.ctypes.data, n, seed, _T_PROMPT, vocab)
    return out


def bf16_to_f32(a: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns to float32 (a data-format helper)."""
    return (a.astype(np.uint32) << 16).view(np.float32)


def f32_to_bf16(a: np.ndarray) -> np.ndarray:
    """Round float32 to bf16 bit patterns, nearest even (a data-format helper)."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32).astype(np.uint64)
    u = u + 0x7FFF + ((u >> 16) & 1)
    return (u >> 16).astype(np.uint16)


@dataclass
class SynthModel:
    """bf16 weights (as uint16 bit patterns) of one synthetic decoder.

    All matrices are row-major ``[out, in]`` (y = W x), stacked over layers.
    """
    shape: DecoderShape
    seed: int
    embed: np.ndarray        # [V, d]
    lm_head: np.ndarray      # [V, d]
    final_norm: np.ndarray   # [d]
    attn_norm: np.ndarray    # [L, d]
    wq: np.ndarray           # [L, d, d]
    wk: np.ndarray           # [L, kv_dim, d]
    wv: np.ndarray           # [L, kv_dim, d]
    wo: np.ndarray           # [L, d, d]
    mlp_norm: np.ndarray     # [L, d]
    wg: np.ndarray           # [L, f, d]
    wu: np.ndarray           # [L, f, d]
    wd: np.ndarray           # [L, d, f]
    scales: np.ndarray = field(default=None)  # [2L] factors of wo (even) / wd (odd)

    def nbytes(self) -> int:
        return sum(getattr(self, k).nbytes for k in
                   ("embed", "lm_head", "final_norm", "attn_norm", "wq", "wk", "wv", "wo", "mlp_norm", "wg", "wu",
                    "wd"))


def make_model(shape: DecoderShape, seed: int = 0, scale_lo: float = 0.05, scale_hi: float = 1.0,
               std: float = 0.02) -> SynthModel:
    """Generate the synthetic decoder of the given shape."""
    L, d, f, V, kv = shape.n_layers, shape.d_model, shape.d_ffn, shape.vocab, shape.kv_dim
    scales = uniform_f64(2 * L, seed, _T_SCALES, scale_lo, scale_hi)

    def stack(rows, cols, which, per_layer_scale=None, gain=False):
        out = np.empty((L, rows, cols) if cols else (L, rows), dtype=np.uint16)
        for l in range(L):
            tid = _T_LAYER0 + l * _T_LAYER_STRIDE + which
            s = 1.0 if per_layer_scale is None else float(per_layer_scale[l])
            if gain:
                out[l] = normal_bf16((rows,), seed, tid, std=0.02, mean=1.0)
            else:
                out[l] = normal_bf16((rows, cols), seed, tid, std=std, scale=s)
        return out

    return SynthModel(
        shape=shape, seed=seed,
        embed=normal_bf16((V, d), seed, _T_EMBED, std=std),
        lm_head=normal_bf16((V, d), seed, _T_LM_HEAD, std=std),
        final_norm=normal_bf16((d,), seed, _T_FINAL_NORM, std=0.02, mean=1.0),
        attn_norm=stack(d, 0, _ATTN_NORM, gain=True),
        wq=stack(d, d, _WQ), wk=stack(kv, d, _WK), wv=stack(kv, d, _WV),
        wo=stack(d, d, _WO, per_layer_scale=scales[0::2]),
        mlp_norm=stack(d, 0, _MLP_NORM, gain=True),
        wg=stack(f, d, _WG), wu=stack(f, d, _WU),
        wd=stack(d, f, _WD, per_layer_scale=scales[1::2]),
        scales=scales,
    )


def make_matrix_bf16(shape, seed: int, stream: int = 0, std: float = 0.02, mean: float = 0.0) -> np.ndarray:
    """A free-standing bf16 array (uint16 bit patterns) for kernel-level tests and micro-benchmarks."""
    return normal_bf16(shape, seed, _T_VECTOR_BASE + stream, std=std, mean=mean)


def make_array_f32(shape, seed: int, stream: int = 0, std: float = 1.0) -> np.ndarray:
    """A float32 array whose entries are bf16-representable N(0, std^2) draws."""
    return bf16_to_f32(make_matrix_bf16(shape, seed, stream, std=std))
