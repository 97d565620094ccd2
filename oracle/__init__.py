"""Python handle on the CPU oracle (``orc.cpp``).

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the
benchmark's CPU-baseline / reference legs.  Nothing on the product path may
import this package, and this package imports nothing of the CUDA library.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "orc.cpp")
_LIB = os.path.join(_HERE, "liborc.so")

USE_CS, USE_RULE1, USE_RULE2 = 1, 2, 4
USE_CS_MLP, RUNNING_C = 8, 16  # extensions beyond Algorithm 1, off by default
ADMG_ALL = USE_CS | USE_RULE1 | USE_RULE2
MODE_AR, MODE_SPEC, MODE_SPEC_MANUAL_MASK = 0, 1, 2
FLAG_NO_ROUNDING = 1
OK, ERR_ARG, ERR_STATE, ERR_OVERFLOW = 0, -1, -2, -4


def build(force: bool = False) -> str:
    """Compile the oracle into ``liborc.so`` next to its source."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["g++", "-O2", "-fopenmp", "-shared", "-fPIC", "-std=c++17", "-o", _LIB, _SRC])
    return _LIB


class Config(ctypes.Structure):
    _fields_ = [(k, ctypes.c_int32) for k in
                ("n_layers", "d_model", "n_heads", "n_kv_heads", "head_dim", "d_ffn", "vocab", "max_seq")] + \
               [("rms_eps", ctypes.c_float), ("rope_theta", ctypes.c_float), ("flags", ctypes.c_uint32)]


class Weights(ctypes.Structure):
    _fields_ = [(k, ctypes.c_void_p) for k in
                ("embed", "lm_head", "final_norm", "attn_norm", "wq", "wk", "wv", "wo", "mlp_norm", "wg", "wu", "wd")]


class AdmgParams(ctypes.Structure):
    _fields_ = [("alpha", ctypes.c_float), ("m", ctypes.c_int32), ("n", ctypes.c_int32), ("flags", ctypes.c_uint32),
                ("alpha_mlp", ctypes.c_float), ("refresh", ctypes.c_int32)]


class GenParams(ctypes.Structure):
    _fields_ = [("mode", ctypes.c_int32), ("draft_len", ctypes.c_int32), ("max_new", ctypes.c_int32),
                ("eos_id", ctypes.c_int32), ("admg", AdmgParams), ("draft_exit_margin", ctypes.c_float),
                ("temperature", ctypes.c_float), ("seed", ctypes.c_uint64)]


class Stats(ctypes.Structure):
    _fields_ = [(k, ctypes.c_int64) for k in
                ("full_passes", "draft_passes", "verify_passes", "rounds", "drafted", "accepted", "prefill_rows")] + \
               [(k, ctypes.c_double) for k in ("ms_prefill", "ms_full", "ms_draft", "ms_verify", "ms_total")]

    def as_dict(self):
        return {k: getattr(self, k) for k, _ in self._fields_}


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        L.orc_cosine.restype = ctypes.c_double
        L.orc_cosine.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64]
        L.orc_last_error.restype = ctypes.c_char_p
        L.orc_uniform.restype = ctypes.c_double
        L.orc_uniform.argtypes = [ctypes.c_uint64, ctypes.c_uint32, ctypes.c_uint32]
        L.orc_sample_cdf.restype = ctypes.c_int32
        L.orc_sample_cdf.argtypes = [ctypes.c_void_p, ctypes.c_int32, ctypes.c_double]
        L.orc_softmax_t.restype = None
        L.orc_softmax_t.argtypes = [ctypes.c_void_p, ctypes.c_int32, ctypes.c_double, ctypes.c_void_p]
        L.orc_spec_accept.restype = ctypes.c_int32
        L.orc_spec_accept.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int32, ctypes.c_int32,
                                      ctypes.c_uint64, ctypes.c_int32, ctypes.c_void_p]
        L.orc_philox4x32_10.restype = None
        L.orc_philox4x32_10.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]
        L.orc_set_sampling.argtypes = [ctypes.c_void_p, ctypes.c_float, ctypes.c_uint64]
        _lib = L
    return _lib


class OracleError(RuntimeError):
    def __init__(self, code, what):
        super().__init__(f"oracle call {what} failed with code {code}")
        self.code = code


def _check(rc, what):
    if rc != 0:
        raise OracleError(rc, what)


def _f32(a):
    return np.ascontiguousarray(a, dtype=np.float32)


def cosine(x, y) -> float:
    x, y = _f32(x), _f32(y)
    assert x.shape == y.shape and x.ndim == 1
    return float(lib().orc_cosine(x.ctypes.data, y.ctypes.data, x.size))


def admg(C, alpha: float, m: int, n: int, flags: int = ADMG_ALL):
    """Algorithm 1.  Returns (remove_attn, remove_mlp) as uint8 arrays indexed by l-1."""
    C = _f32(C)
    L = C.size
    ra, rm = np.zeros(L, np.uint8), np.zeros(L, np.uint8)
    _check(lib().orc_admg(ctypes.c_void_p(C.ctypes.data), ctypes.c_int32(L), ctypes.c_float(alpha), ctypes.c_int32(m),
                          ctypes.c_int32(n), ctypes.c_uint32(flags), ctypes.c_void_p(ra.ctypes.data),
                          ctypes.c_void_p(rm.ctypes.data)), "orc_admg")
    return ra, rm


def admg_ext(C_attn, C_mlp, alpha: float, alpha_mlp: float, m: int, n: int, flags: int):
    """Algorithm 1 plus the optional MLP similarity threshold (``USE_CS_MLP``).  Returns (remove_attn, remove_mlp)."""
    C_attn, C_mlp = _f32(C_attn), _f32(C_mlp)
    L = C_attn.size
    assert C_mlp.size == L
    ra, rm = np.zeros(L, np.uint8), np.zeros(L, np.uint8)
    _check(lib().orc_admg_ext(ctypes.c_void_p(C_attn.ctypes.data), ctypes.c_void_p(C_mlp.ctypes.data), ctypes.c_int32(L),
                              ctypes.c_float(alpha), ctypes.c_float(alpha_mlp), ctypes.c_int32(m), ctypes.c_int32(n),
                              ctypes.c_uint32(flags), ctypes.c_void_p(ra.ctypes.data), ctypes.c_void_p(rm.ctypes.data)),
           "orc_admg_ext")
    return ra, rm


def fused_matvec(x, W, epilogue: int = 0, gain=None, eps: float = 1e-5, W2=None, res=None):
    """One fused sublayer product; see ``orc_fused_matvec``.  Returns (out, cos or None)."""
    x = _f32(x)
    M, n_in = x.shape
    n_out = W.shape[0]
    assert W.dtype == np.uint16 and W.shape[1] == n_in
    out = np.empty((M, n_out), np.float32)
    cosv = np.empty(M, np.float32)
    if res is not None:
        res = _f32(res)
    W = np.ascontiguousarray(W)
    if W2 is not None:
        W2 = np.ascontiguousarray(W2)
    if gain is not None:
        gain = np.ascontiguousarray(gain)
    _check(lib().orc_fused_matvec(
        ctypes.c_void_p(x.ctypes.data), ctypes.c_int32(M), ctypes.c_int32(n_in),
        ctypes.c_void_p(gain.ctypes.data if gain is not None else None), ctypes.c_float(eps),
        ctypes.c_void_p(W.ctypes.data), ctypes.c_void_p(W2.ctypes.data if W2 is not None else None),
        ctypes.c_int32(n_out), ctypes.c_int32(epilogue), ctypes.c_void_p(res.ctypes.data if res is not None else None),
        ctypes.c_void_p(out.ctypes.data), ctypes.c_void_p(cosv.ctypes.data)), "orc_fused_matvec")
    return out, (cosv if epilogue == 2 else None)


DRAW_DRAFT, DRAW_ACCEPT, DRAW_TARGET = 0, 1, 2


def philox4x32_10(counter, key):
    """The counter-based generator behind every random draw: four 32-bit words from a 128-bit counter and a 64-bit key."""
    c = np.ascontiguousarray(counter, dtype=np.uint32)
    k = np.ascontiguousarray(key, dtype=np.uint32)
    assert c.size == 4 and k.size == 2
    out = np.zeros(4, np.uint32)
    lib().orc_philox4x32_10(c.ctypes.data, k.ctypes.data, out.ctypes.data)
    return out


def uniform(seed: int, position: int, kind: int) -> float:
    """The uniform number in (0, 1) of (seed, position of the token being chosen, kind of draw)."""
    return float(lib().orc_uniform(seed, position, kind))


def softmax_t(logits, T: float) -> np.ndarray:
    l = _f32(logits)
    out = np.empty(l.size, np.float64)
    lib().orc_softmax_t(l.ctypes.data, l.size, float(T), out.ctypes.data)
    return out


def sample_cdf(w, u: float) -> int:
    w = np.ascontiguousarray(w, dtype=np.float64)
    return int(lib().orc_sample_cdf(w.ctypes.data, w.size, float(u)))


def spec_accept(p, q, drafts, seed: int, pos0: int):
    """Sampling-based verification of k drafts: p [k+1, V], q [k, V] (float64), drafts [k]. Returns (a, tokens[a+1])."""
    p = np.ascontiguousarray(p, dtype=np.float64)
    q = np.ascontiguousarray(q, dtype=np.float64)
    d = np.ascontiguousarray(drafts, dtype=np.int32)
    k, V = d.size, p.shape[1]
    assert p.shape == (k + 1, V) and (k == 0 or q.shape == (k, V))
    out = np.zeros(k + 1, np.int32)
    a = lib().orc_spec_accept(p.ctypes.data, q.ctypes.data if k else None, d.ctypes.data if k else None, k, V, seed, pos0,
                              out.ctypes.data)
    return int(a), out[: a + 1].copy()


def num_threads() -> int:
    return int(lib().orc_num_threads())


class Oracle:
    """One decoding context of the oracle over a ``synth.SynthModel``-like set of weights."""

    def __init__(self, model, max_seq: int, rms_eps: float = 1e-5, rope_theta: float = 10000.0, flags: int = 0):
        s = model.shape
        self.model = model  # keeps the borrowed weight arrays alive
        self.shape = s
        self.max_seq = max_seq
        self.cfg = Config(s.n_layers, s.d_model, s.n_heads, s.kv_heads, s.head_dim, s.d_ffn, s.vocab, max_seq,
                          rms_eps, rope_theta, flags)
        w = Weights()
        for k, _ in Weights._fields_:
            arr = getattr(model, k)
            assert arr.dtype == np.uint16 and arr.flags["C_CONTIGUOUS"], k
            setattr(w, k, arr.ctypes.data)
        self._w = w
        self._ctx = ctypes.c_void_p()
        _check(lib().orc_create(ctypes.byref(self.cfg), ctypes.byref(w), ctypes.byref(self._ctx)), "orc_create")

    def close(self):
        if self._ctx:
            lib().orc_destroy(self._ctx)
            self._ctx = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- state
    def reset(self):
        _check(lib().orc_reset(self._ctx), "orc_reset")

    def positions(self):
        a, b = ctypes.c_int32(), ctypes.c_int32()
        _check(lib().orc_get_positions(self._ctx, ctypes.byref(a), ctypes.byref(b)), "orc_get_positions")
        return a.value, b.value

    # -- passes
    def prefill(self, tokens) -> int:
        t = np.ascontiguousarray(tokens, dtype=np.int32)
        out = ctypes.c_int32()
        _check(lib().orc_prefill(self._ctx, ctypes.c_void_p(t.ctypes.data), ctypes.c_int32(t.size), ctypes.byref(out)),
               "orc_prefill")
        return out.value

    def similarity(self):
        L = self.shape.n_layers
        ca, cm = np.zeros(L, np.float32), np.zeros(L, np.float32)
        n = ctypes.c_int32()
        _check(lib().orc_get_similarity(self._ctx, ctypes.c_void_p(ca.ctypes.data), ctypes.c_void_p(cm.ctypes.data),
                                        ctypes.byref(n)), "orc_get_similarity")
        return ca, cm, n.value

    def set_skip_mask(self, skip_attn, skip_mlp):
        a = np.ascontiguousarray(skip_attn, dtype=np.uint8)
        b = np.ascontiguousarray(skip_mlp, dtype=np.uint8)
        assert a.size == b.size == self.shape.n_layers
        _check(lib().orc_set_skip_mask(self._ctx, ctypes.c_void_p(a.ctypes.data), ctypes.c_void_p(b.ctypes.data)),
               "orc_set_skip_mask")

    def set_sampling(self, temperature: float, seed: int = 0):
        """temperature 0 = greedy (the default); above 0 every token is drawn, see ``orc_set_sampling``."""
        _check(lib().orc_set_sampling(self._ctx, ctypes.c_float(temperature), ctypes.c_uint64(seed)), "orc_set_sampling")

    def set_running_similarity(self, on: bool):
        _check(lib().orc_set_running_similarity(self._ctx, ctypes.c_int32(1 if on else 0)), "orc_set_running_similarity")

    def admg_update(self, alpha=0.985, m=3, n=2, flags=ADMG_ALL, alpha_mlp=1.0, refresh=0):
        L = self.shape.n_layers
        a, b = np.zeros(L, np.uint8), np.zeros(L, np.uint8)
        p = AdmgParams(alpha, m, n, flags, alpha_mlp, refresh)
        _check(lib().orc_admg_update(self._ctx, ctypes.byref(p), ctypes.c_void_p(a.ctypes.data),
                                     ctypes.c_void_p(b.ctypes.data)), "orc_admg_update")
        return a, b

    def decode_step(self, token: int) -> int:
        out = ctypes.c_int32()
        _check(lib().orc_decode_step(self._ctx, ctypes.c_int32(token), ctypes.byref(out)), "orc_decode_step")
        return out.value

    def draft_step(self, token: int) -> int:
        out = ctypes.c_int32()
        _check(lib().orc_draft_step(self._ctx, ctypes.c_int32(token), ctypes.byref(out)), "orc_draft_step")
        return out.value

    def verify(self, tokens):
        t = np.ascontiguousarray(tokens, dtype=np.int32)
        k = t.size - 1
        out = np.zeros(k + 1, np.int32)
        a = ctypes.c_int32()
        _check(lib().orc_verify(self._ctx, ctypes.c_void_p(t.ctypes.data), ctypes.c_int32(k), ctypes.byref(a),
                                ctypes.c_void_p(out.ctypes.data)), "orc_verify")
        return a.value, out[: a.value + 1].copy()

    def generate(self, prompt, max_new: int, mode: int = MODE_AR, draft_len: int = 4, alpha=0.985, m=3, n=2,
                 flags=ADMG_ALL, eos_id: int = -1, alpha_mlp=1.0, refresh=0, draft_exit_margin=0.0, temperature=0.0, seed=0):
        """Returns (tokens, margins, stats dict)."""
        p = np.ascontiguousarray(prompt, dtype=np.int32)
        gp = GenParams(mode, draft_len, max_new, eos_id, AdmgParams(alpha, m, n, flags, alpha_mlp, refresh), draft_exit_margin,
                       temperature, seed)
        out = np.zeros(max_new, np.int32)
        margins = np.zeros(max_new, np.float32)
        n_out = ctypes.c_int32()
        st = Stats()
        _check(lib().orc_generate(self._ctx, ctypes.c_void_p(p.ctypes.data), ctypes.c_int32(p.size), ctypes.byref(gp),
                                  ctypes.c_void_p(out.ctypes.data), ctypes.byref(n_out), ctypes.byref(st),
                                  ctypes.c_void_p(margins.ctypes.data)), "orc_generate")
        return out[: n_out.value].copy(), margins[: n_out.value].copy(), st.as_dict()

    def stats(self):
        st = Stats()
        _check(lib().orc_get_stats(self._ctx, ctypes.byref(st)), "orc_get_stats")
        return st.as_dict()

    # -- results of the last pass
    def last(self):
        """dict(M, logits [M,V], cos_attn [L,M], cos_mlp [L,M], argmax [M], margin [M])."""
        L, V = self.shape.n_layers, self.shape.vocab
        M = ctypes.c_int32()
        _check(lib().orc_get_last(self._ctx, ctypes.byref(M), None, None, None, None, None), "orc_get_last")
        m = M.value
        logits = np.empty((m, V), np.float32)
        ca, cm = np.empty((L, m), np.float32), np.empty((L, m), np.float32)
        am, mg = np.empty(m, np.int32), np.empty(m, np.float32)
        _check(lib().orc_get_last(self._ctx, ctypes.byref(M), ctypes.c_void_p(logits.ctypes.data),
                                  ctypes.c_void_p(ca.ctypes.data), ctypes.c_void_p(cm.ctypes.data),
                                  ctypes.c_void_p(am.ctypes.data), ctypes.c_void_p(mg.ctypes.data)), "orc_get_last")
        return dict(M=m, logits=logits, cos_attn=ca, cos_mlp=cm, argmax=am, margin=mg)

    def kv(self, layer: int, pos: int):
        kvd = self.shape.kv_dim
        k, v = np.empty(kvd, np.float32), np.empty(kvd, np.float32)
        _check(lib().orc_get_kv(self._ctx, ctypes.c_int32(layer), ctypes.c_int32(pos), ctypes.c_void_p(k.ctypes.data),
                                ctypes.c_void_p(v.ctypes.data)), "orc_get_kv")
        return k, v
