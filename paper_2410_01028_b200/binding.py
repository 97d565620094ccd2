"""ctypes binding of the C ABI in ``include/asd.h``: same names, argument marshalling only."""
from __future__ import annotations

import ctypes
import os

import numpy as np

from . import build as _build

USE_CS, USE_RULE1, USE_RULE2, ADMG_ALL = 1, 2, 4, 7
USE_CS_MLP, RUNNING_C = 8, 16  # extensions beyond Algorithm 1 (see asd_admg_params), off by default
MODE_AR, MODE_SPEC, MODE_SPEC_MANUAL_MASK = 0, 1, 2
EPI_PLAIN, EPI_SWIGLU, EPI_RESIDUAL = 0, 1, 2
PREFILL_AUTO, PREFILL_ROWS, PREFILL_GEMM = 0, 1, 2
OK, ERR_ARG, ERR_STATE, ERR_NOMEM, ERR_OVERFLOW, ERR_CUDA, ERR_DEVICE_TIMEOUT, ERR_IO = 0, -1, -2, -3, -4, -5, -6, -7


class Config(ctypes.Structure):
    _fields_ = [(k, ctypes.c_int32) for k in
                ("n_layers", "d_model", "n_heads", "n_kv_heads", "head_dim", "d_ffn", "vocab", "max_seq", "max_draft")] + \
               [("rms_eps", ctypes.c_float), ("rope_theta", ctypes.c_float)]


class HostWeights(ctypes.Structure):
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
               [(k, ctypes.c_double) for k in ("ms_prefill", "ms_full", "ms_draft", "ms_verify", "ms_total",
                                               "bytes_full", "bytes_draft", "bytes_verify")] + \
               [("kernel_launches", ctypes.c_int64)]

    def as_dict(self):
        return {k: getattr(self, k) for k, _ in self._fields_}


# every symbol include/asd.h declares
EXPORTS = (
    "asd_workspace_bytes", "asd_create", "asd_destroy", "asd_last_error", "asd_load_weights_host",
    "asd_load_weights_file", "asd_reset", "asd_prefill", "asd_prefill_device", "asd_get_similarity", "asd_admg_update",
    "asd_set_skip_mask", "asd_decode_step", "asd_draft_step", "asd_verify", "asd_generate", "asd_generate_device",
    "asd_get_last_cosines", "asd_get_last_margins", "asd_get_last_logits", "asd_set_debug", "asd_get_last_trace", "asd_get_kv", "asd_get_positions", "asd_get_stats",
    "asd_fused_gemv_scratch_bytes", "asd_fused_gemv", "asd_fused_gemv_static", "asd_admg", "asd_admg_ext", "asd_set_running_similarity", "asd_set_prefill_mode", "asd_gemm_bf16", "asd_set_sampling",
)

_lib = None


def lib():
    """Load (building first if the sources are newer) the CUDA library. Fails loudly if that is impossible."""
    global _lib
    if _lib is None:
        path = _build.build()
        L = ctypes.CDLL(path)
        for name in EXPORTS:
            getattr(L, name)  # AttributeError if the library lacks a declared symbol
        L.asd_workspace_bytes.restype = ctypes.c_size_t
        L.asd_fused_gemv_scratch_bytes.restype = ctypes.c_size_t
        L.asd_last_error.restype = ctypes.c_char_p
        L.asd_last_error.argtypes = [ctypes.c_void_p]
        _lib = L
    return _lib


class AsdError(RuntimeError):
    def __init__(self, code, what, detail=""):
        super().__init__(f"{what} failed with code {code}" + (f": {detail}" if detail else ""))
        self.code = code


def _vp(a):
    """void* of a numpy array, a torch tensor, an int address or None."""
    if a is None:
        return ctypes.c_void_p(None)
    if isinstance(a, np.ndarray):
        return ctypes.c_void_p(a.ctypes.data)
    if isinstance(a, int):
        return ctypes.c_void_p(a)
    return ctypes.c_void_p(a.data_ptr())


def make_config(shape, max_seq, max_draft=8, rms_eps=1e-5, rope_theta=10000.0) -> Config:
    kvh = getattr(shape, "kv_heads", None) or shape.n_heads
    return Config(shape.n_layers, shape.d_model, shape.n_heads, kvh, shape.head_dim, shape.d_ffn, shape.vocab, max_seq,
                  max_draft, rms_eps, rope_theta)


def workspace_bytes(cfg: Config) -> int:
    return int(lib().asd_workspace_bytes(ctypes.byref(cfg)))


def admg(C, alpha, m, n, flags=ADMG_ALL):
    """Algorithm 1 as a pure function: (remove_attn, remove_mlp) as uint8 arrays indexed by l-1."""
    C = np.ascontiguousarray(C, dtype=np.float32)
    ra, rm = np.zeros(C.size, np.uint8), np.zeros(C.size, np.uint8)
    p = AdmgParams(alpha, m, n, flags)
    rc = lib().asd_admg(_vp(C), ctypes.c_int32(C.size), ctypes.byref(p), _vp(ra), _vp(rm))
    if rc:
        raise AsdError(rc, "asd_admg")
    return ra, rm


def admg_ext(C_attn, C_mlp, alpha, alpha_mlp, m, n, flags):
    """Algorithm 1 plus the MLP similarity threshold of ``USE_CS_MLP``: (remove_attn, remove_mlp)."""
    C_attn = np.ascontiguousarray(C_attn, dtype=np.float32)
    C_mlp = np.ascontiguousarray(C_mlp, dtype=np.float32)
    assert C_attn.size == C_mlp.size
    ra, rm = np.zeros(C_attn.size, np.uint8), np.zeros(C_attn.size, np.uint8)
    p = AdmgParams(alpha, m, n, flags, alpha_mlp, 0)
    rc = lib().asd_admg_ext(_vp(C_attn), _vp(C_mlp), ctypes.c_int32(C_attn.size), ctypes.byref(p), _vp(ra), _vp(rm))
    if rc:
        raise AsdError(rc, "asd_admg_ext")
    return ra, rm


def fused_gemv_scratch_bytes() -> int:
    return int(lib().asd_fused_gemv_scratch_bytes())


def fused_gemv(x, W, epilogue, out, gain=None, eps=1e-5, cos=None, scratch=None, stream=None):
    """asd_fused_gemv on torch CUDA tensors (x: float32 if gain else bfloat16; W: bfloat16 [n_rows, n_in])."""
    import torch
    M, n_in = x.shape
    n_rows = W.shape[0]
    st = stream if stream is not None else torch.cuda.current_stream().cuda_stream
    rc = lib().asd_fused_gemv(ctypes.c_void_p(st), ctypes.c_int32(M), ctypes.c_int32(n_in), ctypes.c_int32(n_rows),
                              _vp(x), _vp(gain), ctypes.c_float(eps), _vp(W), ctypes.c_int32(epilogue), _vp(out),
                              _vp(cos), _vp(scratch), ctypes.c_size_t(scratch.numel() * scratch.element_size()))
    if rc:
        raise AsdError(rc, "asd_fused_gemv")


def fused_gemv_static(x, W, epilogue, out, gain=None, eps=1e-5, cos=None, stream=None):
    """asd_fused_gemv_static: as ``fused_gemv`` but with the library's built-in scratch array, for callers that
    cannot allocate device memory. Calls that may overlap on the GPU must be ordered on one stream."""
    import torch
    M, n_in = x.shape
    n_rows = W.shape[0]
    st = stream if stream is not None else torch.cuda.current_stream().cuda_stream
    rc = lib().asd_fused_gemv_static(ctypes.c_void_p(st), ctypes.c_int32(M), ctypes.c_int32(n_in),
                                     ctypes.c_int32(n_rows), _vp(x), _vp(gain), ctypes.c_float(eps), _vp(W),
                                     ctypes.c_int32(epilogue), _vp(out), _vp(cos))
    if rc:
        raise AsdError(rc, "asd_fused_gemv_static")


def gemm_bf16(A, W, C, status, stream=None):
    """asd_gemm_bf16 on torch CUDA tensors: C[M, N] (float32) = A[M, K] (bfloat16) @ W[N, K]^T (bfloat16).
    ``status`` is an int32 CUDA tensor of 8 elements; element 0 stays 0 unless a device-side wait expired."""
    import torch
    M, K = A.shape
    N = W.shape[0]
    assert W.shape[1] == K and tuple(C.shape) == (M, N) and status.numel() >= 8
    st = stream if stream is not None else torch.cuda.current_stream().cuda_stream
    rc = lib().asd_gemm_bf16(ctypes.c_void_p(st), ctypes.c_int32(M), ctypes.c_int32(N), ctypes.c_int32(K), _vp(A), _vp(W),
                             _vp(C), _vp(status))
    if rc:
        raise AsdError(rc, "asd_gemm_bf16")


class Decoder:
    """One decoding context. The workspace is a torch uint8 CUDA tensor; work runs on torch's current stream."""

    def __init__(self, shape, max_seq, max_draft=8, rms_eps=1e-5, rope_theta=10000.0, device="cuda:0"):
        import torch
        if not torch.cuda.is_available():
            raise RuntimeError("paper_2410_01028_b200 needs a CUDA device; there is no CPU fallback")
        self._torch = torch
        self.shape = shape
        self.device = torch.device(device)
        self.cfg = make_config(shape, max_seq, max_draft, rms_eps, rope_theta)
        nbytes = workspace_bytes(self.cfg)
        if nbytes == 0:
            raise AsdError(ERR_ARG, "asd_workspace_bytes", "unsupported decoder shape")
        torch.cuda.set_device(self.device)
        self.workspace = torch.empty(nbytes + 256, dtype=torch.uint8, device=self.device)
        base = self.workspace.data_ptr()
        self._ws_ptr = (base + 255) // 256 * 256
        self.stream = torch.cuda.current_stream(self.device).cuda_stream
        self._ctx = ctypes.c_void_p()
        rc = lib().asd_create(ctypes.byref(self.cfg), ctypes.c_void_p(self._ws_ptr), ctypes.c_size_t(nbytes),
                              ctypes.c_void_p(self.stream), ctypes.byref(self._ctx))
        if rc:
            raise AsdError(rc, "asd_create")

    # -- helpers
    def _check(self, rc, what):
        if rc:
            detail = lib().asd_last_error(self._ctx)
            raise AsdError(rc, what, detail.decode() if detail else "")

    def close(self):
        if getattr(self, "_ctx", None):
            lib().asd_destroy(self._ctx)
            self._ctx = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- weights
    def load_weights_host(self, model):
        w = HostWeights()
        keep = []
        for k, _ in HostWeights._fields_:
            arr = np.ascontiguousarray(getattr(model, k))
            assert arr.dtype == np.uint16, k
            keep.append(arr)
            setattr(w, k, arr.ctypes.data)
        self._check(lib().asd_load_weights_host(self._ctx, ctypes.byref(w)), "asd_load_weights_host")

    def load_weights_file(self, path):
        self._check(lib().asd_load_weights_file(self._ctx, path.encode()), "asd_load_weights_file")

    # -- state
    def reset(self):
        self._check(lib().asd_reset(self._ctx), "asd_reset")

    def positions(self):
        a, b = ctypes.c_int32(), ctypes.c_int32()
        self._check(lib().asd_get_positions(self._ctx, ctypes.byref(a), ctypes.byref(b)), "asd_get_positions")
        return a.value, b.value

    def set_debug(self, record_logits=True, trace=False, short_waits=False, missing_arrival=False, no_tagged_handoff=False):
        """record_logits / trace: see asd_set_debug. short_waits and missing_arrival exercise the bounded device waits:
        with both set, the next pass ends with ASD_ERR_DEVICE_TIMEOUT after about a millisecond (see include/asd.h)."""
        flags = ((1 if record_logits else 0) | (2 if trace else 0) | (4 if short_waits else 0) | (8 if missing_arrival else 0)
                 | (16 if no_tagged_handoff else 0))
        self._check(lib().asd_set_debug(self._ctx, ctypes.c_int32(flags)), "asd_set_debug")

    def set_sampling(self, temperature, seed=0):
        """temperature 0 = greedy (default); above 0 every token is drawn and verification keeps M's distribution
        (see asd_set_sampling)."""
        self._check(lib().asd_set_sampling(self._ctx, ctypes.c_float(temperature), ctypes.c_uint64(seed)), "asd_set_sampling")

    def set_prefill_mode(self, mode):
        """PREFILL_AUTO (default), PREFILL_ROWS (row passes, bit-identical to one-row passes) or PREFILL_GEMM."""
        self._check(lib().asd_set_prefill_mode(self._ctx, ctypes.c_int32(mode)), "asd_set_prefill_mode")

    def get_last_trace(self):
        """Per-stage device timeline of the last pass: int64 array [n_stages, 12, n_ctas] (see asd_get_last_trace)."""
        ns, nc = ctypes.c_int32(), ctypes.c_int32()
        self._check(lib().asd_get_last_trace(self._ctx, ctypes.byref(ns), ctypes.byref(nc), None), "asd_get_last_trace")
        out = np.zeros((ns.value, 12, nc.value), np.int64)
        self._check(lib().asd_get_last_trace(self._ctx, ctypes.byref(ns), ctypes.byref(nc), _vp(out)), "asd_get_last_trace")
        return out

    # -- passes
    def prefill(self, tokens) -> int:
        t = np.ascontiguousarray(tokens, dtype=np.int32)
        out = ctypes.c_int32()
        self._check(lib().asd_prefill(self._ctx, _vp(t), ctypes.c_int32(t.size), ctypes.byref(out)), "asd_prefill")
        return out.value

    def prefill_device(self, dev_tokens) -> int:
        out = ctypes.c_int32()
        self._check(lib().asd_prefill_device(self._ctx, _vp(dev_tokens), ctypes.c_int32(dev_tokens.numel()),
                                             ctypes.byref(out)), "asd_prefill_device")
        return out.value

    def get_similarity(self):
        L = self.shape.n_layers
        ca, cm = np.zeros(L, np.float32), np.zeros(L, np.float32)
        n = ctypes.c_int32()
        self._check(lib().asd_get_similarity(self._ctx, _vp(ca), _vp(cm), ctypes.byref(n)), "asd_get_similarity")
        return ca, cm, n.value

    def set_running_similarity(self, on):
        self._check(lib().asd_set_running_similarity(self._ctx, ctypes.c_int32(1 if on else 0)), "asd_set_running_similarity")

    def admg_update(self, alpha=0.985, m=3, n=2, flags=ADMG_ALL, alpha_mlp=1.0, refresh=0):
        L = self.shape.n_layers
        a, b = np.zeros(L, np.uint8), np.zeros(L, np.uint8)
        p = AdmgParams(alpha, m, n, flags, alpha_mlp, refresh)
        self._check(lib().asd_admg_update(self._ctx, ctypes.byref(p), _vp(a), _vp(b)), "asd_admg_update")
        return a, b

    def set_skip_mask(self, skip_attn, skip_mlp):
        a = np.ascontiguousarray(skip_attn, dtype=np.uint8)
        b = np.ascontiguousarray(skip_mlp, dtype=np.uint8)
        assert a.size == b.size == self.shape.n_layers
        self._check(lib().asd_set_skip_mask(self._ctx, _vp(a), _vp(b)), "asd_set_skip_mask")

    def decode_step(self, token: int) -> int:
        out = ctypes.c_int32()
        self._check(lib().asd_decode_step(self._ctx, ctypes.c_int32(token), ctypes.byref(out)), "asd_decode_step")
        return out.value

    def draft_step(self, token: int) -> int:
        out = ctypes.c_int32()
        self._check(lib().asd_draft_step(self._ctx, ctypes.c_int32(token), ctypes.byref(out)), "asd_draft_step")
        return out.value

    def verify(self, tokens):
        t = np.ascontiguousarray(tokens, dtype=np.int32)
        k = t.size - 1
        out = np.zeros(k + 1, np.int32)
        a = ctypes.c_int32()
        self._check(lib().asd_verify(self._ctx, _vp(t), ctypes.c_int32(k), ctypes.byref(a), _vp(out)), "asd_verify")
        return a.value, out[: a.value + 1].copy()

    def _gen_params(self, max_new, mode, draft_len, alpha, m, n, flags, eos_id, alpha_mlp=1.0, refresh=0, draft_exit_margin=0.0,
                    temperature=0.0, seed=0):
        return GenParams(mode, draft_len, max_new, eos_id, AdmgParams(alpha, m, n, flags, alpha_mlp, refresh), draft_exit_margin,
                         temperature, seed)

    def generate(self, prompt, max_new, mode=MODE_AR, draft_len=4, alpha=0.985, m=3, n=2, flags=ADMG_ALL, eos_id=-1,
                 alpha_mlp=1.0, refresh=0, draft_exit_margin=0.0, temperature=0.0, seed=0):
        """Host buffers in, host buffers out. Returns (tokens, stats dict)."""
        p = np.ascontiguousarray(prompt, dtype=np.int32)
        gp = self._gen_params(max_new, mode, draft_len, alpha, m, n, flags, eos_id, alpha_mlp, refresh, draft_exit_margin,
                              temperature, seed)
        out = np.zeros(max_new, np.int32)
        n_out = ctypes.c_int32()
        st = Stats()
        self._check(lib().asd_generate(self._ctx, _vp(p), ctypes.c_int32(p.size), ctypes.byref(gp), _vp(out),
                                       ctypes.byref(n_out), ctypes.byref(st)), "asd_generate")
        return out[: n_out.value].copy(), st.as_dict()

    def generate_device(self, dev_prompt, dev_out, max_new, mode=MODE_AR, draft_len=4, alpha=0.985, m=3, n=2,
                        flags=ADMG_ALL, eos_id=-1, alpha_mlp=1.0, refresh=0, draft_exit_margin=0.0, temperature=0.0, seed=0):
        """Prompt and output are int32 CUDA tensors. Returns (n_out, stats dict)."""
        gp = self._gen_params(max_new, mode, draft_len, alpha, m, n, flags, eos_id, alpha_mlp, refresh, draft_exit_margin,
                              temperature, seed)
        n_out = ctypes.c_int32()
        st = Stats()
        self._check(lib().asd_generate_device(self._ctx, _vp(dev_prompt), ctypes.c_int32(dev_prompt.numel()),
                                              ctypes.byref(gp), _vp(dev_out), ctypes.byref(n_out), ctypes.byref(st)),
                    "asd_generate_device")
        return n_out.value, st.as_dict()

    # -- inspection
    def get_last_cosines(self):
        L = self.shape.n_layers
        M = ctypes.c_int32()
        self._check(lib().asd_get_last_cosines(self._ctx, ctypes.byref(M), None, None), "asd_get_last_cosines")
        ca, cm = np.empty((L, M.value), np.float32), np.empty((L, M.value), np.float32)
        self._check(lib().asd_get_last_cosines(self._ctx, ctypes.byref(M), _vp(ca), _vp(cm)), "asd_get_last_cosines")
        return ca, cm

    def get_last_margins(self):
        M = ctypes.c_int32()
        self._check(lib().asd_get_last_margins(self._ctx, ctypes.byref(M), None), "asd_get_last_margins")
        out = np.empty(M.value, np.float32)
        self._check(lib().asd_get_last_margins(self._ctx, ctypes.byref(M), _vp(out)), "asd_get_last_margins")
        return out

    def get_last_logits(self):
        M = ctypes.c_int32()
        self._check(lib().asd_get_last_logits(self._ctx, ctypes.byref(M), None), "asd_get_last_logits")
        out = np.empty((M.value, self.shape.vocab), np.float32)
        self._check(lib().asd_get_last_logits(self._ctx, ctypes.byref(M), _vp(out)), "asd_get_last_logits")
        return out

    def get_kv(self, layer, pos):
        kvd = self.cfg.n_kv_heads * self.cfg.head_dim
        k, v = np.empty(kvd, np.uint16), np.empty(kvd, np.uint16)
        self._check(lib().asd_get_kv(self._ctx, ctypes.c_int32(layer), ctypes.c_int32(pos), _vp(k), _vp(v)),
                    "asd_get_kv")
        return k, v

    def get_stats(self):
        st = Stats()
        self._check(lib().asd_get_stats(self._ctx, ctypes.byref(st)), "asd_get_stats")
        return st.as_dict()
