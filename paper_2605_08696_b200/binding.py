"""ctypes binding of libsrm.so. Argument marshalling only.

Device memory and streams come from torch; every function below passes raw pointers and sizes
to the C ABI declared in include/srm.h and raises SRMError on a non-zero return code.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass

import numpy as np
import torch

from . import build as _build

EPI_BIAS_GELU, EPI_BIAS_RESIDUAL, EPI_PLAIN = 0, 1, 2
DTYPE_FP32, DTYPE_BF16, DTYPE_FP16 = 0, 1, 2
FLAG_SIMT_GEMM = 1
FLAG_HEAD_PROJ = 2
FLAG_NO_GRAPH = 4
FLAG_GRAPH = 8
FLAG_NO_SPLITK = 16
FLAG_NO_FUSED_TOPK = 32
FLAG_NO_SMALL_BATCH = 64
FLAG_NO_TAIL_SPLIT = 128
FLAG_NO_FUSED_FFN = 256
FLAG_NO_KSLICE = 512
# enum srm_error
ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_ALIGNMENT, ERR_BUFFER_TOO_SMALL, ERR_CTX_OVERFLOW, ERR_CUDA, \
    ERR_DEVICE_STATUS, ERR_STATIC_SCRATCH = -1, -2, -3, -4, -5, -6, -7, -8

# enum srm_tensor
T_E, T_LN1_G, T_LN1_B, T_ALPHA, T_BETA, T_LAMBDA, T_LN2_G, T_LN2_B, T_W1, T_B1, T_W2, T_B2, \
    T_LNF_G, T_LNF_B, T_W_LM, T_W_IN, T_W_OUT, T_ALPHA_COL, T_LAMBDA_COL, T_W_COMB = range(20)
MIXER_MIXED, MIXER_COMBINED, MIXER_KERNEL = 0, 1, 2
_LAYER_TENSORS = {"ln1_g": T_LN1_G, "ln1_b": T_LN1_B, "alpha": T_ALPHA, "beta": T_BETA, "lam": T_LAMBDA,
                  "ln2_g": T_LN2_G, "ln2_b": T_LN2_B, "W1": T_W1, "b1": T_B1, "W2": T_W2, "b2": T_B2}
_GLOBAL_TENSORS = {"E": T_E, "lnf_g": T_LNF_G, "lnf_b": T_LNF_B, "W_lm": T_W_LM}


class SRMError(RuntimeError):
    def __init__(self, code, where):
        self.code = code
        msg = _lib().srm_strerror(code).decode() if _LIB is not None else "?"
        extra = f" (cudaError {_lib().srm_last_cuda_error()})" if code == -6 else ""
        super().__init__(f"{where}: {msg}{extra} [{code}]")


class _Config(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("d_model", C.c_int32), ("n_heads", C.c_int32),
                ("ffn_mult", C.c_int32), ("vocab", C.c_int32), ("n_ctx", C.c_int32),
                ("dtype", C.c_int32), ("state_dtype", C.c_int32), ("ln_eps", C.c_float),
                ("flags", C.c_int32), ("mixer", C.c_int32), ("kernel_size", C.c_int32)]


class _Sampling(C.Structure):
    _fields_ = [("mode", C.c_int32), ("top_k", C.c_int32), ("temperature", C.c_float),
                ("top_p", C.c_float), ("seed", C.c_uint64), ("sample_idx_base", C.c_uint64)]


@dataclass
class Sampling:
    mode: str = "greedy"          # "greedy", "topk" or "topp"
    top_k: int = 50
    temperature: float = 1.0
    seed: int = 0
    sample_idx_base: int = 0
    top_p: float = 1.0

    def c(self) -> _Sampling:
        return _Sampling({"greedy": 0, "topk": 1, "topp": 2}[self.mode], self.top_k, self.temperature, self.top_p,
                         self.seed & 0xFFFFFFFFFFFFFFFF, self.sample_idx_base)


_LIB = None

# every symbol include/srm.h declares: (name, restype, argtypes)
_P, _I32, _I64, _SZ = C.c_void_p, C.c_int32, C.c_int64, C.c_size_t
SYMBOLS = {
    "srm_weights_bytes": (_SZ, [C.POINTER(_Config)]),
    "srm_weight_slot": (C.c_int, [C.POINTER(_Config), _I32, _I32, C.POINTER(_SZ), C.POINTER(_SZ), C.POINTER(_I32)]),
    "srm_state_bytes": (_SZ, [C.POINTER(_Config), _I64]),
    "srm_cache_planes": (_I32, [C.POINTER(_Config)]),
    "srm_workspace_bytes": (_SZ, [C.POINTER(_Config), _I64, _I32]),
    "srm_prefill_workspace_bytes": (_SZ, [C.POINTER(_Config), _I64, _I32]),
    "srm_create": (C.c_int, [C.POINTER(_Config), _P, _SZ, C.POINTER(_P)]),
    "srm_destroy": (C.c_int, [_P]),
    "srm_state_create": (C.c_int, [_P, _I64, _P, _SZ, _P, C.POINTER(_P)]),
    "srm_state_destroy": (C.c_int, [_P]),
    "srm_state_reset": (C.c_int, [_P, _P]),
    "srm_state_pos": (_I64, [_P]),
    "srm_state_set_pos": (C.c_int, [_P, _I64]),
    "srm_state_adopt_positions": (C.c_int, [_P, _I64]),
    "srm_state_is_ragged": (C.c_int, [_P]),
    "srm_state_layer_ptr": (_P, [_P, _I32]),
    "srm_state_last_token_ptr": (_P, [_P]),
    "srm_state_topk_threshold_ptr": (_P, [_P]),
    "srm_state_topk_handed_back": (C.c_int, [_P, _P, C.POINTER(C.c_uint64)]),
    "srm_status": (C.c_int, [_P, _P, C.POINTER(C.c_uint32)]),
    "srm_prefill": (C.c_int, [_P, _P, _P, _I32, C.POINTER(_Sampling), _P, _P, _P, _SZ, _P]),
    "srm_prefill_ragged": (C.c_int, [_P, _P, _P, _I32, _P, C.POINTER(_Sampling), _P, _P, _P, _SZ, _P]),
    "srm_prefill_replicated": (C.c_int, [_P, _P, _P, _I32, _I32, _I32, C.POINTER(_Sampling), _P, _P, _P, _SZ, _P]),
    "srm_decode_step": (C.c_int, [_P, _P, _P, C.POINTER(_Sampling), _I32, _P, _P, _P, _SZ, _P]),
    "srm_generate": (C.c_int, [_P, _P, _I32, _I32, C.POINTER(_Sampling), _P, _I64, _P, _SZ, _P]),
    "srm_decode_step_host": (C.c_int, [_P, _P, _P, C.POINTER(_Sampling), _I32, _P, _P, _SZ, _P]),
    "srm_decode_step_static": (C.c_int, [_P, _P, _P, C.POINTER(_Sampling), _I32, _P, _P, _P]),
    "srm_k_mixer_step": (C.c_int, [_P, _I32, _I32, _I64, _P, _P, _P, _P, _P, _P]),
    "srm_k_final_norm": (C.c_int, [_P, _I64, _P, _P, _P]),
    "srm_k_gemm": (C.c_int, [_P, _I32, _I64, _I64, _I64, _P, _P, _P, _P, _P, _P]),
    "srm_k_gemm_splitk_order_bytes": (_SZ, [_I64, _I64]),
    "srm_k_gemm_splitk": (C.c_int, [_P, _I64, _I64, _I64, _P, _P, _P, _P, _P, _SZ, _P, _P]),
    "srm_k_gemm_splitk_plan": (_I64, [_I64, _I64, _I64, _I32, _I32, C.POINTER(_I64), _I64]),
    "srm_k_ffn_ready_bytes": (_SZ, [_I64, _I64]),
    "srm_k_ffn": (C.c_int, [_P, _I32, _I64, _P, _P, _P, _P, _SZ, _P, _P]),
    "srm_k_ffn_plan": (_I64, [_I64, _I32, _I32, _I32, C.POINTER(_I32), C.POINTER(_I32), _I64, C.POINTER(C.c_double),
                              C.POINTER(C.c_double)]),
    "srm_k_mixer_combined_step": (C.c_int, [_I64, _I32, _I32, _I32, _I32] + [_P] * 11),
    "srm_k_mixer_kernel_step": (C.c_int, [_I64, _I32, _I32, _I32, _I32] + [_P] * 7),
    "srm_k_mixer_combined_scan": (C.c_int, [_I64, _I32, _I32, _I32, _I32, _I32] + [_P] * 11),
    "srm_k_mixer_kernel_scan": (C.c_int, [_I64, _I32, _I32, _I32, _I32, _I32] + [_P] * 7),
    "srm_k_lm_head_greedy": (C.c_int, [_P, _I64, _P, _P, _SZ, _P, _P, _P]),
    "srm_k_select": (C.c_int, [_P, _I64, _P, C.POINTER(_Sampling), _I32, _P, _P, _P]),
    "srm_k_prefill_mixer": (C.c_int, [_P, _I32, _I64, _I32, _P, _P, _P, _P, _P, _P]),
    "srm_k_wait_probe": (C.c_int, [_P, _I64, _P, _P]),
    "srm_profile_enable": (C.c_int, [_P, C.c_int]),
    "srm_profile_read": (C.c_int, [_P, _I32, C.POINTER(C.c_uint64), C.POINTER(C.c_double)]),
    "srm_profile_reset": (C.c_int, [_P]),
    "srm_kernel_launches": (C.c_uint64, []),
    "srm_decode_pass_rows": (_I64, [_I64, _I64]),
    "srm_strerror": (C.c_char_p, [C.c_int]),
    "srm_last_cuda_error": (C.c_int, []),
    "srm_version": (C.c_char_p, []),
}


def lib_path() -> str:
    return _build.LIB_PATH


def load_library(build_if_missing: bool = True):
    """Load libsrm.so (building it with nvcc when absent or stale). There is no fallback:
    without the CUDA library nothing in this package can run."""
    global _LIB
    if _LIB is not None:
        return _LIB
    if build_if_missing and _build.needs_build():
        _build.build_library()
    if not os.path.exists(_build.LIB_PATH):
        raise ImportError(f"{_build.LIB_PATH} is missing; run paper_2605_08696_b200/build.py")
    lib = C.CDLL(_build.LIB_PATH)
    for name, (res, args) in SYMBOLS.items():
        fn = getattr(lib, name)          # AttributeError if the symbol is not exported
        fn.restype, fn.argtypes = res, args
    _LIB = lib
    return lib


def _lib():
    return load_library()


def _check(code, where):
    if code != 0:
        raise SRMError(code, where)


def _ptr(t):
    if t is None:
        return None
    assert t.is_contiguous(), "tensor must be contiguous"
    return C.c_void_p(t.data_ptr())


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _shape_opt(shape, key, default):
    return shape.get(key, default) if isinstance(shape, dict) else getattr(shape, key, default)


def _shape_get(shape, key):
    return shape[key] if isinstance(shape, dict) else getattr(shape, key)


def k_ffn_plan(M: int, d: int, F: int, pairs: int):
    """Work lists of the fused feed-forward kernel (host arithmetic only): returns (lists, makespan, ideal) where
    lists[c] is pair c's sequence of (down, row_block, column_tile)."""
    off = (_I32 * (pairs + 1))()
    n = _lib().srm_k_ffn_plan(M, d, F, pairs, off, None, 0, None, None)
    if n < 0:
        raise SRMError(int(n), "srm_k_ffn_plan")
    items = (_I32 * (3 * n))()
    mk, ideal = C.c_double(), C.c_double()
    _check(min(0, _lib().srm_k_ffn_plan(M, d, F, pairs, off, items, n, C.byref(mk), C.byref(ideal))), "srm_k_ffn_plan")
    lists = [[(items[3 * i], items[3 * i + 1], items[3 * i + 2]) for i in range(off[c], off[c + 1])] for c in range(pairs)]
    return lists, mk.value, ideal.value


def k_wait_probe(status: torch.Tensor, limit_cycles: int, gave_up: torch.Tensor | None = None):
    """A bounded wait on a barrier that nothing completes: must give up after limit_cycles and raise the status bit."""
    _check(_lib().srm_k_wait_probe(_ptr(status), limit_cycles, _ptr(gave_up), _stream()), "srm_k_wait_probe")


def k_mixer_combined_step(t, z, S_row, S_col, alpha_row, alpha_col, beta, lam_row, lam_col, w, y):
    """Recurrent step of a layer with linearly combined heads (srm_k_mixer_combined_step): fp32 CUDA tensors,
    z, y, S_row, S_col [R, d]; alpha_* [h, n_ctx]; beta [n_ctx, d]; lam_* [h]; w [h, 2]. Updates S_row, S_col, y."""
    R, d = z.shape
    h, n_ctx = alpha_row.shape
    _check(_lib().srm_k_mixer_combined_step(R, d, h, t, n_ctx, _ptr(z), _ptr(S_row), _ptr(S_col), _ptr(alpha_row),
                                            _ptr(alpha_col), _ptr(beta), _ptr(lam_row), _ptr(lam_col), _ptr(w), _ptr(y),
                                            _stream()), "srm_k_mixer_combined_step")


def k_mixer_kernel_step(t, z, P, alpha, beta, lam, y):
    """Recurrent step of a layer with a kernel of size k (Eq. 11; srm_k_mixer_kernel_step): fp32 CUDA tensors,
    z, y [R, d]; P [k, R, d]; alpha [k, n_ctx]; beta [n_ctx, d]; lam [k]. Updates P and y."""
    R, d = z.shape
    k, n_ctx = alpha.shape
    _check(_lib().srm_k_mixer_kernel_step(R, d, k, t, n_ctx, _ptr(z), _ptr(P), _ptr(alpha), _ptr(beta), _ptr(lam), _ptr(y),
                                          _stream()), "srm_k_mixer_kernel_step")


def k_mixer_combined_scan(t0, Z, S_row, S_col, alpha_row, alpha_col, beta, lam_row, lam_col, w, Y):
    """Positions t0 .. t0+n-1 of a layer with linearly combined heads (srm_k_mixer_combined_scan): Z, Y [Bp, n, d]."""
    Bp, n, d = Z.shape
    h, n_ctx = alpha_row.shape
    _check(_lib().srm_k_mixer_combined_scan(Bp, n, t0, d, h, n_ctx, _ptr(Z), _ptr(S_row), _ptr(S_col), _ptr(alpha_row),
                                            _ptr(alpha_col), _ptr(beta), _ptr(lam_row), _ptr(lam_col), _ptr(w), _ptr(Y),
                                            _stream()), "srm_k_mixer_combined_scan")


def k_mixer_kernel_scan(t0, Z, P, alpha, beta, lam, Y):
    """Positions t0 .. t0+n-1 of a layer with a kernel of size k (srm_k_mixer_kernel_scan): Z, Y [Bp, n, d], P [k, Bp, d]."""
    Bp, n, d = Z.shape
    k, n_ctx = alpha.shape
    _check(_lib().srm_k_mixer_kernel_scan(Bp, n, t0, d, k, n_ctx, _ptr(Z), _ptr(P), _ptr(alpha), _ptr(beta), _ptr(lam),
                                          _ptr(Y), _stream()), "srm_k_mixer_kernel_scan")


class SRMState:
    """Cache of B samples (device buffer owned here as a torch tensor, borrowed by the library)."""

    def __init__(self, model: "SRM", B: int):
        self.model, self.B = model, B
        nbytes = _lib().srm_state_bytes(C.byref(model.cfg), B)
        if nbytes == 0:
            raise SRMError(-1, "srm_state_bytes")
        self.buf = torch.empty(nbytes, dtype=torch.uint8, device=model.device)
        self.handle = C.c_void_p()
        _check(_lib().srm_state_create(model.handle, B, _ptr(self.buf), nbytes, _stream(), C.byref(self.handle)),
               "srm_state_create")

    def __del__(self):
        if getattr(self, "handle", None) and _LIB is not None:
            _LIB.srm_state_destroy(self.handle)
            self.handle = None

    @property
    def pos(self) -> int:
        return _lib().srm_state_pos(self.handle)

    @pos.setter
    def pos(self, v: int):
        _check(_lib().srm_state_set_pos(self.handle, v), "srm_state_set_pos")

    def reset(self):
        _check(_lib().srm_state_reset(self.handle, _stream()), "srm_state_reset")

    @property
    def ragged(self) -> bool:
        return bool(_lib().srm_state_is_ragged(self.handle))

    def adopt_positions(self, max_pos: int):
        """After copying the buffer of a ragged state into this one: its per-sample positions are valid."""
        _check(_lib().srm_state_adopt_positions(self.handle, max_pos), "srm_state_adopt_positions")

    def status(self) -> int:
        """Synchronises, returns and clears the device status word."""
        f = C.c_uint32(0)
        rc = _lib().srm_status(self.handle, _stream(), C.byref(f))
        if rc not in (0, -7):
            raise SRMError(rc, "srm_status")
        return f.value

    def layer(self, l: int) -> torch.Tensor:
        """View of the cache slab of one layer in the state dtype: [B, d], or [C, B, d] for the mixers that keep
        C > 1 d-vectors per sample and layer."""
        m = self.model
        ptr = _lib().srm_state_layer_ptr(self.handle, l)
        off = ptr - self.buf.data_ptr()
        es = 4 if m.cfg.state_dtype == DTYPE_FP32 else 2
        dt = {DTYPE_FP32: torch.float32, DTYPE_BF16: torch.bfloat16, DTYPE_FP16: torch.float16}[m.cfg.state_dtype]
        n = m.planes * self.B * m.cfg.d_model
        v = self.buf[off: off + n * es].view(dt)
        if m.cfg.mixer == MIXER_MIXED:
            return v.view(self.B, m.cfg.d_model)
        return v.view(m.planes, self.B, m.cfg.d_model)

    def cache(self) -> torch.Tensor:
        """[L, B, d] (or [L, C, B, d]) copy of the whole cache in fp32."""
        return torch.stack([self.layer(l).float() for l in range(self.model.cfg.n_layers)])

    def topk_thresholds(self) -> torch.Tensor:
        """View of the per-sample candidate thresholds of the fused top-k selection, float32 [B] (0 bits: none)."""
        off = _lib().srm_state_topk_threshold_ptr(self.handle) - self.buf.data_ptr()
        return self.buf[off: off + 4 * self.B].view(torch.float32)

    def topk_handed_back(self) -> int:
        """Rows the fused top-k selection handed back to the logits path since the last reset (synchronises)."""
        n = C.c_uint64(0)
        _check(_lib().srm_state_topk_handed_back(self.handle, _stream(), C.byref(n)), "srm_state_topk_handed_back")
        return n.value

    def last_token(self) -> torch.Tensor:
        off = _lib().srm_state_last_token_ptr(self.handle) - self.buf.data_ptr()
        return self.buf[off: off + 4 * self.B].view(torch.int32)


class SRM:
    """Model handle: packs the weight dict into the library's blob layout and owns the blob."""

    def __init__(self, shape, weights: dict, device: str = "cuda:0", state_dtype: str = "fp32", flags: int = 0):
        lib = _lib()
        dt = _shape_get(shape, "dtype")
        if (shape.get("head_proj", False) if isinstance(shape, dict) else getattr(shape, "head_proj", False)):
            flags |= FLAG_HEAD_PROJ
        self.cfg = _Config(_shape_get(shape, "n_layers"), _shape_get(shape, "d_model"), _shape_get(shape, "n_heads"),
                           _shape_get(shape, "ffn_mult"), _shape_get(shape, "vocab"), _shape_get(shape, "n_ctx"),
                           DTYPE_BF16 if dt == "bf16" else DTYPE_FP32,
                           {"fp32": DTYPE_FP32, "bf16": DTYPE_BF16, "fp16": DTYPE_FP16}[state_dtype],
                           _shape_get(shape, "ln_eps"), flags,
                           {"mixed": MIXER_MIXED, "combined": MIXER_COMBINED, "kernel": MIXER_KERNEL}[_shape_opt(shape, "mixer", "mixed")],
                           _shape_opt(shape, "kernel_size", 1))
        self.planes = lib.srm_cache_planes(C.byref(self.cfg))
        self.device = torch.device(device)
        self.act_dtype = torch.bfloat16 if dt == "bf16" else torch.float32
        nbytes = lib.srm_weights_bytes(C.byref(self.cfg))
        if nbytes == 0:
            raise SRMError(-2, "srm_weights_bytes")
        host = torch.zeros(nbytes, dtype=torch.uint8)
        self._slots = {}

        def put(layer, tid, arr):
            off, nb, eb = _SZ(), _SZ(), _I32()
            _check(lib.srm_weight_slot(C.byref(self.cfg), layer, tid, C.byref(off), C.byref(nb), C.byref(eb)),
                   "srm_weight_slot")
            t = torch.from_numpy(np.ascontiguousarray(arr, dtype=np.float32))
            t = t.to(torch.bfloat16) if eb.value == 2 else t
            raw = t.contiguous().view(torch.uint8).reshape(-1)
            assert raw.numel() == nb.value, (layer, tid, raw.numel(), nb.value)
            host[off.value: off.value + nb.value] = raw
            self._slots[(layer, tid)] = (off.value, nb.value, eb.value, tuple(t.shape))

        for name, tid in _GLOBAL_TENSORS.items():
            put(-1, tid, weights[name])
        for l, lw in enumerate(weights["layers"]):
            for name, tid in _LAYER_TENSORS.items():
                put(l, tid, lw[name])
            if flags & FLAG_HEAD_PROJ:
                put(l, T_W_IN, lw["W_in"])
                put(l, T_W_OUT, lw["W_out"])
            if self.cfg.mixer == MIXER_COMBINED:
                put(l, T_ALPHA_COL, lw["alpha_col"])
                put(l, T_LAMBDA_COL, lw["lam_col"])
                put(l, T_W_COMB, lw["w_comb"])
        with torch.cuda.device(self.device):
            self.blob = host.to(self.device)
            self.handle = C.c_void_p()
            _check(lib.srm_create(C.byref(self.cfg), _ptr(self.blob), nbytes, C.byref(self.handle)), "srm_create")

    def __del__(self):
        if getattr(self, "handle", None) and _LIB is not None:
            _LIB.srm_destroy(self.handle)
            self.handle = None

    # ---- buffers ----
    def tensor(self, layer: int, tid: int) -> torch.Tensor:
        """Device view of one tensor of the blob."""
        off, nb, eb, shp = self._slots[(layer, tid)]
        dt = torch.bfloat16 if eb == 2 else torch.float32
        return self.blob[off: off + nb].view(dt).view(shp)

    def new_state(self, B: int) -> SRMState:
        return SRMState(self, B)

    def workspace_bytes(self, B_chunk: int, n_prefill: int = 0) -> int:
        return _lib().srm_workspace_bytes(C.byref(self.cfg), B_chunk, n_prefill)

    def new_workspace(self, B_chunk: int, n_prefill: int = 0, prefill_samples: int = 1) -> torch.Tensor:
        nb = max(self.workspace_bytes(B_chunk, 0),
                 _lib().srm_prefill_workspace_bytes(C.byref(self.cfg), prefill_samples, n_prefill) if n_prefill else 0)
        return torch.empty(nb, dtype=torch.uint8, device=self.device)

    # ---- hot path ----
    def prefill(self, state: SRMState, tokens: torch.Tensor, sampling: Sampling, ws: torch.Tensor,
                want_logits: bool = False):
        B, n = tokens.shape
        assert B == state.B and tokens.dtype == torch.int32
        first = torch.empty(B, dtype=torch.int32, device=self.device)
        logits = torch.empty(B, self.cfg.vocab, dtype=torch.float32, device=self.device) if want_logits else None
        s = sampling.c()
        _check(_lib().srm_prefill(self.handle, state.handle, _ptr(tokens), n, C.byref(s), _ptr(first), _ptr(logits),
                                  _ptr(ws), ws.numel(), _stream()), "srm_prefill")
        return (first, logits) if want_logits else first

    def prefill_ragged(self, state: SRMState, tokens: torch.Tensor, lengths: torch.Tensor, sampling: Sampling,
                       ws: torch.Tensor, want_logits: bool = False):
        """tokens [B, n_max] left-aligned prompts, lengths int32 [B]; afterwards every sample has its own position."""
        B, n = tokens.shape
        assert B == state.B and tokens.dtype == torch.int32 and lengths.dtype == torch.int32 and lengths.numel() == B
        first = torch.empty(B, dtype=torch.int32, device=self.device)
        logits = torch.empty(B, self.cfg.vocab, dtype=torch.float32, device=self.device) if want_logits else None
        s = sampling.c()
        _check(_lib().srm_prefill_ragged(self.handle, state.handle, _ptr(tokens), n, _ptr(lengths), C.byref(s),
                                         _ptr(first), _ptr(logits), _ptr(ws), ws.numel(), _stream()),
               "srm_prefill_ragged")
        return (first, logits) if want_logits else first

    def prefill_replicated(self, state: SRMState, tokens: torch.Tensor, replicas: int, sampling: Sampling,
                           ws: torch.Tensor, want_logits: bool = False):
        """tokens [P, n] distinct prompts; state.B == P * replicas; row p * replicas + j is replica j of prompt p."""
        P_, n = tokens.shape
        assert P_ * replicas == state.B and tokens.dtype == torch.int32
        first = torch.empty(state.B, dtype=torch.int32, device=self.device)
        logits = torch.empty(P_, self.cfg.vocab, dtype=torch.float32, device=self.device) if want_logits else None
        s = sampling.c()
        _check(_lib().srm_prefill_replicated(self.handle, state.handle, _ptr(tokens), P_, n, replicas, C.byref(s),
                                             _ptr(first), _ptr(logits), _ptr(ws), ws.numel(), _stream()),
               "srm_prefill_replicated")
        return (first, logits) if want_logits else first

    def decode_step(self, state: SRMState, tok_in, sampling: Sampling, step: int, ws: torch.Tensor,
                    want_logits: bool = False, tok_out: torch.Tensor | None = None):
        if tok_out is None:
            tok_out = torch.empty(state.B, dtype=torch.int32, device=self.device)
        logits = torch.empty(state.B, self.cfg.vocab, dtype=torch.float32, device=self.device) if want_logits else None
        s = sampling.c()
        _check(_lib().srm_decode_step(self.handle, state.handle, _ptr(tok_in), C.byref(s), step, _ptr(tok_out),
                                      _ptr(logits), _ptr(ws), ws.numel(), _stream()), "srm_decode_step")
        return (tok_out, logits) if want_logits else tok_out

    def generate(self, state: SRMState, steps: int, first_step: int, sampling: Sampling, ws: torch.Tensor,
                 out: torch.Tensor | None = None) -> torch.Tensor:
        if out is None:
            out = torch.empty(state.B, steps, dtype=torch.int32, device=self.device)
        assert out.dtype == torch.int32 and out.stride(1) == 1 and out.shape[1] >= steps     # rows may be strided
        s = sampling.c()
        _check(_lib().srm_generate(self.handle, state.handle, steps, first_step, C.byref(s),
                                   C.c_void_p(out.data_ptr()), out.stride(0),
                                   _ptr(ws), ws.numel(), _stream()), "srm_generate")
        return out

    def decode_step_host(self, state: SRMState, h_tok_in: torch.Tensor, sampling: Sampling, step: int,
                         h_tok_out: torch.Tensor, ws: torch.Tensor):
        """Host-buffer variant: h_tok_in / h_tok_out are CPU int32 tensors (pinned for async copies)."""
        assert not h_tok_in.is_cuda and not h_tok_out.is_cuda
        s = sampling.c()
        _check(_lib().srm_decode_step_host(self.handle, state.handle, _ptr(h_tok_in), C.byref(s), step,
                                           _ptr(h_tok_out), _ptr(ws), ws.numel(), _stream()), "srm_decode_step_host")

    def decode_step_static(self, state: SRMState, tok_in, sampling: Sampling, step: int,
                           want_logits: bool = False, tok_out: torch.Tensor | None = None):
        """srm_decode_step on the library's built-in scratch array (no workspace argument): for callers
        that cannot allocate device memory. Raises SRMError(-8) when the batch does not fit."""
        if tok_out is None:
            tok_out = torch.empty(state.B, dtype=torch.int32, device=self.device)
        logits = torch.empty(state.B, self.cfg.vocab, dtype=torch.float32, device=self.device) if want_logits else None
        s = sampling.c()
        _check(_lib().srm_decode_step_static(self.handle, state.handle, _ptr(tok_in), C.byref(s), step, _ptr(tok_out),
                                             _ptr(logits), _stream()), "srm_decode_step_static")
        return (tok_out, logits) if want_logits else tok_out

    # ---- measurement ----
    KERNEL_CLASSES = ("mixer", "gemm_up", "gemm_down", "gemm_lm", "norm", "select", "prefill_mixer", "gemm_proj",
                      "step_small", "ffn")

    def profile(self, on: bool):
        _check(_lib().srm_profile_enable(self.handle, int(on)), "srm_profile_enable")

    def profile_reset(self):
        _check(_lib().srm_profile_reset(self.handle), "srm_profile_reset")

    def profile_read(self) -> dict:
        """{class name: (launches, total device ms)} since the last reset."""
        out = {}
        for i, name in enumerate(self.KERNEL_CLASSES):
            n, ms = C.c_uint64(), C.c_double()
            _check(_lib().srm_profile_read(self.handle, i, C.byref(n), C.byref(ms)), "srm_profile_read")
            out[name] = (n.value, ms.value)
        return out

    @staticmethod
    def kernel_launches() -> int:
        return _lib().srm_kernel_launches()

    # ---- single kernels ----
    def k_mixer_step(self, layer, t, x, S, a, tok=None, status=None):
        _check(_lib().srm_k_mixer_step(self.handle, layer, t, x.shape[0], _ptr(tok), _ptr(x), _ptr(S), _ptr(a),
                                       _ptr(status), _stream()), "srm_k_mixer_step")

    def k_final_norm(self, x, a):
        _check(_lib().srm_k_final_norm(self.handle, x.shape[0], _ptr(x), _ptr(a), _stream()), "srm_k_final_norm")

    def k_gemm(self, epilogue, A, W, bias, out, status=None):
        M, K = A.shape
        N = W.shape[0]
        _check(_lib().srm_k_gemm(self.handle, epilogue, M, N, K, _ptr(A), _ptr(W), _ptr(bias), _ptr(out),
                                 _ptr(status), _stream()), "srm_k_gemm")

    def k_gemm_splitk(self, A, W, bias, out, order=None, status=None):
        """out += A W^T + bias with K shared out between CTA pairs (raises SRMError -2 when the shape needs no split)."""
        M, K = A.shape
        N = W.shape[0]
        if order is None:
            order = torch.empty(_lib().srm_k_gemm_splitk_order_bytes(M, N), dtype=torch.uint8, device=A.device)
        _check(_lib().srm_k_gemm_splitk(self.handle, M, N, K, _ptr(A), _ptr(W), _ptr(bias), _ptr(out), _ptr(order),
                                        order.numel() * order.element_size(), _ptr(status), _stream()), "srm_k_gemm_splitk")

    def k_ffn(self, layer, a, H, x, ready=None, status=None):
        """The feed-forward block of one layer as one kernel: H = gelu(a W1^T + b1), x += H W2^T + b2."""
        M = a.shape[0]
        if ready is None:
            ready = torch.empty(_lib().srm_k_ffn_ready_bytes(M, H.shape[1]), dtype=torch.uint8, device=a.device)
        _check(_lib().srm_k_ffn(self.handle, layer, M, _ptr(a), _ptr(H), _ptr(x), _ptr(ready),
                                ready.numel() * ready.element_size(), _ptr(status), _stream()), "srm_k_ffn")

    def k_lm_head_greedy(self, a, part, tok, status=None):
        _check(_lib().srm_k_lm_head_greedy(self.handle, a.shape[0], _ptr(a), _ptr(part), part.numel() * part.element_size(),
                                           _ptr(tok), _ptr(status), _stream()), "srm_k_lm_head_greedy")

    def k_select(self, logits, sampling: Sampling, step, tok, status=None):
        s = sampling.c()
        _check(_lib().srm_k_select(self.handle, logits.shape[0], _ptr(logits), C.byref(s), step, _ptr(tok),
                                   _ptr(status), _stream()), "srm_k_select")

    def k_prefill_mixer(self, layer, Bp, n, x, S, a, tok=None, status=None):
        _check(_lib().srm_k_prefill_mixer(self.handle, layer, Bp, n, _ptr(tok), _ptr(x), _ptr(S), _ptr(a),
                                          _ptr(status), _stream()), "srm_k_prefill_mixer")
