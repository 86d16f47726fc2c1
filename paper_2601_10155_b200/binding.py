"""Thin Python binding of liblookat.so: argument marshalling only.

Every function has the name of the C entry point it calls (include/lookat.h)
and hands it raw device pointers of torch CUDA tensors; no step of the method
runs in Python or in torch.  There is no CPU path: a missing library or a
tensor that is not on a CUDA device raises.
"""
from __future__ import annotations

import ctypes
import math
import os

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "liblookat.so")
LIB_DEBUG_PATH = os.path.join(_PKG, "liblookat_debug.so")      # the build whose attend kernels check the codes they read

EXPORTS = [
    "lookat_create", "lookat_destroy", "lookat_last_error", "lookat_is_debug_build", "lookat_fit_codebooks",
    "lookat_encode_keys", "lookat_build_lut", "lookat_attend", "lookat_attend_static", "lookat_attend_pqv",
    "lookat_attend_prefill", "lookat_decode_step", "lookat_decode_step_host",
    "lookat_kernel_launches", "lookat_probe_read_bandwidth", "lookat_selftest_timeout", "lookat_set_prefill_form", "lookat_set_timing", "lookat_attend_kernel_ms", "lookat_attend_kernel_stats",
    # include/lookat_gpt2.h
    "lookat_gpt2_create", "lookat_gpt2_destroy", "lookat_gpt2_last_error", "lookat_gpt2_set_weights", "lookat_gpt2_prefill",
    "lookat_gpt2_decode", "lookat_gpt2_layer_state", "lookat_gpt2_position", "lookat_gpt2_kernel_launches",
    "lookat_gpt2_set_profile", "lookat_gpt2_profile",
    "lookat_linear", "lookat_linear_qkv", "lookat_layernorm", "lookat_embed", "lookat_causal_attention", "lookat_argmax",
]

STATUS = {0: "LOOKAT_OK", 1: "LOOKAT_ERR_INVALID_ARG", 2: "LOOKAT_ERR_UNSUPPORTED",
          3: "LOOKAT_ERR_CUDA", 4: "LOOKAT_ERR_NOMEM", 5: "LOOKAT_ERR_TIMEOUT"}


class LookatError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"{STATUS.get(status, status)}: {message}")
        self.status = status


class lookat_config(ctypes.Structure):
    _fields_ = [("n_q_heads", ctypes.c_int32), ("n_kv_heads", ctypes.c_int32),
                ("d_k", ctypes.c_int32), ("d_v", ctypes.c_int32), ("m", ctypes.c_int32),
                ("K", ctypes.c_int32), ("scale", ctypes.c_float)]


class lookat_gpt2_config(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in ("n_layer", "n_head", "d_model", "vocab", "n_pos", "m", "K", "fit_iters",
                                              "keep_prompt_keys")]


LAYER_FIELDS = ("ln1_g", "ln1_b", "w_qkv", "b_qkv", "w_o", "b_o", "ln2_g", "ln2_b", "w_fc", "b_fc", "w_pr", "b_pr")


class lookat_gpt2_layer(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in LAYER_FIELDS]


_libs = {}


def load_library(debug: bool = False) -> ctypes.CDLL:
    """Loads liblookat.so (built by paper_2601_10155_b200.build), or its debug build; raises if absent."""
    if debug in _libs:
        return _libs[debug]
    path = LIB_DEBUG_PATH if debug else LIB_PATH
    if not os.path.exists(path):
        raise FileNotFoundError(
            f"{path} is missing: run `python -m paper_2601_10155_b200.build{' --debug' if debug else ''}` (needs nvcc). "
            "There is no fallback path.")
    lib = ctypes.CDLL(path)
    vp, i32, i64, u64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_uint64
    lib.lookat_create.argtypes = [ctypes.POINTER(lookat_config), ctypes.c_int, vp, ctypes.POINTER(vp)]
    lib.lookat_create.restype = ctypes.c_int
    lib.lookat_destroy.argtypes = [vp]
    lib.lookat_destroy.restype = None
    lib.lookat_last_error.argtypes = [vp]
    lib.lookat_last_error.restype = ctypes.c_char_p
    lib.lookat_fit_codebooks.argtypes = [vp, vp, i32, i64, i32, u64, vp, vp, vp]
    lib.lookat_fit_codebooks.restype = ctypes.c_int
    lib.lookat_encode_keys.argtypes = [vp, vp, i32, i64, vp, vp, i64, i64, vp]
    lib.lookat_encode_keys.restype = ctypes.c_int
    lib.lookat_build_lut.argtypes = [vp, vp, i32, vp, vp]
    lib.lookat_build_lut.restype = ctypes.c_int
    lib.lookat_attend.argtypes = [vp, vp, vp, vp, vp, vp, i32, i64, vp, i32, vp, vp]
    lib.lookat_attend.restype = ctypes.c_int
    lib.lookat_attend_static.argtypes = [vp, vp, vp, vp, vp, vp, i32, i64, vp, i32, vp, vp]
    lib.lookat_attend_static.restype = ctypes.c_int
    lib.lookat_attend_pqv.argtypes = [vp, vp, vp, vp, vp, vp, vp, i32, i32, i32, i64, vp, vp]
    lib.lookat_attend_pqv.restype = ctypes.c_int
    lib.lookat_attend_prefill.argtypes = [vp, vp, vp, vp, vp, i32, i64, i64, i64, vp, vp]
    lib.lookat_attend_prefill.restype = ctypes.c_int
    lib.lookat_decode_step.argtypes = [vp, vp, vp, vp, vp, vp, i32, i64, i64, i32, vp]
    lib.lookat_decode_step.restype = ctypes.c_int
    lib.lookat_decode_step_host.argtypes = [vp, vp, vp, vp, i32, vp, vp, vp, i64, i64, i32, vp]
    lib.lookat_decode_step_host.restype = ctypes.c_int
    lib.lookat_kernel_launches.argtypes = [vp]
    lib.lookat_kernel_launches.restype = ctypes.c_uint64
    lib.lookat_probe_read_bandwidth.argtypes = [vp, vp, ctypes.c_uint64, i32, ctypes.POINTER(ctypes.c_double)]
    lib.lookat_probe_read_bandwidth.restype = i32
    lib.lookat_selftest_timeout.argtypes = [vp]
    lib.lookat_selftest_timeout.restype = i32
    lib.lookat_set_prefill_form.argtypes = [vp, i32]
    lib.lookat_set_prefill_form.restype = i32
    lib.lookat_set_timing.argtypes = [vp, i32]
    lib.lookat_set_timing.restype = None
    lib.lookat_attend_kernel_ms.argtypes = [vp]
    lib.lookat_attend_kernel_ms.restype = ctypes.c_double
    lib.lookat_attend_kernel_stats.argtypes = [vp, ctypes.POINTER(ctypes.c_double)]
    lib.lookat_attend_kernel_stats.restype = i32
    # the GPT-2 harness (include/lookat_gpt2.h)
    lib.lookat_gpt2_create.argtypes = [ctypes.POINTER(lookat_gpt2_config), ctypes.c_int, vp, i32, i32, ctypes.POINTER(vp)]
    lib.lookat_gpt2_create.restype = i32
    lib.lookat_gpt2_destroy.argtypes = [vp]
    lib.lookat_gpt2_destroy.restype = None
    lib.lookat_gpt2_last_error.argtypes = [vp]
    lib.lookat_gpt2_last_error.restype = ctypes.c_char_p
    lib.lookat_gpt2_set_weights.argtypes = [vp, vp, vp, vp, vp, ctypes.POINTER(lookat_gpt2_layer)]
    lib.lookat_gpt2_set_weights.restype = i32
    lib.lookat_gpt2_prefill.argtypes = [vp, vp, i32, u64, vp]
    lib.lookat_gpt2_prefill.restype = i32
    lib.lookat_gpt2_decode.argtypes = [vp, vp, vp, vp, vp]
    lib.lookat_gpt2_decode.restype = i32
    lib.lookat_gpt2_layer_state.argtypes = [vp, i32, ctypes.POINTER(vp), ctypes.POINTER(vp), ctypes.POINTER(vp), ctypes.POINTER(vp)]
    lib.lookat_gpt2_layer_state.restype = i32
    lib.lookat_gpt2_position.argtypes = [vp]
    lib.lookat_gpt2_position.restype = i32
    lib.lookat_gpt2_kernel_launches.argtypes = [vp]
    lib.lookat_gpt2_kernel_launches.restype = ctypes.c_uint64
    lib.lookat_gpt2_set_profile.argtypes = [vp, i32]
    lib.lookat_gpt2_set_profile.restype = None
    lib.lookat_gpt2_profile.argtypes = [vp, ctypes.POINTER(ctypes.c_double)]
    lib.lookat_gpt2_profile.restype = i32
    lib.lookat_linear.argtypes = [vp, vp, i32, vp, vp, i64, i32, i32, i32, vp, vp, i32]
    lib.lookat_linear.restype = i32
    lib.lookat_linear_qkv.argtypes = [vp, vp, vp, vp, i32, i32, i32, vp, i64, i64, vp, i64, i64, vp, i64, i64]
    lib.lookat_linear_qkv.restype = i32
    lib.lookat_layernorm.argtypes = [vp, vp, vp, vp, i64, i32, vp]
    lib.lookat_layernorm.restype = i32
    lib.lookat_embed.argtypes = [vp, vp, vp, vp, i32, i32, i32, i32, i32, vp]
    lib.lookat_embed.restype = i32
    lib.lookat_causal_attention.argtypes = [vp, vp, vp, vp, i32, i32, i32, i64, vp]
    lib.lookat_causal_attention.restype = i32
    lib.lookat_argmax.argtypes = [vp, vp, i32, i32, vp]
    lib.lookat_argmax.restype = i32
    lib.lookat_is_debug_build.argtypes = []
    lib.lookat_is_debug_build.restype = i32
    _libs[debug] = lib
    return lib


def _dev(t, dtype, name, shape=None):
    if t is None:
        return None
    if not isinstance(t, torch.Tensor) or not t.is_cuda:
        raise TypeError(f"{name} must be a CUDA tensor (the library has no CPU path)")
    if t.dtype != dtype:
        raise TypeError(f"{name} must have dtype {dtype}, got {t.dtype}")
    if not t.is_contiguous():
        raise ValueError(f"{name} must be contiguous")
    if shape is not None and tuple(t.shape) != tuple(shape):
        raise ValueError(f"{name} must have shape {tuple(shape)}, got {tuple(t.shape)}")
    return t.data_ptr()


def _host(t, dtype, name, shape):
    if not isinstance(t, torch.Tensor) or t.is_cuda:
        raise TypeError(f"{name} must be a host tensor")
    if t.dtype != dtype or not t.is_contiguous() or tuple(t.shape) != tuple(shape):
        raise ValueError(f"{name} must be contiguous {dtype} of shape {tuple(shape)}")
    return t.data_ptr()


class Lookat:
    """A library context for one attention shape on one device and stream.

    Method names and argument order are those of the C entry points.
    """

    def __init__(self, n_q_heads, n_kv_heads, d_k, d_v, m, K=256, scale=0.0, device=0, stream=None, debug=False):
        self._lib = load_library(debug)
        self._h = None
        if not torch.cuda.is_available():
            raise RuntimeError("no CUDA device: the LOOKAT library runs on the GPU only")
        self.cfg = lookat_config(n_q_heads, n_kv_heads, d_k, d_v, m, K, scale)
        self.device = torch.device("cuda", device)
        if stream is None:
            stream = torch.cuda.current_stream(self.device)
        self.stream = stream
        h = ctypes.c_void_p()
        st = self._lib.lookat_create(ctypes.byref(self.cfg), device, ctypes.c_void_p(stream.cuda_stream),
                                     ctypes.byref(h))
        if st != 0:
            raise LookatError(st, "lookat_create rejected the configuration or the device")
        self._h = h
        self.scale = scale if scale > 0 else 1.0 / math.sqrt(d_k)

    # -- helpers ---------------------------------------------------------------
    @property
    def d_sub(self):
        return self.cfg.d_k // self.cfg.m

    @property
    def g(self):
        return self.cfg.n_q_heads // self.cfg.n_kv_heads

    def _check(self, st):
        if st != 0:
            raise LookatError(st, self._lib.lookat_last_error(self._h).decode())

    def lookat_last_error(self) -> str:
        return self._lib.lookat_last_error(self._h).decode()

    def close(self):
        if self._h is not None:
            self._lib.lookat_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- the C entry points ------------------------------------------------------
    def lookat_fit_codebooks(self, keys, iters, seed=0, init=None, codebooks=None, distortion=None,
                             want_distortion=False):
        c = self.cfg
        B, H, n, d_k = keys.shape
        if codebooks is None:
            codebooks = torch.empty((c.n_kv_heads, c.m, c.K, self.d_sub), dtype=torch.float32, device=self.device)
        if distortion is None and want_distortion:
            distortion = torch.empty((c.n_kv_heads, c.m, iters + 1), dtype=torch.float64, device=self.device)
        self._check(self._lib.lookat_fit_codebooks(
            self._h, _dev(keys, torch.float16, "keys", (B, c.n_kv_heads, n, c.d_k)), B, n, iters, seed,
            _dev(init, torch.float32, "init", (c.n_kv_heads, c.m, c.K, self.d_sub)),
            _dev(codebooks, torch.float32, "codebooks", (c.n_kv_heads, c.m, c.K, self.d_sub)),
            _dev(distortion, torch.float64, "distortion", (c.n_kv_heads, c.m, iters + 1))))
        return (codebooks, distortion) if distortion is not None else codebooks

    def lookat_encode_keys(self, keys, codebooks, codes=None, L_max=None, pos=0, near_ties=None):
        c = self.cfg
        B, H, n, d_k = keys.shape
        if L_max is None:
            L_max = codes.shape[2] if codes is not None else pos + n
        if codes is None:
            codes = torch.zeros((B, c.n_kv_heads, L_max, c.m), dtype=torch.uint8, device=self.device)
        self._check(self._lib.lookat_encode_keys(
            self._h, _dev(keys, torch.float16, "keys", (B, c.n_kv_heads, n, c.d_k)), B, n,
            _dev(codebooks, torch.float32, "codebooks", (c.n_kv_heads, c.m, c.K, self.d_sub)),
            _dev(codes, torch.uint8, "codes", (B, c.n_kv_heads, L_max, c.m)), L_max, pos,
            _dev(near_ties, torch.int64, "near_ties", (1,))))
        return codes

    def lookat_build_lut(self, q, codebooks, lut=None):
        c = self.cfg
        B = q.shape[0]
        if lut is None:
            lut = torch.empty((B, c.n_q_heads, c.m, c.K), dtype=torch.float32, device=self.device)
        self._check(self._lib.lookat_build_lut(
            self._h, _dev(q, torch.float16, "q", (B, c.n_q_heads, c.d_k)), B,
            _dev(codebooks, torch.float32, "codebooks", (c.n_kv_heads, c.m, c.K, self.d_sub)),
            _dev(lut, torch.float32, "lut", (B, c.n_q_heads, c.m, c.K))))
        return lut

    def lookat_attend(self, codes, v, lut=None, q=None, codebooks=None, seq_lens=None, n_splits=0,
                      out=None, scores_out=None):
        c = self.cfg
        B, H, L_max, m = codes.shape
        if out is None:
            out = torch.empty((B, c.n_q_heads, c.d_v), dtype=torch.float32, device=self.device)
        self._check(self._lib.lookat_attend(
            self._h, _dev(lut, torch.float32, "lut", (B, c.n_q_heads, c.m, c.K)),
            _dev(q, torch.float16, "q", (B, c.n_q_heads, c.d_k)),
            _dev(codebooks, torch.float32, "codebooks", (c.n_kv_heads, c.m, c.K, self.d_sub)),
            _dev(codes, torch.uint8, "codes", (B, c.n_kv_heads, L_max, c.m)),
            _dev(v, torch.float16, "v", (B, c.n_kv_heads, L_max, c.d_v)), B, L_max,
            _dev(seq_lens, torch.int32, "seq_lens", (B,)), n_splits,
            _dev(out, torch.float32, "out", (B, c.n_q_heads, c.d_v)),
            _dev(scores_out, torch.float32, "scores_out", (B, c.n_q_heads, L_max))))
        return out

    def lookat_attend_pqv(self, codes, v_codebooks, v_codes, lut=None, q=None, codebooks=None, seq_lens=None, out=None):
        """Decode attention with product-quantised values as well (weights from the key codes, output from the
        weight histogram over the value codes)."""
        c = self.cfg
        B, H, L_max, m = codes.shape
        _, m_v, K_v, d_vsub = v_codebooks.shape
        if out is None:
            out = torch.empty((B, c.n_q_heads, c.d_v), dtype=torch.float32, device=self.device)
        self._check(self._lib.lookat_attend_pqv(
            self._h, _dev(lut, torch.float32, "lut", (B, c.n_q_heads, c.m, c.K)),
            _dev(q, torch.float16, "q", (B, c.n_q_heads, c.d_k)),
            _dev(codebooks, torch.float32, "codebooks", (c.n_kv_heads, c.m, c.K, self.d_sub)),
            _dev(codes, torch.uint8, "codes", (B, c.n_kv_heads, L_max, c.m)),
            _dev(v_codebooks, torch.float32, "v_codebooks", (c.n_kv_heads, m_v, K_v, c.d_v // m_v)),
            _dev(v_codes, torch.uint8, "v_codes", (B, c.n_kv_heads, L_max, m_v)), m_v, K_v, B, L_max,
            _dev(seq_lens, torch.int32, "seq_lens", (B,)),
            _dev(out, torch.float32, "out", (B, c.n_q_heads, c.d_v))))
        return out

    def lookat_attend_static(self, codes, v, lut=None, q=None, codebooks=None, seq_lens=None, n_splits=0,
                             out=None, scores_out=None):
        """lookat_attend for callers that cannot let the library allocate device memory (a process whose
        own pool owns the device, a latency-critical loop): the kernel's scratch is a fixed array inside
        the library.  `out` should be passed in by such callers; it is created here only for convenience."""
        c = self.cfg
        B, H, L_max, m = codes.shape
        if out is None:
            out = torch.empty((B, c.n_q_heads, c.d_v), dtype=torch.float32, device=self.device)
        self._check(self._lib.lookat_attend_static(
            self._h, _dev(lut, torch.float32, "lut", (B, c.n_q_heads, c.m, c.K)),
            _dev(q, torch.float16, "q", (B, c.n_q_heads, c.d_k)),
            _dev(codebooks, torch.float32, "codebooks", (c.n_kv_heads, c.m, c.K, self.d_sub)),
            _dev(codes, torch.uint8, "codes", (B, c.n_kv_heads, L_max, c.m)),
            _dev(v, torch.float16, "v", (B, c.n_kv_heads, L_max, c.d_v)), B, L_max,
            _dev(seq_lens, torch.int32, "seq_lens", (B,)), n_splits,
            _dev(out, torch.float32, "out", (B, c.n_q_heads, c.d_v)),
            _dev(scores_out, torch.float32, "scores_out", (B, c.n_q_heads, L_max))))
        return out

    def lookat_attend_prefill(self, q, codebooks, codes, v, q_pos0=0, out=None, scores_out=None):
        c = self.cfg
        B, H, L_max, m = codes.shape
        L_q = q.shape[2]
        if out is None:
            out = torch.empty((B, c.n_q_heads, L_q, c.d_v), dtype=torch.float32, device=self.device)
        self._check(self._lib.lookat_attend_prefill(
            self._h, _dev(q, torch.float16, "q", (B, c.n_q_heads, L_q, c.d_k)),
            _dev(codebooks, torch.float32, "codebooks", (c.n_kv_heads, c.m, c.K, self.d_sub)),
            _dev(codes, torch.uint8, "codes", (B, c.n_kv_heads, L_max, c.m)),
            _dev(v, torch.float16, "v", (B, c.n_kv_heads, L_max, c.d_v)), B, L_q, L_max, q_pos0,
            _dev(out, torch.float32, "out", (B, c.n_q_heads, L_q, c.d_v)),
            _dev(scores_out, torch.float32, "scores_out", (B, c.n_q_heads, L_q, L_max))))
        return out

    def lookat_decode_step(self, q, k_new, codebooks, codes, v, pos, out=None, n_splits=0):
        c = self.cfg
        B, H, L_max, m = codes.shape
        if out is None:
            out = torch.empty((B, c.n_q_heads, c.d_v), dtype=torch.float32, device=self.device)
        self._check(self._lib.lookat_decode_step(
            self._h, _dev(q, torch.float16, "q", (B, c.n_q_heads, c.d_k)),
            _dev(k_new, torch.float16, "k_new", (B, c.n_kv_heads, c.d_k)),
            _dev(codebooks, torch.float32, "codebooks", (c.n_kv_heads, c.m, c.K, self.d_sub)),
            _dev(codes, torch.uint8, "codes", (B, c.n_kv_heads, L_max, c.m)),
            _dev(v, torch.float16, "v", (B, c.n_kv_heads, L_max, c.d_v)), B, L_max, pos, n_splits,
            _dev(out, torch.float32, "out", (B, c.n_q_heads, c.d_v))))
        return out

    def lookat_decode_step_host(self, q_host, k_new_host, v_new_host, codebooks, codes, v, pos, out_host,
                                n_splits=0):
        c = self.cfg
        B, H, L_max, m = codes.shape
        self._check(self._lib.lookat_decode_step_host(
            self._h, _host(q_host, torch.float16, "q_host", (B, c.n_q_heads, c.d_k)),
            _host(k_new_host, torch.float16, "k_new_host", (B, c.n_kv_heads, c.d_k)),
            _host(v_new_host, torch.float16, "v_new_host", (B, c.n_kv_heads, c.d_v)), B,
            _dev(codebooks, torch.float32, "codebooks", (c.n_kv_heads, c.m, c.K, self.d_sub)),
            _dev(codes, torch.uint8, "codes", (B, c.n_kv_heads, L_max, c.m)),
            _dev(v, torch.float16, "v", (B, c.n_kv_heads, L_max, c.d_v)), L_max, pos, n_splits,
            _host(out_host, torch.float32, "out_host", (B, c.n_q_heads, c.d_v))))
        return out_host

    def lookat_kernel_launches(self) -> int:
        return int(self._lib.lookat_kernel_launches(self._h))

    def lookat_probe_read_bandwidth(self, buf, reps=5):
        """GB/s of a read-only streaming pass over the device tensor `buf` (measurement aid)."""
        out = ctypes.c_double(0.0)
        self._check(self._lib.lookat_probe_read_bandwidth(self._h, ctypes.c_void_p(buf.data_ptr()),
                                                          ctypes.c_uint64(buf.numel() * buf.element_size()), int(reps),
                                                          ctypes.byref(out)))
        return out.value

    def lookat_selftest_timeout(self):
        self._check(self._lib.lookat_selftest_timeout(self._h))

    def lookat_set_prefill_form(self, form):
        """form: 'auto', 'tables' or 'contraction' (or the header's integer values)."""
        code = {"auto": 0, "tables": 1, "contraction": 2}.get(form, form)
        self._check(self._lib.lookat_set_prefill_form(self._h, int(code)))

    def lookat_set_timing(self, launches):
        """launches >= 1: time up to that many attend launches from now on (True = 64); 0 / False: stop."""
        self._lib.lookat_set_timing(self._h, 64 if launches is True else int(launches))

    def lookat_attend_kernel_stats(self):
        """{'n', 'min', 'median', 'max', 'mean'} of the timed attend launches in milliseconds, or None."""
        st = (ctypes.c_double * 4)()
        n = int(self._lib.lookat_attend_kernel_stats(self._h, st))
        return None if n == 0 else {"n": n, "min": st[0], "median": st[1], "max": st[2], "mean": st[3]}

    def lookat_attend_kernel_ms(self) -> float:
        return float(self._lib.lookat_attend_kernel_ms(self._h))


    # -- the GPT-2 harness's kernels one by one (include/lookat_gpt2.h) ------------
    def lookat_linear(self, x, w_t, bias=None, gelu=False, residual=None, out=None, out_fp16=True):
        M, K = x.shape
        N = w_t.shape[0]
        if out is None:
            out = torch.empty((M, N), dtype=torch.float16 if out_fp16 else torch.float32, device=self.device)
        if x.dtype not in (torch.float16, torch.float32):
            raise TypeError("x must be fp16 or fp32")
        self._check(self._lib.lookat_linear(
            self._h, _dev(x, x.dtype, "x", (M, K)), 1 if x.dtype == torch.float32 else 0, _dev(w_t, torch.float16, "w_t", (N, K)),
            _dev(bias, torch.float16, "bias", (N,)), M, N, K, 1 if gelu else 0, _dev(residual, torch.float32, "residual", (M, N)),
            _dev(out, torch.float16 if out_fp16 else torch.float32, "out", (M, N)), 1 if out_fp16 else 0))
        return out

    def lookat_linear_qkv(self, x, w_t, bias, B, T, n_head, q, k, v, q_off=0, k_off=0, v_off=0):
        d = n_head * 64
        self._check(self._lib.lookat_linear_qkv(
            self._h, _dev(x, torch.float16, "x", (B * T, d)), _dev(w_t, torch.float16, "w_t", (3 * d, d)),
            _dev(bias, torch.float16, "bias", (3 * d,)), B, T, n_head,
            _dev(q, torch.float16, "q"), q.shape[2], q_off, _dev(k, torch.float16, "k"), k.shape[2], k_off,
            _dev(v, torch.float16, "v"), v.shape[2], v_off))
        return q, k, v

    def lookat_layernorm(self, x, gain, bias, out=None):
        rows, d = x.shape
        if out is None:
            out = torch.empty((rows, d), dtype=torch.float16, device=self.device)
        self._check(self._lib.lookat_layernorm(self._h, _dev(x, torch.float32, "x"), _dev(gain, torch.float16, "gain", (d,)),
                                               _dev(bias, torch.float16, "bias", (d,)), rows, d, _dev(out, torch.float16, "out", (rows, d))))
        return out

    def lookat_embed(self, ids, wte, wpe, pos0=0, out=None):
        B, T = ids.shape
        vocab, d = wte.shape
        if out is None:
            out = torch.empty((B, T, d), dtype=torch.float32, device=self.device)
        self._check(self._lib.lookat_embed(self._h, _dev(ids, torch.int32, "ids"), _dev(wte, torch.float16, "wte"),
                                           _dev(wpe, torch.float16, "wpe"), B, T, pos0, d, vocab, _dev(out, torch.float32, "out", (B, T, d))))
        return out

    def lookat_causal_attention(self, q, k, v, out=None):
        B, H, T, dh = q.shape
        if out is None:
            out = torch.empty((B, T, H * dh), dtype=torch.float16, device=self.device)
        self._check(self._lib.lookat_causal_attention(self._h, _dev(q, torch.float16, "q", (B, H, T, 64)), _dev(k, torch.float16, "k", (B, H, T, 64)),
                                                      _dev(v, torch.float16, "v"), B, H, T, v.shape[2], _dev(out, torch.float16, "out", (B, T, H * 64))))
        return out

    def lookat_argmax(self, logits, out=None):
        rows, n = logits.shape
        if out is None:
            out = torch.empty((rows,), dtype=torch.int32, device=self.device)
        self._check(self._lib.lookat_argmax(self._h, _dev(logits, torch.float32, "logits"), rows, n, _dev(out, torch.int32, "out", (rows,))))
        return out


class LookatGpt2:
    """The GPT-2 decoder harness (include/lookat_gpt2.h): argument marshalling only.  `weights` is the dict of fp16
    numpy arrays the seeded generator makes; they are uploaded once and kept alive here."""

    def __init__(self, weights, B, capacity, m, K, fit_iters, device=0, stream=None, keep_prompt_keys=False):
        self._lib = load_library()
        self._h = None
        if not torch.cuda.is_available():
            raise RuntimeError("no CUDA device: the LOOKAT library runs on the GPU only")
        self.device = torch.device("cuda", device)
        if stream is None:
            stream = torch.cuda.current_stream(self.device)
        self.stream = stream
        w = weights
        self.cfg = lookat_gpt2_config(w["n_layer"], w["n_head"], w["d_model"], w["vocab"], w["n_pos"], m, K, fit_iters,
                                      1 if keep_prompt_keys else 0)
        self.B, self.capacity = B, capacity
        h = ctypes.c_void_p()
        st = self._lib.lookat_gpt2_create(ctypes.byref(self.cfg), device, ctypes.c_void_p(stream.cuda_stream), B, capacity, ctypes.byref(h))
        if st != 0:
            raise LookatError(st, "lookat_gpt2_create rejected the configuration or ran out of memory")
        self._h = h
        up = lambda a: torch.from_numpy(a).to(self.device)
        self._keep = {k: up(w[k]) for k in ("wte", "wpe", "lnf_g", "lnf_b")}
        self._layers = [{k: up(lw[k]) for k in LAYER_FIELDS} for lw in w["layers"]]
        arr = (lookat_gpt2_layer * w["n_layer"])()
        for l, lw in enumerate(self._layers):
            for k in LAYER_FIELDS:
                setattr(arr[l], k, lw[k].data_ptr())
        self._check(self._lib.lookat_gpt2_set_weights(self._h, self._keep["wte"].data_ptr(), self._keep["wpe"].data_ptr(),
                                                      self._keep["lnf_g"].data_ptr(), self._keep["lnf_b"].data_ptr(), arr))

    def _check(self, st):
        if st != 0:
            raise LookatError(st, self._lib.lookat_gpt2_last_error(self._h).decode())

    def close(self):
        if self._h is not None:
            self._lib.lookat_gpt2_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def lookat_gpt2_prefill(self, ids, seed=0, want_hidden=False):
        B, T = ids.shape
        hidden = torch.empty((B, T, self.cfg.d_model), dtype=torch.float32, device=self.device) if want_hidden else None
        self._check(self._lib.lookat_gpt2_prefill(self._h, _dev(ids, torch.int32, "ids", (self.B, T)), T, seed,
                                                  None if hidden is None else hidden.data_ptr()))
        return hidden

    def lookat_gpt2_decode(self, ids, want_hidden=False, want_logits=False, want_next=False, logits=None, next_ids=None):
        hidden = torch.empty((self.B, self.cfg.d_model), dtype=torch.float32, device=self.device) if want_hidden else None
        if want_logits and logits is None:
            logits = torch.empty((self.B, self.cfg.vocab), dtype=torch.float32, device=self.device)
        if want_next and next_ids is None:
            next_ids = torch.empty((self.B,), dtype=torch.int32, device=self.device)
        self._check(self._lib.lookat_gpt2_decode(self._h, _dev(ids, torch.int32, "ids", (self.B,)),
                                                 None if hidden is None else hidden.data_ptr(),
                                                 None if logits is None else logits.data_ptr(),
                                                 None if next_ids is None else next_ids.data_ptr()))
        return hidden, logits, next_ids

    def lookat_gpt2_layer_state(self, layer, T=None):
        """(codebooks, codes, values, prompt_keys) of a layer as torch views of the model's own device memory."""
        ptrs = [ctypes.c_void_p() for _ in range(4)]
        self._check(self._lib.lookat_gpt2_layer_state(self._h, layer, *[ctypes.byref(p) for p in ptrs]))
        c = self.cfg

        def view(ptr, shape, dtype):
            if not ptr.value:
                return None
            self.stream.synchronize()
            typestr = {torch.float32: "<f4", torch.float16: "<f2", torch.uint8: "|u1"}[dtype]
            return torch.as_tensor(_RawDeviceArray(ptr.value, shape, typestr), device=self.device).clone()
        H, cap = c.n_head, self.capacity
        return (view(ptrs[0], (H, c.m, c.K, 64 // c.m), torch.float32), view(ptrs[1], (self.B, H, cap, c.m), torch.uint8),
                view(ptrs[2], (self.B, H, cap, 64), torch.float16),
                view(ptrs[3], (self.B, H, T, 64), torch.float16) if T else None)

    def lookat_gpt2_set_profile(self, enabled: bool):
        self._lib.lookat_gpt2_set_profile(self._h, 1 if enabled else 0)

    def lookat_gpt2_profile(self):
        """(steps, {category: milliseconds}) of the decode steps made since profiling was switched on."""
        names = ("embed", "layernorm", "qkv", "attention", "out_proj", "mlp", "lm_head")
        ms = (ctypes.c_double * len(names))()
        steps = int(self._lib.lookat_gpt2_profile(self._h, ms))
        return steps, {n: ms[i] for i, n in enumerate(names)}

    def lookat_gpt2_position(self) -> int:
        return int(self._lib.lookat_gpt2_position(self._h))

    def lookat_gpt2_kernel_launches(self) -> int:
        return int(self._lib.lookat_gpt2_kernel_launches(self._h))


class _RawDeviceArray:
    """A device array of the library seen through the CUDA array interface (no copy, no ownership)."""

    def __init__(self, ptr: int, shape, typestr: str):
        self.__cuda_array_interface__ = {"shape": tuple(int(x) for x in shape), "typestr": typestr, "data": (int(ptr), False),
                                         "version": 2, "strides": None}


# ---- byte accounting of the method (Section 3.4 "Compression Ratio", Section 3.1) ----
def key_bytes_per_token(m: int) -> int:
    """A compressed key is m uint8 indices."""
    return m


def key_compression_ratio(d_k: int, m: int) -> float:
    """fp16 key (2*d_k bytes) over its m code bytes."""
    return 2.0 * d_k / m


def lut_entries(m: int, K: int = 256) -> int:
    return m * K


def kv_cache_bytes_fp16(H: int, L: int, d_k: int) -> int:
    """Uncompressed fp16 KV cache: 2*H*d_k values per token, 2 bytes each."""
    return 4 * H * L * d_k


def attend_bytes_per_token_kvhead(m: int, d_v: int) -> int:
    """What one attend pass must read per cached token and KV head: m code bytes + fp16 V row."""
    return m + 2 * d_v
