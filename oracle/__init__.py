"""numpy front end of the CPU oracle (oracle/lookat_oracle.c).

TEST INFRASTRUCTURE ONLY: the tests, the smoke check and the benchmark's
CPU-baseline leg may import this package; the CUDA library and its Python
binding never do.  Nothing here touches the GPU.

Arrays follow the layouts stated at the top of lookat_oracle.c; fp16 arrays
are numpy float16 and are handed to C as their bit patterns.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "lookat_oracle.c")
_LIB = os.path.join(_HERE, "liblookat_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2 -fopenmp); returns the library path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-std=c99", "-fopenmp", "-fPIC", "-shared",
                               "-ffp-contract=off", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _f16(a):
    a = np.ascontiguousarray(a)
    assert a.dtype == np.float16, a.dtype
    return a


def n_threads() -> int:
    """Threads the OpenMP regions of the oracle will use."""
    return int(_load().oracle_set_num_threads(0))


def set_threads(n: int) -> int:
    """Use n threads from now on (n <= 0: leave as is); returns the setting in force."""
    return int(_load().oracle_set_num_threads(int(n)))


def all_threads() -> int:
    """The cores this process may run on (what OpenMP uses unless told otherwise)."""
    env = os.environ.get("OMP_NUM_THREADS")
    if env:
        return int(env.split(",")[0])
    return len(os.sched_getaffinity(0))


def half_to_double(a: np.ndarray) -> np.ndarray:
    a = _f16(a)
    out = np.empty(a.shape, dtype=np.float64)
    _load().oracle_half_to_double(_p(a), _p(out), ctypes.c_int64(a.size))
    return out


def encode_keys(keys, codebooks, codes=None, L_max=None, pos=0, want_gap=False):
    """keys fp16 [B][H_kv][n][d_k], codebooks fp32 [H_kv][m][K][d_sub].
    Returns codes u8 [B][H_kv][L_max][m] (written at pos..pos+n) and, when
    want_gap, the relative best/second-best gap [B][H_kv][n][m]."""
    keys = _f16(keys)
    codebooks = np.ascontiguousarray(codebooks, dtype=np.float32)
    B, H, n, d_k = keys.shape
    Hc, m, K, d_sub = codebooks.shape
    assert Hc == H and m * d_sub == d_k
    if L_max is None:
        L_max = pos + n
    if codes is None:
        codes = np.zeros((B, H, L_max, m), dtype=np.uint8)
    assert codes.shape == (B, H, L_max, m) and codes.dtype == np.uint8 and codes.flags.c_contiguous
    gap = np.empty((B, H, n, m), dtype=np.float64) if want_gap else None
    _load().oracle_encode_keys(_p(keys), B, H, ctypes.c_int64(n), d_k, m, K, _p(codebooks),
                               _p(codes), ctypes.c_int64(L_max), ctypes.c_int64(pos), _p(gap))
    return (codes, gap) if want_gap else codes


def fit_codebooks(keys, m, K, iters, seed=0, init=None):
    """Lloyd k-means per (KV head, subspace) on keys fp16 [B][H_kv][n][d_k].
    Returns codebooks fp32 [H_kv][m][K][d_sub] and the distortion trace
    fp64 [H_kv][m][iters+1]."""
    keys = _f16(keys)
    B, H, n, d_k = keys.shape
    assert d_k % m == 0
    d_sub = d_k // m
    if init is not None:
        init = np.ascontiguousarray(init, dtype=np.float32)
        assert init.shape == (H, m, K, d_sub)
    books = np.empty((H, m, K, d_sub), dtype=np.float32)
    trace = np.empty((H, m, iters + 1), dtype=np.float64)
    rc = _load().oracle_fit_codebooks(_p(keys), B, H, ctypes.c_int64(n), d_k, m, K, iters,
                                      ctypes.c_uint64(seed), _p(init), _p(books), _p(trace))
    if rc != 0:
        raise ValueError("too many keys for exact 64-bit centroid sums")
    return books, trace


def build_lut(q, codebooks):
    """q fp16 [B][H_q][d_k] -> LUT fp64 [B][H_q][m][K] (unscaled)."""
    q = _f16(q)
    codebooks = np.ascontiguousarray(codebooks, dtype=np.float32)
    B, H_q, d_k = q.shape
    H_kv, m, K, d_sub = codebooks.shape
    assert m * d_sub == d_k and H_q % H_kv == 0
    lut = np.empty((B, H_q, m, K), dtype=np.float64)
    _load().oracle_build_lut(_p(q), B, H_q, H_kv, d_k, m, K, _p(codebooks), _p(lut))
    return lut


def attend(lut, codes, v, seq_lens=None, scale=None, d_k=None, want_scores=False,
           want_alpha=False):
    """lut fp64 [B][H_q][m][K], codes u8 [B][H_kv][L_max][m], v fp16
    [B][H_kv][L_max][d_v].  scale defaults to 1/sqrt(d_k) (d_k required then).
    Returns out fp64 [B][H_q][d_v] (+ raw scores, + alpha when asked)."""
    lut = np.ascontiguousarray(lut, dtype=np.float64)
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    v = _f16(v)
    B, H_q, m, K = lut.shape
    Bc, H_kv, L_max, mc = codes.shape
    assert Bc == B and mc == m and v.shape[:3] == (B, H_kv, L_max) and H_q % H_kv == 0
    assert int(codes.max(initial=0)) < K
    d_v = v.shape[3]
    if scale is None:
        scale = 1.0 / np.sqrt(float(d_k))
    sl = None if seq_lens is None else np.ascontiguousarray(seq_lens, dtype=np.int32)
    out = np.empty((B, H_q, d_v), dtype=np.float64)
    scores = np.full((B, H_q, L_max), np.nan) if want_scores else None
    alpha = np.zeros((B, H_q, L_max)) if want_alpha else None
    _load().oracle_attend(_p(lut), _p(codes), _p(v), B, H_q, H_kv, ctypes.c_int64(L_max), _p(sl),
                          d_v, m, K, ctypes.c_double(scale), _p(out), _p(scores), _p(alpha))
    res = (out,)
    if want_scores:
        res += (scores,)
    if want_alpha:
        res += (alpha,)
    return res if len(res) > 1 else out


def exact_attention(q, keys, v, seq_lens=None, scale=None, want_scores=False):
    """softmax(q K^T * scale) V in fp64 on fp16 inputs; q [B][H_q][d_k],
    keys [B][H_kv][L][d_k], v [B][H_kv][L][d_v]."""
    q, keys, v = _f16(q), _f16(keys), _f16(v)
    B, H_q, d_k = q.shape
    _, H_kv, L_max, _ = keys.shape
    d_v = v.shape[3]
    if scale is None:
        scale = 1.0 / np.sqrt(float(d_k))
    sl = None if seq_lens is None else np.ascontiguousarray(seq_lens, dtype=np.int32)
    out = np.empty((B, H_q, d_v), dtype=np.float64)
    scores = np.full((B, H_q, L_max), np.nan) if want_scores else None
    _load().oracle_exact_attention(_p(q), _p(keys), _p(v), B, H_q, H_kv, ctypes.c_int64(L_max),
                                   _p(sl), d_k, d_v, ctypes.c_double(scale), _p(out), _p(scores))
    return (out, scores) if want_scores else out


def reconstruct_keys(codes, codebooks):
    """k_hat fp64 [B][H_kv][L][d_k] = concatenated centroids the codes name."""
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    codebooks = np.ascontiguousarray(codebooks, dtype=np.float32)
    B, H, L, m = codes.shape
    _, _, K, d_sub = codebooks.shape
    k_hat = np.empty((B, H, L, m * d_sub), dtype=np.float64)
    _load().oracle_reconstruct_keys(_p(codes), B, H, ctypes.c_int64(L), m * d_sub, m, K,
                                    _p(codebooks), _p(k_hat))
    return k_hat


def attend_prefill(q, codebooks, codes, v, q_pos0=0, scale=None, want_scores=False):
    """Causal multi-query attention over the compressed keys: q fp16 [B][H_q][L_q][d_k]; query i stands
    at position q_pos0 + i and attends tokens 0..q_pos0+i.  Returns out fp64 [B][H_q][L_q][d_v]."""
    q = _f16(q)
    codebooks = np.ascontiguousarray(codebooks, dtype=np.float32)
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    v = _f16(v)
    B, H_q, L_q, d_k = q.shape
    H_kv, m, K, d_sub = codebooks.shape
    _, _, L_max, _ = codes.shape
    d_v = v.shape[3]
    assert m * d_sub == d_k and H_q % H_kv == 0 and q_pos0 >= 0 and q_pos0 + L_q <= L_max
    assert int(codes.max(initial=0)) < K
    if scale is None:
        scale = 1.0 / np.sqrt(float(d_k))
    out = np.empty((B, H_q, L_q, d_v), dtype=np.float64)
    scores = np.full((B, H_q, L_q, L_max), np.nan) if want_scores else None
    _load().oracle_attend_prefill(_p(q), _p(codebooks), _p(codes), _p(v), B, H_q, H_kv, ctypes.c_int64(L_q),
                                  ctypes.c_int64(L_max), ctypes.c_int64(q_pos0), d_k, d_v, m, K,
                                  ctypes.c_double(scale), _p(out), _p(scores))
    return (out, scores) if want_scores else out


def decode_step(q, codebooks, codes, v, seq_lens=None, scale=None):
    """Algorithm 1 as a whole: build the tables, then attend."""
    return attend(build_lut(q, codebooks), codes, v, seq_lens=seq_lens, scale=scale,
                  d_k=q.shape[-1])


def attend_pqv(lut, codes, v_codebooks, v_codes, seq_lens=None, scale=None, d_k=None):
    """Decode attention with product-quantised values as well -- the extension Section 5.2 leaves as future work;
    the formulation is this build's own and has no counterpart in the paper.  The weights alpha are those of
    Algorithm 1 (scores from the key codes); the output is o = sum_t alpha_t v^_t with v^_t the value centroids the
    value codes name, taken per value subspace j as sum_c w[j][c] C^V_j[c], w[j][c] = sum of alpha_t over the
    tokens whose code is c (a weight histogram).
    lut fp64 [B][H_q][m][K], codes u8 [B][H_kv][L_max][m], v_codebooks fp32 [H_kv][m_v][K_v][d_vsub],
    v_codes u8 [B][H_kv][L_max][m_v].  Returns out fp64 [B][H_q][m_v * d_vsub]."""
    v_codebooks = np.ascontiguousarray(v_codebooks, dtype=np.float32)
    v_codes = np.ascontiguousarray(v_codes, dtype=np.uint8)
    B, H_q = lut.shape[:2]
    H_kv, m_v, K_v, d_vsub = v_codebooks.shape
    L_max = codes.shape[2]
    assert v_codes.shape == (B, H_kv, L_max, m_v) and int(v_codes.max(initial=0)) < K_v
    g = H_q // H_kv
    dummy = np.zeros((B, H_kv, L_max, 1), dtype=np.float16)
    _, alpha = attend(lut, codes, dummy, seq_lens=seq_lens, scale=scale, d_k=d_k, want_alpha=True)
    out = np.zeros((B, H_q, m_v * d_vsub), dtype=np.float64)
    for b in range(B):
        n = L_max if seq_lens is None else int(seq_lens[b])
        for hq in range(H_q):
            h = hq // g
            for j in range(m_v):
                w = np.zeros(K_v, dtype=np.float64)
                np.add.at(w, v_codes[b, h, :n, j], alpha[b, hq, :n])
                out[b, hq, j * d_vsub:(j + 1) * d_vsub] = w @ v_codebooks[h, j].astype(np.float64)
    return out
