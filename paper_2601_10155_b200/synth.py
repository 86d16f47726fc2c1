"""Seeded synthetic inputs for the LOOKAT decode-attention path.

This module only draws random arrays (numpy, PCG64).  It holds none of the
method's arithmetic (no codebooks, codes, lookup tables, softmax): both the
CUDA path and the CPU oracle receive the arrays produced here, never a seed.

The paper measured on first-layer GPT-2 KV caches of three text samples
(Section 4.1, "Models and Data"); neither the texts nor the weights are
available offline, so the generator below stands in for them with the same
shapes (12 heads of 64 dims, 128..1024 tokens) plus a long-context GQA shape.

Keys and queries of one KV head live near a shared low-rank subspace:

    A = diag(s) G / sqrt(r)            G ~ N(0,1)^{d x r}, fixed per head
    x = fp16( z A^T + 0.1 eps )        z ~ N(0, I_r), eps ~ N(0, I_d)

with per-channel scales ``s`` either log-uniform in [0.5, 4] or heavy tailed
(|Student-t, nu=3| clipped to [0.05, 50]).  Values are fp16 N(0, 1).
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np


@dataclass(frozen=True)
class Workload:
    """Shape of one decode-attention problem (names follow the paper: m
    subspaces, K centroids, L cached tokens, d_k / d_v head dims)."""

    name: str
    seed: int
    B: int
    n_q_heads: int
    n_kv_heads: int
    d_k: int
    d_v: int
    L: int
    m: int
    K: int = 256
    rank: int = 16
    scales: str = "loguniform"      # or "student_t3"
    fit_iters: int = 25
    fit_keys_per_head: int = 0      # 0: fit on all B*L cached keys of the head
    layer: int = 0

    @property
    def g(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    @property
    def d_sub(self) -> int:
        return self.d_k // self.m


# The shapes the benchmark description names.  "gpt2_l128_m4" fits K=256
# centroids on only 128 keys per head, so every key is its own centroid.
WORKLOADS = {
    "gpt2_l128_m4": Workload("gpt2_l128_m4", 1000, 1, 12, 12, 64, 64, 128, 4),
    "gpt2_l128_m4_calib": Workload("gpt2_l128_m4_calib", 1000, 1, 12, 12, 64, 64, 128, 4,
                                   fit_keys_per_head=4096),
    "gpt2_b8_l256_m2": Workload("gpt2_b8_l256_m2", 1001, 8, 12, 12, 64, 64, 256, 2),
    "gpt2_b8_l512_m2": Workload("gpt2_b8_l512_m2", 1001, 8, 12, 12, 64, 64, 512, 2),
    "gpt2_b8_l1024_m2": Workload("gpt2_b8_l1024_m2", 1001, 8, 12, 12, 64, 64, 1024, 2),
    "gpt2_b32_l1024_m4": Workload("gpt2_b32_l1024_m4", 1002, 32, 12, 12, 64, 64, 1024, 4),
    "gqa_32k_m8": Workload("gqa_32k_m8", 1003, 16, 32, 8, 128, 128, 32768, 8, rank=32,
                           scales="student_t3", fit_iters=10, fit_keys_per_head=65536),
    "prefill_4k_m16": Workload("prefill_4k_m16", 1004, 4, 32, 32, 128, 128, 4096, 16, rank=32,
                               fit_iters=10),
    "encode_1m_m16": Workload("encode_1m_m16", 1004, 1, 1, 1, 128, 128, 1048576, 16, rank=32,
                              fit_iters=10, fit_keys_per_head=262144),
}


def head_mixing_matrix(seed: int, layer: int, kv_head: int, d: int, rank: int,
                       scales: str) -> np.ndarray:
    """The fixed d x rank matrix A of one KV head."""
    rng = np.random.default_rng([seed, layer, kv_head])
    G = rng.standard_normal((d, rank))
    if scales == "loguniform":
        s = np.exp(rng.uniform(np.log(0.5), np.log(4.0), d))
    elif scales == "student_t3":
        s = np.clip(np.abs(rng.standard_t(3.0, d)), 0.05, 50.0)
    else:
        raise ValueError(f"unknown scales rule {scales!r}")
    return s[:, None] * G / np.sqrt(rank)


def draw_rows(rng: np.random.Generator, A: np.ndarray, n: int, block: int = 1 << 16) -> np.ndarray:
    """n iid rows  fp16(z A^T + 0.1 eps);  z is drawn before eps, block by block."""
    d, r = A.shape
    out = np.empty((n, d), dtype=np.float16)
    for lo in range(0, n, block):
        hi = min(n, lo + block)
        z = rng.standard_normal((hi - lo, r))
        eps = rng.standard_normal((hi - lo, d))
        out[lo:hi] = (z @ A.T + 0.1 * eps).astype(np.float16)
    return out


def make_keys(w: Workload, n_tokens: int | None = None, stream: int = 1) -> np.ndarray:
    """fp16 keys [B][n_kv_heads][n_tokens][d_k]; rows of a head are iid, batch-major."""
    L = w.L if n_tokens is None else n_tokens
    keys = np.empty((w.B, w.n_kv_heads, L, w.d_k), dtype=np.float16)
    for h in range(w.n_kv_heads):
        A = head_mixing_matrix(w.seed, w.layer, h, w.d_k, w.rank, w.scales)
        rng = np.random.default_rng([w.seed, w.layer, h, stream])
        keys[:, h] = draw_rows(rng, A, w.B * L).reshape(w.B, L, w.d_k)
    return keys


def make_calibration_keys(w: Workload, n: int) -> np.ndarray:
    """A separate draw of n keys per KV head, [1][n_kv_heads][n][d_k], for
    fitting codebooks on keys other than the cached ones."""
    keys = np.empty((1, w.n_kv_heads, n, w.d_k), dtype=np.float16)
    for h in range(w.n_kv_heads):
        A = head_mixing_matrix(w.seed, w.layer, h, w.d_k, w.rank, w.scales)
        rng = np.random.default_rng([w.seed, w.layer, h, 4])
        keys[0, h] = draw_rows(rng, A, n)
    return keys


def make_values(w: Workload, n_tokens: int | None = None) -> np.ndarray:
    """fp16 values [B][n_kv_heads][n_tokens][d_v], iid N(0,1)."""
    L = w.L if n_tokens is None else n_tokens
    v = np.empty((w.B, w.n_kv_heads, L, w.d_v), dtype=np.float16)
    block = 1 << 16
    for h in range(w.n_kv_heads):
        rng = np.random.default_rng([w.seed, w.layer, h, 2])
        buf = np.empty((w.B * L, w.d_v), dtype=np.float16)
        for lo in range(0, w.B * L, block):
            hi = min(w.B * L, lo + block)
            buf[lo:hi] = rng.standard_normal((hi - lo, w.d_v)).astype(np.float16)
        v[:, h] = buf.reshape(w.B, L, w.d_v)
    return v


def make_values_lowrank(w: Workload, n_tokens: int | None = None) -> np.ndarray:
    """fp16 values [B][n_kv_heads][n_tokens][d_v] with the structure of the keys (rows near a rank-`rank` subspace of
    the head, plus noise) instead of iid N(0,1): what a value quantiser can compress.  Only the quantised-values leg
    of the benchmark uses it."""
    L = w.L if n_tokens is None else n_tokens
    v = np.empty((w.B, w.n_kv_heads, L, w.d_v), dtype=np.float16)
    for h in range(w.n_kv_heads):
        A = head_mixing_matrix(w.seed, w.layer, h + 1000, w.d_v, w.rank, w.scales)
        rng = np.random.default_rng([w.seed, w.layer, h, 6])
        v[:, h] = draw_rows(rng, A, w.B * L).reshape(w.B, L, w.d_v)
    return v


def make_queries(w: Workload, q_scale: float = 1.0) -> np.ndarray:
    """fp16 queries [B][n_q_heads][d_k]; query head hq shares the subspace of
    KV head hq // g.  q_scale < 1 flattens the softmax (the plain generator
    gives very peaked attention)."""
    q = np.empty((w.B, w.n_q_heads, w.d_k), dtype=np.float16)
    for hq in range(w.n_q_heads):
        A = head_mixing_matrix(w.seed, w.layer, hq // w.g, w.d_k, w.rank, w.scales)
        rng = np.random.default_rng([w.seed, w.layer, hq, 3])
        rows = draw_rows(rng, A, w.B).astype(np.float64) * q_scale
        q[:, hq] = rows.astype(np.float16)
    return q


def make_prefill_queries(w: Workload, L_q: int, q_scale: float = 1.0) -> np.ndarray:
    """fp16 queries [B][n_q_heads][L_q][d_k] for multi-query (prefill) attention, drawn like the
    decode queries: query head hq shares the subspace of KV head hq // g."""
    q = np.empty((w.B, w.n_q_heads, L_q, w.d_k), dtype=np.float16)
    for hq in range(w.n_q_heads):
        A = head_mixing_matrix(w.seed, w.layer, hq // w.g, w.d_k, w.rank, w.scales)
        rng = np.random.default_rng([w.seed, w.layer, hq, 5])
        rows = draw_rows(rng, A, w.B * L_q).astype(np.float64) * q_scale
        q[:, hq] = rows.astype(np.float16).reshape(w.B, L_q, w.d_k)
    return q


def small_workload(name: str = "small", **kw) -> Workload:
    """A Workload with test-sized defaults; any field can be overridden."""
    base = dict(name=name, seed=7, B=2, n_q_heads=4, n_kv_heads=2, d_k=32, d_v=32,
                L=200, m=4, K=16, rank=8, scales="loguniform", fit_iters=5)
    base.update(kw)
    return Workload(**base)


def gpt2_weights(seed: int, n_layer: int = 12, n_head: int = 12, d_model: int = 768, vocab: int = 50257,
                 n_pos: int = 1088, plain_init: bool = True) -> dict:
    """Random-init GPT-2 shaped weights as fp16 arrays in a plain dict (no arithmetic of the model here).  Linear layers
    are stored transposed, [out][in].  plain_init: GPT-2's own scheme -- N(0, 0.02), residual projections scaled by
    1/sqrt(2 n_layer), zero biases, unit LayerNorm gains.  Otherwise gains and biases are random too, so that a dropped
    bias or gain cannot hide in a test."""
    rng = np.random.default_rng([seed, 77])
    h = lambda a: a.astype(np.float16)
    d = d_model
    nrm = lambda *shape, s=0.02: rng.standard_normal(shape) * s
    gain = (lambda: np.ones(d)) if plain_init else (lambda: 1.0 + 0.2 * rng.standard_normal(d))
    bias = (lambda n: np.zeros(n)) if plain_init else (lambda n: 0.05 * rng.standard_normal(n))
    layers = []
    for _ in range(n_layer):
        layers.append(dict(
            ln1_g=h(gain()), ln1_b=h(bias(d)), w_qkv=h(nrm(3 * d, d)), b_qkv=h(bias(3 * d)),
            w_o=h(nrm(d, d, s=0.02 / np.sqrt(2.0 * n_layer))), b_o=h(bias(d)),
            ln2_g=h(gain()), ln2_b=h(bias(d)), w_fc=h(nrm(4 * d, d)), b_fc=h(bias(4 * d)),
            w_pr=h(nrm(d, 4 * d, s=0.02 / np.sqrt(2.0 * n_layer))), b_pr=h(bias(d))))
    return dict(n_layer=n_layer, n_head=n_head, d_model=d, vocab=vocab, n_pos=n_pos, wte=h(nrm(vocab, d)),
                wpe=h(nrm(n_pos, d, s=0.01)), lnf_g=h(gain()), lnf_b=h(bias(d)), layers=layers)


def token_ids(seed: int, B: int, T: int, vocab: int) -> np.ndarray:
    """Uniform-random token ids int32 [B][T]."""
    return np.random.default_rng([seed, 78]).integers(0, vocab, (B, T), dtype=np.int32)
