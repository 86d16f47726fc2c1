"""CPU oracle of the GPT-2 decoder harness around LOOKAT attention (numpy, fp64).

TEST INFRASTRUCTURE ONLY, like the rest of this package: the tests, the smoke
check and the benchmark's CPU leg may import it; the CUDA library never does.

The paper evaluates on GPT-2 (Section 4.1, "Models and Data": 12 layers, 12
heads, d_model 768, head dim 64) and replaces the key side of attention by
Algorithm 1 at decode time.  This module states that model plainly: token and
position embeddings, pre-LayerNorm blocks (attention, then a 4x MLP with the
tanh-form GELU), a final LayerNorm and the tied output projection.  The prompt
is processed with exact causal attention (Section 3.1); every generated token
attends through the compressed keys: the new key is encoded on append (Section
3.4 "Encoding"), the lookup tables are built from the query (Section 3.5) and
Algorithm 1 gives the attention output.  Matrix products use numpy's matmul in
fp64 (a library primitive as one step); nothing is fused, tiled or reordered.

Weights arrive as fp16 arrays (what the GPU path stores) and are widened
exactly.  Linear layers store W^T, shape [out][in], so y = x W^T^T + b.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

from . import attend, build_lut, encode_keys, fit_codebooks

LN_EPS = 1e-5


@dataclass
class Gpt2Weights:
    """fp16 arrays.  Per layer l: ln1_g/ln1_b [d], w_qkv [3d][d], b_qkv [3d], w_o [d][d], b_o [d],
    ln2_g/ln2_b [d], w_fc [4d][d], b_fc [4d], w_pr [d][4d], b_pr [d]; wte [vocab][d], wpe [n_pos][d], lnf_g/lnf_b [d]."""
    n_layer: int
    n_head: int
    d_model: int
    wte: np.ndarray
    wpe: np.ndarray
    lnf_g: np.ndarray
    lnf_b: np.ndarray
    layers: list          # of dicts with the per-layer arrays

    @classmethod
    def from_dict(cls, d):
        """From the plain dict the seeded generator makes (the same arrays the GPU path uploads)."""
        return cls(n_layer=d["n_layer"], n_head=d["n_head"], d_model=d["d_model"], wte=d["wte"], wpe=d["wpe"],
                   lnf_g=d["lnf_g"], lnf_b=d["lnf_b"], layers=d["layers"])


def f64(a):
    return np.asarray(a).astype(np.float64)


def layer_norm(x, g, b):
    """Per row: (x - mean) / sqrt(var + eps) * g + b with the biased variance."""
    x = f64(x)
    mu = x.mean(axis=-1, keepdims=True)
    var = ((x - mu) ** 2).mean(axis=-1, keepdims=True)
    return (x - mu) / np.sqrt(var + LN_EPS) * f64(g) + f64(b)


def gelu_tanh(x):
    """GPT-2's GELU: 0.5 x (1 + tanh(sqrt(2/pi) (x + 0.044715 x^3)))."""
    x = f64(x)
    return 0.5 * x * (1.0 + np.tanh(np.sqrt(2.0 / np.pi) * (x + 0.044715 * x ** 3)))


def linear(x, w_t, b=None):
    """y = x W + b with W stored transposed: w_t is [out][in]."""
    y = f64(x) @ f64(w_t).T
    return y if b is None else y + f64(b)


def embed(w: Gpt2Weights, ids, pos0: int):
    """ids int [B][T] -> x [B][T][d]: token embedding plus the embedding of positions pos0 .. pos0+T-1."""
    ids = np.asarray(ids)
    T = ids.shape[1]
    return f64(w.wte)[ids] + f64(w.wpe)[pos0:pos0 + T][None]


def split_heads(y, n_head):
    """[B][T][d] -> [B][H][T][d/H]."""
    B, T, d = y.shape
    return y.reshape(B, T, n_head, d // n_head).transpose(0, 2, 1, 3)


def merge_heads(y):
    """[B][H][T][dh] -> [B][T][H*dh]."""
    B, H, T, dh = y.shape
    return y.transpose(0, 2, 1, 3).reshape(B, T, H * dh)


def causal_attention(q, k, v):
    """Exact attention of Section 3.1 with a causal mask: q, k, v [B][H][T][dh] (query i sees keys 0..i)."""
    q, k, v = f64(q), f64(k), f64(v)
    T, dh = q.shape[2], q.shape[3]
    s = np.einsum("bhid,bhjd->bhij", q, k) / np.sqrt(float(dh))
    s = np.where(np.tril(np.ones((T, T), dtype=bool))[None, None], s, -np.inf)
    s = s - s.max(axis=-1, keepdims=True)
    p = np.exp(s)
    p /= p.sum(axis=-1, keepdims=True)
    return np.einsum("bhij,bhjd->bhid", p, v)


def block_mlp(lw, x):
    h = layer_norm(x, lw["ln2_g"], lw["ln2_b"])
    return x + linear(gelu_tanh(linear(h, lw["w_fc"], lw["b_fc"])), lw["w_pr"], lw["b_pr"])


def prefill(w: Gpt2Weights, ids):
    """The prompt with exact causal attention.  Returns the hidden states after the last block [B][T][d] and, per
    layer, the keys and values as the cache stores them (fp16, [B][H][T][dh])."""
    x = embed(w, ids, 0)
    keys, values = [], []
    for lw in w.layers:
        a = layer_norm(x, lw["ln1_g"], lw["ln1_b"])
        qkv = linear(a, lw["w_qkv"], lw["b_qkv"])
        d = w.d_model
        q, k, v = (split_heads(qkv[..., i * d:(i + 1) * d], w.n_head) for i in range(3))
        # the cache holds fp16 keys and values; attention over the prompt reads them as stored
        q16, k16, v16 = (t.astype(np.float16) for t in (q, k, v))
        keys.append(k16)
        values.append(v16)
        att = merge_heads(causal_attention(q16, k16, v16))
        x = x + linear(att, lw["w_o"], lw["b_o"])
        x = block_mlp(lw, x)
    return x, keys, values


def logits_of(w: Gpt2Weights, x_last):
    """Final LayerNorm and the tied output projection for hidden rows [B][d] -> [B][vocab]."""
    return linear(layer_norm(x_last, w.lnf_g, w.lnf_b), w.wte)


class LookatDecoder:
    """Decode-time state: per layer the codebooks (k-means on the prompt's keys of each head), the code cache and the
    fp16 value cache.  step(ids) runs one generated token through every layer with Algorithm 1 in place of q K^T."""

    def __init__(self, w: Gpt2Weights, keys, values, m: int, K: int, iters: int, seed: int, capacity: int):
        self.w, self.m, self.K = w, m, K
        self.pos = keys[0].shape[2]
        self.books, self.codes, self.values = [], [], []
        for l, (k16, v16) in enumerate(zip(keys, values)):
            B, H, T, dh = k16.shape
            books, _ = fit_codebooks(k16, m, K, iters, seed=seed + l)
            codes = np.zeros((B, H, capacity, m), dtype=np.uint8)
            encode_keys(k16, books, codes=codes, L_max=capacity, pos=0)
            vc = np.zeros((B, H, capacity, dh), dtype=np.float16)
            vc[:, :, :T] = v16
            self.books.append(books)
            self.codes.append(codes)
            self.values.append(vc)

    def step(self, ids):
        """ids int [B]: the token at position self.pos of every row.  Returns the hidden rows [B][d] after the last
        block; the caches grow by one token."""
        w, pos = self.w, self.pos
        x = embed(w, np.asarray(ids)[:, None], pos)            # [B][1][d]
        d = w.d_model
        for l, lw in enumerate(w.layers):
            a = layer_norm(x, lw["ln1_g"], lw["ln1_b"])
            qkv = linear(a, lw["w_qkv"], lw["b_qkv"])
            q, k, v = (split_heads(qkv[..., i * d:(i + 1) * d], w.n_head) for i in range(3))   # [B][H][1][dh]
            q16, k16, v16 = (t.astype(np.float16) for t in (q, k, v))
            cap = self.codes[l].shape[2]
            encode_keys(k16, self.books[l], codes=self.codes[l], L_max=cap, pos=pos)       # Section 3.4, on append
            self.values[l][:, :, pos] = v16[:, :, 0]
            lut = build_lut(q16[:, :, 0], self.books[l])                                     # Section 3.5
            lens = np.full(q16.shape[0], pos + 1, dtype=np.int32)
            att = attend(lut, self.codes[l], self.values[l], seq_lens=lens, d_k=q16.shape[-1])   # Algorithm 1
            x = x + linear(att.reshape(att.shape[0], 1, d), lw["w_o"], lw["b_o"])
            x = block_mlp(lw, x)
        self.pos += 1
        return x[:, 0]
