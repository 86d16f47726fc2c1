"""Fidelity metrics of Section 4.2, and a harness that evaluates LOOKAT against exact attention on
the synthetic generator.  CPU only, built on the oracle: TEST INFRASTRUCTURE, never imported by the
CUDA library.

The paper's tables were measured on GPT-2 activations of three texts that are not available here;
the synthetic keys stand in for them, so the figures printed by this module are context, not a
reproduction (the synthetic softmax is far more peaked than a language model's, which lowers the
output cosine; scaling the queries down flattens it).

    python -m oracle.fidelity            # prints one table: m in {2,4,8,16} x sequence length
"""
from __future__ import annotations

import numpy as np

from . import attend, build_lut, encode_keys, exact_attention, fit_codebooks


def cosine_similarity(y_ref: np.ndarray, y: np.ndarray) -> np.ndarray:
    """Section 4.2.1: y_ref . y / (|y_ref| |y|) along the last axis."""
    num = np.sum(y_ref * y, axis=-1)
    den = np.linalg.norm(y_ref, axis=-1) * np.linalg.norm(y, axis=-1)
    return num / den


def kl_divergence(a_ref: np.ndarray, a: np.ndarray, eps: float = 1e-300) -> np.ndarray:
    """Section 4.2.2: sum_i a_ref_i log(a_ref_i / a_i) along the last axis (natural log; terms with
    a_ref_i = 0 contribute nothing)."""
    a_ref = np.asarray(a_ref, dtype=np.float64)
    a = np.asarray(a, dtype=np.float64)
    with np.errstate(divide="ignore", invalid="ignore"):
        t = np.where(a_ref > 0, a_ref * (np.log(np.maximum(a_ref, eps)) - np.log(np.maximum(a, eps))), 0.0)
    return t.sum(axis=-1)


def _ranks(x: np.ndarray) -> np.ndarray:
    """Average ranks (ties share the mean of their positions) along the last axis."""
    x = np.asarray(x)
    out = np.empty(x.shape, dtype=np.float64)
    flat, oflat = x.reshape(-1, x.shape[-1]), out.reshape(-1, x.shape[-1])
    for row, orow in zip(flat, oflat):
        order = np.argsort(row, kind="stable")
        sorted_row = row[order]
        ranks = np.empty(len(row))
        i = 0
        while i < len(row):
            j = i
            while j + 1 < len(row) and sorted_row[j + 1] == sorted_row[i]:
                j += 1
            ranks[order[i:j + 1]] = 0.5 * (i + j)
            i = j + 1
        orow[:] = ranks
    return out


def spearman_rho(s_ref: np.ndarray, s: np.ndarray) -> np.ndarray:
    """Section 4.2.3: Pearson correlation of the ranks along the last axis."""
    r1, r2 = _ranks(s_ref), _ranks(s)
    r1 = r1 - r1.mean(axis=-1, keepdims=True)
    r2 = r2 - r2.mean(axis=-1, keepdims=True)
    return np.sum(r1 * r2, axis=-1) / np.sqrt(np.sum(r1 * r1, axis=-1) * np.sum(r2 * r2, axis=-1))


def topk_overlap(a_ref: np.ndarray, a: np.ndarray, k: int = 5) -> np.ndarray:
    """Section 4.2.4: |TopK(a_ref) ∩ TopK(a)| / k along the last axis."""
    top_ref = np.argsort(-a_ref, axis=-1, kind="stable")[..., :k]
    top = np.argsort(-a, axis=-1, kind="stable")[..., :k]
    hits = (top_ref[..., :, None] == top[..., None, :]).any(axis=-1).sum(axis=-1)
    return hits / float(k)


def _softmax(s: np.ndarray, scale: float) -> np.ndarray:
    x = s * scale
    x = x - x.max(axis=-1, keepdims=True)
    e = np.exp(x)
    return e / e.sum(axis=-1, keepdims=True)


def evaluate(keys, v, q, m: int, K: int = 256, iters: int = 25, seed: int = 0, calib=None) -> dict:
    """LOOKAT with m subspaces against exact attention for one decode query per head.
    keys [B][H_kv][L][d_k], v [B][H_kv][L][d_v], q [B][H_q][d_k] (fp16).  Codebooks are fitted on
    `calib` (same layout) or, if None, on the cached keys themselves.  Returns mean and std over
    (batch row, head) of the four metrics of Section 4.2."""
    d_k = keys.shape[-1]
    books, _ = fit_codebooks(keys if calib is None else calib, m, K, iters, seed=seed)
    codes = encode_keys(keys, books)
    out, s_hat = attend(build_lut(q, books), codes, v, d_k=d_k, want_scores=True)
    ref, s = exact_attention(q, keys, v, want_scores=True)
    scale = 1.0 / np.sqrt(d_k)
    a_ref, a = _softmax(s, scale), _softmax(s_hat, scale)
    metrics = {"cosine": cosine_similarity(ref, out), "kl": kl_divergence(a_ref, a),
               "spearman": spearman_rho(s, s_hat), "top5": topk_overlap(a_ref, a, 5)}
    res = {k: (float(np.mean(val)), float(np.std(val))) for k, val in metrics.items()}
    res["compression"] = 2.0 * d_k / m
    return res


def main():
    from paper_2601_10155_b200 import synth
    print("LOOKAT vs exact attention on the synthetic generator (GPT-2 shapes: 12 heads, d = 64, K = 256, "
          "25 Lloyd iterations, codebooks fitted on a separate 4096-key draw per head; batch 4)")
    print(f"{'m':>3} {'L':>5} {'q scale':>8} {'compr':>6} {'cosine':>14} {'KL (nats)':>14} {'Spearman':>14} {'top-5':>14}")
    for q_scale in (1.0, 0.1):
        for m in (2, 4, 8, 16):
            for L in (128, 512, 1024):
                w = synth.small_workload(name="fid", seed=1000, B=4, n_q_heads=12, n_kv_heads=12, d_k=64,
                                         d_v=64, L=L, m=m, K=256, rank=16)
                keys, v, q = synth.make_keys(w), synth.make_values(w), synth.make_queries(w, q_scale)
                r = evaluate(keys, v, q, m, calib=synth.make_calibration_keys(w, 4096))
                cells = "  ".join(f"{r[k][0]:6.3f}±{r[k][1]:5.3f}" for k in ("cosine", "kl", "spearman", "top5"))
                print(f"{m:>3} {L:>5} {q_scale:>8} {r['compression']:>5.0f}x  {cells}")


if __name__ == "__main__":
    main()
