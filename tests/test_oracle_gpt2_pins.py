"""Pins of the decoder oracle (oracle/gpt2.py) against what mathematics and library routines fix: LayerNorm moments
and a written-out formula, the tanh-form GELU against its scalar formula and the erf form, linear layers against plain
loops, causal attention against scipy's softmax row by row and closed forms, the cached prompt pass against a
from-scratch recomputation, and the LOOKAT decode step against exact attention over the keys its codes name.
CPU only."""
import math

import numpy as np
import scipy.special

import oracle
from oracle import gpt2
from paper_2601_10155_b200 import synth


def test_layer_norm_moments_and_written_out_formula():
    rng = np.random.default_rng(0)
    x = rng.standard_normal((5, 48)) * 3 + 2
    g, b = rng.standard_normal(48), rng.standard_normal(48)
    y = gpt2.layer_norm(x, np.ones(48), np.zeros(48))
    assert np.abs(y.mean(-1)).max() < 1e-12
    var = x.var(-1)                                        # biased
    np.testing.assert_allclose(y.var(-1), var / (var + gpt2.LN_EPS), rtol=1e-12)
    yy = gpt2.layer_norm(x, g, b)
    for r in range(5):
        mu = sum(x[r]) / 48
        v = sum((t - mu) ** 2 for t in x[r]) / 48
        for c in range(48):
            assert abs(yy[r, c] - ((x[r, c] - mu) / math.sqrt(v + 1e-5) * g[c] + b[c])) < 1e-12
    # a constant row has no direction: the output is the bias
    np.testing.assert_allclose(gpt2.layer_norm(np.full((1, 8), 7.0), g[:8], b[:8])[0], b[:8], atol=1e-12)


def test_gelu_tanh_form():
    xs = np.linspace(-6, 6, 241)
    y = gpt2.gelu_tanh(xs)
    for x, v in zip(xs, y):
        ref = 0.5 * x * (1 + math.tanh(math.sqrt(2 / math.pi) * (x + 0.044715 * x ** 3)))
        assert abs(v - ref) < 1e-15
    assert gpt2.gelu_tanh(np.array([0.0]))[0] == 0.0
    assert abs(gpt2.gelu_tanh(np.array([10.0]))[0] - 10.0) < 1e-12 and abs(gpt2.gelu_tanh(np.array([-10.0]))[0]) < 1e-12
    # the tanh form approximates x Phi(x): they differ by less than 1e-3 everywhere
    erf_form = 0.5 * xs * (1 + scipy.special.erf(xs / math.sqrt(2)))
    assert np.abs(y - erf_form).max() < 1e-3


def test_linear_against_loops():
    rng = np.random.default_rng(1)
    x = rng.standard_normal((3, 7)).astype(np.float16)
    w_t = rng.standard_normal((5, 7)).astype(np.float16)
    b = rng.standard_normal(5).astype(np.float16)
    y = gpt2.linear(x, w_t, b)
    for r in range(3):
        for o in range(5):
            ref = sum(float(x[r, i]) * float(w_t[o, i]) for i in range(7)) + float(b[o])
            assert abs(y[r, o] - ref) < 1e-12


def test_causal_attention_closed_forms_and_scipy():
    rng = np.random.default_rng(2)
    q, k, v = (rng.standard_normal((2, 3, 9, 8)) for _ in range(3))
    out = gpt2.causal_attention(q, k, v)
    np.testing.assert_allclose(out[:, :, 0], v[:, :, 0], atol=1e-12)          # the first query sees one token
    for i in (1, 4, 8):
        s = np.einsum("bhd,bhjd->bhj", q[:, :, i], k[:, :, :i + 1]) / math.sqrt(8)
        p = scipy.special.softmax(s, axis=-1)
        np.testing.assert_allclose(out[:, :, i], np.einsum("bhj,bhjd->bhd", p, v[:, :, :i + 1]), atol=1e-12)
    # q = 0: uniform weights, the running mean of the values
    out0 = gpt2.causal_attention(np.zeros_like(q), k, v)
    np.testing.assert_allclose(out0, np.cumsum(v, axis=2) / np.arange(1, 10)[None, None, :, None], atol=1e-12)


def _toy(seed=3, n_layer=2, n_head=2, d=16, vocab=37, n_pos=24):
    wd = synth.gpt2_weights(seed, n_layer=n_layer, n_head=n_head, d_model=d, vocab=vocab, n_pos=n_pos, plain_init=False)
    return gpt2.Gpt2Weights.from_dict(wd)


def test_prompt_pass_is_causal_and_matches_a_from_scratch_restatement():
    w = _toy()
    ids = synth.token_ids(5, 2, 10, 37)
    x, keys, values = gpt2.prefill(w, ids)
    # causality: the hidden state at position t depends on tokens 0..t only
    x7, _, _ = gpt2.prefill(w, ids[:, :7])
    np.testing.assert_allclose(x[:, :7], x7, atol=1e-12)
    # restated per (row, head, position) with plain loops over the stored fp16 q, k, v of layer 0
    lw = w.layers[0]
    emb = w.wte.astype(np.float64)[ids] + w.wpe.astype(np.float64)[:10][None]
    a = gpt2.layer_norm(emb, lw["ln1_g"], lw["ln1_b"])
    qkv = a @ lw["w_qkv"].astype(np.float64).T + lw["b_qkv"].astype(np.float64)
    b, t, h = 1, 6, 1
    dh = 8
    q = qkv[b, t, h * dh:(h + 1) * dh].astype(np.float16).astype(np.float64)
    s = [float(q @ keys[0][b, h, j].astype(np.float64)) / math.sqrt(dh) for j in range(t + 1)]
    p = scipy.special.softmax(np.array(s))
    att = sum(p[j] * values[0][b, h, j].astype(np.float64) for j in range(t + 1))
    full = gpt2.merge_heads(gpt2.causal_attention(
        gpt2.split_heads(qkv[..., :16], 2).astype(np.float16), keys[0], values[0]))
    np.testing.assert_allclose(full[b, t, h * dh:(h + 1) * dh], att, atol=1e-12)
    np.testing.assert_array_equal(keys[0], gpt2.split_heads(qkv[..., 16:32], 2).astype(np.float16))


def test_decode_step_equals_exact_attention_over_the_keys_its_codes_name():
    """K at least the number of prompt keys per head: every prompt key is its own centroid (distortion 0), so
    Algorithm 1 over the prompt is exact attention; the appended keys are the centroids their codes name.  The decode
    step must therefore equal exact attention with the appended keys replaced by those centroids."""
    w = _toy(seed=4)
    B, T0, steps, m, K = 2, 6, 3, 2, 32                        # 12 prompt keys per head < K
    ids = synth.token_ids(6, B, T0 + steps, 37)
    x, keys, values = gpt2.prefill(w, ids[:, :T0])
    dec = gpt2.LookatDecoder(w, keys, values, m=m, K=K, iters=3, seed=11, capacity=T0 + steps)
    for l in range(w.n_layer):
        np.testing.assert_array_equal(oracle.reconstruct_keys(dec.codes[l][:, :, :T0], dec.books[l]),
                                      keys[l].astype(np.float64))
    for t in range(steps):
        pos = T0 + t
        # the reference runs the same layers with plain softmax attention over k_hat
        xr = gpt2.embed(w, ids[:, pos:pos + 1], pos)
        codes_before = [c.copy() for c in dec.codes]
        x_step = dec.step(ids[:, pos])
        for l, lw in enumerate(w.layers):
            a = gpt2.layer_norm(xr, lw["ln1_g"], lw["ln1_b"])
            qkv = gpt2.linear(a, lw["w_qkv"], lw["b_qkv"])
            q = gpt2.split_heads(qkv[..., :16], 2).astype(np.float16).astype(np.float64)       # [B][H][1][dh]
            k_hat = oracle.reconstruct_keys(dec.codes[l][:, :, :pos + 1], dec.books[l])        # [B][H][pos+1][dh]
            v = dec.values[l][:, :, :pos + 1].astype(np.float64)
            s = np.einsum("bhd,bhjd->bhj", q[:, :, 0], k_hat) / math.sqrt(8)
            att = np.einsum("bhj,bhjd->bhd", scipy.special.softmax(s, axis=-1), v).reshape(B, 1, 16)
            xr = xr + gpt2.linear(att, lw["w_o"], lw["b_o"])
            xr = gpt2.block_mlp(lw, xr)
            assert np.array_equal(codes_before[l][:, :, :pos], dec.codes[l][:, :, :pos])      # earlier codes untouched
        np.testing.assert_allclose(x_step, xr[:, 0], atol=1e-10)
    logits = gpt2.logits_of(w, x_step)
    assert logits.shape == (B, 37) and np.isfinite(logits).all()
