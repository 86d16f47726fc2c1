"""The GPT-2 decoder harness on the GPU against the decoder oracle (oracle/gpt2.py), through the C ABI of
include/lookat_gpt2.h: every kernel of the harness on its own, then the model -- the prompt pass with exact attention,
codebooks and codes of every layer, and teacher-forced decode steps with Algorithm 1 in every layer.

Tolerances.  The oracle works in fp64 on the same fp16 weights.  The GPU rounds what a product reads to fp16 (relative
2^-11 = 4.9e-4 per element, independent across the K terms of a dot product) and accumulates in fp32; outputs stored
as fp16 add one more rounding (2^-11 of the value).  A single kernel fed the oracle's own inputs is therefore held to
2e-3 of the output's rms plus 1e-3 of each value.  Through the model the roundings of about five products per block add up like a random
walk: after L blocks about sqrt(5 L) * 5e-4 of the residual stream's scale; 12 blocks give 4e-3, the tests allow 2e-2.
Where an integer decision hangs on floating point (a key's code), the codes are compared on the GPU's own fp16 keys.
"""
import numpy as np
import pytest
import torch

import oracle
from oracle import gpt2 as ref
from paper_2601_10155_b200 import synth
from paper_2601_10155_b200.binding import Lookat, LookatGpt2

pytestmark = pytest.mark.gpu


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def close(got, want, rel, what=""):
    """|got - want| <= rel * rms(want) + 1e-3 * |want| element by element: an error budget against the scale of the
    whole output plus the rounding of an fp16 result (2^-11 of its own magnitude, twice)"""
    got, want = np.asarray(got, dtype=np.float64), np.asarray(want, dtype=np.float64)
    scale = float(np.sqrt((want ** 2).mean())) + 1e-30
    excess = np.abs(got - want) - 1e-3 * np.abs(want)
    assert float(excess.max()) <= rel * scale, \
        f"{what}: error {float(np.abs(got - want).max()):.3e} against scale {scale:.3e} (allowed {rel:g} of it plus 1e-3 relative)"


@pytest.fixture(scope="module")
def lk():
    return Lookat(4, 4, 64, 64, 4, 16)


@pytest.mark.parametrize("M,N,K", [(200, 384, 128), (128, 128, 64), (129, 200, 72), (1000, 768, 768), (333, 3072, 768), (257, 768, 3072),
                                   (32, 384, 128), (1, 96, 64), (17, 100, 1032), (32, 2304, 768),
                                   (32, 768, 3072),      # one-token product, K in 8 slices over a thread-block cluster
                                   (32, 9491, 768),      # ... 32 columns per CTA (wide output), ragged last column group
                                   (5, 20011, 136),      # ... wide, one slice, K not a multiple of 32
                                   (32, 8, 8)])          # ... the smallest
@pytest.mark.parametrize("mode", ["plain_fp16", "gelu_fp16", "residual_fp32"])
def test_linear_matches_oracle(lk, M, N, K, mode):
    rng = np.random.default_rng(M * 31 + N * 7 + K)
    x = (rng.standard_normal((M, K)) * 1.5).astype(np.float16)
    w_t = (rng.standard_normal((N, K)) * 0.05).astype(np.float16)
    b = (rng.standard_normal(N) * 0.5).astype(np.float16)
    res = rng.standard_normal((M, N)).astype(np.float32)
    want = ref.linear(x, w_t, b)
    if mode == "plain_fp16":
        got = lk.lookat_linear(dev(x), dev(w_t), dev(b))
    elif mode == "gelu_fp16":
        want = ref.gelu_tanh(want)
        got = lk.lookat_linear(dev(x), dev(w_t), dev(b), gelu=True)
    else:
        want = want + res
        r = dev(res)
        got = lk.lookat_linear(dev(x), dev(w_t), dev(b), residual=r, out=r, out_fp16=False)     # in place, as the model does
    torch.cuda.synchronize()
    close(got.float().cpu().numpy(), want, 2e-3, f"linear {M}x{N}x{K} {mode}")


def test_linear_takes_fp32_rows_for_a_decode_step(lk):
    rng = np.random.default_rng(3)
    x = rng.standard_normal((32, 768)).astype(np.float32)
    w_t = (rng.standard_normal((768, 768)) * 0.03).astype(np.float16)
    got = lk.lookat_linear(dev(x), dev(w_t), None, out_fp16=False)
    close(got.cpu().numpy(), ref.linear(x.astype(np.float16), w_t), 2e-3, "fp32 rows")


@pytest.mark.parametrize("B,T", [(2, 100), (3, 1), (1, 64)])
def test_fused_qkv_projection_scatters_head_major(lk, B, T):
    H, d = 4, 256
    rng = np.random.default_rng(B * 100 + T)
    x = rng.standard_normal((B * T, d)).astype(np.float16)
    w_t = (rng.standard_normal((3 * d, d)) * 0.06).astype(np.float16)
    b = (rng.standard_normal(3 * d) * 0.3).astype(np.float16)
    cap, off = T + 5, 3
    q = torch.zeros((B, H, T, 64), dtype=torch.float16, device="cuda")
    k = torch.zeros((B, H, T, 64), dtype=torch.float16, device="cuda")
    v = torch.full((B, H, cap, 64), 7.0, dtype=torch.float16, device="cuda")
    lk.lookat_linear_qkv(dev(x), dev(w_t), dev(b), B, T, H, q, k, v, v_off=off)
    y = ref.linear(x, w_t, b).reshape(B, T, 3 * d)
    for i, got in enumerate((q, k, v[:, :, off:off + T])):
        close(got.float().cpu().numpy(), ref.split_heads(y[..., i * d:(i + 1) * d], H), 2e-3, f"third {i}")
    assert float(v[:, :, :off].min()) == 7.0 and float(v[:, :, off + T:].min()) == 7.0     # nothing outside the rows written


def test_layernorm_embed_argmax_match_oracle(lk):
    rng = np.random.default_rng(5)
    x = (rng.standard_normal((77, 768)) * 3 + 1).astype(np.float32)
    g, b = (1 + 0.3 * rng.standard_normal(768)).astype(np.float16), rng.standard_normal(768).astype(np.float16)
    close(lk.lookat_layernorm(dev(x), dev(g), dev(b)).float().cpu().numpy(), ref.layer_norm(x, g, b), 2e-3, "layernorm")
    x2 = rng.standard_normal((5, 128)).astype(np.float32)
    close(lk.lookat_layernorm(dev(x2), dev(g[:128]), dev(b[:128])).float().cpu().numpy(), ref.layer_norm(x2, g[:128], b[:128]), 2e-3, "layernorm 128")
    wd = synth.gpt2_weights(1, n_layer=1, n_head=2, d_model=128, vocab=300, n_pos=40)
    ids = synth.token_ids(2, 3, 9, 300)
    got = lk.lookat_embed(dev(ids), dev(wd["wte"]), dev(wd["wpe"]), pos0=4).cpu().numpy()
    want = ref.f64(wd["wte"])[ids] + ref.f64(wd["wpe"])[4:13][None]
    assert np.abs(got - want).max() <= 1e-6
    logits = rng.standard_normal((6, 50257)).astype(np.float32)
    logits[2, 100] = logits[2, 40000] = 50.0                       # a tie: the first index wins
    assert np.array_equal(lk.lookat_argmax(dev(logits)).cpu().numpy(), logits.argmax(axis=1))


@pytest.mark.parametrize("B,H,T", [(2, 3, 200), (1, 2, 64), (1, 1, 65), (2, 2, 1), (1, 12, 300)])
def test_causal_attention_matches_oracle(lk, B, H, T):
    rng = np.random.default_rng(B * 1000 + H * 100 + T)
    q = (rng.standard_normal((B, H, T, 64)) * 1.5).astype(np.float16)
    k = (rng.standard_normal((B, H, T, 64)) * 1.5).astype(np.float16)
    cap = T + 3
    v = np.zeros((B, H, cap, 64), dtype=np.float16)
    v[:, :, :T] = rng.standard_normal((B, H, T, 64)).astype(np.float16)
    got = lk.lookat_causal_attention(dev(q), dev(k), dev(v)).float().cpu().numpy()
    want = ref.merge_heads(ref.causal_attention(q, k, v[:, :, :T]))
    assert np.abs(got - want).max() <= 2e-3                         # the attention outputs' bound, as for Algorithm 1


def _model(n_layer, n_head, vocab, B, T0, steps, m, K, seed):
    wd = synth.gpt2_weights(seed, n_layer=n_layer, n_head=n_head, d_model=64 * n_head, vocab=vocab, n_pos=T0 + steps + 2,
                            plain_init=False)
    ids = synth.token_ids(seed + 1, B, T0 + steps, vocab)
    gpu = LookatGpt2(wd, B, T0 + steps, m, K, fit_iters=4, keep_prompt_keys=True)
    return wd, ids, gpu


@pytest.mark.parametrize("n_layer,n_head,B,T0,steps,m,K", [(2, 12, 2, 150, 4, 4, 64),      # two blocks at full width
                                                          (12, 4, 3, 70, 5, 4, 32)])       # twelve blocks, narrower
def test_decoder_matches_oracle_teacher_forced(n_layer, n_head, B, T0, steps, m, K):
    vocab = 1000
    wd, ids, gpu = _model(n_layer, n_head, vocab, B, T0, steps, m, K, seed=21)
    w = ref.Gpt2Weights.from_dict(wd)
    hidden = gpu.lookat_gpt2_prefill(dev(ids[:, :T0]), seed=5, want_hidden=True)
    torch.cuda.synchronize()
    x_ref, keys_ref, values_ref = ref.prefill(w, ids[:, :T0])
    close(hidden.cpu().numpy(), x_ref, 2e-2, "prompt pass, residual stream")
    # per layer: the GPU's fp16 keys are the oracle's up to fp16 rounding of slightly different fp32 values; codebooks and
    # codes are compared on the GPU's OWN keys (verified hand-off), where they must be the oracle's bit for bit
    dec_keys, dec_vals = [], []
    for l in range(n_layer):
        books, codes, values, pkeys = gpu.lookat_gpt2_layer_state(l, T=T0)
        pk = pkeys.cpu().numpy()
        close(pk.astype(np.float64), keys_ref[l].astype(np.float64), 2e-2, f"layer {l} keys")
        close(values[:, :, :T0].float().cpu().numpy(), values_ref[l].astype(np.float64), 2e-2, f"layer {l} values")
        rb, _ = oracle.fit_codebooks(pk, m, K, 4, seed=5 + l)
        one, _ = oracle.fit_codebooks(pk, m, K, 1, seed=5 + l)
        rc, gap = oracle.encode_keys(pk, rb, want_gap=True)
        near = (gap > 0) & (gap < 1e-6)
        if np.array_equal(books.cpu().numpy(), rb):
            assert not ((codes[:, :, :T0].cpu().numpy() != rc) & ~near).any(), f"layer {l} codes"
        else:
            # a near-tie decision in an assignment pass may split two valid Lloyd runs: the codes must then be the nearest
            # centroids of the GPU's own codebooks
            gb = books.cpu().numpy()
            rc2, gap2 = oracle.encode_keys(pk, gb, want_gap=True)
            assert not ((codes[:, :, :T0].cpu().numpy() != rc2) & ~((gap2 > 0) & (gap2 < 1e-6))).any(), f"layer {l} codes"
        dec_keys.append(pk)
        dec_vals.append(values[:, :, :T0].cpu().numpy())
    # decode, teacher forced: the oracle continues from the GPU's caches (its own k-means on the GPU's keys, seeds as the
    # GPU's), so that a code that legitimately differs through rounded keys cannot masquerade as an error of a step
    dec = ref.LookatDecoder(w, dec_keys, dec_vals, m=m, K=K, iters=4, seed=5, capacity=T0 + steps)
    for t in range(steps):
        hid, logits, nxt = gpu.lookat_gpt2_decode(dev(ids[:, T0 + t]), want_hidden=True, want_logits=True, want_next=True)
        torch.cuda.synchronize()
        x_step = dec.step(ids[:, T0 + t])
        close(hid.cpu().numpy(), x_step, 2e-2, f"decode step {t}, residual stream")
        lg_ref = ref.logits_of(w, x_step)
        close(logits.cpu().numpy(), lg_ref, 2e-2, f"decode step {t}, logits")
        assert np.array_equal(nxt.cpu().numpy(), logits.cpu().numpy().argmax(axis=1))
    assert gpu.lookat_gpt2_position() == T0 + steps
