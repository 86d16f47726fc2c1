"""Parity at the full size of the benchmark workload (`gqa_32k_m8`: batch 16, 32 query heads on 8 KV
heads, d = 128, 32768 cached tokens, m = 8), in the launch configuration bench.py times
(`lookat_decode_step`, library-chosen chunking), on sampled rows the oracle can compute one by one;
plus properties that hold at any size.  Also the 1M-key encode shape on a subset the oracle can do,
and the causal prefill launch of config 4 in its three forms on sampled queries.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2601_10155_b200 import synth
from paper_2601_10155_b200.binding import Lookat

pytestmark = pytest.mark.gpu

SCORE_TOL = 1e-4
OUT_TOL = 2e-3


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


@pytest.fixture(scope="module")
def gqa_32k():
    w = synth.WORKLOADS["gqa_32k_m8"]
    keys, v, q = synth.make_keys(w), synth.make_values(w), synth.make_queries(w)
    # codebooks from the ORACLE's k-means on a small calibration draw (nothing the oracle is fed
    # comes from the GPU): 2 Lloyd iterations on 4096 keys per head
    books, _ = oracle.fit_codebooks(synth.make_calibration_keys(w, 4096), w.m, w.K, iters=2, seed=w.seed)
    lk = Lookat(w.n_q_heads, w.n_kv_heads, w.d_k, w.d_v, w.m, w.K)
    books_d, v_d = dev(books), dev(v)
    codes_d = lk.lookat_encode_keys(dev(keys), books_d)
    torch.cuda.synchronize()
    return dict(w=w, keys=keys, v=v, q=q, books=books, lk=lk, books_d=books_d, v_d=v_d, codes_d=codes_d)


def test_full_size_decode_step_on_sampled_rows(gqa_32k):
    s = gqa_32k
    w, lk = s["w"], s["lk"]
    rows = [(0, 0), (7, 3), (15, 7)]                       # (batch row, KV head)
    L = w.L
    # hand-off: the sampled rows get the oracle's codes (GPU codes are checked against them first)
    for b, h in rows:
        ref_codes, gap = oracle.encode_keys(s["keys"][b:b + 1, h:h + 1], s["books"][h:h + 1], want_gap=True)
        got = s["codes_d"][b, h].cpu().numpy()
        diff = got != ref_codes[0, 0]
        near = (gap[0, 0] > 0) & (gap[0, 0] < 1e-6)
        assert not (diff & ~near).any()
        s["codes_d"][b, h] = dev(ref_codes[0, 0])
    # the newest key is appended again by the step itself (same value, same code)
    k_new = dev(s["keys"][:, :, L - 1])
    for q_scale in (1.0, 0.1):
        q = synth.make_queries(w, q_scale)
        out = lk.lookat_decode_step(dev(q), k_new, s["books_d"], s["codes_d"], s["v_d"], L - 1)
        torch.cuda.synchronize()
        out = out.cpu().numpy()
        assert np.isfinite(out).all()
        for b, h in rows:
            codes_row = s["codes_d"][b, h].cpu().numpy()[None, None]
            hq = slice(h * w.g, (h + 1) * w.g)
            lut = oracle.build_lut(q[b:b + 1, hq], s["books"][h:h + 1])
            ref = oracle.attend(lut, codes_row, s["v"][b:b + 1, h:h + 1], d_k=w.d_k)
            assert np.abs(out[b, hq] - ref[0]).max() <= OUT_TOL


def test_full_size_scores_on_a_sampled_row(gqa_32k):
    s = gqa_32k
    w, lk = s["w"], s["lk"]
    b, h = 3, 5
    scores = torch.full((w.B, w.n_q_heads, w.L), float("nan"), device="cuda")
    lk.lookat_attend(s["codes_d"], s["v_d"], q=dev(s["q"]), codebooks=s["books_d"], scores_out=scores)
    torch.cuda.synchronize()
    hq = slice(h * w.g, (h + 1) * w.g)
    got = scores[b, hq].cpu().numpy().astype(np.float64)
    codes_row = s["codes_d"][b, h].cpu().numpy()[None, None]
    lut = oracle.build_lut(s["q"][b:b + 1, hq], s["books"][h:h + 1])
    _, ref = oracle.attend(lut, codes_row, s["v"][b:b + 1, h:h + 1], d_k=w.d_k, want_scores=True)
    assert np.all(np.abs(got - ref[0]) <= SCORE_TOL * (1 + np.abs(ref[0])))
    assert not torch.isnan(scores).any()


def test_full_size_properties(gqa_32k):
    s = gqa_32k
    w, lk = s["w"], s["lk"]
    # q = 0: every table is 0, the weights are uniform, every output row is the mean of its V rows
    out0 = lk.lookat_attend(s["codes_d"], s["v_d"], q=torch.zeros_like(dev(s["q"])), codebooks=s["books_d"])
    mean_v = s["v_d"].float().mean(dim=2).repeat_interleave(w.g, dim=1)
    assert float((out0 - mean_v).abs().max()) <= 1e-4
    # the chunking chosen by the library and explicit chunk counts give the same result
    q_d = dev(synth.make_queries(w, 0.1))
    ref = lk.lookat_attend(s["codes_d"], s["v_d"], q=q_d, codebooks=s["books_d"])
    for n_splits in (1, 5, 32):
        o = lk.lookat_attend(s["codes_d"], s["v_d"], q=q_d, codebooks=s["books_d"], n_splits=n_splits)
        assert float((o - ref).abs().max()) <= 2e-5
    # heads of a group with the same query give the same output
    q2 = synth.make_queries(w, 0.1)
    q2[:, 1] = q2[:, 0]
    o = lk.lookat_attend(s["codes_d"], s["v_d"], q=dev(q2), codebooks=s["books_d"]).cpu().numpy()
    assert np.array_equal(o[:, 0], o[:, 1])
    # ragged rows: a row cut to 1000 tokens equals attending over a cache of 1000 tokens
    sl = torch.full((w.B,), w.L, dtype=torch.int32, device="cuda")
    sl[2] = 1000
    sl[9] = 0
    o_r = lk.lookat_attend(s["codes_d"], s["v_d"], q=q_d, codebooks=s["books_d"], seq_lens=sl)
    short = lk.lookat_attend(s["codes_d"][2:3, :, :1008].contiguous(), s["v_d"][2:3, :, :1008].contiguous(),
                             q=q_d[2:3].contiguous(), codebooks=s["books_d"],
                             seq_lens=torch.tensor([1000], dtype=torch.int32, device="cuda"))
    assert float((o_r[2] - short[0]).abs().max()) <= 2e-5
    assert float(o_r[9].abs().max()) == 0.0
    assert float((o_r[0] - ref[0]).abs().max()) <= 2e-5


def test_full_size_attention_with_quantised_values(gqa_32k):
    """`lookat_attend_pqv` in the launch configuration bench.py times (16 rows, 32,768 tokens, m = m_v = 8): the
    value codebooks are the oracle's k-means on 4096 values per head, the value codes the GPU encoder's (the
    sampled rows get the oracle's codes, checked against the GPU's first), the tables come from q inside the call;
    sampled (row, KV head) units against the oracle, plus properties that need no oracle."""
    s = gqa_32k
    w, lk = s["w"], s["lk"]
    m_v = w.m
    v_books, _ = oracle.fit_codebooks(s["v"][:1, :, :4096], m_v, 256, iters=2, seed=w.seed + 1)
    lv = Lookat(w.n_kv_heads, w.n_kv_heads, w.d_v, w.d_v, m_v, 256)
    v_books_d = dev(v_books)
    v_codes_d = lv.lookat_encode_keys(s["v_d"], v_books_d)
    rows = [(0, 0), (6, 5), (15, 7)]
    for b, h in rows:
        ref_codes, gap = oracle.encode_keys(s["v"][b:b + 1, h:h + 1], v_books[h:h + 1], want_gap=True)
        got = v_codes_d[b, h].cpu().numpy()
        assert not ((got != ref_codes[0, 0]) & ~((gap[0, 0] > 0) & (gap[0, 0] < 1e-6))).any()
        v_codes_d[b, h] = dev(ref_codes[0, 0])
    for q_scale in (1.0, 0.1):
        q = synth.make_queries(w, q_scale)
        out = lk.lookat_attend_pqv(s["codes_d"], v_books_d, v_codes_d, q=dev(q), codebooks=s["books_d"]).cpu().numpy()
        assert np.isfinite(out).all()
        for b, h in rows:
            hq = slice(h * w.g, (h + 1) * w.g)
            lut = oracle.build_lut(q[b:b + 1, hq], s["books"][h:h + 1])
            codes = s["codes_d"][b:b + 1, h:h + 1].cpu().numpy()
            ref = oracle.attend_pqv(lut, codes, v_books[h:h + 1], v_codes_d[b:b + 1, h:h + 1].cpu().numpy(), d_k=w.d_k)
            assert np.abs(out[b, hq] - ref[0]).max() <= OUT_TOL
    # bit-reproducible: the histogram adds are integer adds, whatever order they land in
    q_d = dev(synth.make_queries(w, 0.1))
    o1 = lk.lookat_attend_pqv(s["codes_d"], v_books_d, v_codes_d, q=q_d, codebooks=s["books_d"])
    o2 = lk.lookat_attend_pqv(s["codes_d"], v_books_d, v_codes_d, q=q_d, codebooks=s["books_d"])
    assert torch.equal(o1, o2)
    # q = 0: uniform weights, the output is the mean of the dequantised values
    o0 = lk.lookat_attend_pqv(s["codes_d"], v_books_d, v_codes_d, q=torch.zeros_like(q_d), codebooks=s["books_d"])
    b, h = 3, 2
    vc = v_codes_d[b, h].long()                             # [L][m_v]
    deq = torch.cat([v_books_d[h, j][vc[:, j]] for j in range(m_v)], dim=1)      # [L][d_v]
    assert float((o0[b, h * w.g] - deq.double().mean(dim=0).float()).abs().max()) <= 1e-4
    # a row cut short by seq_lens equals attending over a cache of that length
    sl = torch.full((w.B,), w.L, dtype=torch.int32, device="cuda")
    sl[2], sl[9] = 5000, 0
    o_r = lk.lookat_attend_pqv(s["codes_d"], v_books_d, v_codes_d, q=q_d, codebooks=s["books_d"], seq_lens=sl)
    short = lk.lookat_attend_pqv(s["codes_d"][2:3, :, :5000].contiguous(), v_books_d, v_codes_d[2:3, :, :5000].contiguous(),
                                 q=q_d[2:3].contiguous(), codebooks=s["books_d"])
    assert float((o_r[2] - short[0]).abs().max()) <= 2e-5
    assert float(o_r[9].abs().max()) == 0.0
    assert torch.equal(o_r[0], o1[0])


def test_encode_shape_of_the_1m_key_workload_on_a_subset():
    """d_k = 128, m = 16 (d_sub = 8), K = 256: 65,536 of the 1,048,576 keys against codebooks taken
    from the first keys by the start rule (0 Lloyd iterations), checked in full against the oracle."""
    w = synth.WORKLOADS["encode_1m_m16"]
    n = 65536
    keys = synth.make_keys(w, n_tokens=n)
    books, _ = oracle.fit_codebooks(keys[:, :, :16384], w.m, w.K, iters=0, seed=w.seed)
    ref, gap = oracle.encode_keys(keys, books, want_gap=True)
    lk = Lookat(w.n_q_heads, w.n_kv_heads, w.d_k, w.d_v, w.m, w.K)
    ties = torch.zeros(1, dtype=torch.int64, device="cuda")
    books_gpu = lk.lookat_fit_codebooks(dev(keys[:, :, :16384]), 0, seed=w.seed)
    assert np.array_equal(books_gpu.cpu().numpy(), books)
    codes = lk.lookat_encode_keys(dev(keys), dev(books), near_ties=ties).cpu().numpy()
    near = (gap > 0) & (gap < 1e-6)
    assert not ((codes != ref) & ~near).any()
    assert int(ties.item()) == int(near.sum())


# ------------------------------------------------------------------ causal prefill at the config-4 size
@pytest.fixture(scope="module")
def prefill_4k():
    w = synth.WORKLOADS["prefill_4k_m16"]
    keys, v = synth.make_keys(w), synth.make_values(w)
    q = synth.make_prefill_queries(w, w.L)
    books, _ = oracle.fit_codebooks(synth.make_calibration_keys(w, 2048), w.m, w.K, iters=2, seed=w.seed)
    lk = Lookat(w.n_q_heads, w.n_kv_heads, w.d_k, w.d_v, w.m, w.K)
    codes_d = lk.lookat_encode_keys(dev(keys), dev(books))
    torch.cuda.synchronize()
    return dict(w=w, keys=keys, v=v, q=q, books=books, lk=lk, codes_d=codes_d)


@pytest.mark.parametrize("form", ["contraction", "tables"])
def test_full_size_prefill_on_sampled_rows(prefill_4k, form):
    """The whole config-4 launch (batch 4, 32 heads, 4096 causal queries over 4096 tokens) as bench.py times it;
    sampled (row, head, query) triples against the oracle, tile and chunk edges among them; and a closed form
    for every head: the first query sees one token, so its output is that token's value row."""
    s = prefill_4k
    w, lk = s["w"], s["lk"]
    heads = [(0, 0), (1, 13), (3, 31)]
    queries = [0, 1, 63, 64, 127, 128, 129, 1000, 2047, 2048, 4032, 4095]
    # hand-off: the sampled heads get the oracle's codes (the GPU's are checked against them first)
    for b, h in heads:
        ref_codes, gap = oracle.encode_keys(s["keys"][b:b + 1, h:h + 1], s["books"][h:h + 1], want_gap=True)
        got = s["codes_d"][b, h].cpu().numpy()
        near = (gap[0, 0] > 0) & (gap[0, 0] < 1e-6)
        assert not ((got != ref_codes[0, 0]) & ~near).any()
        s["codes_d"][b, h] = dev(ref_codes[0, 0])
    lk.lookat_set_prefill_form(form)
    out = lk.lookat_attend_prefill(dev(s["q"]), dev(s["books"]), s["codes_d"], dev(s["v"]))
    torch.cuda.synchronize()
    lk.lookat_set_prefill_form("auto")
    out = out.cpu().numpy()
    assert np.isfinite(out).all()
    assert np.abs(out[:, :, 0] - s["v"][:, :, 0].astype(np.float32)).max() <= 1e-3
    for b, h in heads:
        codes_row = s["codes_d"][b, h].cpu().numpy()[None, None]
        for i in queries:
            ref = oracle.attend_prefill(s["q"][b:b + 1, h:h + 1, i:i + 1], s["books"][h:h + 1], codes_row,
                                        s["v"][b:b + 1, h:h + 1], q_pos0=i)
            assert np.abs(out[b, h, i] - ref[0, 0, 0]).max() <= OUT_TOL, (form, b, h, i)


def test_prefill_with_16_subspaces_on_64_dim_heads_at_a_gpt2_prompt_size():
    """The paper's 16-subspace setting on GPT-2 heads (d_k 64, sub-vectors of 4 dims) over a prompt of 1024 tokens, batch 8,
    12 heads, in the contraction form (two centroids per 8-dim group of a rebuilt key row): sampled (row, head, query)
    triples against the oracle, every first query against its closed form, and the two forms against each other."""
    w = synth.small_workload(B=8, n_q_heads=12, n_kv_heads=12, d_k=64, d_v=64, m=16, K=256, L=1024, rank=16)
    keys, v = synth.make_keys(w), synth.make_values(w)
    q = synth.make_prefill_queries(w, w.L)
    books, _ = oracle.fit_codebooks(keys[:, :, :512], w.m, w.K, iters=2, seed=11)
    lk = Lookat(w.n_q_heads, w.n_kv_heads, w.d_k, w.d_v, w.m, w.K)
    codes_d = lk.lookat_encode_keys(dev(keys), dev(books))
    heads = [(0, 0), (3, 7), (7, 11)]
    for b, h in heads:
        ref_codes, gap = oracle.encode_keys(keys[b:b + 1, h:h + 1], books[h:h + 1], want_gap=True)
        got = codes_d[b, h].cpu().numpy()
        near = (gap[0, 0] > 0) & (gap[0, 0] < 1e-6)
        assert not ((got != ref_codes[0, 0]) & ~near).any()
        codes_d[b, h] = dev(ref_codes[0, 0])
    outs = {}
    for form in ("contraction", "tables"):
        lk.lookat_set_prefill_form(form)
        outs[form] = lk.lookat_attend_prefill(dev(q), dev(books), codes_d, dev(v)).cpu().numpy()
    lk.lookat_set_prefill_form("auto")
    out = outs["contraction"]
    assert np.isfinite(out).all()
    assert np.abs(out[:, :, 0] - v[:, :, 0].astype(np.float32)).max() <= 1e-3
    assert np.abs(out - outs["tables"]).max() <= 2 * OUT_TOL
    for b, h in heads:
        codes_row = codes_d[b, h].cpu().numpy()[None, None]
        for i in (0, 1, 63, 64, 127, 128, 255, 256, 700, 1023):
            ref = oracle.attend_prefill(q[b:b + 1, h:h + 1, i:i + 1], books[h:h + 1], codes_row, v[b:b + 1, h:h + 1], q_pos0=i)
            assert np.abs(out[b, h, i] - ref[0, 0, 0]).max() <= OUT_TOL, (b, h, i)


# ------------------------------------------------------------------ k-means at the sizes the benchmark fits
def _fit_against_oracle(w, keys, lk, iters, head, subspaces, seed):
    """GPU k-means on the whole problem, the oracle's on `subspaces` (consecutive, starting at 0) of KV head `head`
    -- the start rule depends on (head, subspace) only through head * m + subspace, so head 0 keeps its starts when
    the oracle is given just the first subspaces.  One Lloyd step must agree bit for bit (exact integer means)
    unless the oracle flags a near tie in that assignment; the full run must be bit-identical, or -- where a near-tie
    decision split the two runs -- end at the same distortion to 1e-4 relative."""
    assert head == 0 and list(subspaces) == list(range(len(subspaces)))
    d_sub, ms = w.d_sub, len(subspaces)
    sub = np.ascontiguousarray(keys[:, :1, :, :ms * d_sub])
    keys_d = dev(keys)
    one_gpu = lk.lookat_fit_codebooks(keys_d, 1, seed=seed).cpu().numpy()[0, :ms]
    books_gpu, trace_gpu = lk.lookat_fit_codebooks(keys_d, iters, seed=seed, want_distortion=True)
    books_gpu, trace_gpu = books_gpu.cpu().numpy()[0, :ms], trace_gpu.cpu().numpy()[0, :ms]
    start, _ = oracle.fit_codebooks(sub, ms, w.K, 0, seed=seed)
    _, gap0 = oracle.encode_keys(sub, start, want_gap=True)
    one, _ = oracle.fit_codebooks(sub, ms, w.K, 1, seed=seed)
    if not ((gap0 > 0) & (gap0 < 1e-6)).any():
        assert np.array_equal(one_gpu, one[0]), "one Lloyd step differs from the oracle"
    ref, ref_trace = oracle.fit_codebooks(sub, ms, w.K, iters, seed=seed)
    if np.array_equal(books_gpu, ref[0]):
        np.testing.assert_allclose(trace_gpu, ref_trace[0], rtol=1e-11, atol=1e-300)
    else:
        np.testing.assert_allclose(trace_gpu[:, -1], ref_trace[0, :, -1], rtol=1e-4)
    assert np.all(trace_gpu[:, 1:] <= trace_gpu[:, :-1] * (1 + 1e-7))
    return sub, ref


def test_fit_at_the_benchmark_size_on_two_subspaces():
    """Config 3 as bench.py fits it: 8 KV heads x 8 subspaces of 16 dims, 65,536 keys per head (16 rows x 4096), 10
    Lloyd iterations in one call; KV head 0, subspaces 0 and 1 against the oracle.  Then the near-tie counter of the bulk
    encoder on those keys against the oracle's count."""
    w = synth.WORKLOADS["gqa_32k_m8"]
    keys = synth.make_keys(w, n_tokens=w.fit_keys_per_head // w.B)
    lk = Lookat(w.n_q_heads, w.n_kv_heads, w.d_k, w.d_v, w.m, w.K)
    sub, ref = _fit_against_oracle(w, keys, lk, w.fit_iters, 0, (0, 1), w.seed)
    ref_codes, gap = oracle.encode_keys(sub, ref, want_gap=True)
    near = (gap > 0) & (gap < 1e-6)
    l2 = Lookat(1, 1, 2 * w.d_sub, w.d_v, 2, w.K)
    ties = torch.zeros(1, dtype=torch.int64, device="cuda")
    codes = l2.lookat_encode_keys(dev(sub), dev(ref), near_ties=ties).cpu().numpy()
    assert not ((codes != ref_codes) & ~near).any()
    assert int(ties.item()) == int(near.sum())


def test_refit_at_the_1m_key_workload_size_on_one_subspace():
    """Config 4's refit as bench.py runs it: one head, 16 subspaces of 8 dims, 262,144 keys, 10 Lloyd iterations --
    256 CTAs add into the sums of every problem; subspace 0 against the oracle."""
    w = synth.WORKLOADS["encode_1m_m16"]
    keys = synth.make_keys(w, n_tokens=w.fit_keys_per_head)
    lk = Lookat(w.n_q_heads, w.n_kv_heads, w.d_k, w.d_v, w.m, w.K)
    _fit_against_oracle(w, keys, lk, w.fit_iters, 0, (0,), w.seed)


# ------------------------------------------------------------------ the generation loop of config 2 at its size
def test_generation_loop_at_the_gpt2_decoder_size():
    """One attention layer of BASELINE config 2 at size: batch 32 x 12 heads, d = 64, m = 4, a cache with room for 1088
    tokens that `lookat_decode_step` grows from 1024 to 1028 (append-encode + Algorithm 1 per step, one launch).  Per
    step: the appended codes of every row bit-exact against the oracle's (near ties excused), and the outputs of sampled
    (row, head) pairs against the oracle within 2e-3."""
    w = synth.WORKLOADS["gpt2_b32_l1024_m4"]
    L0, L_cap, steps = w.L, w.L + 64, 4
    keys, v = synth.make_keys(w, n_tokens=L_cap), synth.make_values(w, n_tokens=L_cap)
    books, _ = oracle.fit_codebooks(synth.make_calibration_keys(w, 4096), w.m, w.K, iters=2, seed=w.seed)
    lk = Lookat(w.n_q_heads, w.n_kv_heads, w.d_k, w.d_v, w.m, w.K)
    books_d, v_d = dev(books), dev(v)
    cache = torch.zeros((w.B, w.n_kv_heads, L_cap, w.m), dtype=torch.uint8, device="cuda")
    lk.lookat_encode_keys(dev(keys[:, :, :L0]), books_d, codes=cache, pos=0)          # prefill encode
    ref_cache, gap = oracle.encode_keys(keys, books, want_gap=True)                       # every key, appended ones too
    near = (gap > 0) & (gap < 1e-6)
    got = cache.cpu().numpy()
    assert not ((got[:, :, :L0] != ref_cache[:, :, :L0]) & ~near[:, :, :L0].any(axis=-1, keepdims=True)).any()
    cache[:, :, :L0] = dev(ref_cache[:, :, :L0])            # hand-off: attention below reads the oracle's codes
    rng = np.random.default_rng(5)
    for t in range(steps):
        pos = L0 + t
        q = synth.make_queries(synth.Workload(**{**w.__dict__, "seed": w.seed + 100 * t}), (1.0, 0.1, 0.5, 0.3)[t])
        out = lk.lookat_decode_step(dev(q), dev(keys[:, :, pos]), books_d, cache, v_d, pos)
        torch.cuda.synchronize()
        out = out.cpu().numpy()
        new = cache[:, :, pos].cpu().numpy()
        assert not ((new != ref_cache[:, :, pos]) & ~near[:, :, pos]).any(), f"appended codes differ at step {t}"
        assert float(cache[:, :, pos + 1:].max()) == 0, "a step wrote beyond its token"
        cache[:, :, pos] = dev(ref_cache[:, :, pos])
        for b, h in [(0, 0), (31, 11)] + [(int(rng.integers(w.B)), int(rng.integers(w.n_q_heads))) for _ in range(2)]:
            lut = oracle.build_lut(q[b:b + 1, h:h + 1], books[h:h + 1])
            ref = oracle.attend(lut, ref_cache[b:b + 1, h:h + 1, :pos + 1], v[b:b + 1, h:h + 1, :pos + 1], d_k=w.d_k)
            assert np.abs(out[b, h] - ref[0, 0]).max() <= OUT_TOL, (t, b, h)
