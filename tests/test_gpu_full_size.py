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


@pytest.mark.parametrize("form", ["contraction", "contraction_mma_sync", "tables"])
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
