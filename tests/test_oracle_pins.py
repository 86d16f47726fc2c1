"""Pins for the CPU oracle: every oracle routine is checked against something
the paper or the mathematics fixes, computed here WITHOUT the oracle (numpy /
scipy routines, closed forms, brute force in Python loops).

Citations are to the paper: Section 3.1 (attention), 3.4 (prototype learning,
encoding), 3.5 (lookup tables, lookup-and-sum, Algorithm 1).
"""
import itertools

import numpy as np
import pytest
import scipy.special
from scipy.cluster.vq import kmeans2

import oracle
from paper_2601_10155_b200 import synth


def _rand_problem(seed, B=2, H_q=4, H_kv=2, d_k=16, d_v=8, L=37, m=4, K=16, q_scale=1.0):
    w = synth.small_workload(seed=seed, B=B, n_q_heads=H_q, n_kv_heads=H_kv, d_k=d_k, d_v=d_v,
                             L=L, m=m, K=K, rank=4)
    keys = synth.make_keys(w)
    v = synth.make_values(w)
    q = synth.make_queries(w, q_scale)
    rng = np.random.default_rng(seed + 99)
    books = rng.standard_normal((H_kv, m, K, d_k // m)).astype(np.float32)
    return w, keys, v, q, books


def _softmax_attention_numpy(scores, v, scale, g):
    """Independent statement of the Algorithm 1 continuation: softmax then weighted sum."""
    B, H_q, L = scores.shape
    out = np.empty((B, H_q, v.shape[-1]))
    for b in range(B):
        for hq in range(H_q):
            a = scipy.special.softmax(scores[b, hq] * scale)
            out[b, hq] = a @ v[b, hq // g].astype(np.float64)
    return out


# ---------------------------------------------------------------- fp16 widening
def test_half_to_double_matches_numpy_for_every_bit_pattern():
    bits = np.arange(65536, dtype=np.uint16).view(np.float16)
    got = oracle.half_to_double(bits)
    ref = bits.astype(np.float64)
    finite = ~np.isnan(ref)
    assert np.array_equal(got[finite], ref[finite])
    assert np.isnan(got[~finite]).all()


# ---------------------------------------------------------------- encoding (Section 3.4)
def test_encode_matches_brute_force_argmin():
    rng = np.random.default_rng(0)
    B, H, n, d_k, m, K = 2, 2, 13, 8, 4, 7
    keys = rng.standard_normal((B, H, n, d_k)).astype(np.float16)
    books = rng.standard_normal((H, m, K, d_k // m)).astype(np.float32)
    codes = oracle.encode_keys(keys, books)
    d_sub = d_k // m
    for b, h, t, j in itertools.product(range(B), range(H), range(n), range(m)):
        x = [float(keys[b, h, t, j * d_sub + i]) for i in range(d_sub)]
        best, best_c = None, None
        for c in range(K):
            d = sum((x[i] - float(books[h, j, c, i])) ** 2 for i in range(d_sub))
            if best is None or d < best:
                best, best_c = d, c
        assert codes[b, h, t, j] == best_c


def test_encode_lowest_index_wins_exact_ties_and_gap_is_zero():
    # centroids 1 and 3 are identical and nearest; centroid 0 and 2 are far.
    books = np.zeros((1, 1, 4, 2), dtype=np.float32)
    books[0, 0, 0] = [10, 10]
    books[0, 0, 1] = [1, 1]
    books[0, 0, 2] = [-10, 3]
    books[0, 0, 3] = [1, 1]
    keys = np.array([[[[1.25, 0.75]]]], dtype=np.float16)
    codes, gap = oracle.encode_keys(keys, books, want_gap=True)
    assert codes[0, 0, 0, 0] == 1
    assert gap[0, 0, 0, 0] == 0.0
    # symmetric tie between two different centroids: x is equidistant from 0 and 2.
    books2 = np.array([[[[0.0], [5.0], [2.0]]]], dtype=np.float32)
    keys2 = np.array([[[[1.0]]]], dtype=np.float16)
    assert oracle.encode_keys(keys2, books2)[0, 0, 0, 0] == 0


def test_encode_of_a_centroid_returns_its_index_and_writes_at_pos():
    rng = np.random.default_rng(3)
    H, m, K, d_sub = 2, 2, 16, 4
    # well separated, fp16-representable centroids
    books = (rng.integers(-8, 8, (H, m, K, d_sub)) + 32 * np.arange(K)[None, None, :, None]).astype(np.float32)
    pick = rng.integers(0, K, (1, H, 5, m))
    keys = np.empty((1, H, 5, m * d_sub), dtype=np.float16)
    for h, t, j in itertools.product(range(H), range(5), range(m)):
        keys[0, h, t, j * d_sub:(j + 1) * d_sub] = books[h, j, pick[0, h, t, j]]
    codes = np.full((1, H, 12, m), 255, dtype=np.uint8)
    oracle.encode_keys(keys, books, codes=codes, L_max=12, pos=3)
    assert np.array_equal(codes[:, :, 3:8], pick.astype(np.uint8))
    assert (codes[:, :, :3] == 255).all() and (codes[:, :, 8:] == 255).all()


def test_near_tie_gap_definition():
    books = np.array([[[[0.0], [2.0 + 1e-6]]]], dtype=np.float32)
    keys = np.array([[[[1.0]]]], dtype=np.float16)
    codes, gap = oracle.encode_keys(keys, books, want_gap=True)
    d1 = 1.0
    d2 = (float(books[0, 0, 1, 0]) - 1.0) ** 2
    assert codes[0, 0, 0, 0] == 0
    assert gap[0, 0, 0, 0] == pytest.approx((d2 - d1) / d2, rel=1e-12)


# ---------------------------------------------------------------- lookup tables (Section 3.5)
def test_lut_matches_numpy_einsum():
    w, keys, v, q, books = _rand_problem(1)
    lut = oracle.build_lut(q, books)
    g = w.g
    qs = q.astype(np.float64).reshape(w.B, w.n_q_heads, w.m, w.d_sub)
    ref = np.einsum("bhji,hjci->bhjc", qs, np.repeat(books.astype(np.float64), g, axis=0))
    np.testing.assert_allclose(lut, ref, rtol=1e-13, atol=1e-13)


def test_lookup_sum_equals_dot_with_reconstructed_key():
    """sum_j LUT_j[code_j] == q . k_hat to 1e-9 relative (denominator sum |q_i k_hat_i|)."""
    for seed, (m, K, d_k) in enumerate([(4, 16, 16), (2, 256, 64), (8, 33, 64), (64, 5, 64)]):
        w, keys, v, q, books = _rand_problem(10 + seed, d_k=d_k, m=m, K=K, L=50)
        codes = oracle.encode_keys(keys, books)
        lut = oracle.build_lut(q, books)
        _, scores = oracle.attend(lut, codes, v, d_k=d_k, want_scores=True)
        # reconstruction written here with numpy indexing, not the oracle's routine
        d_sub = d_k // m
        k_hat = np.empty((w.B, w.n_kv_heads, w.L, d_k))
        for h in range(w.n_kv_heads):
            for j in range(m):
                k_hat[:, h, :, j * d_sub:(j + 1) * d_sub] = books[h, j][codes[:, h, :, j]]
        np.testing.assert_array_equal(k_hat, oracle.reconstruct_keys(codes, books))
        q64 = q.astype(np.float64)
        for hq in range(w.n_q_heads):
            kh = k_hat[:, hq // w.g]
            ref = np.einsum("bd,bld->bl", q64[:, hq], kh)
            den = np.einsum("bd,bld->bl", np.abs(q64[:, hq]), np.abs(kh))
            assert np.all(np.abs(scores[:, hq] - ref) <= 1e-9 * den + 1e-300)


# ---------------------------------------------------------------- Algorithm 1 as a whole
def test_attend_matches_numpy_softmax_weighted_sum():
    w, keys, v, q, books = _rand_problem(2, L=61, q_scale=0.3)
    codes = oracle.encode_keys(keys, books)
    lut = oracle.build_lut(q, books)
    out, scores, alpha = oracle.attend(lut, codes, v, d_k=w.d_k, want_scores=True, want_alpha=True)
    ref = _softmax_attention_numpy(scores, v, 1.0 / np.sqrt(w.d_k), w.g)
    np.testing.assert_allclose(out, ref, rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(alpha.sum(-1), 1.0, rtol=1e-13)


def test_lookat_reduces_to_exact_attention_when_codebooks_list_every_value():
    """m = d_k (d_sub = 1) and each codebook holds every distinct channel value:
    k_hat = k, so Algorithm 1 equals the attention of Section 3.1."""
    rng = np.random.default_rng(5)
    B, H_q, H_kv, d_k, d_v, L, K = 2, 4, 2, 8, 8, 40, 11
    levels = (rng.permutation(64)[:K] - 32) / 8.0           # K distinct fp16-exact levels
    keys = rng.choice(levels, size=(B, H_kv, L, d_k)).astype(np.float16)
    q = rng.standard_normal((B, H_q, d_k)).astype(np.float16)
    v = rng.standard_normal((B, H_kv, L, d_v)).astype(np.float16)
    books = np.broadcast_to(levels.astype(np.float32)[None, None, :, None], (H_kv, d_k, K, 1)).copy()
    codes, gap = oracle.encode_keys(keys, books, want_gap=True)
    assert np.array_equal(books[0, 0, :, 0][codes[:, 0, :, 0]], keys[:, 0, :, 0].astype(np.float32))
    out = oracle.attend(oracle.build_lut(q, books), codes, v, d_k=d_k)
    exact, s_exact = oracle.exact_attention(q, keys, v, want_scores=True)
    np.testing.assert_allclose(out, exact, rtol=1e-12, atol=1e-14)
    # and the exact routine itself against numpy
    s_ref = np.einsum("bhd,bhld->bhl", q.astype(np.float64),
                      np.repeat(keys.astype(np.float64), H_q // H_kv, axis=1))
    np.testing.assert_allclose(s_exact, s_ref, rtol=1e-13, atol=1e-13)
    np.testing.assert_allclose(exact, _softmax_attention_numpy(s_ref, v, d_k ** -0.5, H_q // H_kv),
                               rtol=1e-12, atol=1e-14)


def test_fewer_keys_than_centroids_is_the_exact_case_too():
    """N <= K: the strided init makes every key a centroid, distortion is 0 at once."""
    w = synth.small_workload(B=1, n_q_heads=3, n_kv_heads=3, d_k=16, d_v=8, L=20, m=2, K=32)
    keys, v, q = synth.make_keys(w), synth.make_values(w), synth.make_queries(w)
    books, trace = oracle.fit_codebooks(keys, w.m, w.K, iters=3, seed=11)
    assert np.all(trace == 0.0)
    codes = oracle.encode_keys(keys, books)
    out = oracle.attend(oracle.build_lut(q, books), codes, v, d_k=w.d_k)
    np.testing.assert_allclose(out, oracle.exact_attention(q, keys, v), rtol=1e-12, atol=1e-14)
    # duplicates of a centroid never win: only the first N indices (in init order) are used
    assert len(np.unique(codes[0, 0, :, 0])) == w.L or len(np.unique(keys[0, 0, :, :8], axis=0)) < w.L


def test_softmax_closed_forms():
    w, keys, v, q, books = _rand_problem(4, L=33)
    codes = oracle.encode_keys(keys, books)
    v64 = v.astype(np.float64)
    # q = 0 -> all tables 0 -> uniform weights -> mean of V
    out0 = oracle.attend(oracle.build_lut(np.zeros_like(q), books), codes, v, d_k=w.d_k)
    for hq in range(w.n_q_heads):
        np.testing.assert_allclose(out0[:, hq], v64[:, hq // w.g].mean(1), rtol=1e-13, atol=1e-15)
    # all codes equal -> mean of V as well
    same = np.zeros_like(codes) + 3
    lut = oracle.build_lut(q, books)
    out_same = oracle.attend(lut, same, v, d_k=w.d_k)
    np.testing.assert_allclose(out_same, out0, rtol=1e-12, atol=1e-14)
    # one token -> that token's value
    out1 = oracle.attend(lut, codes, v, seq_lens=np.ones(w.B, np.int32), d_k=w.d_k)
    for hq in range(w.n_q_heads):
        np.testing.assert_array_equal(out1[:, hq], v64[:, hq // w.g, 0])
    # seq_len 0 -> zeros (convention); ragged lengths use only the prefix
    sl = np.array([0, 17], np.int32)
    out_r = oracle.attend(lut, codes, v, seq_lens=sl, d_k=w.d_k)
    assert np.all(out_r[0] == 0)
    out_prefix = oracle.attend(lut[1:], codes[1:, :, :17], v[1:, :, :17], d_k=w.d_k)
    np.testing.assert_allclose(out_r[1:], out_prefix, rtol=1e-13)


def test_softmax_invariances():
    w, keys, v, q, books = _rand_problem(6, L=45, q_scale=0.5)
    codes = oracle.encode_keys(keys, books)
    lut = oracle.build_lut(q, books)
    out = oracle.attend(lut, codes, v, d_k=w.d_k)
    # a constant added to one table shifts every score alike
    lut2 = lut.copy()
    lut2[:, :, 1, :] += 3.75
    np.testing.assert_allclose(oracle.attend(lut2, codes, v, d_k=w.d_k), out, rtol=1e-11, atol=1e-13)
    # permuting tokens (codes and values together) changes nothing
    perm = np.random.default_rng(0).permutation(w.L)
    np.testing.assert_allclose(oracle.attend(lut, codes[:, :, perm], v[:, :, perm], d_k=w.d_k), out,
                               rtol=1e-11, atol=1e-13)
    # explicit scale: doubling the tables equals doubling the scale
    a = oracle.attend(2 * lut, codes, v, scale=0.25)
    b = oracle.attend(lut, codes, v, scale=0.5)
    np.testing.assert_allclose(a, b, rtol=1e-12)


def test_gqa_heads_of_a_group_share_the_kv_head():
    w, keys, v, q, books = _rand_problem(8, H_q=8, H_kv=2, L=29)
    q[:, 1] = q[:, 0]
    q[:, 2] = q[:, 0]                       # heads 0..3 belong to KV head 0
    codes = oracle.encode_keys(keys, books)
    out = oracle.attend(oracle.build_lut(q, books), codes, v, d_k=w.d_k)
    np.testing.assert_array_equal(out[:, 1], out[:, 0])
    np.testing.assert_array_equal(out[:, 2], out[:, 0])
    # same result as multi-head attention against replicated KV heads
    g = w.g
    out_mha = oracle.attend(oracle.build_lut(q, np.repeat(books, g, 0)), np.repeat(codes, g, 1),
                            np.repeat(v, g, 1), d_k=w.d_k)
    np.testing.assert_array_equal(out, out_mha)


# ---------------------------------------------------------------- prototype learning (Section 3.4)
def test_kmeans_distortion_never_increases():
    w = synth.small_workload(B=2, n_q_heads=2, n_kv_heads=2, d_k=32, L=700, m=4, K=32)
    keys = synth.make_keys(w)
    books, trace = oracle.fit_codebooks(keys, w.m, w.K, iters=12, seed=5)
    assert np.all(trace[..., 1:] <= trace[..., :-1] * (1 + 1e-7))
    assert np.all(trace[..., -1] < trace[..., 0])
    # the trace is the objective of Section 3.4 evaluated at the returned codebooks
    codes = oracle.encode_keys(keys, books)
    k64 = keys.astype(np.float64)
    for h in range(2):
        for j in range(w.m):
            x = k64[:, h, :, j * 8:(j + 1) * 8]
            c = books[h, j].astype(np.float64)[codes[:, h, :, j]]
            assert np.sum((x - c) ** 2) == pytest.approx(trace[h, j, -1], rel=1e-12)


def test_kmeans_with_one_centroid_is_the_mean():
    w = synth.small_workload(B=3, n_q_heads=2, n_kv_heads=2, d_k=8, L=101, m=2, K=1)
    keys = synth.make_keys(w)
    books, trace = oracle.fit_codebooks(keys, 2, 1, iters=2, seed=1)
    k64 = keys.astype(np.float64)                     # sums of 303 fp16 values are exact in fp64
    for h in range(2):
        mean = k64[:, h].reshape(-1, 8).sum(0) / 303.0
        np.testing.assert_array_equal(books[h, :, 0, :].reshape(-1), mean.astype(np.float32))
    assert np.all(trace[..., 2] <= trace[..., 1])
    assert trace[0, 0, 1] == trace[0, 0, 2]


def test_kmeans_planted_mixture_is_a_fixed_point_and_matches_scipy_lloyd_step():
    rng = np.random.default_rng(12)
    K, d_sub, per = 6, 4, 40
    centres = (rng.permutation(K)[:, None] * 16.0 + rng.integers(-2, 3, (K, d_sub))).astype(np.float64)
    pts = centres[:, None, :] + rng.integers(-8, 9, (K, per, d_sub)) / 16.0
    perm = rng.permutation(K * per)
    x = pts.reshape(-1, d_sub)[perm]
    keys = x.astype(np.float16).reshape(1, 1, K * per, d_sub)
    assert np.array_equal(keys.astype(np.float64).reshape(-1, d_sub), x)     # fp16-exact data
    true_means = np.stack([x[(perm // per) == c].mean(0) for c in range(K)])
    init = true_means.astype(np.float32).reshape(1, 1, K, d_sub)
    books, trace = oracle.fit_codebooks(keys, 1, K, iters=3, init=init)
    np.testing.assert_array_equal(books, init)
    assert trace[0, 0, 0] == trace[0, 0, 3]
    # one Lloyd step from a perturbed start: scipy's kmeans2 (iter=1, given centroids) is the
    # textbook assignment + mean update
    start = (centres + 1.5).astype(np.float32)
    books1, _ = oracle.fit_codebooks(keys, 1, K, iters=1, init=start.reshape(1, 1, K, d_sub))
    ref, _ = kmeans2(x, start.astype(np.float64), iter=1, minit="matrix")
    np.testing.assert_allclose(books1[0, 0], ref, rtol=1e-6, atol=1e-6)


def test_kmeans_init_rule_and_empty_clusters():
    # N = 5 keys, K = 8: rows repeat; centroids 5..7 duplicate 0..2 (in init order) and stay unused
    rng = np.random.default_rng(2)
    keys = rng.standard_normal((1, 1, 5, 4)).astype(np.float16)
    seed = 1234
    books, trace = oracle.fit_codebooks(keys, 2, 8, iters=2, seed=seed)
    for j in range(2):
        off = (seed + 0x9E3779B97F4A7C15 * (j + 1)) % (1 << 64) % 5
        for c in range(8):
            r = (off + c) % 5
            np.testing.assert_array_equal(books[0, j, c], keys[0, 0, r, 2 * j:2 * j + 2].astype(np.float32))
    assert np.all(trace == 0)
    codes = oracle.encode_keys(keys, books)
    assert codes.max() < 5


# ---------------------------------------------------------------- causal multi-query (prefill)
def test_prefill_is_algorithm_1_per_query_and_exact_attention_in_the_exact_case():
    rng = np.random.default_rng(21)
    B, H_q, H_kv, d_k, d_v, L, K = 2, 4, 2, 8, 8, 23, 9
    levels = (rng.permutation(64)[:K] - 32) / 8.0
    keys = rng.choice(levels, size=(B, H_kv, L, d_k)).astype(np.float16)
    v = rng.standard_normal((B, H_kv, L, d_v)).astype(np.float16)
    qs = (0.5 * rng.standard_normal((B, H_q, 7, d_k))).astype(np.float16)
    books = np.broadcast_to(levels.astype(np.float32)[None, None, :, None], (H_kv, d_k, K, 1)).copy()
    codes = oracle.encode_keys(keys, books)
    q_pos0 = L - 7
    out, scores = oracle.attend_prefill(qs, books, codes, v, q_pos0=q_pos0, want_scores=True)
    g = H_q // H_kv
    for i in range(7):
        n = q_pos0 + i + 1
        # the decode routine on the prefix (itself pinned above) ...
        ref = oracle.attend(oracle.build_lut(qs[:, :, i], books), codes[:, :, :n], v[:, :, :n], d_k=d_k)
        np.testing.assert_allclose(out[:, :, i], ref, rtol=1e-12, atol=1e-14)
        # ... and plain causal softmax attention written with numpy (codebooks reproduce the keys exactly)
        s_ref = np.einsum("bhd,bhld->bhl", qs[:, :, i].astype(np.float64),
                          np.repeat(keys[:, :, :n].astype(np.float64), g, axis=1))
        np.testing.assert_allclose(scores[:, :, i, :n], s_ref, rtol=1e-12, atol=1e-13)
        assert np.isnan(scores[:, :, i, n:]).all()
        np.testing.assert_allclose(out[:, :, i], _softmax_attention_numpy(s_ref, v[:, :, :n], d_k ** -0.5, g),
                                   rtol=1e-12, atol=1e-14)


def test_value_pq_attention_is_attention_over_the_reconstructed_values():
    """The weight-histogram form equals sum_t alpha_t v^_t written out with numpy, and when every value sub-vector is
    itself a centroid (value codebooks list the values) it is Algorithm 1 on the fp16 values."""
    rng = np.random.default_rng(5)
    B, H_q, H_kv, L, d_k, m, K, m_v, d_vsub = 2, 4, 2, 40, 16, 4, 8, 2, 4
    books = rng.standard_normal((H_kv, m, K, d_k // m)).astype(np.float32)
    codes = rng.integers(0, K, (B, H_kv, L, m), dtype=np.uint8)
    q = rng.standard_normal((B, H_q, d_k)).astype(np.float16)
    lut = oracle.build_lut(q, books)
    v_books = rng.standard_normal((H_kv, m_v, 16, d_vsub)).astype(np.float32)
    v_codes = rng.integers(0, 16, (B, H_kv, L, m_v), dtype=np.uint8)
    seq_lens = np.array([L, 23], np.int32)
    out = oracle.attend_pqv(lut, codes, v_books, v_codes, seq_lens=seq_lens, d_k=d_k)
    # written out: softmax of the lookup sums, times the reconstructed values
    g = H_q // H_kv
    for b in range(B):
        n = int(seq_lens[b])
        for hq in range(H_q):
            h = hq // g
            s = np.array([sum(lut[b, hq, j, codes[b, h, t, j]] for j in range(m)) for t in range(n)]) / np.sqrt(d_k)
            a = np.exp(s - s.max())
            a /= a.sum()
            v_hat = np.concatenate([v_books[h, j][v_codes[b, h, :n, j]] for j in range(m_v)], axis=1).astype(np.float64)
            assert np.allclose(out[b, hq], a @ v_hat, rtol=1e-12, atol=1e-12)
    # exact case: 16 distinct fp16 value rows per (head, subspace), every token takes one of them
    v_books16 = v_books.astype(np.float16).astype(np.float32)
    v = np.concatenate([v_books16[:, j][np.arange(H_kv)[None, :, None], v_codes[:, :, :, j]] for j in range(m_v)],
                       axis=3).astype(np.float16)
    ref = oracle.attend(lut, codes, v, seq_lens=seq_lens, d_k=d_k)
    assert np.allclose(oracle.attend_pqv(lut, codes, v_books16, v_codes, seq_lens=seq_lens, d_k=d_k), ref,
                       rtol=1e-12, atol=1e-12)
