"""GPU parity: every C-ABI call of the CUDA library against the CPU oracle on
the same seeded inputs.  Stages are checked with a verified hand-off: attend
is fed the ORACLE's codes and codebooks, so one stage's permitted deviations
(near-tie codes) cannot leak into the next stage's comparison.

Tolerances (stated by the benchmark spec): codes bit-exact except near ties (relative
distance gap in (0, 1e-6)); raw scores |d| <= 1e-4 (1 + |s|); outputs <= 2e-3
max abs.  Tables: |d| <= 1e-5 (1 + |lut|).
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2601_10155_b200 import synth
from paper_2601_10155_b200.binding import Lookat, LookatError

pytestmark = pytest.mark.gpu

SCORE_TOL = 1e-4
OUT_TOL = 2e-3
LUT_TOL = 1e-5


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def ctx_for(w, **kw):
    return Lookat(w.n_q_heads, w.n_kv_heads, w.d_k, w.d_v, w.m, w.K, **kw)


def random_books(w, seed):
    rng = np.random.default_rng(seed)
    return rng.standard_normal((w.n_kv_heads, w.m, w.K, w.d_sub)).astype(np.float32)


def check_codes(gpu_codes, ref_codes, gap):
    """Bit-exact outside the oracle's near-tie flags; returns (#mismatch inside, #flags)."""
    diff = gpu_codes != ref_codes
    near = (gap > 0) & (gap < 1e-6)
    outside = diff & ~near
    assert outside.sum() == 0, f"{outside.sum()} code mismatches that are not near ties"
    return int((diff & near).sum()), int(near.sum())


def check_attend(w, lk, q, books, codes, v, seq_lens=None, n_splits=0, scale=None):
    lut64 = oracle.build_lut(q, books)
    ref_out, ref_s = oracle.attend(lut64, codes, v, seq_lens=seq_lens, scale=scale, d_k=w.d_k,
                                   want_scores=True)
    scores = torch.full((w.B, w.n_q_heads, codes.shape[2]), float("nan"), device="cuda")
    out = lk.lookat_attend(dev(codes), dev(v), q=dev(q), codebooks=dev(books),
                           seq_lens=None if seq_lens is None else dev(np.asarray(seq_lens, np.int32)),
                           n_splits=n_splits, scores_out=scores)
    torch.cuda.synchronize()
    out = out.cpu().numpy().astype(np.float64)
    s = scores.cpu().numpy().astype(np.float64)
    valid = ~np.isnan(ref_s)
    assert np.array_equal(np.isnan(s), ~valid), "scores written outside seq_len or missing inside"
    err_s = np.abs(s[valid] - ref_s[valid]) / (1 + np.abs(ref_s[valid]))
    assert err_s.max(initial=0) <= SCORE_TOL, f"score error {err_s.max()}"
    err_o = np.abs(out - ref_out).max()
    assert err_o <= OUT_TOL, f"output error {err_o}"
    return err_o


# ------------------------------------------------------------------ tables
@pytest.mark.parametrize("shape", [
    dict(B=2, n_q_heads=4, n_kv_heads=2, d_k=32, m=4, K=16),
    dict(B=3, n_q_heads=12, n_kv_heads=12, d_k=64, m=2, K=256),
    dict(B=2, n_q_heads=8, n_kv_heads=2, d_k=128, m=8, K=256),
    dict(B=1, n_q_heads=3, n_kv_heads=1, d_k=24, m=8, K=7),          # d_sub = 3
    dict(B=1, n_q_heads=2, n_kv_heads=2, d_k=16, m=16, K=255),       # d_sub = 1
])
def test_build_lut_matches_oracle(shape):
    w = synth.small_workload(**shape)
    q = synth.make_queries(w)
    books = random_books(w, 1)
    lk = ctx_for(w)
    lut = lk.lookat_build_lut(dev(q), dev(books)).cpu().numpy()
    ref = oracle.build_lut(q, books)
    assert np.all(np.abs(lut - ref) <= LUT_TOL * (1 + np.abs(ref)))
    # fp64 accumulation then one rounding: equal to the rounded oracle table
    assert np.array_equal(lut, ref.astype(np.float32))


# ------------------------------------------------------------------ encoding
@pytest.mark.parametrize("shape", [
    dict(B=2, n_kv_heads=2, n_q_heads=2, d_k=32, m=4, K=16, L=300),        # d_sub 8, tile kernel
    dict(B=1, n_kv_heads=3, n_q_heads=3, d_k=64, m=4, K=256, L=1500),      # d_sub 16
    dict(B=2, n_kv_heads=2, n_q_heads=2, d_k=64, m=2, K=256, L=700),       # d_sub 32
    dict(B=1, n_kv_heads=2, n_q_heads=2, d_k=64, m=16, K=200, L=900),      # d_sub 4
    dict(B=1, n_kv_heads=2, n_q_heads=2, d_k=24, m=8, K=31, L=5000),       # d_sub 3, generic kernel
    dict(B=1, n_kv_heads=1, n_q_heads=1, d_k=128, m=1, K=64, L=2100),      # d_sub 128, generic kernel
    dict(B=2, n_kv_heads=2, n_q_heads=2, d_k=16, m=16, K=256, L=800),      # d_sub 1
    dict(B=4, n_kv_heads=2, n_q_heads=2, d_k=64, m=4, K=256, L=3),         # few keys: warp kernel
])
def test_encode_matches_oracle(shape):
    w = synth.small_workload(**shape)
    keys = synth.make_keys(w)
    books, _ = oracle.fit_codebooks(keys[:, :, :min(w.L, 512)], w.m, w.K, iters=2, seed=3)
    ref, gap = oracle.encode_keys(keys, books, want_gap=True)
    lk = ctx_for(w)
    ties = torch.zeros(1, dtype=torch.int64, device="cuda")
    codes = lk.lookat_encode_keys(dev(keys), dev(books), near_ties=ties).cpu().numpy()
    inside, flagged = check_codes(codes, ref, gap)
    assert int(ties.item()) == flagged


def test_encode_duplicate_centroids_and_exact_ties_take_lowest_index():
    w = synth.small_workload(B=1, n_kv_heads=2, n_q_heads=2, d_k=32, m=4, K=64, L=2000)
    keys = synth.make_keys(w)
    books, _ = oracle.fit_codebooks(keys[:, :, :256], w.m, 32, iters=1, seed=1)
    books = np.concatenate([books, books], axis=2)             # every centroid twice
    ref, gap = oracle.encode_keys(keys, books, want_gap=True)
    assert ref.max() < 32 and np.all(gap == 0)
    lk = ctx_for(w)
    for n in (2000, 5):                                          # tile kernel and warp kernel
        codes = lk.lookat_encode_keys(dev(keys[:, :, :n]), dev(books)).cpu().numpy()
        assert np.array_equal(codes, ref[:, :, :n])


@pytest.mark.parametrize("d_sub", [8, 16, 32])
@pytest.mark.parametrize("K", [203, 256])
def test_encode_on_adversarial_scales_equals_the_fp64_argmin(d_sub, K):
    """The tensor-core search must hand every key it cannot decide to the exact rule: keys of mixed
    scale (zero, tiny, huge), centroids of very different norms, pairs of centroids one fp32 step
    apart, keys that sit exactly on a centroid, and a codebook outside fp16 range."""
    m = 4
    w = synth.small_workload(B=1, n_kv_heads=2, n_q_heads=2, d_k=m * d_sub, m=m, K=K, L=4133)
    rng = np.random.default_rng(77 + d_sub + K)
    keys = synth.make_keys(w).astype(np.float32)
    scale = rng.choice([0.0, 1e-4, 1e-2, 1.0, 1.0, 30.0], size=(1, 2, w.L, 1))
    keys = (keys * scale).astype(np.float16)
    books = rng.standard_normal((2, m, K, d_sub)).astype(np.float32)
    books *= rng.choice([1e-3, 0.1, 1.0, 1.0, 25.0], size=(2, m, K, 1)).astype(np.float32)
    books[:, :, 1::7] = np.nextafter(books[:, :, 0::7][:, :, :books[:, :, 1::7].shape[2]], np.float32(np.inf))
    sub = keys.reshape(1, 2, w.L, m, d_sub)
    for j in range(m):                                            # some centroids are keys themselves
        books[:, j, 5:K:11] = sub[0, :, 100:100 + len(range(5, K, 11)), j].astype(np.float32)
    lk = ctx_for(w)
    for trial, bk in enumerate((books, books * np.float32(3000.0))):   # second pass: |c| beyond fp16 range
        ref, gap = oracle.encode_keys(keys, bk, want_gap=True)
        ties = torch.zeros(1, dtype=torch.int64, device="cuda")
        codes = lk.lookat_encode_keys(dev(keys), dev(bk), near_ties=ties).cpu().numpy()
        check_codes(codes, ref, gap)


def test_encode_appends_at_odd_positions_without_touching_neighbours():
    w = synth.small_workload(B=2, n_kv_heads=2, n_q_heads=2, d_k=32, m=4, K=16, L=64)
    keys = synth.make_keys(w)
    books = random_books(w, 5)
    lk = ctx_for(w)
    cache = torch.full((w.B, w.n_kv_heads, 101, w.m), 255, dtype=torch.uint8, device="cuda")
    ref = np.full((w.B, w.n_kv_heads, 101, w.m), 255, dtype=np.uint8)
    for pos, n in ((0, 1), (1, 1), (2, 5), (7, 30), (37, 1), (100, 1)):
        lk.lookat_encode_keys(dev(keys[:, :, :n]), dev(books), codes=cache, pos=pos)
        oracle.encode_keys(keys[:, :, :n], books, codes=ref, L_max=101, pos=pos)
    assert np.array_equal(cache.cpu().numpy(), ref)
    with pytest.raises(LookatError):
        lk.lookat_encode_keys(dev(keys[:, :, :2]), dev(books), codes=cache, pos=100)


# ------------------------------------------------------------------ k-means
@pytest.mark.parametrize("shape,iters", [
    (dict(B=2, n_kv_heads=2, n_q_heads=2, d_k=32, m=4, K=32, L=900), 6),
    (dict(B=1, n_kv_heads=3, n_q_heads=3, d_k=64, m=4, K=256, L=128), 4),      # N < K: every key a centroid
    (dict(B=8, n_kv_heads=2, n_q_heads=2, d_k=64, m=2, K=256, L=512), 5),
    (dict(B=1, n_kv_heads=1, n_q_heads=1, d_k=24, m=8, K=9, L=700), 7),        # d_sub 3
    (dict(B=3, n_kv_heads=2, n_q_heads=2, d_k=16, m=2, K=1, L=101), 2),        # K = 1: the mean
])
def test_fit_matches_oracle(shape, iters):
    w = synth.small_workload(**shape)
    keys = synth.make_keys(w)
    lk = ctx_for(w)
    books, trace = lk.lookat_fit_codebooks(dev(keys), iters, seed=17, want_distortion=True)
    books, trace = books.cpu().numpy(), trace.cpu().numpy()
    ref_books, ref_trace = oracle.fit_codebooks(keys, w.m, w.K, iters, seed=17)
    # single step from the same start: assignments, hence exact means, must agree bit for bit
    one, _ = oracle.fit_codebooks(keys, w.m, w.K, 1, seed=17)
    one_gpu = lk.lookat_fit_codebooks(dev(keys), 1, seed=17).cpu().numpy()
    assert np.array_equal(one_gpu, one)
    if np.array_equal(books, ref_books):
        np.testing.assert_allclose(trace, ref_trace, rtol=1e-11, atol=1e-300)
    else:
        # only a near-tie decision may split the two runs; both are valid Lloyd runs
        np.testing.assert_allclose(trace[..., -1], ref_trace[..., -1], rtol=1e-4)
    assert np.all(trace[..., 1:] <= trace[..., :-1] * (1 + 1e-7))


def test_fit_with_given_start_and_fixed_point():
    rng = np.random.default_rng(12)
    K, d_sub, per = 6, 4, 40
    centres = (rng.permutation(K)[:, None] * 16.0 + rng.integers(-2, 3, (K, d_sub))).astype(np.float64)
    pts = centres[:, None, :] + rng.integers(-8, 9, (K, per, d_sub)) / 16.0
    perm = rng.permutation(K * per)
    x = pts.reshape(-1, d_sub)[perm]
    keys = x.astype(np.float16).reshape(1, 1, K * per, d_sub)
    true_means = np.stack([x[(perm // per) == c].mean(0) for c in range(K)]).astype(np.float32)
    lk = Lookat(1, 1, d_sub, 8, 1, K)
    init = dev(true_means.reshape(1, 1, K, d_sub))
    books = lk.lookat_fit_codebooks(dev(keys), 3, init=init).cpu().numpy()
    assert np.array_equal(books[0, 0], true_means)


# ------------------------------------------------------------------ attend
ATTEND_SHAPES = [
    # streaming kernel: d_v in {64,128}, m in {1,2,4,8,16}
    dict(B=2, n_q_heads=8, n_kv_heads=2, d_k=128, d_v=128, m=8, K=256, L=1000),      # g=4
    dict(B=2, n_q_heads=12, n_kv_heads=12, d_k=64, d_v=64, m=4, K=256, L=129),       # g=1
    dict(B=3, n_q_heads=4, n_kv_heads=2, d_k=64, d_v=64, m=2, K=256, L=1025),        # g=2
    dict(B=1, n_q_heads=3, n_kv_heads=1, d_k=64, d_v=128, m=16, K=255, L=333),       # g=3, K=255
    dict(B=1, n_q_heads=16, n_kv_heads=2, d_k=64, d_v=64, m=1, K=16, L=4097),        # g=8: two head groups
    dict(B=2, n_q_heads=6, n_kv_heads=1, d_k=32, d_v=128, m=4, K=2, L=48),           # g=6: 4 + 2
    # generic kernel: other d_v / m / odd row pitch
    dict(B=2, n_q_heads=4, n_kv_heads=2, d_k=32, d_v=8, m=4, K=16, L=200),
    dict(B=1, n_q_heads=2, n_kv_heads=2, d_k=64, d_v=64, m=64, K=11, L=127),         # m = d_k
    dict(B=2, n_q_heads=2, n_kv_heads=1, d_k=8, d_v=200, m=8, K=256, L=31),
    dict(B=1, n_q_heads=2, n_kv_heads=2, d_k=64, d_v=64, m=4, K=256, L=7),           # L*m not a multiple of 16
]


@pytest.mark.parametrize("shape", ATTEND_SHAPES)
@pytest.mark.parametrize("q_scale", [1.0, 0.1, 0.0])
def test_attend_matches_oracle(shape, q_scale):
    w = synth.small_workload(**shape)
    keys, v, q = synth.make_keys(w), synth.make_values(w), synth.make_queries(w, q_scale)
    books, _ = oracle.fit_codebooks(keys[:, :, :min(w.L, 400)], w.m, w.K, iters=2, seed=3)
    codes = oracle.encode_keys(keys, books)
    lk = ctx_for(w)
    check_attend(w, lk, q, books, codes, v)


@pytest.mark.parametrize("shape", [ATTEND_SHAPES[0], ATTEND_SHAPES[2], ATTEND_SHAPES[6]])
def test_attend_is_independent_of_the_split_count_and_handles_ragged_rows(shape):
    w = synth.small_workload(**shape)
    keys, v, q = synth.make_keys(w), synth.make_values(w), synth.make_queries(w, 0.3)
    books = random_books(w, 2)
    codes = oracle.encode_keys(keys, books)
    lk = ctx_for(w)
    seq_lens = [0, w.L, 1][:w.B] if w.B <= 3 else None
    outs = []
    for n_splits in (1, 2, 3, 7, 64, 0):
        check_attend(w, lk, q, books, codes, v, seq_lens=seq_lens, n_splits=n_splits)
        out = lk.lookat_attend(dev(codes), dev(v), q=dev(q), codebooks=dev(books), n_splits=n_splits)
        outs.append(out.cpu().numpy())
    for o in outs[1:]:
        np.testing.assert_allclose(o, outs[0], rtol=0, atol=2e-5)
    for L_row in (1, 15, 16, 17, w.L - 1):
        check_attend(w, lk, q, books, codes, v, seq_lens=[L_row] * w.B, n_splits=3)


# Rows above 8192 tokens take the long-row kernel (attend_stream_kernel: bulk-copy ring, one table set, ranges cut
# from the flat tile sequence); shapes chosen so that ranges lie inside a unit, cross one border, or span several units.
LONG_SHAPES = [
    dict(B=1, n_q_heads=4, n_kv_heads=1, d_k=64, d_v=64, m=4, K=64, L=8300),         # one unit over all CTAs: 3-4 tiles each
    dict(B=3, n_q_heads=6, n_kv_heads=2, d_k=128, d_v=128, m=8, K=256, L=8500),      # g = 3; six units, ragged rows below
    dict(B=2, n_q_heads=16, n_kv_heads=2, d_k=64, d_v=128, m=16, K=255, L=8209),     # g = 8: two head groups; m = 16; odd L
    dict(B=2, n_q_heads=2, n_kv_heads=2, d_k=32, d_v=64, m=1, K=16, L=12000),        # m = 1, g = 1
    dict(B=40, n_q_heads=8, n_kv_heads=4, d_k=32, d_v=64, m=2, K=32, L=8224),        # 160 units: every range spans two borders
]


@pytest.mark.parametrize("shape", LONG_SHAPES)
def test_attend_on_long_rows_matches_oracle(shape):
    w = synth.small_workload(**shape)
    keys, v, q = synth.make_keys(w), synth.make_values(w), synth.make_queries(w, 0.3)
    books = random_books(w, 6)
    codes = oracle.encode_keys(keys, books)
    lk = ctx_for(w)
    check_attend(w, lk, q, books, codes, v)
    # ragged rows: empty, full, one token into the last tile, and (larger batches) lengths all over the place
    rng = np.random.default_rng(w.L)
    seq_lens = ([0, w.L, w.L - 15] * w.B)[:w.B] if w.B <= 3 else list(rng.integers(0, w.L + 1, w.B))
    check_attend(w, lk, q, books, codes, v, seq_lens=seq_lens)
    if w.B <= 3:
        for n_splits in (1, 5, 64):
            check_attend(w, lk, q, books, codes, v, seq_lens=seq_lens, n_splits=n_splits)


@pytest.mark.parametrize("shape", [LONG_SHAPES[1], LONG_SHAPES[3], LONG_SHAPES[4]])
def test_long_rows_on_the_cp_async_ring(shape, monkeypatch):
    """The long-row kernel's other copy path (16-byte cp.async pieces into padded rows; taken where the driver offers no
    tensor maps or the caches have 2^31 rows or more), forced by the library's environment switch: attention, ragged
    rows and a decode step against the oracle."""
    monkeypatch.setenv("LOOKAT_NO_TENSOR_MAPS", "1")
    w = synth.small_workload(**shape)
    keys, v, q = synth.make_keys(w), synth.make_values(w), synth.make_queries(w, 0.3)
    books = random_books(w, 6)
    codes = oracle.encode_keys(keys, books)
    lk = ctx_for(w)
    check_attend(w, lk, q, books, codes, v)
    rng = np.random.default_rng(w.L + 1)
    seq_lens = ([0, w.L, w.L - 15] * w.B)[:w.B] if w.B <= 3 else list(rng.integers(0, w.L + 1, w.B))
    check_attend(w, lk, q, books, codes, v, seq_lens=seq_lens)
    pos = w.L - 1
    cache = codes.copy()
    cache[:, :, pos] = 201 % w.K
    codes_dev = dev(cache)
    out = lk.lookat_decode_step(dev(q), dev(np.ascontiguousarray(keys[:, :, pos])), dev(books), codes_dev, dev(v), pos)
    torch.cuda.synchronize()
    assert np.array_equal(codes_dev.cpu().numpy(), codes)
    ref = oracle.attend(oracle.build_lut(q, books), codes, v, d_k=w.d_k)
    assert np.abs(out.cpu().numpy() - ref).max() <= OUT_TOL


@pytest.mark.parametrize("shape", LONG_SHAPES[:4])
@pytest.mark.parametrize("pos_from_end", [1, 16, 50])
def test_decode_step_on_long_rows(shape, pos_from_end):
    """The append inside the long-row kernel, with the cache filled to the end of its rows or a little short of it.  Where
    one unit is cut among all CTAs the new token's tile is among the first tiles its CTA copies (encoded before the ring
    is primed); elsewhere it lies far down a range (encoded while the first tiles are in flight)."""
    w = synth.small_workload(**shape)
    keys, v, q = synth.make_keys(w), synth.make_values(w), synth.make_queries(w, 0.4)
    books = random_books(w, 8)
    pos = w.L - pos_from_end
    ref_codes, gap = oracle.encode_keys(keys[:, :, :pos + 1], books, want_gap=True)
    assert not ((gap[:, :, pos] > 0) & (gap[:, :, pos] < 1e-6)).any()
    cache = np.zeros((w.B, w.n_kv_heads, w.L, w.m), np.uint8)
    cache[:, :, :pos] = ref_codes[:, :, :pos]
    cache[:, :, pos:] = 201 % w.K                      # stale codes where the new key goes and beyond
    lk = ctx_for(w)
    codes_dev = dev(cache)
    out = lk.lookat_decode_step(dev(q), dev(np.ascontiguousarray(keys[:, :, pos])), dev(books), codes_dev, dev(v), pos)
    torch.cuda.synchronize()
    got = codes_dev.cpu().numpy()
    assert np.array_equal(got[:, :, :pos + 1], ref_codes)          # row pos written, bit-exact
    assert np.all(got[:, :, pos + 1:] == 201 % w.K)                 # nothing beyond it touched
    ref = oracle.attend(oracle.build_lut(q, books), ref_codes, v[:, :, :pos + 1], d_k=w.d_k)
    assert np.abs(out.cpu().numpy() - ref).max() <= OUT_TOL


def test_attend_with_prebuilt_tables_and_explicit_scale():
    w = synth.small_workload(B=2, n_q_heads=8, n_kv_heads=2, d_k=64, d_v=64, m=4, K=64, L=500)
    keys, v, q = synth.make_keys(w), synth.make_values(w), synth.make_queries(w, 0.5)
    books = random_books(w, 9)
    codes = oracle.encode_keys(keys, books)
    lk = ctx_for(w, scale=0.05)
    lut = lk.lookat_build_lut(dev(q), dev(books))
    out = lk.lookat_attend(dev(codes), dev(v), lut=lut).cpu().numpy()
    ref = oracle.attend(oracle.build_lut(q, books), codes, v, scale=0.05)
    assert np.abs(out - ref).max() <= OUT_TOL
    check_attend(w, lk, q, books, codes, v, scale=0.05)


def test_exactness_special_case_on_the_gpu():
    """N <= K: the fitted codebooks hold every key, ADC attention equals exact attention."""
    w = synth.WORKLOADS["gpt2_l128_m4"]
    keys, v, q = synth.make_keys(w), synth.make_values(w), synth.make_queries(w)
    lk = ctx_for(w)
    books = lk.lookat_fit_codebooks(dev(keys), w.fit_iters, seed=w.seed)
    codes = lk.lookat_encode_keys(dev(keys), books)
    out = lk.lookat_attend(codes, dev(v), q=dev(q), codebooks=books).cpu().numpy()
    exact = oracle.exact_attention(q, keys, v)
    assert np.abs(out - exact).max() <= OUT_TOL
    assert np.array_equal(codes.cpu().numpy(), oracle.encode_keys(keys, books.cpu().numpy()))


def test_gpt2_shapes_end_to_end_with_handoff():
    """The 64x configuration (m=2) at L=1024, batch 8: GPU codebooks vs oracle, codes vs oracle,
    then attend on the oracle's codes."""
    w = synth.WORKLOADS["gpt2_b8_l1024_m2"]
    keys, v, q = synth.make_keys(w), synth.make_values(w), synth.make_queries(w)
    lk = ctx_for(w)
    iters = 3
    books_gpu = lk.lookat_fit_codebooks(dev(keys), iters, seed=w.seed).cpu().numpy()
    books, _ = oracle.fit_codebooks(keys, w.m, w.K, iters, seed=w.seed)
    ref_codes, gap = oracle.encode_keys(keys, books, want_gap=True)
    codes = lk.lookat_encode_keys(dev(keys), dev(books)).cpu().numpy()
    check_codes(codes, ref_codes, gap)
    if not ((gap > 0) & (gap < 1e-6)).any():
        assert np.array_equal(books_gpu, books)
    for q_scale in (1.0, 0.1):
        check_attend(w, lk, synth.make_queries(w, q_scale), books, ref_codes, v)


@pytest.mark.parametrize("shape", [
    dict(B=3, n_q_heads=8, n_kv_heads=2, d_k=64, d_v=64, m=4, K=64, L=300),        # streaming kernel, fused append
    dict(B=2, n_q_heads=16, n_kv_heads=2, d_k=128, d_v=128, m=8, K=256, L=2000),   # g = 8: two head groups per KV head
    dict(B=2, n_q_heads=4, n_kv_heads=2, d_k=32, d_v=8, m=4, K=16, L=100),         # generic kernel: separate encode
    dict(B=2, n_q_heads=4, n_kv_heads=2, d_k=64, d_v=64, m=2, K=200, L=200),       # g = 2, sub-vectors of 32 dims, K < 256
    dict(B=1, n_q_heads=12, n_kv_heads=12, d_k=64, d_v=64, m=8, K=256, L=900),     # g = 1, m = 8: distances do not fit beside the partials
    dict(B=40, n_q_heads=4, n_kv_heads=2, d_k=64, d_v=128, m=4, K=256, L=1500),    # several units per round (separate append pass)
])
@pytest.mark.parametrize("pos_from_end", [1, 2, 17])
def test_decode_step_on_device_appends_then_attends(shape, pos_from_end):
    w = synth.small_workload(**shape)
    keys, v, q = synth.make_keys(w), synth.make_values(w), synth.make_queries(w, 0.4)
    books, _ = oracle.fit_codebooks(keys[:, :, :256], w.m, w.K, iters=2, seed=5)
    pos = w.L - pos_from_end
    ref_codes, gap = oracle.encode_keys(keys[:, :, :pos + 1], books, want_gap=True)
    assert not ((gap[:, :, pos] > 0) & (gap[:, :, pos] < 1e-6)).any()
    cache = np.zeros((w.B, w.n_kv_heads, w.L, w.m), np.uint8)
    cache[:, :, :pos] = ref_codes[:, :, :pos]
    cache[:, :, pos:] = 201 % w.K                      # stale codes where the new key goes and beyond
    lk = ctx_for(w)
    codes_dev = dev(cache)
    out = lk.lookat_decode_step(dev(q), dev(np.ascontiguousarray(keys[:, :, pos])), dev(books), codes_dev, dev(v), pos)
    torch.cuda.synchronize()
    got = codes_dev.cpu().numpy()
    assert np.array_equal(got[:, :, :pos + 1], ref_codes)          # row pos written, bit-exact
    assert np.all(got[:, :, pos + 1:] == 201 % w.K)                 # nothing beyond it touched
    ref = oracle.attend(oracle.build_lut(q, books), ref_codes, v[:, :, :pos + 1], d_k=w.d_k)
    assert np.abs(out.cpu().numpy() - ref).max() <= OUT_TOL
    # and once more: the cache now holds the new code already
    out2 = lk.lookat_decode_step(dev(q), dev(np.ascontiguousarray(keys[:, :, pos])), dev(books), codes_dev, dev(v), pos)
    assert np.abs(out2.cpu().numpy() - ref).max() <= OUT_TOL


def test_decode_steps_grow_the_cache_like_a_generation_loop():
    """GPT-2 shapes, several decode steps in a row: each step appends one key and value row and attends
    over everything so far; after every step codes and output equal the oracle's."""
    w = synth.small_workload(B=4, n_q_heads=12, n_kv_heads=12, d_k=64, d_v=64, m=4, K=256, L=70, rank=16)
    keys, v = synth.make_keys(w), synth.make_values(w)
    books, _ = oracle.fit_codebooks(keys[:, :, :60], w.m, w.K, iters=3, seed=2)
    L_max = 80                                            # 80 * 4 code bytes: rows stay 16-byte aligned
    lk = ctx_for(w)
    start = 61
    ref_cache = np.zeros((w.B, w.n_kv_heads, L_max, w.m), np.uint8)
    oracle.encode_keys(keys[:, :, :start], books, codes=ref_cache, L_max=L_max, pos=0)
    codes_dev = dev(ref_cache)
    v_cache = np.zeros((w.B, w.n_kv_heads, L_max, w.d_v), np.float16)
    v_cache[:, :, :start] = v[:, :, :start]
    v_dev = dev(v_cache)
    for step, pos in enumerate(range(start, w.L)):
        wq = synth.small_workload(seed=100 + step, B=w.B, n_q_heads=12, n_kv_heads=12, d_k=64, rank=16)
        q = synth.make_queries(wq, 0.5)
        v_dev[:, :, pos] = dev(v[:, :, pos])              # the caller stores the value row
        out = lk.lookat_decode_step(dev(q), dev(np.ascontiguousarray(keys[:, :, pos])), dev(books), codes_dev,
                                    v_dev, pos)
        oracle.encode_keys(keys[:, :, pos:pos + 1], books, codes=ref_cache, L_max=L_max, pos=pos)
        ref = oracle.attend(oracle.build_lut(q, books), ref_cache[:, :, :pos + 1], v[:, :, :pos + 1], d_k=w.d_k)
        assert np.array_equal(codes_dev.cpu().numpy(), ref_cache)
        assert np.abs(out.cpu().numpy() - ref).max() <= OUT_TOL


@pytest.mark.parametrize("pinned", [True, False])
def test_decode_step_from_host_buffers(pinned):
    """Pinned buffers are addressed by the kernel in place; pageable ones go through staging copies."""
    pin = (lambda t: t.pin_memory()) if pinned else (lambda t: t)
    w = synth.small_workload(B=3, n_q_heads=8, n_kv_heads=2, d_k=64, d_v=64, m=4, K=64, L=300)
    keys, v, q = synth.make_keys(w), synth.make_values(w), synth.make_queries(w, 0.4)
    books = random_books(w, 4)
    lk = ctx_for(w)
    L_max = 320
    codes_ref = np.zeros((w.B, w.n_kv_heads, L_max, w.m), np.uint8)
    oracle.encode_keys(keys, books, codes=codes_ref, L_max=L_max, pos=0)
    v_cache = np.zeros((w.B, w.n_kv_heads, L_max, w.d_v), np.float16)
    v_cache[:, :, :w.L - 1] = v[:, :, :w.L - 1]
    codes_dev = dev(codes_ref)
    codes_dev[:, :, w.L - 1] = 77                      # the step must write this row
    v_dev = dev(v_cache)
    out_host = pin(torch.empty((w.B, w.n_q_heads, w.d_v), dtype=torch.float32))
    lk.lookat_decode_step_host(pin(torch.from_numpy(q)),
                               pin(torch.from_numpy(np.ascontiguousarray(keys[:, :, w.L - 1]))),
                               pin(torch.from_numpy(np.ascontiguousarray(v[:, :, w.L - 1]))),
                               dev(books), codes_dev, v_dev, w.L - 1, out_host)
    assert np.array_equal(codes_dev.cpu().numpy()[:, :, :w.L], codes_ref[:, :, :w.L])
    assert np.array_equal(v_dev.cpu().numpy()[:, :, w.L - 1], v[:, :, w.L - 1])
    ref = oracle.attend(oracle.build_lut(q, books), codes_ref[:, :, :w.L], v, d_k=w.d_k)
    assert np.abs(out_host.numpy() - ref).max() <= OUT_TOL


def test_invalid_arguments_are_rejected_without_launching():
    w = synth.small_workload()
    lk = ctx_for(w)
    before = lk.lookat_kernel_launches()
    codes = torch.zeros((w.B, w.n_kv_heads, 32, w.m), dtype=torch.uint8, device="cuda")
    v = torch.zeros((w.B, w.n_kv_heads, 32, w.d_v), dtype=torch.float16, device="cuda")
    with pytest.raises(LookatError):
        lk.lookat_attend(codes, v)                                       # neither lut nor (q, codebooks)
    with pytest.raises(LookatError):
        lk.lookat_attend(codes, v, n_splits=-1, lut=torch.zeros((w.B, w.n_q_heads, w.m, w.K), device="cuda"))
    with pytest.raises((TypeError, ValueError)):
        lk.lookat_attend(codes.cpu(), v)                                  # host tensor: no CPU path
    assert lk.lookat_kernel_launches() == before
    for bad in (dict(m=3), dict(K=0), dict(K=257), dict(n_kv_heads=3)):
        kw = dict(n_q_heads=4, n_kv_heads=2, d_k=32, d_v=32, m=4, K=16)
        kw.update(bad)
        with pytest.raises(LookatError):
            Lookat(**kw)


# ------------------------------------------------------------------ causal multi-query (prefill)
@pytest.mark.parametrize("shape,L_q,q_pos0", [
    (dict(B=2, n_q_heads=4, n_kv_heads=2, d_k=64, d_v=64, m=4, K=256, L=150), 150, 0),      # whole prompt
    (dict(B=1, n_q_heads=8, n_kv_heads=2, d_k=128, d_v=128, m=8, K=256, L=200), 37, 163),   # a late slice
    (dict(B=1, n_q_heads=2, n_kv_heads=2, d_k=128, d_v=128, m=16, K=256, L=130), 130, 0),   # tables of 8 queries
    (dict(B=2, n_q_heads=2, n_kv_heads=1, d_k=32, d_v=32, m=2, K=16, L=70), 1, 69),         # one query = a decode step
    (dict(B=1, n_q_heads=3, n_kv_heads=3, d_k=24, d_v=16, m=8, K=7, L=65), 65, 0),          # d_sub 3, small K
    (dict(B=1, n_q_heads=2, n_kv_heads=1, d_k=128, d_v=64, m=16, K=200, L=450), 300, 150),  # 3 query tiles, ragged, K < 256
    (dict(B=1, n_q_heads=2, n_kv_heads=2, d_k=64, d_v=128, m=8, K=256, L=257), 257, 0),     # d_k 64; one row in the last tile
    (dict(B=1, n_q_heads=2, n_kv_heads=2, d_k=64, d_v=64, m=16, K=256, L=90), 90, 0),       # d_sub 4: two centroids per 8-dim group
    (dict(B=2, n_q_heads=4, n_kv_heads=2, d_k=64, d_v=128, m=16, K=100, L=333), 200, 133),  # d_sub 4, grouped heads, ragged, K < 256
    (dict(B=1, n_q_heads=2, n_kv_heads=1, d_k=128, d_v=64, m=32, K=16, L=80), 80, 0),        # 32 subspaces: tables only
    (dict(B=1, n_q_heads=4, n_kv_heads=1, d_k=64, d_v=128, m=2, K=16, L=300), 259, 41),     # m 2: a CTA's last token has an odd index
])
@pytest.mark.parametrize("q_scale", [1.0, 0.1])
@pytest.mark.parametrize("form", ["tables", "contraction"])
def test_attend_prefill_matches_oracle(shape, L_q, q_pos0, q_scale, form):
    w = synth.small_workload(**shape)
    keys, v = synth.make_keys(w), synth.make_values(w)
    q = synth.make_prefill_queries(w, L_q, q_scale)
    books, _ = oracle.fit_codebooks(keys[:, :, :min(w.L, 300)], w.m, w.K, iters=2, seed=3)
    codes = oracle.encode_keys(keys, books)
    lk = ctx_for(w)
    lk.lookat_set_prefill_form(form)
    scores = torch.full((w.B, w.n_q_heads, L_q, w.L), float("nan"), device="cuda")
    covered = w.d_k in (64, 128) and w.d_v in (64, 128) and (w.d_sub % 8 == 0 or w.d_sub == 4) and w.m <= 16
    if form != "tables" and not covered:
        with pytest.raises(LookatError):
            lk.lookat_attend_prefill(dev(q), dev(books), dev(codes), dev(v), q_pos0=q_pos0, scores_out=scores)
        return
    ref, ref_s = oracle.attend_prefill(q, books, codes, v, q_pos0=q_pos0, want_scores=True)
    out = lk.lookat_attend_prefill(dev(q), dev(books), dev(codes), dev(v), q_pos0=q_pos0, scores_out=scores)
    torch.cuda.synchronize()
    s = scores.cpu().numpy().astype(np.float64)
    visible = ~np.isnan(ref_s)
    assert np.array_equal(np.isnan(s), ~visible), "scores written for hidden pairs or missing for visible ones"
    assert np.all(np.abs(s[visible] - ref_s[visible]) <= SCORE_TOL * (1 + np.abs(ref_s[visible])))
    assert np.abs(out.cpu().numpy() - ref).max() <= OUT_TOL
    # without the validation output the kernel is another instantiation: same result
    out2 = lk.lookat_attend_prefill(dev(q), dev(books), dev(codes), dev(v), q_pos0=q_pos0)
    assert float((out2 - out).abs().max()) <= 1e-6
    # the last query of a whole prompt is a decode step over the same cache
    if q_pos0 + L_q == w.L:
        dec = lk.lookat_attend(dev(codes), dev(v), q=dev(np.ascontiguousarray(q[:, :, -1])), codebooks=dev(books))
        # the contraction form rounds each weight to fp16 once (relative 2^-12 = 2.4e-4, values up to ~4) where decode
        # keeps two planes; both sit inside OUT_TOL of the oracle, and well inside it of each other
        assert float((dec - out[:, :, -1]).abs().max()) <= (2e-5 if form == "tables" else 6e-4)


@pytest.mark.parametrize("seed", range(8))
def test_attend_prefill_contraction_on_random_shapes(seed):
    """Shapes drawn at random inside what the tensor-core forms cover: grouped heads, codebooks small enough for two
    CTAs per SM, query slices that start and end anywhere; both contraction kernels against the oracle, twice
    (the second call reuses the context's scratch)."""
    rng = np.random.default_rng(9000 + seed)
    d_k, d_v = int(rng.choice([64, 128])), int(rng.choice([64, 128]))
    d_sub = int(rng.choice([4, 8, 16, 32]))
    d_sub = max(d_sub, d_k // 16)                         # at most 16 subspaces
    H_kv = int(rng.choice([1, 2, 3]))
    g = int(rng.choice([1, 2, 4]))
    K = int(rng.choice([16, 64, 200, 256]))
    L = int(rng.integers(70, 700))
    L_q = int(rng.integers(1, L + 1))
    q_pos0 = int(rng.integers(0, L - L_q + 1))
    B = int(rng.choice([1, 2, 3]))
    L += (-L * (d_k // d_sub)) % 4 and 1                  # the contraction form copies codes four bytes at a time
    w = synth.small_workload(B=B, n_q_heads=H_kv * g, n_kv_heads=H_kv, d_k=d_k, d_v=d_v, m=d_k // d_sub, K=K, L=L)
    keys, v = synth.make_keys(w), synth.make_values(w)
    q = synth.make_prefill_queries(w, L_q, float(rng.choice([1.0, 0.2])))
    books, _ = oracle.fit_codebooks(keys[:, :, :min(w.L, 300)], w.m, w.K, iters=1, seed=3)
    codes = oracle.encode_keys(keys, books)
    ref = oracle.attend_prefill(q, books, codes, v, q_pos0=q_pos0)
    lk = ctx_for(w)
    for form in ("contraction",):
        lk.lookat_set_prefill_form(form)
        for _ in range(2):
            out = lk.lookat_attend_prefill(dev(q), dev(books), dev(codes), dev(v), q_pos0=q_pos0)
            assert np.abs(out.cpu().numpy() - ref).max() <= OUT_TOL, (form, shape_of(w), L_q, q_pos0)


def shape_of(w):
    return dict(B=w.B, H_q=w.n_q_heads, H_kv=w.n_kv_heads, d_k=w.d_k, d_v=w.d_v, m=w.m, K=w.K, L=w.L)


def test_a_wait_that_runs_out_is_reported_once_and_the_context_stays_usable():
    """The bounded-wait status, without hanging anything: a self-test kernel's only wait can never be satisfied and
    gives up after 4096 polls; the next prefill call reports the time-out and clears it; the one after runs."""
    w = synth.small_workload(B=1, n_q_heads=2, n_kv_heads=2, d_k=64, d_v=64, m=8, K=64, L=200)
    keys, v = synth.make_keys(w), synth.make_values(w)
    q = synth.make_prefill_queries(w, 100, 1.0)
    books, _ = oracle.fit_codebooks(keys[:, :, :200], w.m, w.K, iters=1, seed=3)
    codes = oracle.encode_keys(keys, books)
    ref = oracle.attend_prefill(q, books, codes, v, q_pos0=100)
    lk = ctx_for(w)
    args = (dev(q), dev(books), dev(codes), dev(v))
    out = lk.lookat_attend_prefill(*args, q_pos0=100)
    assert np.abs(out.cpu().numpy() - ref).max() <= OUT_TOL
    lk.lookat_selftest_timeout()
    torch.cuda.synchronize()
    with pytest.raises(LookatError) as err:
        lk.lookat_attend_prefill(*args, q_pos0=100)
    assert err.value.status == 5                                   # LOOKAT_ERR_TIMEOUT
    out = lk.lookat_attend_prefill(*args, q_pos0=100)              # reported once; the context is usable
    assert np.abs(out.cpu().numpy() - ref).max() <= OUT_TOL


def test_read_bandwidth_probe_reports_a_plausible_figure():
    w = synth.small_workload(B=1, n_q_heads=1, n_kv_heads=1, d_k=64, d_v=64, m=8, K=16, L=64)
    lk = ctx_for(w)
    buf = torch.ones(1 << 28, dtype=torch.uint8, device="cuda")            # 256 MiB: larger than L2
    gbs = lk.lookat_probe_read_bandwidth(buf, reps=3)
    assert 1000.0 < gbs < 12000.0, gbs
    with pytest.raises(LookatError):
        lk.lookat_probe_read_bandwidth(buf[1:17], reps=1)                 # misaligned


# ------------------------------------------------------------------ product-quantised values (beyond the paper)
@pytest.mark.parametrize("shape,m_v", [
    (dict(B=2, n_q_heads=8, n_kv_heads=2, d_k=128, d_v=128, m=8, K=256, L=9000), 8),     # grouped heads, two chunks, ragged
    (dict(B=3, n_q_heads=3, n_kv_heads=3, d_k=64, d_v=64, m=4, K=64, L=777), 16),        # d_vsub 4
    (dict(B=1, n_q_heads=6, n_kv_heads=1, d_k=32, d_v=32, m=2, K=16, L=300), 2),         # 6 heads: groups of 4 + 2
    (dict(B=2, n_q_heads=2, n_kv_heads=2, d_k=64, d_v=128, m=16, K=200, L=100), 4),      # K < 256
    (dict(B=1, n_q_heads=2, n_kv_heads=1, d_k=64, d_v=24, m=8, K=256, L=5000), 8),       # pairs of heads; d_vsub 3
    (dict(B=1, n_q_heads=1, n_kv_heads=1, d_k=32, d_v=32, m=2, K=256, L=20000), 4),      # one unit over five CTAs
    (dict(B=1, n_q_heads=4, n_kv_heads=1, d_k=64, d_v=64, m=16, K=256, L=4500), 16),     # rows not doubled, small blocks
])
@pytest.mark.parametrize("q_scale", [1.0, 0.1])
def test_attend_with_quantised_values_matches_oracle(shape, m_v, q_scale):
    w = synth.small_workload(**shape)
    keys, v, q = synth.make_keys(w), synth.make_values(w), synth.make_queries(w, q_scale)
    books, _ = oracle.fit_codebooks(keys[:, :, :min(w.L, 300)], w.m, w.K, iters=2, seed=3)
    codes = oracle.encode_keys(keys, books)
    K_v = 256 if w.L >= 300 else 64
    v_books, _ = oracle.fit_codebooks(v[:, :, :min(w.L, 300)], m_v, K_v, iters=2, seed=4)     # values are encoded like keys
    v_codes = oracle.encode_keys(v, v_books)
    seq_lens = np.array([w.L - 5 * b for b in range(w.B)], np.int32)
    lut = oracle.build_lut(q, books)
    ref = oracle.attend_pqv(lut, codes, v_books, v_codes, seq_lens=seq_lens, d_k=w.d_k)
    lk = ctx_for(w)
    out = lk.lookat_attend_pqv(dev(codes), dev(v_books), dev(v_codes), q=dev(q), codebooks=dev(books),
                               seq_lens=dev(seq_lens))
    assert np.abs(out.cpu().numpy() - ref).max() <= OUT_TOL
    out2 = lk.lookat_attend_pqv(dev(codes), dev(v_books), dev(v_codes), lut=dev(lut.astype(np.float32)),
                                seq_lens=dev(seq_lens))
    assert np.abs(out2.cpu().numpy() - ref).max() <= OUT_TOL
    # the value codes and codebooks of the GPU's own encoder give the same codes as the oracle's (values are keys to it)
    lv = Lookat(w.n_kv_heads, w.n_kv_heads, w.d_v, w.d_v, m_v, K_v)
    ref_gap = oracle.encode_keys(v, v_books, want_gap=True)[1]
    got = lv.lookat_encode_keys(dev(v), dev(v_books)).cpu().numpy()
    check_codes(got, v_codes, ref_gap)


@pytest.mark.parametrize("direction", [1, -1])
def test_attend_with_quantised_values_rescales_its_histograms(direction):
    """Scores that rise (fall) steadily along the sequence: with rising scores every block of tokens moves the
    running maximum far up, so the fixed-point weight histograms are rescaled at every block; with falling scores the
    first block fixes maximum and scale and everything later adds weights that are tiny against it.  The tables are
    handed in directly: with m = 2, table 0 = delta * c and table 1 = 256 * delta * c, token t with codes
    (t mod 256, t div 256) scores delta * t."""
    L, d_v, m_v = 20000, 64, 8
    w = synth.small_workload(B=1, n_q_heads=4, n_kv_heads=1, d_k=32, d_v=d_v, m=2, K=256, L=L)
    v = synth.make_values(w)
    v_books, _ = oracle.fit_codebooks(v[:, :, :400], m_v, 256, iters=2, seed=5)
    v_codes = oracle.encode_keys(v, v_books)
    t = np.arange(L)
    codes = np.stack([t % 256, t // 256], axis=-1).astype(np.uint8)[None, None]
    c = np.arange(256, dtype=np.float64)
    lut = np.zeros((1, 4, 2, 256))
    for h in range(4):
        delta = direction * (h + 1) * 0.004               # over 20,000 tokens: 80 to 320, times 1/sqrt(32) in the exponent
        lut[0, h, 0], lut[0, h, 1] = delta * c, 256 * delta * c
    lut = lut.astype(np.float32).astype(np.float64)        # both sides start from the same fp32 tables
    ref = oracle.attend_pqv(lut, codes, v_books, v_codes, seq_lens=np.array([L], np.int32), d_k=w.d_k)
    out = ctx_for(w).lookat_attend_pqv(dev(codes), dev(v_books), dev(v_codes), lut=dev(lut.astype(np.float32)))
    assert np.abs(out.cpu().numpy() - ref).max() <= OUT_TOL
