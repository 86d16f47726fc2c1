"""The debug build of the library (liblookat_debug.so, -DLOOKAT_DEBUG): its attend kernels check every code they read
from a cache.  A code >= K is clamped to K - 1 before it is used as an index -- so no address outside a table is ever
formed here -- and the context's status word records it; lookat_last_error reports it after the stream has drained.
The normal build does not check (a code >= K there is the caller's error) and is not given such codes."""
import numpy as np
import pytest
import torch

import oracle
from paper_2601_10155_b200 import synth
from paper_2601_10155_b200.binding import Lookat, load_library

pytestmark = pytest.mark.gpu


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def test_the_two_builds_say_which_they_are():
    assert load_library().lookat_is_debug_build() == 0
    assert load_library(debug=True).lookat_is_debug_build() == 1


@pytest.mark.parametrize("shape", [
    dict(B=2, n_q_heads=4, n_kv_heads=2, d_k=32, d_v=8, m=4, K=16, L=200),       # any-shape kernel (d_v 8), K < 256
    dict(B=2, n_q_heads=4, n_kv_heads=2, d_k=64, d_v=64, m=4, K=16, L=300),      # streaming kernel, K < 256
])
def test_debug_build_clamps_and_reports_codes_beyond_K(shape):
    w = synth.small_workload(**shape)
    keys, v, q = synth.make_keys(w), synth.make_values(w), synth.make_queries(w, 0.3)
    books, _ = oracle.fit_codebooks(keys, w.m, w.K, iters=2, seed=1)
    codes = oracle.encode_keys(keys, books)
    lk = Lookat(w.n_q_heads, w.n_kv_heads, w.d_k, w.d_v, w.m, w.K, debug=True)
    lut = lk.lookat_build_lut(dev(q), dev(books))
    # clean codes: same result as the oracle, nothing reported
    out = lk.lookat_attend(dev(codes), dev(v), lut=lut)
    torch.cuda.synchronize()
    ref = oracle.attend(oracle.build_lut(q, books), codes, v, d_k=w.d_k)
    assert np.abs(out.cpu().numpy() - ref).max() <= 2e-3
    assert lk.lookat_last_error() == ""
    # a few codes beyond K (the largest byte among them, in the last subspace too): clamped to K - 1 and reported
    bad = codes.copy()
    bad[0, 0, 5, 0], bad[1, 1, w.L - 1, w.m - 1], bad[0, 1, 77, 2] = 200, 255, w.K
    clamped = np.minimum(bad, w.K - 1)
    out = lk.lookat_attend(dev(bad), dev(v), lut=lut)
    torch.cuda.synchronize()
    ref = oracle.attend(oracle.build_lut(q, books), clamped, v, d_k=w.d_k)
    assert np.abs(out.cpu().numpy() - ref).max() <= 2e-3
    assert "code >= K" in lk.lookat_last_error()
    assert lk.lookat_last_error().startswith("debug check")       # the text stays until the next error; the word is cleared
    out = lk.lookat_attend(dev(codes), dev(v), lut=lut)
    torch.cuda.synchronize()
    assert np.abs(out.cpu().numpy() - oracle.attend(oracle.build_lut(q, books), codes, v, d_k=w.d_k)).max() <= 2e-3


def test_debug_build_checks_key_and_value_codes_of_the_quantised_values_path():
    w = synth.small_workload(B=1, n_q_heads=4, n_kv_heads=2, d_k=64, d_v=64, m=4, K=32, L=500)
    keys, v, q = synth.make_keys(w), synth.make_values(w), synth.make_queries(w, 0.3)
    books, _ = oracle.fit_codebooks(keys, w.m, w.K, iters=2, seed=1)
    codes = oracle.encode_keys(keys, books)
    v_books, _ = oracle.fit_codebooks(v, 4, 64, iters=2, seed=2)
    v_codes = oracle.encode_keys(v, v_books)
    lk = Lookat(w.n_q_heads, w.n_kv_heads, w.d_k, w.d_v, w.m, w.K, debug=True)
    out = lk.lookat_attend_pqv(dev(codes), dev(v_books), dev(v_codes), q=dev(q), codebooks=dev(books))
    torch.cuda.synchronize()
    ref = oracle.attend_pqv(oracle.build_lut(q, books), codes, v_books, v_codes, d_k=w.d_k)
    assert np.abs(out.cpu().numpy() - ref).max() <= 2e-3 and lk.lookat_last_error() == ""
    bad_k, bad_v = codes.copy(), v_codes.copy()
    bad_k[0, 1, 123, 3] = 90
    bad_v[0, 0, 499, 0] = 64
    out = lk.lookat_attend_pqv(dev(bad_k), dev(v_books), dev(bad_v), q=dev(q), codebooks=dev(books))
    torch.cuda.synchronize()
    ref = oracle.attend_pqv(oracle.build_lut(q, books), np.minimum(bad_k, w.K - 1), v_books, np.minimum(bad_v, 63), d_k=w.d_k)
    assert np.abs(out.cpu().numpy() - ref).max() <= 2e-3
    assert "code >= K" in lk.lookat_last_error()
