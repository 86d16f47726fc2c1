"""lookat_attend_static: the attend entry point for callers that cannot let the library allocate
(their own pool owns the device memory, or they cannot take the synchronisation of cudaMalloc in a
decode loop).  Its scratch is a fixed array inside the library, so its results must equal those of
lookat_attend and of the oracle, call after call, whatever ran before on the device, and the amount
of free device memory must not move across a call.

Collected last on purpose (file name): a failure here cannot hide the other tests' results.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2601_10155_b200 import synth
from paper_2601_10155_b200.binding import Lookat, LookatError

pytestmark = pytest.mark.gpu

OUT_TOL = 2e-3          # the output tolerance of the parity tests
SCORE_TOL = 1e-4        # |ds| <= SCORE_TOL * (1 + |s|)


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def _problem(seed, B, L):
    """Inputs made on the CPU only: generator keys, the oracle's codebooks and the oracle's codes."""
    w = synth.small_workload(seed=seed, B=B, n_q_heads=8, n_kv_heads=2, d_k=128, d_v=128, L=L, m=8, K=256,
                             rank=32, scales="student_t3")
    keys, v, q = synth.make_keys(w), synth.make_values(w), synth.make_queries(w, 0.3)
    books, _ = oracle.fit_codebooks(keys[:, :, :600], w.m, w.K, iters=1, seed=seed)
    codes = oracle.encode_keys(keys, books)
    return w, q, books, codes, v


def _warm_up_the_module():
    """One call on a context of its own: the CUDA runtime loads the library's module (kernel images and the fixed
    array) on first use, which is not an allocation of the entry point under test."""
    w, q, books, codes, v = _problem(9, 1, 64)
    lk = Lookat(w.n_q_heads, w.n_kv_heads, w.d_k, w.d_v, w.m, w.K)
    lk.lookat_attend_static(dev(codes), dev(v), q=dev(q), codebooks=dev(books))
    torch.cuda.synchronize()
    lk.close()


def test_static_scratch_variant_matches_oracle_and_lookat_attend_on_two_calls_in_a_row():
    _warm_up_the_module()
    # two different problems back to back: the second call finds the first call's partials and
    # counters in the shared array and must not be affected by them
    for seed, B, L in ((1, 3, 1500), (2, 2, 4104)):
        w, q, books, codes, v = _problem(seed, B, L)
        ref, ref_s = oracle.attend(oracle.build_lut(q, books), codes, v, d_k=w.d_k, want_scores=True)
        q_d, books_d, codes_d, v_d = dev(q), dev(books), dev(codes), dev(v)
        # a fresh context: the static entry point runs first, so nothing it uses can be context scratch
        lk = Lookat(w.n_q_heads, w.n_kv_heads, w.d_k, w.d_v, w.m, w.K)
        out = torch.full((w.B, w.n_q_heads, w.d_v), float("nan"), device="cuda")
        scores = torch.full((w.B, w.n_q_heads, w.L), float("nan"), device="cuda")
        torch.cuda.synchronize()
        for call in range(2):
            free_before, _ = torch.cuda.mem_get_info()
            lk.lookat_attend_static(codes_d, v_d, q=q_d, codebooks=books_d, out=out, scores_out=scores if call else None)
            torch.cuda.synchronize()
            free_after, _ = torch.cuda.mem_get_info()
            assert free_after == free_before, "the call changed the amount of free device memory"
            assert np.abs(out.cpu().numpy() - ref).max() <= OUT_TOL
        s = scores.cpu().numpy().astype(np.float64)
        assert np.all(np.abs(s - ref_s) <= SCORE_TOL * (1 + np.abs(ref_s)))
        # the allocating entry point gives the same result
        same = lk.lookat_attend(codes_d, v_d, q=q_d, codebooks=books_d)
        assert float((out - same).abs().max()) <= OUT_TOL
        # ready tables, ragged rows and a forced chunk count go through the same scratch
        lut = lk.lookat_build_lut(q_d, books_d)
        sl = np.array([L, 17, 0][:B], dtype=np.int32)
        ref2 = oracle.attend(oracle.build_lut(q, books), codes, v, seq_lens=sl, d_k=w.d_k)
        ref2[sl == 0] = 0.0                                 # a row without tokens gives zeros
        out2 = lk.lookat_attend_static(codes_d, v_d, lut=lut, seq_lens=dev(sl), n_splits=5)
        torch.cuda.synchronize()
        assert np.abs(out2.cpu().numpy() - ref2).max() <= OUT_TOL
        same2 = lk.lookat_attend(codes_d, v_d, lut=lut, seq_lens=dev(sl), n_splits=5)
        assert float((out2 - same2).abs().max()) <= OUT_TOL


def test_static_scratch_variant_rejects_what_does_not_fit():
    w, q, books, codes, v = _problem(3, 2, 4096)
    lk = Lookat(w.n_q_heads, w.n_kv_heads, w.d_k, w.d_v, w.m, w.K)
    before = lk.lookat_kernel_launches()
    with pytest.raises(LookatError) as err:          # 4 units x 256 chunks: partials beyond the 2 MiB array
        lk.lookat_attend_static(dev(codes), dev(v), q=dev(q), codebooks=dev(books), n_splits=256)
    assert err.value.status == 2 and "fixed" in str(err.value)
    assert lk.lookat_kernel_launches() == before
