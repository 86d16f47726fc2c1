"""lookat_attend_static: the attend entry point for callers that cannot let the library allocate
(their own pool owns the device memory, or they cannot take the synchronisation of cudaMalloc in a
decode loop).  Its scratch is a fixed array inside the library, so its results must equal those of
lookat_attend, call after call, whatever ran before on the device.

Collected last on purpose (file name): a failure here cannot hide the other tests' results.
"""
import numpy as np
import pytest
import torch

from paper_2601_10155_b200 import synth
from paper_2601_10155_b200.binding import Lookat, LookatError

pytestmark = pytest.mark.gpu

OUT_TOL = 2e-3          # the output tolerance of the parity tests


def _problem(seed, B, L):
    w = synth.small_workload(seed=seed, B=B, n_q_heads=8, n_kv_heads=2, d_k=128, d_v=128, L=L, m=8, K=256,
                             rank=32, scales="student_t3")
    rng = np.random.default_rng(seed)
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
    books = dev(rng.standard_normal((w.n_kv_heads, w.m, w.K, w.d_sub)).astype(np.float32))
    codes = dev(rng.integers(0, w.K, (w.B, w.n_kv_heads, w.L, w.m), dtype=np.uint8))
    return w, dev(synth.make_queries(w, 0.3)), books, codes, dev(synth.make_values(w))


def test_static_scratch_variant_matches_lookat_attend_on_two_calls_in_a_row():
    # two different problems back to back: the second call finds the first call's partials and
    # counters in the shared array and must not be affected by them
    for seed, B, L in ((1, 3, 1500), (2, 2, 4104)):
        w, q, books, codes, v = _problem(seed, B, L)
        lk = Lookat(w.n_q_heads, w.n_kv_heads, w.d_k, w.d_v, w.m, w.K)
        ref = lk.lookat_attend(codes, v, q=q, codebooks=books)
        out = torch.full_like(ref, float("nan"))
        for _ in range(2):
            lk.lookat_attend_static(codes, v, q=q, codebooks=books, out=out)
            torch.cuda.synchronize()
            assert float((out - ref).abs().max()) <= OUT_TOL
        # ready tables, ragged rows and a forced chunk count go through the same scratch
        lut = lk.lookat_build_lut(q, books)
        sl = torch.tensor([L, 17, 0][:B], dtype=torch.int32, device="cuda")
        ref2 = lk.lookat_attend(codes, v, lut=lut, seq_lens=sl, n_splits=5)
        out2 = lk.lookat_attend_static(codes, v, lut=lut, seq_lens=sl, n_splits=5)
        torch.cuda.synchronize()
        assert float((out2 - ref2).abs().max()) <= OUT_TOL


def test_static_scratch_variant_rejects_what_does_not_fit():
    w, q, books, codes, v = _problem(3, 2, 4096)
    lk = Lookat(w.n_q_heads, w.n_kv_heads, w.d_k, w.d_v, w.m, w.K)
    before = lk.lookat_kernel_launches()
    with pytest.raises(LookatError) as err:          # 4 units x 256 chunks: partials beyond the 2 MiB array
        lk.lookat_attend_static(codes, v, q=q, codebooks=books, n_splits=256)
    assert err.value.status == 2 and "fixed" in str(err.value)
    assert lk.lookat_kernel_launches() == before
