"""CPU-side checks: the C-ABI library builds, loads and exports what the header
declares; byte accounting against the counts the paper prints; the input
generator is deterministic; the binding has no CPU path."""
import ctypes
import os
import re

import numpy as np
import pytest

from paper_2601_10155_b200 import binding, build, synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib_path():
    return build.build()


def _declared_functions():
    names = set()
    for header in sorted(os.listdir(os.path.join(ROOT, "include"))):
        text = open(os.path.join(ROOT, "include", header)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        names |= set(re.findall(r"\b(lookat_[a-z0-9_]+)\s*\(", text))
    return sorted(names)


def test_library_exports_every_declared_symbol(lib_path):
    lib = ctypes.CDLL(lib_path)
    names = _declared_functions()
    assert {"lookat_fit_codebooks", "lookat_encode_keys", "lookat_build_lut", "lookat_attend"} <= set(names)
    for name in names:
        assert hasattr(lib, name), f"{name} is declared in include/ but not exported"
    assert sorted(binding.EXPORTS) == names


def test_create_rejects_bad_configurations_before_touching_a_device(lib_path):
    lib = binding.load_library()
    h = ctypes.c_void_p()
    for kw in (dict(m=3), dict(K=0), dict(K=257), dict(n_kv_heads=3), dict(d_k=0), dict(scale=-1.0)):
        base = dict(n_q_heads=4, n_kv_heads=2, d_k=32, d_v=32, m=4, K=16, scale=0.0)
        base.update(kw)
        cfg = binding.lookat_config(*[base[k] for k in ("n_q_heads", "n_kv_heads", "d_k", "d_v", "m", "K", "scale")])
        assert lib.lookat_create(ctypes.byref(cfg), 0, None, ctypes.byref(h)) == 1
    assert lib.lookat_create(None, 0, None, ctypes.byref(h)) == 1
    assert lib.lookat_last_error(None) == b"context is NULL"


def test_binding_has_no_cpu_path():
    import torch
    if torch.cuda.is_available():
        pytest.skip("checks the behaviour on a box without a GPU")
    with pytest.raises(RuntimeError):
        binding.Lookat(4, 2, 32, 32, 4, 16)


def test_counts_the_paper_prints():
    fns = {"key_bytes_per_token": binding.key_bytes_per_token,
           "key_compression_ratio": binding.key_compression_ratio,
           "lut_entries": binding.lut_entries,
           "kv_cache_bytes_fp16": binding.kv_cache_bytes_fp16}
    rows = 0
    for line in open(os.path.join(ROOT, "tests", "golden", "paper_counts.txt")):
        if line.startswith("#") or not line.strip():
            continue
        name, args, value = line.split()[:3]
        kwargs = {k: int(x) for k, x in (a.split("=") for a in args.split(","))}
        assert fns[name](**kwargs) == float(value), line
        rows += 1
    assert rows == 10
    # the long-context configuration: 8 code bytes against a 256-byte fp16 key, 264 bytes per token read
    assert binding.key_compression_ratio(128, 8) == 32
    assert binding.attend_bytes_per_token_kvhead(8, 128) == 264


def test_generator_is_deterministic_and_shaped():
    w = synth.small_workload(B=2, n_q_heads=4, n_kv_heads=2, d_k=16, d_v=8, L=33, m=4, K=8)
    k1, k2 = synth.make_keys(w), synth.make_keys(w)
    assert k1.dtype == np.float16 and k1.shape == (2, 2, 33, 16) and np.array_equal(k1, k2)
    assert synth.make_values(w).shape == (2, 2, 33, 8)
    q = synth.make_queries(w)
    assert q.shape == (2, 4, 16)
    assert np.array_equal(synth.make_queries(w, 0.0), np.zeros_like(q))
    # keys of one head are iid rows: a longer draw extends nothing it shares a stream with
    assert not np.array_equal(synth.make_keys(w, stream=1), synth.make_calibration_keys(w, 66).reshape(2, 2, 33, 16))
    for name, wl in synth.WORKLOADS.items():
        assert wl.d_k % wl.m == 0 and wl.n_q_heads % wl.n_kv_heads == 0, name
