"""Benchmark of the LOOKAT decode-attention hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl lookat|reference] [--workload NAME]

One step = one decode step of the whole batch: encode the newest key of every
(batch row, KV head) into the code cache, build the lookup tables for the
step's queries, and attend (ADC scores, softmax, value sum, chunk merge) over
all cached tokens.  Codebooks are fitted and the cache is encoded once before
the timed region (offline calibration and prefill); their device times are
reported under "setup".  Metric: tokens*heads scored per second
(B * H_q * L / step time), whole job.

With N > 1 (torchrun, one rank per GPU) every rank runs its own replica of
the workload; there is no exchange between ranks on this path.

--impl reference times the CPU oracle (tests' reference implementation) on
the host cores for the same step on a bounded sample of the workload.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2601_10155_b200 import synth  # noqa: E402

METRIC = "adc_decode_attention_tokens_heads_per_s"
UNIT = "tokens*heads/s"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) per (token, KV head) pair of one
# attend_stream_kernel launch, from an ncu capture of the batch-4 case of gqa_32k_m8
# (278,003,200 + 4,173,056 bytes over 1,048,576 pairs; traffic grows in proportion to the pairs).
ATTEND_DRAM_BYTES_PER_PAIR = {"gqa_32k_m8": 282176256 / 1048576}
ATTEND_TRAFFIC_SOURCE = ("ncu capture of attend_stream_kernel<8,128,2,true> (bulk-copy ring) on gqa_32k_m8 at batch 4 "
                         "(profiles/attend_stream_kernel_gqa_32k_m8_batch4_ncu.md), scaled by the pair count")
SMALL_WORKLOADS = ["gpt2_l128_m4", "gpt2_b8_l256_m2", "gpt2_b8_l512_m2", "gpt2_b8_l1024_m2", "gpt2_b32_l1024_m4"]
MIN_TIMED_SECONDS = 0.25


def measured_peak(key: str, fallback: float):
    """A figure of MEASURED_PEAKS.json ("of measured"), else the stated fallback ("of fallback")."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)[key]), "of measured"
    except Exception:
        return fallback, "of fallback"


def measured_peak_gbs():
    peak, which = measured_peak("hbm_gbs", FALLBACK_HBM_GBS)
    return peak, which[3:]


# ----------------------------------------------------------------------------- clocks
class ClockSampler:
    """Samples SM clock and clock-event reasons of one GPU through NVML from a thread."""

    REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown",
               0x40: "hw_thermal_slowdown", 0x80: "hw_power_brake_slowdown", 0x2: "applications_clocks_setting"}

    def __init__(self, device_index: int):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        self._h = None
        try:
            import pynvml
            import torch
            pynvml.nvmlInit()
            self._nv = pynvml
            uuid = str(torch.cuda.get_device_properties(device_index).uuid)
            if not uuid.startswith("GPU-"):
                uuid = "GPU-" + uuid
            try:
                self._h = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode())
            except Exception:
                self._h = pynvml.nvmlDeviceGetHandleByIndex(device_index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self._h = None

    def sample(self):
        if self._h is None:
            return
        nv = self._nv
        try:
            self.samples.append(int(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM)))
            try:
                bits = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self._h))
            except Exception:
                bits = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._h))
            for bit, name in self.REASONS.items():
                if bits & bit:
                    self.reasons.add(name)
        except Exception:
            pass

    def _run(self):
        while not self._stop.is_set():
            self.sample()
            time.sleep(0.002)

    def start(self):
        self._stop.clear()
        self._thread = threading.Thread(target=self._run, daemon=True)
        self._thread.start()

    def stop(self):
        self._stop.set()
        if self._thread:
            self._thread.join()

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0}
        return {"sm_mhz": int(np.median(self.samples)), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


# ----------------------------------------------------------------------------- CPU oracle leg
def oracle_step_sample(w, rows: int):
    """Inputs of the oracle's decode step for the first `rows` batch rows, all made on the CPU
    (generator + the oracle's own k-means and encoder on a small calibration draw)."""
    import oracle
    wr = synth.Workload(**{**w.__dict__, "B": rows})
    keys, v, q = synth.make_keys(wr), synth.make_values(wr), synth.make_queries(wr)
    calib = synth.make_calibration_keys(wr, 2048)
    books, _ = oracle.fit_codebooks(calib, w.m, w.K, iters=1, seed=w.seed)
    codes = oracle.encode_keys(keys, books)
    return wr, keys, v, q, books, codes


def oracle_step(wr, keys, v, q, books, codes):
    """The same step the GPU times: encode the newest key, build tables, attend."""
    import oracle
    L = wr.L
    oracle.encode_keys(keys[:, :, L - 1:L], books, codes=codes, L_max=L, pos=L - 1)
    return oracle.decode_step(q, books, codes, v)


def time_oracle(w, budget_s: float = 12.0):
    import oracle
    rows = 1
    sample = oracle_step_sample(w, rows)
    t0 = time.perf_counter()
    oracle_step(*sample)
    t1 = time.perf_counter() - t0
    reps = int(max(1, min(20, budget_s / max(t1, 1e-3))))
    t0 = time.perf_counter()
    for _ in range(reps):
        oracle_step(*sample)
    dt = (time.perf_counter() - t0) / reps
    units = rows * w.n_q_heads * w.L
    return {"value": units / dt, "unit": UNIT, "cores": oracle.n_threads(), "kind": "oracle",
            "sample": f"{rows} of {w.B} batch rows ({w.n_q_heads} query heads x {w.L} tokens), "
                      f"mean of {reps} steps of {dt * 1e3:.1f} ms; fp64, OpenMP over (row, head)"}


def time_oracle_configs(budget_s: float = 2.0):
    """The oracle's decode step (tables + attend, the newest key encoded first) on the GPT-2 shaped workloads and one
    batch row of the long-context one, with one thread and with all of them: tokens*heads per second each."""
    import oracle
    out = {}
    cases = [("gpt2_l128_m4", None), ("gpt2_b8_l1024_m2", None), ("gpt2_b32_l1024_m4", None), ("gqa_32k_m8", 1)]
    for name, rows in cases:
        w = synth.WORKLOADS[name]
        sample = oracle_step_sample(w, rows or w.B)
        units = (rows or w.B) * w.n_q_heads * w.L
        res = {"sample": f"{rows or w.B} of {w.B} batch rows"}
        for label, nthreads in (("threads_1", 1), ("threads_all", oracle.all_threads())):
            oracle.set_threads(nthreads)
            oracle_step(*sample)
            t0 = time.perf_counter()
            reps = 0
            while reps < 50 and (reps == 0 or time.perf_counter() - t0 < budget_s / 2):
                oracle_step(*sample)
                reps += 1
            dt = (time.perf_counter() - t0) / reps
            res[label] = {"value": units / dt, "unit": UNIT, "cores": nthreads, "ms_per_step": dt * 1e3, "reps": reps}
        out[name] = res
    oracle.set_threads(oracle.all_threads())
    return out


def run_reference(args, w):
    """--impl reference: the CPU oracle, as it stands, on the host cores."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    rows = 1
    sample = oracle_step_sample(w, rows)
    for _ in range(args.warmup):
        oracle_step(*sample)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_step(*sample)
    dt = (time.perf_counter() - t0) / args.steps
    units = rows * w.n_q_heads * w.L
    value = units / dt
    sample_txt = (f"each step: {rows} of {w.B} batch rows ({w.n_q_heads} query heads x {w.L} tokens); "
                  "fp64, OpenMP over (row, head)")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": workload_config(w),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.n_threads(), "kind": "oracle",
                             "sample": sample_txt},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def rank_workload(w, rank: int):
    """The replica a rank runs: same shape, its own inputs (seed offset by rank)."""
    return synth.Workload(**{**w.__dict__, "seed": w.seed + 7919 * rank})


def max_over_ranks(values, device):
    """Element-wise maximum of a list of floats over all ranks (identity without a process group)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return [float(x) for x in values]
    t = torch.tensor(values, dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t]


def job_value(w, world: int, ms_per_step: float) -> float:
    """Whole-job tokens*heads per second: every rank scores B*H_q*L pairs per step."""
    return w.B * w.n_q_heads * w.L * world / (ms_per_step * 1e-3)


L2_BYTES = 126e6


def input_sets_needed(w) -> int:
    """Copies of (codes, V) to rotate through so that successive steps never find their inputs in L2."""
    per_set = w.B * w.n_kv_heads * w.L * (w.m + 2 * w.d_v)
    return 1 if per_set > 2 * L2_BYTES else int(np.ceil(2.5 * L2_BYTES / per_set))


def workload_config(w):
    sets = input_sets_needed(w)
    l2 = ("inputs larger than L2 (codes + V >> 126 MB), no flush needed" if sets == 1 else
          f"rotating through {sets} copies of codes + V ({sets * w.B * w.n_kv_heads * w.L * (w.m + 2 * w.d_v) / 1e6:.0f} MB), "
          "so every step reads from HBM")
    return {"workload": w.name, "batch": w.B, "n_q_heads": w.n_q_heads, "n_kv_heads": w.n_kv_heads,
            "d_k": w.d_k, "d_v": w.d_v, "seq_len": w.L, "m": w.m, "K": w.K, "v_dtype": "fp16",
            "codebooks": f"fp32, {w.fit_iters} Lloyd iterations on "
                         f"{w.fit_keys_per_head or w.B * w.L} keys per KV head",
            "l2": l2}


# ----------------------------------------------------------------------------- GPU leg
def time_prefill(device_index: int, steps: int = 5, batch: int = 0, heads: int = 0, form: str = "auto"):
    """Causal multi-query attention (lookat_attend_prefill) on the prefill_4k_m16 shape: batch 4, 32 heads,
    4096 queries over 4096 cached tokens, d = 128, m = 16.  The contraction forms are bound by the tensor
    cores: per visible (query, token) pair 2 * d_k MACs of scores (two fp16 planes of each centroid) and
    d_v MACs of the value sum; the table form by its m shared-memory gathers per pair."""
    import torch

    from paper_2601_10155_b200.binding import Lookat
    w = synth.WORKLOADS["prefill_4k_m16"]
    if batch > 0 or heads > 0:                             # smaller cases for profiler captures
        w = synth.Workload(**{**w.__dict__, "B": batch or w.B, "n_q_heads": heads or w.n_q_heads,
                              "n_kv_heads": heads or w.n_kv_heads,
                              "name": f"{w.name}_b{batch or w.B}_h{heads or w.n_q_heads}"})
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
    lk = Lookat(w.n_q_heads, w.n_kv_heads, w.d_k, w.d_v, w.m, w.K, device=device_index)
    lk.lookat_set_prefill_form(form)
    keys = dev(synth.make_keys(w))
    v = dev(synth.make_values(w))
    q = dev(synth.make_prefill_queries(w, w.L))
    books = lk.lookat_fit_codebooks(keys, w.fit_iters, seed=w.seed)          # per head, on its 16,384 keys
    codes = lk.lookat_encode_keys(keys, books)
    out = torch.empty((w.B, w.n_q_heads, w.L, w.d_v), dtype=torch.float32, device="cuda")
    for _ in range(2):
        lk.lookat_attend_prefill(q, books, codes, v, out=out)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record()
    for _ in range(steps):
        lk.lookat_attend_prefill(q, books, codes, v, out=out)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    pairs = w.B * w.n_q_heads * w.L * (w.L + 1) // 2
    res = {"workload": w.name, "form": form, "ms": ms, "pairs_per_s": pairs / (ms * 1e-3), "steps": steps}
    if form == "tables":
        props = torch.cuda.get_device_properties(device_index)
        smem_peak = props.multi_processor_count * 128 * 1.965e9 / 1e9      # GB/s at the maximum SM clock
        achieved = pairs * w.m * 4 / (ms * 1e-3) / 1e9
        res["roofline"] = {"bound": "smem", "achieved": achieved, "peak": smem_peak, "unit": "GB/s",
                           "frac": achieved / smem_peak,
                           "note": "gather bytes (m x 4 B per pair) over 128 B/clk/SM x SMs x 1965 MHz"}
    else:
        peak, which = measured_peak("bf16_tflops", 1590.0)                 # fp16 and bf16 run at the same rate
        achieved = pairs * 2.0 * (2 * w.d_k + w.d_v) / (ms * 1e-3) / 1e12
        res["roofline"] = {"bound": "tensor", "achieved": achieved, "peak": peak, "unit": "TFLOP/s",
                           "frac": achieved / peak,
                           "note": f"2 x (2 d_k + d_v) flop per visible pair; peak: cuBLAS bf16 burst, {which}"}
    return res


def time_encode_1m(device_index: int):
    """Bulk encoding at the size of BASELINE config 4: one KV head, 1,048,576 keys of d = 128, m = 16 (d_sub 8),
    codebooks = the seeded start rule on the first 262,144 keys (no Lloyd iteration); then a refit of 10 iterations
    on those 262,144 keys.  Bounds: HBM (keys in, codes out) and the tensor pipe (2 fp16 planes per centroid)."""
    import torch

    from paper_2601_10155_b200.binding import Lookat
    w = synth.WORKLOADS["encode_1m_m16"]
    lk = Lookat(w.n_q_heads, w.n_kv_heads, w.d_k, w.d_v, w.m, w.K, device=device_index)
    keys = torch.from_numpy(np.ascontiguousarray(synth.make_keys(w))).cuda()
    sample = keys[:, :, :w.fit_keys_per_head].contiguous()
    books0 = lk.lookat_fit_codebooks(sample, 0, seed=w.seed)
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
    for attempt in range(2):                               # the second pass is timed
        ev[0].record()
        codes = lk.lookat_encode_keys(keys, books0)
        ev[1].record()
        books = lk.lookat_fit_codebooks(sample, w.fit_iters, seed=w.seed)
        ev[2].record()
    torch.cuda.synchronize()
    enc_ms, fit_ms = ev[0].elapsed_time(ev[1]), ev[1].elapsed_time(ev[2])
    n = w.B * w.n_kv_heads * w.L
    hbm_peak, which = measured_peak("hbm_gbs", FALLBACK_HBM_GBS)
    tensor_peak, _ = measured_peak("bf16_tflops", 1590.0)
    bytes_moved = n * (w.d_k * 2 + w.m)
    flops = 2.0 * n * w.K * w.d_k * 2                      # two fp16 planes per centroid
    del codes, books
    return {"workload": w.name, "encode_ms": enc_ms, "keys_per_s": n / (enc_ms * 1e-3),
            "hbm_frac": bytes_moved / (enc_ms * 1e-3) / 1e9 / hbm_peak,
            "tensor_frac": flops / (enc_ms * 1e-3) / 1e12 / tensor_peak, "peaks": which,
            "refit_ms": fit_ms, "refit": f"{w.fit_iters} Lloyd iterations on {w.fit_keys_per_head} keys"}


def time_pqv(lk, w, q, books, codes, v, steps: int, sm_mhz: float):
    """Beyond the paper (its Section 5.2 names value compression as future work): the same decode attention with
    the values product-quantised too (m_v = m subspaces, K = 256), `lookat_attend_pqv`.  Per (token, KV head) pair it
    reads m + m_v bytes instead of m + 2 d_v; the codes of one copy fit in L2, so the step rotates through copies."""
    import torch

    from paper_2601_10155_b200.binding import Lookat
    m_v = w.m
    lv = Lookat(w.n_kv_heads, w.n_kv_heads, w.d_v, w.d_v, m_v, 256, device=lk.device.index)
    n_fit = w.fit_keys_per_head or w.B * w.L
    sample = v[:, :, :max(1, n_fit // w.B)].contiguous()
    v_books = lv.lookat_fit_codebooks(sample, w.fit_iters, seed=w.seed + 1)       # values are encoded like keys
    v_codes = lv.lookat_encode_keys(v, v_books)
    bytes_per_copy = codes.numel() + v_codes.numel()
    n_sets = max(2, int(np.ceil(3 * L2_BYTES / bytes_per_copy)))                  # every step reads from HBM
    sets = [(codes.clone(), v_codes.clone()) for _ in range(n_sets)]
    out = torch.empty((w.B, w.n_q_heads, w.d_v), dtype=torch.float32, device="cuda")
    for i in range(3):
        lk.lookat_attend_pqv(sets[i % n_sets][0], v_books, sets[i % n_sets][1], q=q, codebooks=books, out=out)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record()
    for i in range(steps):
        lk.lookat_attend_pqv(sets[i % n_sets][0], v_books, sets[i % n_sets][1], q=q, codebooks=books, out=out)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    pairs = w.B * w.n_kv_heads * w.L
    peak, which = measured_peak("hbm_gbs", FALLBACK_HBM_GBS)
    achieved = pairs * (w.m + m_v) / (ms * 1e-3) / 1e9
    smem_bytes = w.B * w.n_q_heads * w.L * (w.m * 4 + m_v * 4)
    smem_peak = 148 * 128 * sm_mhz * 1e6 / 1e9
    # what the compression costs in accuracy on these inputs: against the fp16-V result of the same step
    ref = lk.lookat_attend(codes, v, q=q, codebooks=books)
    err = float((out - ref).abs().max())
    # the same comparison on values a quantiser can compress (rows near a low-rank subspace, like the keys): 2 batch rows
    structured = None
    try:
        rows = min(2, w.B)
        wl = synth.Workload(**{**w.__dict__, "B": rows})
        v_lr = torch.from_numpy(synth.make_values_lowrank(wl)).cuda()
        books_lr = lv.lookat_fit_codebooks(v_lr[:, :, :max(1, n_fit // rows)].contiguous(), w.fit_iters, seed=w.seed + 2)
        codes_lr = lv.lookat_encode_keys(v_lr, books_lr)
        q2, c2 = q[:rows].contiguous(), codes[:rows].contiguous()
        o_pq = lk.lookat_attend_pqv(c2, books_lr, codes_lr, q=q2, codebooks=books)
        o_fp = lk.lookat_attend(c2, v_lr, q=q2, codebooks=books)
        structured = {"values": "fp16(z A^T + 0.1 eps), rank as the keys", "batch_rows": rows,
                      "max_abs_diff_to_fp16_values": float((o_pq - o_fp).abs().max()),
                      "rms_of_fp16_values_output": float(o_fp.pow(2).mean().sqrt()),
                      "relative_rms_error": float((o_pq - o_fp).pow(2).mean().sqrt() / o_fp.pow(2).mean().sqrt())}
        del v_lr, codes_lr
    except Exception as exc:
        structured = {"error": str(exc)[:200]}
    return {"ms_per_step": ms, "tokens_heads_per_s": w.B * w.n_q_heads * w.L / (ms * 1e-3), "m_v": m_v, "K_v": 256,
            "structured_values": structured,
            "launches_per_step": 2, "l2": f"{n_sets} copies of the codes in rotation",
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                         "note": f"(m + m_v) bytes per (token, KV head) pair; peak {which}.  The kernel is bound by its "
                                 "table reads and histogram adds in shared memory, not by HBM: see shared_memory"},
            # 4 bytes read and 4 bytes added per (token, query head, subspace), against 128 bytes per clock and SM
            "shared_memory": {"bytes_per_step": smem_bytes, "achieved_gbs": smem_bytes / (ms * 1e-3) / 1e9,
                              "peak_gbs": smem_peak, "frac": smem_bytes / (ms * 1e-3) / 1e9 / smem_peak,
                              "note": "peak = 148 SMs x 128 B/clk x the median SM clock sampled during the timed decode steps"},
            "max_abs_diff_to_fp16_values": err,
            "note": "value compression is not part of the paper's method (its Section 5.2: future work)"}


def timed_blocks(run_block, sync, min_seconds: float = MIN_TIMED_SECONDS, max_blocks: int = 400):
    """Calls run_block() (one block of steps, enqueued on the current stream) between CUDA events until min_seconds of
    device time have been timed; returns the blocks' durations in milliseconds."""
    import torch
    times = []
    while len(times) < max_blocks and (not times or sum(times) < min_seconds * 1e3):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        run_block()
        e1.record()
        sync()
        times.append(e0.elapsed_time(e1))
    return times


def time_small_config(name: str, device_index: int):
    """One GPT-2 shaped decode step (`lookat_decode_step`: append-encode, tables, scores, softmax, value sum, merge in
    one launch) timed as a CUDA graph of back-to-back steps that rotate through enough copies of codes + V that every
    step reads from HBM; beside it the same loop as plain host calls.  Codebooks: the workload's Lloyd iterations on the
    cached keys."""
    import torch

    from paper_2601_10155_b200.binding import Lookat
    w = synth.WORKLOADS[name]
    side = torch.cuda.Stream(device=device_index)
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
    with torch.cuda.stream(side):
        lk = Lookat(w.n_q_heads, w.n_kv_heads, w.d_k, w.d_v, w.m, w.K, device=device_index, stream=side)
        keys, v, q = dev(synth.make_keys(w)), dev(synth.make_values(w)), dev(synth.make_queries(w))
        n_fit = w.fit_keys_per_head or w.B * w.L
        books = lk.lookat_fit_codebooks(keys[:, :, :max(1, n_fit // w.B)].contiguous(), w.fit_iters, seed=w.seed)
        codes = lk.lookat_encode_keys(keys, books)
        n_sets = input_sets_needed(w)
        cs = [codes.clone() for _ in range(n_sets)]
        vs = [v.clone() for _ in range(n_sets)]
        new_k = keys[:, :, w.L - 1].contiguous()
        out = torch.empty((w.B, w.n_q_heads, w.d_v), dtype=torch.float32, device="cuda")

        def step(i):
            lk.lookat_decode_step(q, new_k, books, cs[i % n_sets], vs[i % n_sets], w.L - 1, out=out)

        for i in range(max(3, min(n_sets, 16))):
            step(i)
        side.synchronize()
        launches0 = lk.lookat_kernel_launches()
        step(0)
        launches_per_step = lk.lookat_kernel_launches() - launches0
        n_in = max(n_sets, 32)
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            for i in range(n_in):
                step(i)
        graph.replay()
        side.synchronize()
        g_ms = timed_blocks(graph.replay, side.synchronize)
        h_ms = timed_blocks(lambda: [step(i) for i in range(n_in)], side.synchronize, min_seconds=0.05)
    ms = float(np.median(g_ms)) / n_in
    alg = w.B * w.n_kv_heads * w.L * (w.m + 2 * w.d_v) + books.numel() * 4
    peak, which = measured_peak("hbm_gbs", FALLBACK_HBM_GBS)
    gbs = alg / (ms * 1e-3) / 1e9
    return {"ms_per_step": ms, "us_per_step": ms * 1e3, "tokens_heads_per_s": w.B * w.n_q_heads * w.L / (ms * 1e-3),
            "algorithmic_bytes": int(alg), "hbm_gbs": gbs, "frac_of_measured_peak": gbs / peak,
            "frac_of_nominal_8tbs": gbs / NOMINAL_HBM_GBS, "peak_source": which,
            "ms_per_step_host_calls": float(np.median(h_ms)) / n_in, "launches_per_step": int(launches_per_step),
            "timing": f"CUDA graph of {n_in} steps, median of {len(g_ms)} replays", "l2": workload_config(w)["l2"],
            "batch": w.B, "heads": w.n_q_heads, "seq_len": w.L, "m": w.m}


def time_c2_replay(device_index: int, layers: int = 12, steps: int = 64):
    """The attention of BASELINE config 2 replayed: 12 layers with their own head generators and codebooks (25 Lloyd
    iterations on the layer's 32,768 prefill keys per head), batch 32 x 12 heads, caches with room for 1088 tokens that
    64 decode steps grow from 1024 to 1088; every layer-step is one `lookat_decode_step` (the new key encoded on
    append, then Algorithm 1 over the cache).  768 launches captured as one CUDA graph; 634 MB of codes + V per
    token-step over the 12 layers, so every layer-step reads from HBM."""
    import torch

    from paper_2601_10155_b200.binding import Lookat
    base = synth.WORKLOADS["gpt2_b32_l1024_m4"]
    L0, cap = base.L, base.L + steps
    side = torch.cuda.Stream(device=device_index)
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
    with torch.cuda.stream(side):
        lk = Lookat(base.n_q_heads, base.n_kv_heads, base.d_k, base.d_v, base.m, base.K, device=device_index, stream=side)
        per_layer = []
        fit_ms = 0.0
        for layer in range(layers):
            w = synth.Workload(**{**base.__dict__, "layer": layer})
            keys = dev(synth.make_keys(w, n_tokens=cap))
            v = dev(synth.make_values(w, n_tokens=cap))
            q = dev(synth.make_queries(w))
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            books = lk.lookat_fit_codebooks(keys[:, :, :L0].contiguous(), w.fit_iters, seed=w.seed)
            e1.record()
            cache = torch.zeros((w.B, w.n_kv_heads, cap, w.m), dtype=torch.uint8, device="cuda")
            lk.lookat_encode_keys(keys[:, :, :L0].contiguous(), books, codes=cache, pos=0)
            new_keys = keys[:, :, L0:].permute(2, 0, 1, 3).contiguous()       # [step][B][H][d_k]
            side.synchronize()
            fit_ms += e0.elapsed_time(e1)
            per_layer.append((q, new_keys, books, cache, v))
            del keys
        out = torch.empty((base.B, base.n_q_heads, base.d_v), dtype=torch.float32, device="cuda")

        def replay():
            for t in range(steps):
                for q, new_keys, books, cache, v in per_layer:
                    lk.lookat_decode_step(q, new_keys[t], books, cache, v, L0 + t, out=out)

        replay()                                            # also grows the context's scratch to its final size
        side.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            replay()
        graph.replay()
        side.synchronize()
        g_ms = timed_blocks(graph.replay, side.synchronize)
        h_ms = timed_blocks(replay, side.synchronize, min_seconds=0.05)
    total_ms = float(np.median(g_ms))
    n = layers * steps
    pairs = sum(base.B * base.n_kv_heads * (L0 + t + 1) for t in range(steps)) * layers
    alg = pairs * (base.m + 2 * base.d_v) + n * per_layer[0][2].numel() * 4
    peak, which = measured_peak("hbm_gbs", FALLBACK_HBM_GBS)
    gbs = alg / (total_ms * 1e-3) / 1e9
    return {"layers": layers, "steps": steps, "batch": base.B, "heads": base.n_q_heads, "seq_len": f"{L0} -> {cap}",
            "total_ms": total_ms, "us_per_layer_step": total_ms * 1e3 / n, "ms_per_generated_token": total_ms / steps,
            "tokens_heads_per_s": pairs * (base.n_q_heads // base.n_kv_heads) / (total_ms * 1e-3),
            "algorithmic_bytes": int(alg), "hbm_gbs": gbs, "frac_of_measured_peak": gbs / peak,
            "frac_of_nominal_8tbs": gbs / NOMINAL_HBM_GBS, "peak_source": which,
            "total_ms_host_calls": float(np.median(h_ms)), "launches": n,
            "timing": f"one CUDA graph of {n} launches, median of {len(g_ms)} replays",
            "setup_fit_ms_all_layers": fit_ms}


def time_gpt2_decoder(device_index: int, steps: int = 64, profile_steps: int = 8):
    """BASELINE config 2 end to end: the 12-layer GPT-2-small decoder (d_model 768, 12 heads, MLP 3072, vocab 50257,
    random-init fp16 weights, uniform-random prompt ids), batch 32, a prompt of 1024 tokens processed with exact
    attention, codebooks (m = 4, K = 256, 25 Lloyd iterations) fitted per layer and head on the prompt's keys, then 64
    tokens generated greedily with the new key encoded on append and Algorithm 1 in every layer.  Every kernel is this
    library's own.  A few more steps are then decoded with per-category events to show where a step's time goes."""
    import torch

    from paper_2601_10155_b200.binding import LookatGpt2
    B, T0, vocab = 32, 1024, 50257
    cap = T0 + steps + profile_steps
    wd = synth.gpt2_weights(1002, n_pos=cap)
    ids = torch.from_numpy(synth.token_ids(1002, B, T0 + 1, vocab)).cuda()
    model = LookatGpt2(wd, B, cap, m=4, K=256, fit_iters=25, device=device_index)
    prompt = ids[:, :T0].contiguous()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
    model.lookat_gpt2_prefill(prompt, seed=1002)                 # first pass: scratch grows, clocks come up
    torch.cuda.synchronize()
    launches0 = model.lookat_gpt2_kernel_launches()
    ev[0].record()
    model.lookat_gpt2_prefill(prompt, seed=1002)
    ev[1].record()
    torch.cuda.synchronize()
    prefill_launches = model.lookat_gpt2_kernel_launches() - launches0
    nxt = [torch.empty((B,), dtype=torch.int32, device="cuda") for _ in range(2)]
    cur = ids[:, T0].contiguous()
    launches0 = model.lookat_gpt2_kernel_launches()
    ev[2].record()
    for t in range(steps):
        model.lookat_gpt2_decode(cur, want_next=True, next_ids=nxt[t & 1])
        cur = nxt[t & 1]
    ev[3].record()
    torch.cuda.synchronize()
    step_launches = (model.lookat_gpt2_kernel_launches() - launches0) // steps
    model.lookat_gpt2_set_profile(True)
    for t in range(profile_steps):
        model.lookat_gpt2_decode(cur, want_next=True, next_ids=nxt[t & 1])
        cur = nxt[t & 1]
    torch.cuda.synchronize()
    n_prof, cats = model.lookat_gpt2_profile()
    model.lookat_gpt2_set_profile(False)
    total = sum(cats.values()) or 1.0
    prefill_ms, decode_ms = ev[0].elapsed_time(ev[1]), ev[2].elapsed_time(ev[3])
    params = sum(int(np.prod(a.shape)) for lw in wd["layers"] for a in lw.values()) + int(np.prod(wd["wte"].shape))
    return {"model": "GPT-2 small shape, random-init fp16", "batch": B, "prompt_tokens": T0, "generated_tokens": steps,
            "m": 4, "K": 256, "fit_iters": 25,
            "prefill_ms": prefill_ms, "prefill_tokens_per_s": B * T0 / (prefill_ms * 1e-3), "prefill_launches": int(prefill_launches),
            "prefill_includes": "12 x (products, exact causal attention, k-means on 32,768 keys per head, encoding)",
            "ms_per_generated_token": decode_ms / steps, "generated_tokens_per_s": B * steps / (decode_ms * 1e-3),
            "launches_per_token": int(step_launches),
            "weight_bytes_per_token": int(params * 2),
            "weights_gbs": params * 2 / (decode_ms / steps * 1e-3) / 1e9,
            "share_of_step": {k: v / total for k, v in cats.items()},
            "share_measured_over_steps": int(n_prof), "sampling": "greedy (argmax on the device), ids fed back without a host copy"}


def run_lookat(args, w):
    import torch
    import torch.distributed as dist

    from paper_2601_10155_b200.binding import Lookat

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    # every rank runs the same replica shape on its own inputs (seed offset by rank)
    wr = rank_workload(w, rank)
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
    lk = Lookat(w.n_q_heads, w.n_kv_heads, w.d_k, w.d_v, w.m, w.K, device=local_rank)

    t_gen = time.perf_counter()
    keys = dev(synth.make_keys(wr))
    v = dev(synth.make_values(wr))
    q_np = synth.make_queries(wr)
    q = dev(q_np)
    t_gen = time.perf_counter() - t_gen

    # ---- setup: calibration (k-means) and prefill encoding, timed but outside the step ----
    n_fit = w.fit_keys_per_head or w.B * w.L
    per_row = max(1, n_fit // w.B)
    fit_keys = keys[:, :, :per_row].contiguous()
    # the first pass is not timed (first-call allocations, clocks coming up); of the three that follow the median counts
    # (the k-means is some thirty short launches: a host that is held up for a moment shows in a single timing)
    passes = []
    for attempt in range(4):
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
        ev[0].record()
        books = lk.lookat_fit_codebooks(fit_keys, w.fit_iters, seed=w.seed)
        ev[1].record()
        ties = torch.zeros(1, dtype=torch.int64, device="cuda")
        codes = lk.lookat_encode_keys(keys, books, near_ties=ties)
        ev[2].record()
        torch.cuda.synchronize()
        if attempt:
            passes.append((ev[0].elapsed_time(ev[1]), ev[1].elapsed_time(ev[2])))
    fit_ms, enc_ms = float(np.median([p[0] for p in passes])), float(np.median([p[1] for p in passes]))
    del fit_keys

    L = w.L
    new_k = keys[:, :, L - 1:L].contiguous()              # the newest key of every (row, KV head)
    out = torch.empty((w.B, w.n_q_heads, w.d_v), dtype=torch.float32, device="cuda")

    new_k3 = new_k.reshape(w.B, w.n_kv_heads, w.d_k)
    # small workloads: rotate through enough copies of the cache that no step finds it in L2
    n_sets = input_sets_needed(w)
    code_sets = [codes] + [codes.clone() for _ in range(n_sets - 1)]
    v_sets = [v] + [v.clone() for _ in range(n_sets - 1)]
    turn = [0]

    def step():
        # append (encode the newest key) and Algorithm 1 (tables, lookup-sum, softmax, value sum)
        i = turn[0] = (turn[0] + 1) % n_sets
        lk.lookat_decode_step(q, new_k3, books, code_sets[i], v_sets[i], L - 1, out=out, n_splits=args.splits)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(local_rank)
    for _ in range(max(args.warmup, 3)):
        step()
    barrier()
    # a block = exactly `steps` steps between two events; blocks are repeated until MIN_TIMED_SECONDS have been timed
    # (every rank runs the same number: the count is fixed from one untimed block), the median block is reported
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        step()
    e1.record()
    barrier()
    (probe_ms,) = max_over_ranks([e0.elapsed_time(e1)], "cuda")
    n_blocks = int(min(400, max(1, np.ceil(MIN_TIMED_SECONDS * 1e3 / max(probe_ms, 1e-3)))))
    launches0 = lk.lookat_kernel_launches()
    lk.lookat_set_timing(min(args.steps * n_blocks, 40000))
    block_ms = []
    sampler.start()
    for _ in range(n_blocks):
        e0.record()
        for _ in range(args.steps):
            step()
        e1.record()
        barrier()
        block_ms.append(e0.elapsed_time(e1))
    sampler.sample()
    sampler.stop()
    lk.lookat_set_timing(0)
    kstats = lk.lookat_attend_kernel_stats()
    launches = (lk.lookat_kernel_launches() - launches0) // n_blocks
    elapsed_ms, attend_ms = max_over_ranks([float(np.median(block_ms)), kstats["median"]], "cuda")

    # ---- end to end: host buffers in, host buffer out, through the C-ABI call ----
    q_host = torch.from_numpy(q_np).pin_memory()
    k_host = new_k.reshape(w.B, w.n_kv_heads, w.d_k).cpu().pin_memory()
    v_host = v[:, :, L - 1].contiguous().cpu().pin_memory()
    out_host = torch.empty((w.B, w.n_q_heads, w.d_v), dtype=torch.float32).pin_memory()
    for _ in range(3):
        lk.lookat_decode_step_host(q_host, k_host, v_host, books, codes, v, L - 1, out_host, n_splits=args.splits)
    barrier()
    e2e_steps = args.steps
    t0 = time.perf_counter()
    e0.record()
    for _ in range(e2e_steps):
        lk.lookat_decode_step_host(q_host, k_host, v_host, books, codes, v, L - 1, out_host, n_splits=args.splits)
    e1.record()
    torch.cuda.synchronize()
    e2e_ms = max(e0.elapsed_time(e1), (time.perf_counter() - t0) * 1e3)
    (e2e_ms,) = max_over_ranks([e2e_ms], "cuda")
    step()
    torch.cuda.synchronize()
    same = bool(torch.allclose(out_host.cuda(), out, rtol=0, atol=1e-5))
    # read ceiling of this GPU, same process and clocks: a read-only streaming pass over the V cache (>> L2)
    read_ceiling = lk.lookat_probe_read_bandwidth(v, reps=5) if v.numel() * 2 >= (1 << 28) else None
    pqv = None
    if world == 1 and args.pqv:
        try:
            pqv = time_pqv(lk, w, q, books, codes, v, min(args.steps, 50), sampler.summary()["sm_mhz"] or sampler.max_mhz or 1965)
        except Exception as exc:
            pqv = {"error": str(exc)[:200]}

    if rank == 0:
        units_per_step = w.B * w.n_q_heads * L * world
        ms_per_step = elapsed_ms / args.steps
        value = job_value(w, world, ms_per_step)
        peak, peak_kind = measured_peak_gbs()
        alg_bytes = (w.m + 2 * w.d_v) * w.B * w.n_kv_heads * L           # per attend launch
        achieved = alg_bytes / (attend_ms * 1e-3) / 1e9
        per_pair = ATTEND_DRAM_BYTES_PER_PAIR.get(args.workload)
        traffic = None if per_pair is None else int(per_pair * w.B * w.n_kv_heads * L)
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": workload_config(w),
            "roofline": {"bound": "hbm", "kernel": "attend_stream_kernel", "achieved": achieved, "peak": peak,
                         "unit": "GB/s", "frac": achieved / peak, "peak_source": f"of {peak_kind}",
                         "traffic": traffic, "traffic_source": ATTEND_TRAFFIC_SOURCE if traffic else None,
                         "algorithmic_bytes_per_launch": alg_bytes,
                         "kernel_ms": attend_ms, "kernel_ms_min": kstats["min"], "kernel_ms_median": kstats["median"],
                         "kernel_ms_max": kstats["max"], "kernel_ms_mean": kstats["mean"], "kernel_launches_timed": kstats["n"],
                         "frac_of_nominal_8tbs": achieved / NOMINAL_HBM_GBS,
                         "read_ceiling_gbs": read_ceiling,
                         "frac_of_read_ceiling": None if not read_ceiling else achieved / read_ceiling},
            "e2e": {"value": units_per_step / (e2e_ms / e2e_steps * 1e-3), "unit": UNIT,
                    "h2d_bytes_per_step": int(q_host.numel() * 2 + k_host.numel() * 2 + v_host.numel() * 2),
                    "d2h_bytes_per_step": int(out_host.numel() * 4), "ms_per_step": e2e_ms / e2e_steps,
                    "matches_device_path": same},
            "gpu_launches": int(launches),
            "blocks": n_blocks, "block_ms_min": float(min(block_ms)), "block_ms_max": float(max(block_ms)),
            "timing": f"median of {n_blocks} blocks of {args.steps} steps (CUDA events, barrier between blocks)",
            "clocks": sampler.summary(),
            "step_hbm_gbs": (alg_bytes + books.numel() * 4) / (ms_per_step * 1e-3) / 1e9,
            "setup": {"fit_ms": fit_ms, "bulk_encode_ms": enc_ms,
                      "bulk_encode_keys_per_s": w.B * w.n_kv_heads * L / (enc_ms * 1e-3),
                      "near_ties": int(ties.item()), "input_generation_s": t_gen},
        }
        if world == 1 and not args.no_cpu_baseline:
            line["cpu_baseline"] = time_oracle(w)
            try:
                line["cpu_baseline_configs"] = time_oracle_configs()
            except Exception as exc:
                line["cpu_baseline_configs"] = {"error": str(exc)[:200]}
        if pqv is not None:
            line["pqv"] = pqv
        if world == 1 and args.prefill:
            keys = v = codes = code_sets = v_sets = None
            torch.cuda.empty_cache()
            try:
                line["prefill"] = time_prefill(local_rank)
            except Exception as exc:                      # the decode line stands on its own
                line["prefill"] = {"error": str(exc)[:200]}
            try:
                line["encode_1m"] = time_encode_1m(local_rank)
            except Exception as exc:
                line["encode_1m"] = {"error": str(exc)[:200]}
        if world == 1 and args.small:
            keys = v = codes = code_sets = v_sets = None
            torch.cuda.empty_cache()
            small = {}
            for name in SMALL_WORKLOADS:
                try:
                    small[name] = time_small_config(name, local_rank)
                except Exception as exc:
                    small[name] = {"error": str(exc)[:200]}
                torch.cuda.empty_cache()
            line["small_configs"] = small
            try:
                line["c2_replay"] = time_c2_replay(local_rank)
            except Exception as exc:
                line["c2_replay"] = {"error": str(exc)[:200]}
            torch.cuda.empty_cache()
            try:
                line["gpt2_decoder"] = time_gpt2_decoder(local_rank)
            except Exception as exc:
                line["gpt2_decoder"] = {"error": str(exc)[:200]}
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="lookat", choices=["lookat", "reference"])
    ap.add_argument("--workload", default="gqa_32k_m8", choices=sorted(synth.WORKLOADS))
    ap.add_argument("--splits", type=int, default=0, help="sequence chunks per row (0: library default)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-prefill", dest="prefill", action="store_false",
                    help="skip the extra timing of the causal multi-query kernel")
    ap.add_argument("--no-pqv", dest="pqv", action="store_false",
                    help="skip the extra leg that times decode attention with product-quantised values")
    ap.add_argument("--no-small", dest="small", action="store_false",
                    help="skip the GPT-2 shaped decode steps and the 12-layer x 64-step replay")
    ap.add_argument("--only-gpt2", action="store_true", help="time only the GPT-2 decoder harness (prints its object alone)")
    ap.add_argument("--only-prefill", action="store_true",
                    help="time only the causal multi-query kernel (prints its object alone)")
    ap.add_argument("--prefill-batch", type=int, default=0, help="smaller prefill case: batch rows")
    ap.add_argument("--prefill-heads", type=int, default=0, help="smaller prefill case: heads")
    ap.add_argument("--prefill-form", default="auto", choices=["auto", "tables", "contraction"],
                    help="which kernel lookat_attend_prefill uses in the prefill timing")
    ap.add_argument("--batch", type=int, default=0,
                    help="override the workload's batch size (smaller cases for profiler captures)")
    args = ap.parse_args()
    w = synth.WORKLOADS[args.workload]
    if args.batch > 0:
        w = synth.Workload(**{**w.__dict__, "B": args.batch, "name": f"{w.name}_b{args.batch}"})
    if args.only_gpt2:
        print(json.dumps(time_gpt2_decoder(int(os.environ.get("LOCAL_RANK", "0")))), flush=True)
        return
    if args.only_prefill:
        print(json.dumps(time_prefill(int(os.environ.get("LOCAL_RANK", "0")), steps=max(1, min(args.steps, 5)),
                                      batch=args.prefill_batch, heads=args.prefill_heads, form=args.prefill_form)), flush=True)
    elif args.impl == "reference":
        run_reference(args, w)
    else:
        run_lookat(args, w)


if __name__ == "__main__":
    main()
