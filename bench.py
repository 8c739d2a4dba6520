#!/usr/bin/env python
"""Benchmark of the fused attention forward pass on B200 (one JSON line on stdout).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config IDX] [--impl reference]

The default workload is the largest single-GPU configuration (index 4: 128K tokens, grouped
heads, causal), whose timed region of K launches lasts seconds: the clock samples fall inside it
and the GPU runs under its power cap, as it does in production.  `per_config` holds a full record
of all five configurations (back-to-back mean, per-launch minimum and median of 20 launches after
10 warm-ups as in Section 5.1 of the paper, clock samples of its own window, roofline fractions
against the measured burst and sustained peaks).

A step is one pass of the whole hot path (one `fa_forward` launch) over one
batch of the workload.  `value` is effective-GEMM throughput (Section 5.1 of the
paper: 2*H*Lq*Lk*(dk+dv)/T) counted over VISIBLE (query, key) pairs only; the
paper's own convention (full Lq*Lk rectangle even when causal) is reported as
`value_paper_convention`.  Inputs are synthetic Gaussians already resident in
HBM; several input sets are rotated so that the footprint between two uses of
the same set exceeds L2.  `e2e` is the same metric through `fa_forward_host`
with pinned host buffers (copies inside the timed region).

`--impl reference` times the fp64 CPU oracle instead (a deliberately slow
program; parity and the roofline fraction are the headline, not that ratio).
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2609_21264_b200 import launch, metrics, workloads  # noqa: E402

L2_BYTES = 126 * 1024 * 1024
# Paper, Table 6: Llama-3 8B shape (32/8 heads, d=128, causal, S=2048) on XDNA 2: 34076 us.
PAPER_SECONDS = {"llama3_8b_gqa_s2048": 34076e-6}
# dram__bytes_read.sum + dram__bytes_write.sum of one launch of the dominant kernel on each configuration, each taken
# from a one-pass ncu capture of this program on that configuration at full size (a one-pass metric list saves and
# restores no device memory, so the full workload can be captured); the commands and figures are under profiles/.
# Reads below the compulsory bytes mean that part of a rotating input set was still in L2; writes below the output
# size mean that the launch ended with its last outputs still in L2.
NCU_DRAM_BYTES_PER_LAUNCH = {
    "bert_base_mha_s512": 2.42e6 + 0.0,
    "llama3_8b_gqa_s2048": 25.23e6 + 0.0,
    "llama2_7b_mha_b4_s8192": 923.00e6 + 253.69e6,
    "deepseek_v2_mha_s4096_d192_128": 569.05e6 + 121.60e6,
    "long_context_gqa_s131072": 3.14e9 + 1.06e9,
}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": p["hbm_gbs"], "bf16_tflops": p["bf16_tflops"],
                "bf16_tflops_sustained": p.get("bf16_tflops_sustained", p["bf16_tflops"]),
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML while the timed region runs (read-only)."""

    def __init__(self, index: int, period_s: float = 0.005):
        super().__init__(daemon=True)
        self.index, self.period = index, period_s
        self.samples, self.max_mhz = [], None          # (time, MHz, set of reasons)
        self.window = [None, None]                     # timed region, marked by the caller
        self._halt = threading.Event()
        self.error = None

    def run(self):
        try:
            import pynvml as nv
            nv.nvmlInit()
            h = nv.nvmlDeviceGetHandleByIndex(self.index)
            self.max_mhz = nv.nvmlDeviceGetMaxClockInfo(h, nv.NVML_CLOCK_SM)
            names = {
                getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8): "hw_slowdown",
                getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
                getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
                getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4): "sw_power_cap",
            }
            get_reasons = getattr(nv, "nvmlDeviceGetCurrentClocksEventReasons", None) or \
                getattr(nv, "nvmlDeviceGetCurrentClocksThrottleReasons")
            while not self._halt.is_set():
                mhz = nv.nvmlDeviceGetClockInfo(h, nv.NVML_CLOCK_SM)
                mask = get_reasons(h)
                self.samples.append((time.perf_counter(), mhz,
                                     {name for bit, name in names.items() if bit and (mask & bit)}))
                time.sleep(self.period)
        except Exception as ex:  # pragma: no cover
            self.error = repr(ex)

    def wait_ready(self, timeout_s: float = 3.0):
        t_end = time.perf_counter() + timeout_s
        while not self.samples and self.error is None and time.perf_counter() < t_end:
            time.sleep(0.002)

    def mark(self, which: int):
        self.window[which] = time.perf_counter()

    def stop(self):
        self._halt.set()
        self.join(timeout=2.0)
        t0, t1 = self.window
        inside = [x for x in self.samples if t0 is not None and t1 is not None and t0 <= x[0] <= t1]
        note = "samples taken inside the timed region"
        if not inside:      # region shorter than one sampling period: the warm-up ran the same launches just before
            inside = [x for x in self.samples if t1 is None or x[0] <= t1][-3:]
            note = "timed region shorter than the sampling period: last samples of the warm-up (same launches)"
        mhz = sorted(x[1] for x in inside)
        reasons = set().union(*[x[2] for x in inside]) if inside else set()
        return {"sm_mhz": (mhz[len(mhz) // 2] if mhz else None), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(reasons), "samples": len(mhz), "window": note,
                **({"error": self.error} if self.error else {})}


def physical_gpu_index(local_index: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_index])
        except Exception:
            return local_index
    return local_index


def make_device_sets(w, n_sets, device):
    """n_sets independent (Q, K, V, O, lse) sets of synthetic bf16 Gaussians on the device."""
    import torch
    g = torch.Generator(device=device)
    g.manual_seed(w.seed)
    qs, ks, vs, os_ = w.shapes()
    sets = []
    for _ in range(n_sets):
        q = (torch.randn(qs, generator=g, device=device, dtype=torch.float32) * w.sigma).to(torch.bfloat16)
        k = (torch.randn(ks, generator=g, device=device, dtype=torch.float32) * w.sigma).to(torch.bfloat16)
        if w.k_mult != 1.0:
            k = k * w.k_mult
        v = (torch.randn(vs, generator=g, device=device, dtype=torch.float32) * w.sigma).to(torch.bfloat16)
        o = torch.empty(os_, device=device, dtype=torch.bfloat16)
        lse = torch.empty(os_[:3], device=device, dtype=torch.float32)
        sets.append((q.contiguous(), k.contiguous(), v.contiguous(), o, lse))
    return sets


def host_inputs(w):
    """(Q, K, V) bf16 bit patterns (uint16 numpy arrays) of the workload's shapes and distribution, drawn on the host
    with torch's seeded generator: the same recipe as workloads.make_inputs (i.i.d. N(0, sigma^2) rounded to bf16, K
    times k_mult) from a faster generator, for the timing legs, which need the distribution and not the very bits the
    parity tests are stored against."""
    import numpy as np
    import torch
    g = torch.Generator().manual_seed(w.seed)
    out = []
    for shape, mult in zip(w.shapes()[:3], (1.0, w.k_mult, 1.0)):
        x = torch.empty(shape, dtype=torch.bfloat16)
        flat = x.view(-1)
        step = 1 << 26
        for o in range(0, flat.numel(), step):
            n = min(step, flat.numel() - o)
            chunk = torch.randn(n, generator=g, dtype=torch.float32) * w.sigma
            flat[o:o + n] = chunk.to(torch.bfloat16)
        if mult != 1.0:
            x = x * mult
        out.append(x.view(torch.int16).numpy().view(np.uint16))
    return tuple(out)


def workload_numbers(w):
    fl_alg = metrics.flops_algorithmic(w.B, w.Hq, w.Sq, w.Sk, w.dqk, w.dv, w.causal)
    fl_pap = metrics.flops_paper(w.B, w.Hq, w.Sq, w.Sk, w.dqk, w.dv)
    nbytes = metrics.bytes_compulsory(w.B, w.Hq, w.Hkv, w.Sq, w.Sk, w.dqk, w.dv)
    return fl_alg, fl_pap, nbytes


def n_sets_for(w):
    _, _, nbytes = workload_numbers(w)
    return max(2, min(16, -(-2 * L2_BYTES // nbytes))) if nbytes < 2 * L2_BYTES else 1


def run_device_timed(binding, h, w, sets, steps, warmup, world, sampler=None):
    """Time `steps` launches (after `warmup`) with CUDA events on the launching stream; seconds."""
    import torch
    stream = torch.cuda.current_stream()

    def one(i):
        q, k, v, o, lse = sets[i % len(sets)]
        st = binding.fa_forward(h, q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(), lse.data_ptr(),
                                w.B, w.Hq, w.Hkv, w.Sq, w.Sk, w.dqk, w.dv, w.causal, w.scale,
                                stream.cuda_stream)
        if st != binding.FA_OK:
            raise binding.FaError(st, "fa_forward")

    for i in range(warmup):
        one(i)
    torch.cuda.synchronize()
    launch.barrier(world)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    n0 = binding.fa_launch_count(h)
    if sampler is not None:
        sampler.mark(0)
    e0.record(stream)
    for i in range(steps):
        one(warmup + i)
    e1.record(stream)
    torch.cuda.synchronize()
    if sampler is not None:
        sampler.mark(1)
    launch.barrier(world)
    st, detail = binding.fa_last_status(h)
    if st != binding.FA_OK:
        raise binding.FaError(st, "device status (site 0x%x)" % detail)
    return e0.elapsed_time(e1) * 1e-3, binding.fa_launch_count(h) - n0


def run_e2e_timed(binding, h, w, steps, warmup, world, host=None):
    """Same metric through fa_forward_host: pinned host buffers, copies inside the timed region."""
    import numpy as np
    import torch
    Q, K, V = host if host is not None else host_inputs(w)
    pin = [torch.from_numpy(a.view(np.int16)).pin_memory() for a in (Q, K, V)]
    o = torch.empty(w.shapes()[3], dtype=torch.int16).pin_memory()
    lse = torch.empty(w.shapes()[3][:3], dtype=torch.float32).pin_memory()
    stream = torch.cuda.current_stream()

    def one():
        st = binding.fa_forward_host(h, pin[0].data_ptr(), pin[1].data_ptr(), pin[2].data_ptr(), o.data_ptr(),
                                     lse.data_ptr(), w.B, w.Hq, w.Hkv, w.Sq, w.Sk, w.dqk, w.dv, w.causal,
                                     w.scale, stream.cuda_stream)
        if st != binding.FA_OK:
            raise binding.FaError(st, "fa_forward_host")

    for _ in range(max(1, warmup)):
        one()
    torch.cuda.synchronize()
    launch.barrier(world)
    t0 = time.perf_counter()
    for _ in range(steps):
        one()                       # synchronises the stream itself before returning
    torch.cuda.synchronize()
    dt = time.perf_counter() - t0
    launch.barrier(world)
    h2d = sum(int(t.numel()) * t.element_size() for t in pin)
    d2h = int(o.numel()) * 2 + int(lse.numel()) * 4
    return dt, h2d, d2h, float(lse.double().mean())


def oracle_timed(w, budget_s=20.0, host=None):
    """The fp64 oracle on the host cores over a bounded sample of query rows of the workload."""
    import numpy as np
    import oracle
    Q, K, V = host if host is not None else host_inputs(w)
    rng = np.random.default_rng(0)
    threads = oracle.num_threads()

    def rows_sample(n):
        return np.stack([rng.integers(w.B, size=n), rng.integers(w.Hq, size=n), rng.integers(w.Sq, size=n)],
                        axis=1).astype(np.int64)

    def pairs_of(rows):
        i = rows[:, 2]
        vis = np.minimum(w.Sk, np.maximum(0, i + (w.Sk - w.Sq) + 1)) if w.causal else np.full(len(i), w.Sk)
        return int(vis.sum())

    probe = rows_sample(64 * threads)
    t0 = time.perf_counter()
    oracle.attention(Q, K, V, causal=w.causal, scale=w.scale, rows=probe)
    dt = time.perf_counter() - t0
    rate = pairs_of(probe) / max(dt, 1e-6)                   # visible pairs per second
    total_pairs = w.B * w.Hq * metrics.visible_pairs(w.Sq, w.Sk, w.causal)
    if total_pairs / rate <= budget_s:
        t0 = time.perf_counter()
        oracle.attention(Q, K, V, causal=w.causal, scale=w.scale)
        dt = time.perf_counter() - t0
        pairs, sample = total_pairs, "whole workload (%d rows)" % (w.B * w.Hq * w.Sq)
    else:
        n = max(threads, int(budget_s * rate / (total_pairs / (w.B * w.Hq * w.Sq))))
        rows = rows_sample(n)
        t0 = time.perf_counter()
        oracle.attention(Q, K, V, causal=w.causal, scale=w.scale, rows=rows)
        dt = time.perf_counter() - t0
        pairs, sample = pairs_of(rows), ("%d random query rows of the workload; the rate over the whole workload is "
                                         "extrapolated from them (every row is an independent problem)" % n)
    flops = 2 * pairs * (w.dqk + w.dv)
    return {"value": flops / dt / 1e12, "unit": "TFLOP_GEMM/s", "cores": threads, "kind": "oracle",
            "sample": sample, "seconds": dt}


# Few queries over a long K/V sequence with grouped heads (B, Hq, Hkv, Sq, Sk, d): decoding.
DECODE_SHAPES = ((8, 32, 8, 1, 8192, 128), (64, 32, 8, 1, 4096, 128), (1, 32, 8, 16, 131072, 128), (4, 32, 8, 128, 8192, 128))


def time_libraries(binding, h, device, only=None):
    """Library attention kernels on the same GPU and shapes, for context: PyTorch's
    scaled_dot_product_attention with each of its fused back ends, and flash_attn where it is
    installed.  One input set per shape (the library kernels and ours see the same L2 state);
    a back end that refuses a shape is recorded with its message."""
    import torch
    import torch.nn.functional as F
    from torch.nn.attention import SDPBackend, sdpa_kernel
    try:
        from flash_attn import flash_attn_func
    except Exception:                                   # not installed, or no kernels for this GPU
        flash_attn_func = None

    def timed(f, k):
        for _ in range(3):
            f()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(k):
            f()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) * 1e-3 / k

    def one_shape(name, B, Hq, Hkv, Sq, Sk, dqk, dv, causal, scale, flops, kv_bytes):
        gen = torch.Generator(device=device).manual_seed(7)
        q = torch.randn((B, Hq, Sq, dqk), generator=gen, device=device).to(torch.bfloat16)
        k = torch.randn((B, Hkv, Sk, dqk), generator=gen, device=device).to(torch.bfloat16)
        v = torch.randn((B, Hkv, Sk, dv), generator=gen, device=device).to(torch.bfloat16)
        n = max(3, min(100, int(0.2 / max(flops / 0.5e15, kv_bytes / 3e12, 1e-5))))
        row = {"workload": name, "steps": n}

        def record(key, f):
            try:
                t = timed(f, n)
                row[key] = {"us": t * 1e6, "tflops_algorithmic": flops / t / 1e12, "kv_read_gbs": kv_bytes / t / 1e9}
            except Exception as e:                      # this back end has no kernel for the shape
                torch.cuda.synchronize()
                row[key] = {"error": str(e).splitlines()[0][:160]}

        record("ours", lambda: binding.forward(h, q, k, v, causal=causal, scale=scale))
        for key, be in (("torch_sdpa_cudnn", SDPBackend.CUDNN_ATTENTION), ("torch_sdpa_flash", SDPBackend.FLASH_ATTENTION),
                        ("torch_sdpa_efficient", SDPBackend.EFFICIENT_ATTENTION)):
            def f(be=be):
                with sdpa_kernel([be]):
                    return F.scaled_dot_product_attention(q, k, v, is_causal=causal, scale=scale, enable_gqa=(Hq != Hkv))
            record(key, f)
        if flash_attn_func is not None:
            qt, kt, vt = (x.transpose(1, 2).contiguous() for x in (q, k, v))      # [B, S, H, d]
            record("flash_attn", lambda: flash_attn_func(qt, kt, vt, softmax_scale=scale, causal=causal))
        return row

    rows = []
    if only is not None:            # a custom shape: that shape alone
        fa, _, _ = workload_numbers(only)
        return [one_shape(only.name, only.B, only.Hq, only.Hkv, only.Sq, only.Sk, only.dqk, only.dv, only.causal, only.scale, fa,
                          2 * only.B * only.Hkv * only.Sk * (only.dqk + only.dv))]
    for wc in workloads.CONFIGS:
        fa, _, _ = workload_numbers(wc)
        rows.append(one_shape(wc.name, wc.B, wc.Hq, wc.Hkv, wc.Sq, wc.Sk, wc.dqk, wc.dv, wc.causal, wc.scale, fa,
                              2 * wc.B * wc.Hkv * wc.Sk * (wc.dqk + wc.dv)))
        torch.cuda.empty_cache()
    for (B, Hq, Hkv, Sq, Sk, d) in DECODE_SHAPES:
        rows.append(one_shape("decode_b%d_h%d_%d_q%d_k%d_d%d" % (B, Hq, Hkv, Sq, Sk, d), B, Hq, Hkv, Sq, Sk, d, d, False,
                              d ** -0.5, 4.0 * B * Hq * Sq * Sk * d, 2 * B * Hkv * Sk * 2 * d))
        torch.cuda.empty_cache()
    return rows


def l2_note(w):
    n_sets = n_sets_for(w)
    _, _, nbytes = workload_numbers(w)
    return ("rotating %d input sets (%.0f MB in total, L2 is 126 MB)" % (n_sets, n_sets * nbytes / 1e6) if n_sets > 1 else
            "one input set of %.0f MB (larger than the 126 MB L2)" % (nbytes / 1e6))


def config_dict(w, world=1):
    """The workload as both arms print it (identical for the same workload and N)."""
    return {"workload": w.name, "B": w.B, "Hq": w.Hq, "Hkv": w.Hkv, "Sq": w.Sq, "Sk": w.Sk, "dqk": w.dqk,
            "dv": w.dv, "causal": w.causal, "scale": w.scale, "inputs": "bf16 N(0,1), seeded",
            "flop_convention": "value counts visible (i,j) pairs only; value_paper_convention counts Sq*Sk",
            "l2": l2_note(w), "parallelism": "replicas x%d, no collective" % world}


def per_launch_times(binding, h, w, sets, launches, warmup):
    """Duration of every one of `launches` launches after `warmup` (an event pair around each, on the launching
    stream; the handle launches the ordinary way, so consecutive launches do not overlap); seconds."""
    import torch
    stream = torch.cuda.current_stream()

    def one(i):
        q, k, v, o, lse = sets[i % len(sets)]
        st = binding.fa_forward(h, q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(), lse.data_ptr(),
                                w.B, w.Hq, w.Hkv, w.Sq, w.Sk, w.dqk, w.dv, w.causal, w.scale, stream.cuda_stream)
        if st != binding.FA_OK:
            raise binding.FaError(st, "fa_forward")

    for i in range(warmup):
        one(i)
    torch.cuda.synchronize()
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(launches)]
    for i, (e0, e1) in enumerate(ev):
        e0.record(stream)
        one(warmup + i)
        e1.record(stream)
    torch.cuda.synchronize()
    return sorted(e0.elapsed_time(e1) * 1e-3 for e0, e1 in ev)


def roofline_of(w, t_step, peaks, kernel):
    """Roofline record of one launch of `w` that takes t_step seconds: against the measured burst peak (a kernel timed
    alone) and the sustained one (a kernel inside a long, power-capped region); `frac` takes the one that applies."""
    fl_alg, _, nbytes = workload_numbers(w)
    t_tensor_burst = fl_alg / (peaks["bf16_tflops"] * 1e12)
    t_hbm = nbytes / (peaks["hbm_gbs"] * 1e9)
    bound = "tensor" if t_tensor_burst >= t_hbm else "hbm"
    traffic = NCU_DRAM_BYTES_PER_LAUNCH.get(w.name)
    r = {"bound": bound, "kernel": kernel, "avg_launch_us": t_step * 1e6, "traffic": traffic,
         "algorithmic_flops_per_launch": fl_alg, "compulsory_bytes_per_launch": nbytes,
         "frac_of_nominal_2250_tflops": fl_alg / t_step / 2.25e15}
    if bound == "tensor":
        ach = fl_alg / t_step / 1e12
        r.update({"achieved": ach, "unit": "TFLOP/s", "frac_burst": ach / peaks["bf16_tflops"],
                  "frac_sustained": ach / peaks["bf16_tflops_sustained"]})
    else:
        ach = nbytes / t_step / 1e9
        r.update({"achieved": ach, "unit": "GB/s", "frac_burst": ach / peaks["hbm_gbs"], "frac_sustained": ach / peaks["hbm_gbs"]})
    return r


def measure_config(binding, h, h_plain, w, device, peaks, gpu_index, steps=None, warmup=None, world=1):
    """Full record of one configuration: back-to-back mean over a timed region with its own clock samples, per-launch
    minimum and median (Section 5.1's protocol: 10 warm-ups, 20 timed launches), roofline fractions."""
    import torch
    fl_alg, fl_pap, nbytes = workload_numbers(w)
    sets = make_device_sets(w, n_sets_for(w), device)
    if steps is None:
        steps = max(20, min(2000, int(0.5 / max(fl_alg / 1.0e15, 1e-5))))
    if warmup is None:
        warmup = max(3, min(50, steps // 10))
    sampler = ClockSampler(gpu_index, period_s=0.002)
    sampler.start()
    sampler.wait_ready()
    seconds, launches = run_device_timed(binding, h, w, sets, steps, warmup, world, sampler)
    clocks = sampler.stop()
    seconds = launch.max_over_ranks(seconds, world, device)
    t = seconds / steps
    kernel = binding.fa_last_kernel_name(h)
    each = per_launch_times(binding, h_plain, w, sets, 20, 10)
    del sets
    torch.cuda.empty_cache()
    long_region = seconds > 0.25          # long enough for the power cap to set the clock
    roof = roofline_of(w, t, peaks, kernel)
    roof["frac"] = roof["frac_sustained"] if long_region else roof["frac_burst"]
    roof["peak"] = (peaks["bf16_tflops_sustained"] if long_region else peaks["bf16_tflops"]) if roof["bound"] == "tensor" else peaks["hbm_gbs"]
    roof["peak_source"] = "%s (%s: the timed region lasted %.2f s)" % (peaks["source"], "sustained" if long_region else "burst", seconds)
    rec = {"workload": w.name, "kernel": kernel, "steps": steps, "warmup": warmup, "us": t * 1e6,
           "tflops_algorithmic": fl_alg / t / 1e12, "tflops_paper_convention": fl_pap / t / 1e12,
           "per_launch_us_min": each[0] * 1e6, "per_launch_us_median": each[len(each) // 2] * 1e6,
           "per_launch_note": "20 launches after 10 warm-ups, an event pair around each, launched without programmatic "
                              "stream serialisation (no overlap between consecutive launches); 'us' is the mean of "
                              "back-to-back launches, whose tails overlap",
           "bound": roof["bound"], "frac_burst": roof["frac_burst"], "frac_sustained": roof["frac_sustained"],
           "frac_of_nominal_2250": fl_alg / t / 2.25e15,
           "dram_traffic_bytes_per_launch": roof["traffic"], "compulsory_bytes_per_launch": nbytes, "clocks": clocks,
           "us_x_sm_mhz": (t * 1e6 * clocks["sm_mhz"]) if clocks.get("sm_mhz") else None}
    return rec, roof, seconds, launches, steps, warmup


def run_reference(args, w, rank, world):
    """Reference arm: the CPU oracle, rank 0 only."""
    if rank != 0:
        return
    import numpy as np
    import oracle
    Q, K, V = host_inputs(w)
    threads = oracle.num_threads()
    rows_total = w.B * w.Hq * w.Sq
    rng = np.random.default_rng(0)
    # size one step so that steps+warmup steps end within ~2 minutes
    probe = np.stack([rng.integers(w.B, size=256), rng.integers(w.Hq, size=256), rng.integers(w.Sq, size=256)],
                     axis=1).astype(np.int64)
    t0 = time.perf_counter()
    oracle.attention(Q, K, V, causal=w.causal, scale=w.scale, rows=probe)
    per_row = (time.perf_counter() - t0) / 256
    budget_per_step = 120.0 / max(1, args.steps + args.warmup)
    n = int(min(rows_total, max(threads, budget_per_step / per_row)))
    whole = n >= rows_total
    rows = None if whole else np.stack([rng.integers(w.B, size=n), rng.integers(w.Hq, size=n),
                                        rng.integers(w.Sq, size=n)], axis=1).astype(np.int64)
    if whole:
        pairs = w.B * w.Hq * metrics.visible_pairs(w.Sq, w.Sk, w.causal)
    else:
        i = rows[:, 2]
        pairs = int((np.minimum(w.Sk, np.maximum(0, i + (w.Sk - w.Sq) + 1)) if w.causal
                     else np.full(n, w.Sk)).sum())
    for _ in range(args.warmup):
        oracle.attention(Q, K, V, causal=w.causal, scale=w.scale, rows=rows)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle.attention(Q, K, V, causal=w.causal, scale=w.scale, rows=rows)
    dt = time.perf_counter() - t0
    value = 2 * pairs * (w.dqk + w.dv) * args.steps / dt / 1e12
    sample = "whole workload" if whole else "%d random query rows per step" % n
    line = {"impl": "reference", "metric": "attention_fwd_tflop_gemm_per_s", "value": value,
            "unit": "TFLOP_GEMM/s", "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": dt / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": config_dict(w, max(1, args.gpus)),
            "cpu_baseline": {"value": value, "unit": "TFLOP_GEMM/s", "cores": threads, "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": value, "unit": "TFLOP_GEMM/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def plan_ab(binding, device, gpu_index):
    """The planner's choices against the alternatives it rejected, on the five configurations and on items of every
    length: every case with the library's own plan and with each kernel forced through the FA_FLAG_* overrides."""
    import torch
    variants = (("planned", 0), ("two_tiles_per_item", binding.FA_FLAG_NO_PERSISTENT | binding.FA_FLAG_NO_STREAM_KERNEL),
                ("persistent", binding.FA_FLAG_FORCE_PERSISTENT | binding.FA_FLAG_NO_STREAM_KERNEL),
                ("stream", binding.FA_FLAG_STREAM_KERNEL | binding.FA_FLAG_NO_PERSISTENT),
                ("stream_persistent", binding.FA_FLAG_STREAM_KERNEL | binding.FA_FLAG_FORCE_PERSISTENT),
                ("two_cta", binding.FA_FLAG_TWO_CTA_KERNEL),
                ("two_cta_four_tiles", binding.FA_FLAG_QUAD_KERNEL))
    handles = {name: binding.fa_create(device=device.index, flags=flags) for name, flags in variants}
    cases = list(workloads.CONFIGS)
    for (B, Hq, Hkv, S, causal) in ((64, 32, 8, 128, True), (32, 32, 8, 256, True), (16, 32, 8, 512, True), (8, 32, 8, 1024, True),
                                    (8, 32, 8, 2048, True), (4, 32, 8, 4096, True), (2, 32, 8, 16384, True), (4, 32, 8, 2048, False)):
        cases.append(workloads.Workload("b%d_h%d_%d_s%d_%s" % (B, Hq, Hkv, S, "causal" if causal else "full"), B, Hq, Hkv, S, S, 128, 128,
                                        causal, 128 ** -0.5))
    rows = []
    for w in cases:
        fl_alg, _, _ = workload_numbers(w)
        sets = make_device_sets(w, n_sets_for(w), device)
        k = max(5, min(300, int(0.3 / max(fl_alg / 1.0e15, 1e-5))))
        row = {"workload": w.name}
        for name, h in handles.items():
            try:
                sec, _ = run_device_timed(binding, h, w, sets, k, 3, 1)
                row[name] = {"us": sec / k * 1e6, "tflops_algorithmic": fl_alg / (sec / k) / 1e12, "kernel": binding.fa_last_kernel_name(h)}
            except binding.FaError as e:
                row[name] = {"error": str(e)}
        timed = {n: r["us"] for n, r in row.items() if isinstance(r, dict) and "us" in r and n != "planned"}
        row["best"] = min(timed, key=timed.get) if timed else None
        row["planned_over_best"] = row["planned"]["us"] / min(timed.values()) if timed and "us" in row["planned"] else None
        rows.append(row)
        del sets
        torch.cuda.empty_cache()
    for h in handles.values():
        binding.fa_destroy(h)
    return rows


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--config", type=int, default=4,
                    help="index into the five benchmark configurations (default: the largest, 128K tokens)")
    ap.add_argument("--shape", default=None,
                    help="time a custom shape instead of --config, e.g. "
                         "B=1,Hq=16,Hkv=16,S=8192,dqk=128,dv=128,causal=1 (used for small ncu captures)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-sweep", action="store_true", help="skip the records of the other configurations (key 'per_config')")
    ap.add_argument("--table6", action="store_true",
                    help="also time the twelve attention shapes of the paper's Table 6 (key 'table6')")
    ap.add_argument("--eight-bit", action="store_true",
                    help="time the 8-bit variants on the workload (keys 'block_scaled_e4m3', 'mx_e4m3') even with --no-sweep")
    ap.add_argument("--no-decode", action="store_true", help="skip the grouped-head decode step and the packed batches (keys 'decode', 'packed_batches')")
    ap.add_argument("--plan-ab", action="store_true",
                    help="also time every configuration, and items of every length, with each kernel forced, next to the "
                         "library's own choice (key 'plan_ab')")
    ap.add_argument("--libraries", action="store_true",
                    help="also time the attention kernels of the libraries in the image (torch SDPA back ends, flash_attn) "
                         "on the five configurations and a few decode shapes, for context (key 'libraries')")
    ap.add_argument("--flags", type=int, default=0,
                    help="fa_config.flags of the handle that runs the workload (FA_FLAG_* bits, e.g. 1024 for the kernel with "
                         "four query tiles per pair of SMs); for A/B timing and ncu captures of a kernel the planner does not pick")
    args = ap.parse_args()
    w = workloads.config(args.config)
    if args.shape:
        kv = dict(item.split("=") for item in args.shape.split(","))
        S = int(kv.get("S", 2048))
        dqk = int(kv.get("dqk", 128))
        w = workloads.Workload("custom_" + args.shape.replace(",", "_").replace("=", ""), int(kv.get("B", 1)),
                               int(kv.get("Hq", 16)), int(kv.get("Hkv", kv.get("Hq", 16))),
                               int(kv.get("Sq", S)), int(kv.get("Sk", S)), dqk, int(kv.get("dv", dqk)),
                               bool(int(kv.get("causal", 1))), dqk ** -0.5)

    if args.impl == "reference":
        rank, world, _ = launch.env_rank()
        args.steps = args.steps if args.steps is not None else 3
        args.warmup = args.warmup if args.warmup is not None else 1
        run_reference(args, w, rank, world)
        return

    import torch
    from paper_2609_21264_b200 import binding

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    rank, world, local = launch.init_process_group("nccl")
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    if world != args.gpus and rank == 0:
        print("warning: --gpus %d but WORLD_SIZE=%d" % (args.gpus, world), file=sys.stderr)

    fl_alg, fl_pap, nbytes = workload_numbers(w)
    default_steps = max(20, min(2000, int(0.25 / max(fl_alg / 1.0e15, 1e-5))))
    steps = args.steps if args.steps is not None else default_steps
    warmup = args.warmup if args.warmup is not None else max(3, min(50, steps // 10))
    warmup = max(3, warmup)

    gpu_index = physical_gpu_index(local)
    peaks = load_peaks()
    h = binding.fa_create(device=local, flags=args.flags)
    h_plain = binding.fa_create(device=local, flags=args.flags | binding.FA_FLAG_NO_DEPENDENT_LAUNCH)
    rec, roofline, seconds, launches, steps, warmup = measure_config(binding, h, h_plain, w, device, peaks, gpu_index, steps, warmup, world)
    t_step = seconds / steps
    clocks = rec["clocks"]

    value = world * fl_alg / t_step / 1e12
    line = {"metric": "attention_fwd_tflop_gemm_per_s", "value": value, "unit": "TFLOP_GEMM/s",
            "n_gpus": world, "steps": steps, "warmup": warmup, "ms_per_step": t_step * 1e3,
            "higher_is_better": True, "scaling": "weak",
            "vs_baseline": (PAPER_SECONDS[w.name] / t_step if (w.name in PAPER_SECONDS and world == 1) else None),
            "dtype": "bf16", "data": "synthetic",
            "config": config_dict(w, world),
            "value_paper_convention": world * fl_pap / t_step / 1e12,
            "paper_context": "3.62 TFLOP_GEMM/s on XDNA 2 (paper's headline, other hardware and shape)",
            "per_launch_us_min": rec["per_launch_us_min"], "per_launch_us_median": rec["per_launch_us_median"],
            "roofline": roofline, "clocks": clocks, "gpu_launches": int(launches)}
    if args.flags:
        line["config"]["handle_flags"] = args.flags

    if (args.eight_bit or not args.no_sweep) and world == 1 and w.dqk == 128 and w.dv == 128:
        # the block-scaled e4m3 variant on the same shape (N(0, sigma^2) rounded to e4m3, unit scales), for context
        gen = torch.Generator(device=device).manual_seed(w.seed)
        q8, k8, v8 = (torch.randn(shape, generator=gen, device=device).mul_(w.sigma).to(torch.float8_e4m3fn).view(torch.uint8)
                      for shape in w.shapes()[:3])
        o8 = torch.empty((w.B, w.Hq, w.Sq, 128), dtype=torch.bfloat16, device=device)
        l8 = torch.empty((w.B, w.Hq, w.Sq), dtype=torch.float32, device=device)
        k = max(5, min(200, int(0.3 / max(fl_alg / 1.0e15, 1e-5))))
        cs = torch.cuda.current_stream().cuda_stream

        def one8():
            st8 = binding.fa_forward_fp8(h, q8.data_ptr(), k8.data_ptr(), v8.data_ptr(), None, None, None, o8.data_ptr(),
                                         l8.data_ptr(), w.B, w.Hq, w.Hkv, w.Sq, w.Sk, 128, w.causal, w.scale, cs)
            if st8 != binding.FA_OK:
                raise binding.FaError(st8, "fa_forward_fp8")

        for _ in range(3):
            one8()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(k):
            one8()
        e1.record()
        torch.cuda.synchronize()
        t8 = e0.elapsed_time(e1) * 1e-3 / k
        line["block_scaled_e4m3"] = {"workload": w.name, "us": t8 * 1e6, "tflops_algorithmic": fl_alg / t8 / 1e12,
                                     "speedup_over_bf16": t_step / t8, "steps": k, "kernel": binding.fa_last_kernel_name(h),
                                     "note": "fa_forward_fp8, N(0,sigma^2) rounded to e4m3, unit scales, one input set"}
        # the MX form of the same operands (e8m0 scales per 32 elements inside the MMA; unit scale atoms here)
        n_qt, n_kt = (w.Sq + 127) // 128, (w.Sk + 127) // 128
        qa = torch.full((w.B, w.Hq, n_qt, 512), 127, dtype=torch.uint8, device=device)
        ka = torch.full((w.B, w.Hkv, n_kt, 512), 127, dtype=torch.uint8, device=device)

        def one_mx():
            stx = binding.fa_forward_mxfp8(h, q8.data_ptr(), k8.data_ptr(), v8.data_ptr(), qa.data_ptr(), ka.data_ptr(), ka.data_ptr(),
                                           o8.data_ptr(), l8.data_ptr(), w.B, w.Hq, w.Hkv, w.Sq, w.Sk, 128, w.causal, w.scale, cs)
            if stx != binding.FA_OK:
                raise binding.FaError(stx, "fa_forward_mxfp8")

        for _ in range(3):
            one_mx()
        torch.cuda.synchronize()
        e0.record()
        for _ in range(k):
            one_mx()
        e1.record()
        torch.cuda.synchronize()
        tx = e0.elapsed_time(e1) * 1e-3 / k
        line["mx_e4m3"] = {"workload": w.name, "us": tx * 1e6, "tflops_algorithmic": fl_alg / tx / 1e12,
                           "speedup_over_bf16": t_step / tx, "steps": k, "kernel": binding.fa_last_kernel_name(h),
                           "note": "fa_forward_mxfp8, the same codes with unit e8m0 scale atoms"}
        del qa, ka
        del q8, k8, v8, o8, l8

    if not args.no_decode and world == 1:
        # Decoding with grouped heads (few queries over a long K/V sequence): bound by the K/V read, so the
        # figure of merit is bytes per second against the measured copy bandwidth.  bf16 and e4m3 K/V.
        dB, dHq, dHkv, dSq, dSk = 64, 32, 8, 1, 4096
        gen = torch.Generator(device=device).manual_seed(11)
        qd = torch.randn((dB, dHq, dSq, 128), generator=gen, device=device).to(torch.bfloat16)
        kd = torch.randn((dB, dHkv, dSk, 128), generator=gen, device=device).to(torch.bfloat16)
        vd = torch.randn((dB, dHkv, dSk, 128), generator=gen, device=device).to(torch.bfloat16)
        od = torch.empty_like(qd)
        ld = torch.empty((dB, dHq, dSq), dtype=torch.float32, device=device)
        cs = torch.cuda.current_stream().cuda_stream

        def timed_launches(f, k=20):
            for _ in range(3):
                f()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(k):
                f()
            e1.record()
            torch.cuda.synchronize()
            return e0.elapsed_time(e1) * 1e-3 / k

        def dec16():
            st = binding.fa_forward(h, qd.data_ptr(), kd.data_ptr(), vd.data_ptr(), od.data_ptr(), ld.data_ptr(),
                                    dB, dHq, dHkv, dSq, dSk, 128, 128, False, 0.0, cs)
            if st != binding.FA_OK:
                raise binding.FaError(st, "fa_forward")

        t16 = timed_launches(dec16)
        plan = binding.fa_plan(torch.cuda.get_device_properties(device).multi_processor_count, dB, dHq, dHkv, dSq, dSk, 128, 128, False)
        bytes16 = 2 * (2 * dB * dHkv * dSk * 128 + 2 * dB * dHq * dSq * 128) + 4 * dB * dHq * dSq
        q8, k8, v8 = (x.to(torch.float8_e4m3fn).view(torch.uint8) for x in (qd, kd, vd))

        def dec8():
            st = binding.fa_forward_fp8(h, q8.data_ptr(), k8.data_ptr(), v8.data_ptr(), None, None, None, od.data_ptr(),
                                        ld.data_ptr(), dB, dHq, dHkv, dSq, dSk, 128, False, 0.0, cs)
            if st != binding.FA_OK:
                raise binding.FaError(st, "fa_forward_fp8")

        t8 = timed_launches(dec8)
        bytes8 = 2 * dB * dHkv * dSk * 128 + dB * dHq * dSq * 128 * 3 + 4 * dB * dHq * dSq
        line["decode"] = {"workload": "B=%d Hq=%d Hkv=%d Sq=%d Sk=%d d=128 non-causal" % (dB, dHq, dHkv, dSq, dSk),
                          "heads_per_tile": plan["heads_per_tile"], "kv_splits": plan["kv_splits"],
                          "bf16": {"us": t16 * 1e6, "compulsory_bytes": bytes16, "gbs": bytes16 / t16 / 1e9,
                                   "frac_of_measured_hbm": bytes16 / t16 / 1e9 / peaks["hbm_gbs"]},
                          "e4m3": {"us": t8 * 1e6, "compulsory_bytes": bytes8, "gbs": bytes8 / t8 / 1e9,
                                   "frac_of_measured_hbm": bytes8 / t8 / 1e9 / peaks["hbm_gbs"]},
                          "note": "inputs larger than L2 (1.07 GB / 0.54 GB of K and V); 20 launches each after 3 warm-up launches"}
        del qd, kd, vd, od, ld, q8, k8, v8
        torch.cuda.empty_cache()

        # Packed batches of sequences of different lengths (fa_forward_varlen; Hq 32 / Hkv 8, d 128, causal):
        # one batch of equal sequences (comparable with the fixed-length call) and one of mixed lengths.
        import numpy as np
        packed = []
        for pname, lens in (("8 x 2048 tokens", [2048] * 8),
                            ("64 sequences of 64..2048 tokens", [int(x) for x in np.random.RandomState(5).randint(64, 2049, 64)])):
            tq = int(sum(lens))
            qp = torch.randn((tq, 32, 128), generator=gen, device=device).to(torch.bfloat16)
            kp = torch.randn((tq, 8, 128), generator=gen, device=device).to(torch.bfloat16)
            vp = torch.randn((tq, 8, 128), generator=gen, device=device).to(torch.bfloat16)
            op = torch.empty_like(qp)
            lp = torch.empty((32, tq), dtype=torch.float32, device=device)
            cu = torch.tensor(np.concatenate([[0], np.cumsum(lens)]), dtype=torch.int32, device=device)

            def packed_call():
                st = binding.fa_forward_varlen(h, qp.data_ptr(), kp.data_ptr(), vp.data_ptr(), op.data_ptr(), lp.data_ptr(),
                                               cu.data_ptr(), cu.data_ptr(), len(lens), tq, tq, max(lens), 32, 8, 128, 128,
                                               True, 0.0, cs)
                if st != binding.FA_OK:
                    raise binding.FaError(st, "fa_forward_varlen")

            tp = timed_launches(packed_call)
            flp = 4.0 * 128 * 32 * sum(l * (l + 1) // 2 for l in lens)
            packed.append({"workload": pname, "total_tokens": tq, "us": tp * 1e6, "tflops_algorithmic": flp / tp / 1e12,
                           "kernel": binding.fa_last_kernel_name(h)})
            del qp, kp, vp, op, lp, cu
        line["packed_batches"] = {"cases": packed, "note": "Hq 32 / Hkv 8, d 128, causal, lengths on the device; "
                                  "20 launches each after 3 warm-up launches"}
        torch.cuda.empty_cache()

    host = None
    if (not args.no_e2e) or (rank == 0 and world == 1 and not args.no_cpu_baseline):
        host = host_inputs(w)
    if not args.no_e2e:
        e2e_steps = max(3, min(steps, 50, int(4.0 / max(t_step * 3, 1e-4)) + 3))
        dt, h2d, d2h, _ = run_e2e_timed(binding, h, w, e2e_steps, 3 if t_step < 0.05 else 1, world, host)
        dt = launch.max_over_ranks(dt, world, device)
        line["e2e"] = {"value": world * fl_alg * e2e_steps / dt / 1e12, "unit": "TFLOP_GEMM/s",
                       "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": e2e_steps,
                       "ms_per_step": dt / e2e_steps * 1e3,
                       "api": "fa_forward_host: pinned host buffers, both copies inside the timed region"}

    if not args.no_sweep and world == 1:
        per = []
        for idx, wc in enumerate(workloads.CONFIGS):
            if wc.name == w.name:
                r = dict(rec)
            else:
                r, _, _, _, _, _ = measure_config(binding, h, h_plain, wc, device, peaks, gpu_index)
            r["config"] = idx
            per.append(r)
        line["per_config"] = per

    if args.plan_ab and world == 1:
        line["plan_ab"] = plan_ab(binding, device, gpu_index)

    if args.table6 and world == 1:
        rows = []
        for wc, paper_us in workloads.TABLE6:
            fa, fp, nb = workload_numbers(wc)
            ss = make_device_sets(wc, n_sets_for(wc), device)
            k = max(3, min(200, int(0.3 / max(fa / 1.0e15, 1e-5))))
            sec, _ = run_device_timed(binding, h, wc, ss, k, 3, 1)
            t = sec / k
            rows.append({"workload": wc.name, "us": t * 1e6, "tflops_paper_convention": fp / t / 1e12,
                         "tflops_algorithmic": fa / t / 1e12, "paper_xdna2_us": paper_us,
                         "paper_xdna2_tflops": fp / (paper_us * 1e-6) / 1e12})
            del ss
            torch.cuda.empty_cache()
        line["table6"] = rows

    if args.libraries and world == 1:
        line["libraries"] = time_libraries(binding, h, device, only=w if args.shape else None)

    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        line["cpu_baseline"] = oracle_timed(w, host=host)

    binding.fa_destroy(h)
    binding.fa_destroy(h_plain)
    if rank == 0:
        print(json.dumps(line), flush=True)
    launch.destroy(world)


if __name__ == "__main__":
    main()
