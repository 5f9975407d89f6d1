#!/usr/bin/env python
"""Benchmark of the DiffQKV decode path on B200: KV-cache GB/s and fraction of the HBM roofline.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--quick]

Headline workload: long-context DiffQKV decode (batch 4, 32/4/8 heads, d 128, 32768 cached tokens,
bf16).  One step = one ``diffqkv_decode`` call (split kernel + combine kernel) over the whole batch.
The line printed by rank 0 also carries the GQA twin (n_k = n_v), the other decode configurations,
the roofline of the split kernel and the CPU oracle timed on the host cores.

The timed region is exactly ``--steps`` steps between barriers; when that is shorter than 50 ms it is repeated as
separate groups and the median group is reported (minimum and maximum beside it).  The last key of the line,
``summary``, repeats the headline figures of every configuration in short form.

With N > 1 every rank runs the same workload on its own GPU (the path has no exchange step:
replicas only), the timed region is bracketed by barriers and the slowest rank's time is used.
``--impl reference`` times the float64 CPU oracle instead (rank 0 only).
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

METRIC = "decode_kv_cache_bandwidth"
UNIT = "GB/s"
L2_BYTES = 126 * 1024 * 1024


def split_kernel_dram_bytes():
    """dram__bytes_read.sum + dram__bytes_write.sum of one launch of the split kernel on the headline workload, as
    recorded (with a hash of the kernel's source) when the counters were last taken; None once the kernel's source
    no longer matches that hash, so that a stale figure is never printed."""
    import hashlib
    rec = os.path.join(ROOT, "profiles", "decode_tma_kernel_cfg3.json")
    src = os.path.join(ROOT, "paper_2501_13629_b200", "csrc", "decode_tma.cu")
    try:
        with open(rec) as f:
            d = json.load(f)
        with open(src, "rb") as f:
            h = hashlib.sha256(f.read()).hexdigest()
        return float(d["dram_bytes_per_launch"]) if d.get("source_sha256") == h else None
    except Exception:
        return None


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d["bf16_tflops"]),
                "bf16_tflops_sustained": float(d.get("bf16_tflops_sustained", d["bf16_tflops"])),
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


def kv_bytes(cfg, seqlens) -> float:
    """Algorithmic bytes of one decode step: every cached K and V element once."""
    return float(np.sum(seqlens.astype(np.int64))) * (cfg.n_k * cfg.d_qk + cfg.n_v * cfg.d_v) * \
        (2 if cfg.dtype == "bf16" else 4)


class ClockSampler:
    """Polls SM clock and throttle reasons through NVML (read-only) while the timed region runs."""

    def __init__(self, index: int):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self._nv = pynvml
            self._h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self._nv = None

    def _run(self):
        nv = self._nv
        names = {
            "hw_slowdown": getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8),
            "hw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40),
            "sw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20),
            "sw_power_cap": getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4),
        }
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM)))
                try:
                    mask = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self._h))
                except Exception:
                    mask = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._h))
                for k, bit in names.items():
                    if mask & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            self._stop.wait(0.01)

    def __enter__(self):
        if self._nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": 0}
        return {"sm_mhz": float(np.median(self.samples)), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


# ----------------------------------------------------------------------------- GPU arm
class DecodeCase:
    """One decode workload resident on the device, with `rotate` distinct copies of the cache so that
    consecutive steps never find their cache lines in L2."""

    def __init__(self, api, cfg, device, host_inputs=None, rotate=None):
        import torch
        from paper_2501_13629_b200 import workloads as W
        self.api, self.cfg, self.torch = api, cfg, torch
        if host_inputs is not None:
            inp = host_inputs
            self.seqlens_host = inp.seqlens
            k, v = W.to_torch(inp.k, device), W.to_torch(inp.v, device)
            q = W.to_torch(inp.q, device)
            pt = None if inp.page_table is None else torch.from_numpy(inp.page_table).to(device)
            num_blocks = inp.num_pages if pt is not None else cfg.batch
            max_seqlen, ks, vs = inp.max_seqlen, inp.k_strides, inp.v_strides
        else:  # large pools: same recipe (i.i.d. N(0,1) rounded to the storage type), drawn on the device
            dt = torch.bfloat16 if cfg.dtype == "bf16" else torch.float32
            g = torch.Generator(device=device)
            g.manual_seed(cfg.seed)
            self.seqlens_host = W.draw_lengths(cfg)
            q = torch.randn((cfg.batch, cfg.n_q, cfg.d_qk), generator=g, device=device).to(dt)
            if cfg.page_size:
                table, num_blocks = W.shuffled_page_table(self.seqlens_host, cfg.page_size, cfg.seed)
                pt = torch.from_numpy(table).to(device)
                k = torch.empty((num_blocks, cfg.n_k, cfg.page_size, cfg.d_qk), dtype=dt, device=device)
                v = torch.empty((num_blocks, cfg.n_v, cfg.page_size, cfg.d_v), dtype=dt, device=device)
                max_seqlen = int(table.shape[1]) * cfg.page_size
            else:
                pt, num_blocks, max_seqlen = None, cfg.batch, cfg.kv_len
                k = torch.empty((cfg.batch, cfg.n_k, cfg.kv_len, cfg.d_qk), dtype=dt, device=device)
                v = torch.empty((cfg.batch, cfg.n_v, cfg.kv_len, cfg.d_v), dtype=dt, device=device)
            for t in (k, v):  # fill in slices to bound temporary memory
                flat = t.view(-1)
                step = 1 << 28
                for lo in range(0, flat.numel(), step):
                    n = min(step, flat.numel() - lo)
                    flat[lo:lo + n] = torch.randn(n, generator=g, device=device).to(dt)
            ks = (k.stride(0), k.stride(1), k.stride(2))
            vs = (v.stride(0), v.stride(1), v.stride(2))
        self.bytes = kv_bytes(cfg, self.seqlens_host)
        pool_bytes = (k.numel() + v.numel()) * k.element_size()
        if rotate is None:
            rotate = 1 if pool_bytes > 4 * L2_BYTES else min(64, int(np.ceil(4 * L2_BYTES / pool_bytes)))
        self.rotate = rotate
        seqlens = torch.from_numpy(self.seqlens_host).to(device)
        self.caches = []
        for r in range(rotate):
            kk, vv = (k, v) if r == 0 else (k.clone(), v.clone())
            self.caches.append(api.KVCache(kk, vv, seqlens, int(max_seqlen), page_table=pt,
                                           page_size=cfg.page_size, k_strides=ks, v_strides=vs,
                                           num_blocks=num_blocks))
        self.q = q
        out_dt = torch.bfloat16 if cfg.dtype == "bf16" else torch.float32
        self.shape = api.make_shape(cfg.batch, cfg.n_q, cfg.n_k, cfg.n_v, cfg.d_qk, cfg.d_v, q.dtype, out_dt, cfg.scale)
        nbytes = api.diffqkv_decode_workspace_bytes(self.shape, int(max_seqlen), 0)
        self.workspace = torch.empty(max(nbytes, 256), dtype=torch.uint8, device=device)
        self.out = torch.empty((cfg.batch, cfg.n_q, cfg.d_v), dtype=out_dt, device=device)
        self.status = torch.zeros(1, dtype=torch.int32, device=device)
        self.working_set = pool_bytes * rotate
        self._i = 0
        # the library call per cache copy with its argument structs built once, as a C caller keeps them: a step of
        # 15-25 us would otherwise be bounded by the Python marshalling (14-16 us per call), not by the GPU
        self.calls = [api.bind_decode(self.q, c, cfg.n_k, cfg.n_v, cfg.scale, self.workspace, self.out,
                                      dev_status=self.status, gqa=cfg.n_k == cfg.n_v) for c in self.caches]

    def step(self, q=None, out=None):
        cfg = self.cfg
        if q is None and out is None:
            self.calls[self._i % self.rotate]()
            self._i += 1
            return
        cache = self.caches[self._i % self.rotate]
        self._i += 1
        fn = self.api.gqa_decode if cfg.n_k == cfg.n_v else None
        if fn is not None:
            fn(self.q if q is None else q, cache, cfg.n_k, cfg.scale, workspace=self.workspace,
               out=self.out if out is None else out, dev_status=self.status)
        else:
            self.api.diffqkv_decode(self.q if q is None else q, cache, cfg.n_k, cfg.n_v, cfg.scale,
                                    workspace=self.workspace, out=self.out if out is None else out,
                                    dev_status=self.status)

    def time_steps(self, steps, warmup, barrier=None):
        """Device time of `steps` consecutive steps, in ms (CUDA events on the launching stream)."""
        torch = self.torch
        for _ in range(warmup):
            self.step()
        torch.cuda.synchronize()
        if barrier:
            barrier()
        start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        start.record()
        for _ in range(steps):
            self.step()
        end.record()
        torch.cuda.synchronize()
        if barrier:
            barrier()
        return start.elapsed_time(end)

    def time_groups(self, steps, warmup, barrier=None, reduce_max=None, min_total_ms=50.0, max_groups=25):
        """Groups of exactly `steps` steps, each bracketed like time_steps (warm-up before the first only).  One group
        when it lasts min_total_ms or more; otherwise as many as make up that time (at most max_groups), so that a
        short timed region is not one sample.  Every group time is the slowest rank's (`reduce_max`)."""
        reduce_max = reduce_max or (lambda x: x)
        first = reduce_max(self.time_steps(steps, warmup, barrier))
        n = 1 if first >= min_total_ms else int(min(max_groups, np.ceil(min_total_ms / max(first, 1e-6))))
        return [first] + [reduce_max(self.time_steps(steps, 0, barrier)) for _ in range(n - 1)]

    def launches_per_step(self):
        """Kernels the library launches for one step (2: split + combine; 1: the rows are merged on chip)."""
        n0 = self.api.launch_count()
        self.step()
        self.torch.cuda.synchronize()
        return self.api.launch_count() - n0

    def time_split_and_combine(self, steps):
        """Mean durations of the split kernel and of the combine kernel, each timed alone: the library records an
        event before and after the split kernel, a third event follows the call.  The events between the two
        kernels keep them from overlapping, so the two figures add up to more than an untimed step."""
        torch, api = self.torch, self.api
        trip = [tuple(torch.cuda.Event(enable_timing=True) for _ in range(3)) for _ in range(steps)]
        for t in trip:
            for e in t:
                e.record()  # creates the underlying CUDA events
        torch.cuda.synchronize()
        for a, b, c in trip:
            api.set_split_events(a, b)
            self.step()
            c.record()
        api.set_split_events(None, None)
        torch.cuda.synchronize()
        return (float(np.mean([a.elapsed_time(b) for a, b, _ in trip])),
                float(np.mean([b.elapsed_time(c) for _, b, c in trip])))

    def time_split_kernel(self, steps):
        """Average duration of the split kernel alone: the library records an event pair around it."""
        torch, api = self.torch, self.api
        pairs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        for a, b in pairs:
            a.record()  # creates the underlying CUDA events
            b.record()
        torch.cuda.synchronize()
        for a, b in pairs:
            api.set_split_events(a, b)
            self.step()
        api.set_split_events(None, None)
        torch.cuda.synchronize()
        return float(np.mean([a.elapsed_time(b) for a, b in pairs]))

    def time_e2e(self, steps, warmup):
        """Same step through the C-ABI call that takes HOST buffers (diffqkv_decode_host): pinned q copied to the
        device and the output copied back inside the timed region, which ends with a stream synchronisation every
        step (the KV cache is decode state and stays resident)."""
        torch = self.torch
        q_host = self.q.cpu().pin_memory()
        out_host = torch.empty(self.out.shape, dtype=self.out.dtype).pin_memory()
        q_dev = torch.empty_like(self.q)
        cfg = self.cfg
        # one library call with host buffers per step: copy q in, split + combine kernels, copy the output back;
        # the argument structs are built once per cache copy, as a C caller would keep them
        calls = [self.api.bind_decode_host(q_host, q_dev, cache, cfg.n_k, cfg.n_v, cfg.scale, self.workspace, self.out,
                                           out_host, dev_status=self.status) for cache in self.caches]
        stream = torch.cuda.current_stream()
        for i in range(warmup + steps):
            if i == warmup:
                torch.cuda.synchronize()
                t0 = time.perf_counter()
            calls[i % self.rotate]()
            stream.synchronize()
        dt = time.perf_counter() - t0
        return dt * 1e3, q_host.numel() * q_host.element_size(), out_host.numel() * out_host.element_size()


def time_prefill(api, W, device, peaks, steps):
    """Config 4 (batch 2 x 8192 tokens, 32/4/8 heads, d 128, hidden 2048): the augmented-Q projection and the causal
    prefill (cache update + attention), each timed with CUDA events.  Inputs are drawn on the device with the
    recipe of the host generator (hidden N(0, 0.02), weights N(0, 1/fan_in), K and V N(0,1), all bf16)."""
    import torch
    cfg = W.CFG4
    T, d_q0 = cfg.batch * cfg.seq, cfg.n_q * cfg.d_qk
    g = torch.Generator(device=device)
    g.manual_seed(cfg.seed)

    def rn(*shape, std=1.0):
        return (torch.randn(shape, generator=g, device=device) * std).to(torch.bfloat16)

    h = rn(T, cfg.d_model, std=cfg.h_std)
    w_q = rn(d_q0, cfg.d_model, std=cfg.d_model ** -0.5)
    w_g, w_u = rn(cfg.d_aug, d_q0, std=d_q0 ** -0.5), rn(cfg.d_aug, d_q0, std=d_q0 ** -0.5)
    w_d = rn(d_q0, cfg.d_aug, std=cfg.d_aug ** -0.5)
    ws = torch.empty(api.diffqkv_augq_workspace_bytes(T, d_q0, cfg.d_aug), dtype=torch.uint8, device=device)
    q = torch.empty(T, d_q0, dtype=torch.bfloat16, device=device)
    status = torch.zeros(1, dtype=torch.int32, device=device)
    k_new = rn(cfg.batch, cfg.seq, cfg.n_k, cfg.d_qk)
    v_new = rn(cfg.batch, cfg.seq, cfg.n_v, cfg.d_v)
    k = torch.zeros(cfg.batch, cfg.n_k, cfg.seq, cfg.d_qk, dtype=torch.bfloat16, device=device)
    v = torch.zeros(cfg.batch, cfg.n_v, cfg.seq, cfg.d_v, dtype=torch.bfloat16, device=device)
    cache = api.KVCache(k, v, torch.zeros(cfg.batch, dtype=torch.int32, device=device), cfg.seq)
    out = torch.empty(cfg.batch, cfg.seq, cfg.n_q, cfg.d_v, dtype=torch.bfloat16, device=device)
    q4 = q.view(cfg.batch, cfg.seq, cfg.n_q, cfg.d_qk)

    groups = {}

    def timed(fn, name=None):
        """Mean time of `steps` back-to-back calls, the fastest of three such groups, each after a short idle (the
        dense kernels run into the power cap within tens of milliseconds, and what a group gets depends on what ran
        before it); all three are kept under `groups`."""
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        means = []
        for _ in range(3):
            time.sleep(0.3)  # let the power-averaging window drain: each group is a burst measurement
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            for _ in range(steps):
                fn()
            b.record()
            torch.cuda.synchronize()
            means.append(a.elapsed_time(b) / steps)
        if name:
            groups[name] = means
        return min(means)

    with ClockSampler(device.index or 0) as ck_a:
        augq_ms = timed(lambda: api.diffqkv_augq(h, w_q, w_g, w_u, w_d, workspace=ws, q_out=q, dev_status=status), "augq")
    with ClockSampler(device.index or 0) as ck_p:
        attn_ms = timed(lambda: api.diffqkv_prefill(q4, k_new, v_new, cache, cfg.scale, out=out, dev_status=status),
                        "attention")
    assert int(status.item()) == 0, "device status reported an error"
    # the projections around it in the listing: k = rope(h W_K^T), v = h W_V^T (rotary tables for positions 0 .. seq - 1)
    w_k = rn(cfg.n_k * cfg.d_qk, cfg.d_model, std=cfg.d_model ** -0.5)
    w_v = rn(cfg.n_v * cfg.d_v, cfg.d_model, std=cfg.d_model ** -0.5)
    pos = torch.arange(cfg.seq, device=device, dtype=torch.float64).repeat(cfg.batch)
    inv = torch.pow(torch.tensor(50000.0, dtype=torch.float64, device=device),
                    -2.0 * torch.arange(cfg.d_qk // 2, device=device, dtype=torch.float64) / cfg.d_qk)
    ang = pos[:, None] * inv[None, :]
    cos, sin = torch.cos(ang).float().contiguous(), torch.sin(ang).float().contiguous()
    k_out = torch.empty(T, cfg.n_k * cfg.d_qk, dtype=torch.bfloat16, device=device)
    v_out = torch.empty(T, cfg.n_v * cfg.d_v, dtype=torch.bfloat16, device=device)

    def kv_proj():
        api.diffqkv_project(h, w_k, cfg.d_qk, cos, sin, out=k_out, dev_status=status)
        api.diffqkv_project(h, w_v, out=v_out, dev_status=status)

    kv_ms = timed(kv_proj)
    augq_rope_ms = timed(lambda: api.diffqkv_augq_rope(h, w_q, w_g, w_u, w_d, cfg.d_qk, cos, sin, workspace=ws, q_out=q,
                                                       dev_status=status))
    augq_flops = 2.0 * T * (cfg.d_model * d_q0 + 2 * d_q0 * cfg.d_aug + cfg.d_aug * d_q0)
    attn_flops = 2.0 * cfg.batch * cfg.n_q * (cfg.seq * (cfg.seq + 1) / 2) * (cfg.d_qk + cfg.d_v)
    res = {}
    for name, ms, fl in (("augq", augq_ms, augq_flops), ("attention", attn_ms, attn_flops)):
        tf = fl / ms / 1e9
        res[name] = {"ms": ms, "TFLOP/s": tf, "flops": fl, "bound": "tensor",
                     "frac_of_measured_bf16_burst": tf / peaks["bf16_tflops"],
                     "frac_of_measured_bf16_sustained": tf / peaks["bf16_tflops_sustained"]}
    res["augq"]["clocks"], res["attention"]["clocks"] = ck_a.summary(), ck_p.summary()
    for name, means in groups.items():
        res[name]["ms_of_each_group"] = means
        res[name]["timing"] = f"fastest of 3 groups of {steps} calls, 0.3 s idle before each group (burst regime)"
    kv_flops = 2.0 * T * cfg.d_model * (cfg.n_k * cfg.d_qk + cfg.n_v * cfg.d_v)
    res["kv_projection_rope"] = {"ms": kv_ms, "TFLOP/s": kv_flops / kv_ms / 1e9, "flops": kv_flops,
                                 "note": "k = rope(h W_K^T) and v = h W_V^T, two launches"}
    res["augq_rope"] = {"ms": augq_rope_ms, "TFLOP/s": augq_flops / augq_rope_ms / 1e9}
    res["attention"]["note"] = "causal flops (lower triangle incl. diagonal); time includes the cache-update kernel"
    res["working_set"] = "weights 92 MB + activations 0.5 GB per step: larger than L2"
    # the same causal attention with SIGMA-1.5B's heads (32 query / 4 K / 16 V heads of 64 channels)
    d64, nk64, nv64 = 64, 4, 16
    q64 = rn(cfg.batch, cfg.seq, cfg.n_q, d64)
    k64n, v64n = rn(cfg.batch, cfg.seq, nk64, d64), rn(cfg.batch, cfg.seq, nv64, d64)
    cache64 = api.KVCache(torch.zeros(cfg.batch, nk64, cfg.seq, d64, dtype=torch.bfloat16, device=device),
                          torch.zeros(cfg.batch, nv64, cfg.seq, d64, dtype=torch.bfloat16, device=device),
                          torch.zeros(cfg.batch, dtype=torch.int32, device=device), cfg.seq)
    out64 = torch.empty(cfg.batch, cfg.seq, cfg.n_q, d64, dtype=torch.bfloat16, device=device)
    ms64 = timed(lambda: api.diffqkv_prefill(q64, k64n, v64n, cache64, d64 ** -0.5, out=out64, dev_status=status))
    assert int(status.item()) == 0, "device status reported an error"
    fl64 = 2.0 * cfg.batch * cfg.n_q * (cfg.seq * (cfg.seq + 1) / 2) * (2 * d64)
    res["attention_sigma1p5b_heads_d64"] = {"ms": ms64, "TFLOP/s": fl64 / ms64 / 1e9, "flops": fl64,
                                            "heads": "32 query / 4 K / 16 V, 64 channels"}
    del q64, k64n, v64n, cache64, out64
    # keys cached at half the value width (d_qk 64, d_v 128; queries folded through the K feed-forward layer first)
    w_kup = rn(cfg.n_k, cfg.d_v, 64, std=64 ** -0.5)
    qh = torch.empty(cfg.batch, cfg.seq, cfg.n_q, 64, dtype=torch.bfloat16, device=device)
    kh_new = rn(cfg.batch, cfg.seq, cfg.n_k, 64)
    cache_h = api.KVCache(torch.zeros(cfg.batch, cfg.n_k, cfg.seq, 64, dtype=torch.bfloat16, device=device), v,
                          torch.zeros(cfg.batch, dtype=torch.int32, device=device), cfg.seq)
    fold_ms = timed(lambda: api.diffqkv_fold_k_up(q4, w_kup, out=qh))
    ms_h = timed(lambda: api.diffqkv_prefill(qh, kh_new, v_new, cache_h, cfg.scale, out=out, dev_status=status))
    assert int(status.item()) == 0, "device status reported an error"
    fl_h = 2.0 * cfg.batch * cfg.n_q * (cfg.seq * (cfg.seq + 1) / 2) * (64 + cfg.d_v)
    res["attention_half_width_keys"] = {"ms": ms_h, "TFLOP/s": fl_h / ms_h / 1e9, "flops": fl_h, "fold_k_up_ms": fold_ms,
                                        "heads": "32 query / 4 K / 8 V, d_qk 64, d_v 128"}
    return res


def time_augq_decode(api, W, device, steps):
    """The augmented-Q projection of one decode step (config 4's widths, one row per sequence): three launches that
    stream the 92 MB of weights; four weight sets are rotated so that none is found in L2."""
    import torch
    cfg = W.CFG4
    d_q0 = cfg.n_q * cfg.d_qk
    g = torch.Generator(device=device)
    g.manual_seed(cfg.seed + 7)

    def rn(*shape, std=1.0):
        return (torch.randn(shape, generator=g, device=device) * std).to(torch.bfloat16)

    sets = [(rn(d_q0, cfg.d_model, std=cfg.d_model ** -0.5), rn(cfg.d_aug, d_q0, std=d_q0 ** -0.5),
             rn(cfg.d_aug, d_q0, std=d_q0 ** -0.5), rn(d_q0, cfg.d_aug, std=cfg.d_aug ** -0.5)) for _ in range(4)]
    wbytes = float(sum(w.numel() * 2 for w in sets[0]))
    res = {"weight_bytes": wbytes, "rows": {}}
    for T in (4, 16, 64):
        h = rn(T, cfg.d_model, std=cfg.h_std)
        ws = torch.empty(max(api.diffqkv_augq_workspace_bytes(T, d_q0, cfg.d_aug), 256), dtype=torch.uint8, device=device)
        q = torch.empty(T, d_q0, dtype=torch.bfloat16, device=device)
        i = [0]

        def step():
            api.diffqkv_augq(h, *sets[i[0] % 4], workspace=ws, q_out=q)
            i[0] += 1

        for _ in range(10):
            step()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(steps):
            step()
        b.record()
        torch.cuda.synchronize()
        ms = a.elapsed_time(b) / steps
        res["rows"][str(T)] = {"us_per_step": ms * 1e3, "weights_GB/s": wbytes / ms / 1e6}
    return res


def time_decode_step(api, W, device, host, steps):
    """One decode step of the whole attention block on the headline shape (config 3: batch 4, 32/4/8 heads, d 128,
    32768 cached tokens; hidden 2048 and the aug-Q widths of config 4): diffqkv_decode_frontend (q = rope(aug-Q(h)),
    k = rope(h W_K^T) and v = h W_V^T written into the cache as token 32767), then diffqkv_decode over the 32768 tokens.  Weights and caches are rotated
    out of L2; every product runs in this library's kernels."""
    import dataclasses
    import torch
    cfg, c4 = host.cfg, W.CFG4
    case = DecodeCase(api, cfg, device, host_inputs=host)
    d_q0 = cfg.n_q * cfg.d_qk
    g = torch.Generator(device=device)
    g.manual_seed(cfg.seed + 11)

    def rn(*shape, std=1.0):
        return (torch.randn(shape, generator=g, device=device) * std).to(torch.bfloat16)

    sets = [(rn(d_q0, c4.d_model, std=c4.d_model ** -0.5), rn(c4.d_aug, d_q0, std=d_q0 ** -0.5),
             rn(c4.d_aug, d_q0, std=d_q0 ** -0.5), rn(d_q0, c4.d_aug, std=c4.d_aug ** -0.5),
             rn(cfg.n_k * cfg.d_qk, c4.d_model, std=c4.d_model ** -0.5),
             rn(cfg.n_v * cfg.d_v, c4.d_model, std=c4.d_model ** -0.5)) for _ in range(4)]
    T = cfg.batch
    h = rn(T, c4.d_model, std=c4.h_std)
    pos = torch.full((T,), cfg.kv_len - 1, device=device, dtype=torch.float64)
    inv = torch.pow(torch.tensor(50000.0, dtype=torch.float64, device=device),
                    -2.0 * torch.arange(cfg.d_qk // 2, device=device, dtype=torch.float64) / cfg.d_qk)
    ang = pos[:, None] * inv[None, :]
    cos, sin = torch.cos(ang).float().contiguous(), torch.sin(ang).float().contiguous()
    ws = torch.empty(1 << 22, dtype=torch.uint8, device=device)  # far more than the few rows need
    q = torch.empty(T, d_q0, dtype=torch.bfloat16, device=device)
    before = torch.from_numpy(case.seqlens_host - 1).to(device)  # the new token becomes the last cached one
    appends = [dataclasses.replace(c, seqlens=before) for c in case.caches]
    i = [0]

    def step():
        w_q, w_g, w_u, w_d, w_k, w_v = sets[i[0] % 4]
        r = i[0] % case.rotate
        i[0] += 1
        api.diffqkv_decode_frontend(h, w_q, w_g, w_u, w_d, w_k, w_v, appends[r], cfg.n_q, cfg.d_qk, cfg.d_v, cos, sin,
                                    workspace=ws, q_out=q.view(T, cfg.n_q, cfg.d_qk), dev_status=case.status)
        api.diffqkv_decode(q.view(T, cfg.n_q, cfg.d_qk), case.caches[r], cfg.n_k, cfg.n_v, cfg.scale,
                           workspace=case.workspace, out=case.out, dev_status=case.status)

    for _ in range(10):
        step()
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    l0 = api.launch_count()
    a.record()
    for _ in range(steps):
        step()
    b.record()
    torch.cuda.synchronize()
    assert int(case.status.item()) == 0, "device status reported an error"
    ms = a.elapsed_time(b) / steps
    wbytes = float(sum(w.numel() * 2 for w in sets[0]))
    return {"us_per_step": ms * 1e3, "kernels_per_step": (api.launch_count() - l0) // steps,
            "weight_bytes": wbytes, "kv_bytes": case.bytes, "GB/s": (wbytes + case.bytes) / ms / 1e6,
            "tokens_per_s_per_layer": cfg.batch / (ms * 1e-3)}


def time_sigma_table(api, W, device, steps):
    """The paper's own efficiency experiment in shape (appendix table of split / combine / total kernel times):
    SIGMA-1.5B attention heads (32 query, 4 K, 16 V heads, head dimension 64) against the standard model's 16 K /
    16 V heads at prefix lengths 2k, 4k, 16k and 32k (batch 8, bf16 cache drawn on the device).  Per shape: the split
    kernel and the combine kernel each timed alone (events between them), and one whole untimed-inside decode step;
    per prefix: the relative reduction of each, beside the reduction of the cache bytes."""
    import dataclasses
    rows = []
    for prefix in (2048, 4096, 16384, 32768):
        row = {"prefix": prefix}
        for name, n_k, n_v in (("sigma", 4, 16), ("std", 16, 16)):
            cfg = dataclasses.replace(W.SIGMA15B, name=f"{name}_{prefix}", batch=8, n_k=n_k, n_v=n_v, kv_len=prefix)
            case = DecodeCase(api, cfg, device)
            ms = case.time_steps(steps, 20) / steps
            split_ms, combine_ms = case.time_split_and_combine(min(steps, 100))
            kernels = case.launches_per_step()
            row[name] = {"us_per_step": ms * 1e3, "split_us": split_ms * 1e3,
                         "combine_us": combine_ms * 1e3 if kernels > 1 else None, "kernels_per_step": kernels,
                         "GB/s": case.bytes / ms / 1e6, "kv_bytes": case.bytes, "rotate": case.rotate}
            if kernels == 1:
                row[name]["note"] = "the rows' blocks merge on chip (thread-block clusters): no combine kernel"
            del case
        for key, out in (("us_per_step", "time_reduction_pct"), ("split_us", "split_reduction_pct"),
                         ("combine_us", "combine_reduction_pct")):
            a, b = row["sigma"][key], row["std"][key]
            row[out] = 100.0 * (1.0 - a / b) if a is not None and b is not None else None
        row["bytes_reduction_pct"] = 100.0 * (1.0 - row["sigma"]["kv_bytes"] / row["std"]["kv_bytes"])
        rows.append(row)
    return rows


def time_context_sweep(api, W, device, steps):
    """DiffQKV (32 query / 4 K / 8 V heads) against its GQA twin (8 K / 8 V heads) over the context length, batch 4,
    d 128, bf16 cache drawn on the device: one decode step each; the bytes model predicts 25 % less time."""
    import dataclasses
    rows = []
    for ctx in (4096, 8192, 16384, 32768, 65536, 131072):
        row = {"context": ctx}
        for name, cfg in (("diffqkv", W.CFG3), ("gqa", W.CFG3.gqa_twin())):
            case = DecodeCase(api, dataclasses.replace(cfg, name=f"{name}_{ctx}", kv_len=ctx), device)
            ms = case.time_steps(steps, 20) / steps
            row[name] = {"us_per_step": ms * 1e3, "GB/s": case.bytes / ms / 1e6, "rotate": case.rotate,
                         "kernels_per_step": case.launches_per_step()}
            del case
        row["speedup"] = row["gqa"]["us_per_step"] / row["diffqkv"]["us_per_step"]
        rows.append(row)
    return rows


def time_fp32_mode(api, W, device, steps):
    """The fp32 mode beyond the second-level cache: config 1's heads (16 query / 2 K / 4 V, 64 channels, fp32 cache) at
    batch 4 and 65536 tokens, 403 MB of cache per step, on the generic path's unit kernel (plain loads, fp32 FMAs,
    every K and V row read once for the eight query heads of its unit) and its combine kernel."""
    import dataclasses
    cfg = dataclasses.replace(W.CFG1, name="fp32_b4_64k", batch=4, kv_len=65536, seed=1500)
    case = DecodeCase(api, cfg, device)
    ms = case.time_steps(steps, 5) / steps
    return {"ms_per_step": ms, "GB/s": case.bytes / ms / 1e6, "kv_bytes": case.bytes, "rotate": case.rotate,
            "shape": "batch 4, 16/2/4 heads, d 64, 65536 tokens, fp32 cache"}


def time_topk(api, W, device, host, steps, topk=100):
    """Selective V fetching on the headline workload: the K cache is streamed once, of V only `topk` rows per query
    head are read.  Algorithmic bytes = K bytes + gathered V rows; the fp32 scores and the per-16-token maxima are
    scratch (written once, read where the selection needs them) and reported apart."""
    import torch
    cfg = host.cfg
    case = DecodeCase(api, cfg, device, host_inputs=host)
    shape = case.shape
    nbytes = int(api._lib.diffqkv_decode_topk_workspace_bytes(__import__("ctypes").byref(shape), case.caches[0].max_seqlen, topk))
    ws = torch.empty(nbytes, dtype=torch.uint8, device=device)
    i = [0]

    def step():
        cache = case.caches[i[0] % case.rotate]
        i[0] += 1
        api.diffqkv_decode_topk(case.q, cache, cfg.n_k, cfg.n_v, cfg.scale, topk, workspace=ws, out=case.out,
                                dev_status=case.status)

    for _ in range(20):
        step()
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(steps):
        step()
    b.record()
    torch.cuda.synchronize()
    ms = a.elapsed_time(b) / steps
    assert int(case.status.item()) == 0
    tokens = float(np.sum(host.seqlens.astype(np.int64)))
    k_bytes = tokens * cfg.n_k * cfg.d_qk * 2
    v_bytes = float(cfg.batch * cfg.n_q * topk * cfg.d_v * 2)
    scratch_bytes = tokens * cfg.n_q * 4 * (1 + 1 / 16)
    return {"topk": topk, "ms_per_step": ms, "k_bytes": k_bytes, "v_bytes_gathered": v_bytes,
            "scratch_bytes_written": scratch_bytes, "GB/s": (k_bytes + v_bytes) / ms / 1e6,
            "k_stream_GB/s": k_bytes / ms / 1e6}


def summarize(line, peaks):
    """The figures the benchmark definition asks for, in one short object: decode GB/s per configuration with the
    fractions of the measured copy peak and of the 8 TB/s nominal figure, the prefill leg's TFLOP/s against the
    measured bf16 burst peak, and DiffQKV against GQA at 32K context."""
    o = line.get("others", {})
    r3 = lambda x: None if x is None else round(float(x), 3)  # noqa: E731

    def gbs(v):
        return None if v is None else {"GB/s": round(v, 1), "of_measured": r3(v / peaks["hbm_gbs"]), "of_8TBs": r3(v / 8000.0)}

    out = {"cfg3": gbs(line["value"] / line["n_gpus"]), "cfg3_us_per_step": r3(line["ms_per_step"] * 1e3),
           "cfg3_us_per_step_min": r3(line["timed_groups"]["ms_per_step_min"] * 1e3)}
    for key, name in (("cfg2_b16_4k", "cfg2"), ("cfg2_b16_4k_gqa", "cfg2_gqa"), ("cfg1_small_f32", "cfg1"),
                      ("cfg5_paged_varlen", "cfg5"), ("cfg3_gqa_twin", "cfg3_gqa")):
        if key in o:
            out[name] = gbs(o[key]["GB/s"])
    if "diffqkv_vs_gqa_speedup_32k" in line:
        out["diffqkv_vs_gqa_32k"] = r3(line["diffqkv_vs_gqa_speedup_32k"])
    for row in o.get("diffqkv_vs_gqa_over_context", []):
        if row["context"] in (4096, 8192):
            out[f"diffqkv_vs_gqa_{row['context'] // 1024}k"] = r3(row["speedup"])
    c4 = o.get("cfg4_prefill_8k")
    if c4:
        for name in ("augq", "attention"):
            out["cfg4_" + name] = {"TFLOP/s": round(c4[name]["TFLOP/s"], 1), "ms": r3(c4[name]["ms"]),
                                   "of_measured_burst": r3(c4[name]["frac_of_measured_bf16_burst"])}
    if "fp32_b4_64k" in o:
        out["fp32_64k"] = gbs(o["fp32_b4_64k"]["GB/s"])
    if "cfg3_selective_v_top100" in o:
        out["cfg3_top100_us"] = r3(o["cfg3_selective_v_top100"]["ms_per_step"] * 1e3)
    if line.get("e2e"):
        out["e2e_GB/s"] = round(line["e2e"]["value"], 1)
    if line.get("roofline"):
        out["split_kernel_frac_of_measured"] = r3(line["roofline"]["frac"])
    return out


def max_over_ranks(value: float, device) -> float:
    """The slowest rank's value (all-reduce MAX over the default process group; identity without one)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def run_ours(args):
    import torch
    from paper_2501_13629_b200 import api, workloads as W

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    barrier = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=device)
        barrier = lambda: (dist.barrier(), torch.cuda.synchronize())  # noqa: E731
    peaks = measured_peaks()
    api.set_tail_reserve(args.tail_reserve)
    if args.workload == "prefill":  # the config 4 leg alone (the command profilers wrap for the tensor-core kernels)
        if rank == 0:
            print(json.dumps({"workload": W.CFG4.name, **time_prefill(api, W, device, peaks, max(1, min(args.steps, 20)))}))
        return

    cfg = W.CFG3
    host = W.make_decode_inputs(cfg)
    if args.workload == "augq_decode":  # the projection chain at decode row counts alone (the command profilers wrap)
        if rank == 0:
            print(json.dumps({"workload": "cfg4 widths, 4 / 16 / 64 rows",
                              **time_augq_decode(api, W, device, max(1, min(args.steps, 200)))}))
        return
    if args.workload == "cfg2":  # config 2 and its GQA twin alone (short rows: merged on chip; the command profilers wrap)
        if rank == 0:
            res = {"workload": W.CFG2.name}
            steps = max(1, min(args.steps, 2000))
            for c in (W.CFG2, W.CFG2.gqa_twin()):
                cs = DecodeCase(api, c, device, host_inputs=W.make_decode_inputs(c))
                c_ms = cs.time_steps(steps, args.warmup) / steps
                res[c.name] = {"ms_per_step": c_ms, "GB/s": cs.bytes / c_ms / 1e6, "kv_bytes": cs.bytes,
                               "rotate": cs.rotate, "kernels_per_step": cs.launches_per_step()}
                del cs
            print(json.dumps(res))
        return
    if args.workload == "fp32":  # the fp32 mode alone (the command profilers wrap)
        if rank == 0:
            print(json.dumps({"workload": "fp32_b4_64k", **time_fp32_mode(api, W, device, max(1, min(args.steps, 50)))}))
        return
    if args.workload == "topk":  # selective V fetching on the headline workload alone (the command profilers wrap)
        if rank == 0:
            print(json.dumps({"workload": cfg.name + " top-100 / top-1024",
                              "top100": time_topk(api, W, device, host, max(1, min(args.steps, 300)), 100),
                              "top1024": time_topk(api, W, device, host, max(1, min(args.steps, 300)), 1024)}))
        return
    case = DecodeCase(api, cfg, device, host_inputs=host)
    launches0 = api.launch_count()
    case.step()
    launches_per_step = api.launch_count() - launches0
    with ClockSampler(local_rank) as clocks:
        groups = case.time_groups(args.steps, args.warmup, barrier, lambda x: max_over_ranks(x, device))
    assert int(case.status.item()) == 0, "device status reported an error"
    # every group is exactly `steps` steps between barriers, slowest rank; the line reports the median group
    ms_per_step = float(np.median(groups)) / args.steps
    value = world * case.bytes / (ms_per_step * 1e-3) / 1e9

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": "cfg3: DiffQKV decode batch 4, n_q 32, n_k 4, n_v 8, d 128, KV length 32768, bf16 "
                               "cache [batch, head, seq, dim], one query token per sequence",
                   "kv_bytes_per_step": case.bytes, "parallelism": "replicas" if world > 1 else "single",
                   "l2": f"inputs larger than L2: {case.rotate} distinct cache copies rotated, "
                         f"working set {case.working_set / 1e6:.0f} MB"},
        "gpu_launches": launches_per_step * args.steps,
        "timed_groups": {"groups": len(groups), "steps_each": args.steps,
                         "ms_per_step_median": ms_per_step, "ms_per_step_min": float(np.min(groups)) / args.steps,
                         "ms_per_step_max": float(np.max(groups)) / args.steps,
                         "note": "groups of exactly `steps` steps, repeated until 50 ms are timed; value = median group"},
        "clocks": clocks.summary(),
        "tokens_per_s_per_layer": world * cfg.batch / (ms_per_step * 1e-3),
        "frac_of_8TBs_nominal": value / world / 8000.0,
        "frac_of_measured_hbm": value / world / peaks["hbm_gbs"],
    }

    e2e = None
    if not args.profile:  # every rank runs the end-to-end loop at the same time; the slowest one counts
        n_e2e = min(max(args.steps, 200), 500)  # a short --steps would leave this host-timed figure to a few samples
        if barrier:
            barrier()
        e2e_ms, h2d, d2h = case.time_e2e(n_e2e, min(args.warmup, 20))
        e2e_step = max_over_ranks(e2e_ms, device) / n_e2e
        e2e = {"value": world * case.bytes / (e2e_step * 1e-3) / 1e9, "unit": UNIT,
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "ms_per_step": e2e_step,
               "note": "one diffqkv_decode_host call per step: pinned q copied in, split + combine, out copied back, stream "
                       "synchronised; the KV cache is resident state"}
    if rank == 0 and args.profile:
        print(json.dumps(line))
    elif rank == 0:
        # roofline of the dominant (split) kernel, timed alone by events the library records around it
        k_ms = case.time_split_kernel(min(max(args.steps, 100), 200))
        ach = case.bytes / (k_ms * 1e-3) / 1e9
        line["roofline"] = {"bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                            "frac": ach / peaks["hbm_gbs"], "traffic": split_kernel_dram_bytes(),
                            "kernel": "decode split kernel",
                            "kernel_ms": k_ms, "peak_source": peaks["source"] + " (burst copy)"}
        line["e2e"] = e2e
        others = {}
        so = max(args.steps, 300)  # steps for the other configurations: their figures should not hinge on a short --steps
        if not args.quick and world == 1:
            twin = DecodeCase(api, cfg.gqa_twin(), device, host_inputs=W.make_decode_inputs(cfg.gqa_twin()))
            t_ms = twin.time_steps(so, args.warmup) / so
            others["cfg3_gqa_twin"] = {"ms_per_step": t_ms, "GB/s": twin.bytes / t_ms / 1e6,
                                       "tokens_per_s_per_layer": cfg.batch / (t_ms * 1e-3)}
            line["diffqkv_vs_gqa_speedup_32k"] = t_ms / ms_per_step
            del twin
            tk = time_topk(api, W, device, host, 300)
            tk["speedup_vs_full_v"] = ms_per_step / tk["ms_per_step"]
            others["cfg3_selective_v_top100"] = tk
            for c in (W.CFG2, W.CFG2.gqa_twin(), W.CFG1):
                cs = DecodeCase(api, c, device, host_inputs=W.make_decode_inputs(c))
                c_ms = cs.time_steps(so, args.warmup) / so
                others[c.name] = {"ms_per_step": c_ms, "GB/s": cs.bytes / c_ms / 1e6, "rotate": cs.rotate,
                                  "kernels_per_step": cs.launches_per_step()}
                del cs
            torch.cuda.empty_cache()
            others["fp32_b4_64k"] = time_fp32_mode(api, W, device, max(5, min(args.steps, 50)))
            torch.cuda.empty_cache()
            c5 = DecodeCase(api, W.CFG5, device)
            n5 = max(5, min(args.steps, 30))
            c5_ms = c5.time_steps(n5, 3) / n5
            others[W.CFG5.name] = {"ms_per_step": c5_ms, "GB/s": c5.bytes / c5_ms / 1e6,
                                   "kv_bytes": c5.bytes, "frac_of_measured_hbm": c5.bytes / c5_ms / 1e6 / peaks["hbm_gbs"]}
            del c5
            torch.cuda.empty_cache()
            others[W.CFG4.name] = time_prefill(api, W, device, peaks, max(5, min(args.steps, 20)))
            torch.cuda.empty_cache()
            others["augq_at_decode"] = time_augq_decode(api, W, device, 200)
            others["decode_step_cfg3"] = time_decode_step(api, W, device, host, 200)
            torch.cuda.empty_cache()
            others["sigma1p5b_vs_std_heads"] = time_sigma_table(api, W, device, 300)
            torch.cuda.empty_cache()
            others["diffqkv_vs_gqa_over_context"] = time_context_sweep(api, W, device, 200)
        line["others"] = others
        if world == 1:
            line["cpu_baseline"] = cpu_baseline(host, budget_s=12.0)
        line["summary"] = summarize(line, peaks)  # last on the line, so that it survives a truncated tail
        print(json.dumps(line))
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
        dist.destroy_process_group()


# ----------------------------------------------------------------------------- oracle arm
def _time_oracle_pairs(oracle, host, pairs):
    cfg = host.cfg
    cache = oracle.Cache(host.k, host.v, host.k_strides, host.v_strides, host.seqlens, host.page_table,
                         cfg.page_size)
    t0 = time.perf_counter()
    oracle.decode(host.q, cache, cfg.n_q, cfg.n_k, cfg.n_v, cfg.d_qk, cfg.d_v, cfg.scale, pairs=pairs)
    return time.perf_counter() - t0


def _all_pairs(cfg):
    return np.array([(b, h) for b in range(cfg.batch) for h in range(cfg.n_q)], dtype=np.int32)


def cpu_baseline(host, budget_s=20.0):
    """The float64 oracle, as it stands, on the host cores, on a bounded sample of the same workload."""
    import oracle
    cores = oracle.set_threads(0)
    cfg = host.cfg
    pairs = _all_pairs(cfg)
    t1 = _time_oracle_pairs(oracle, host, pairs)  # the whole workload once (also warms the page cache)
    reps = int(max(1, min(200, budget_s / max(t1, 1e-6))))
    t0 = time.perf_counter()
    for _ in range(reps):
        _time_oracle_pairs(oracle, host, pairs)
    dt = (time.perf_counter() - t0) / reps
    return {"value": kv_bytes(cfg, host.seqlens) / dt / 1e9, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"all {len(pairs)} (sequence, query head) rows of cfg3 at the full 32768-token context, "
                      f"{reps} repetitions, {dt:.3f} s each", "seconds": dt * reps}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    from paper_2501_13629_b200 import workloads as W
    oracle.build()
    cores = oracle.set_threads(0)
    cfg = W.CFG3
    host = W.make_decode_inputs(cfg)
    pairs = _all_pairs(cfg)
    t_row = _time_oracle_pairs(oracle, host, pairs[:cores]) / 1.0  # wall time of `cores` rows in parallel
    budget = float(args.budget_s)
    total_steps = args.steps + args.warmup
    per_step_rows = int(max(1, min(len(pairs), (budget / total_steps / max(t_row, 1e-6)) * cores)))
    sample = pairs[:per_step_rows]
    for _ in range(args.warmup):
        _time_oracle_pairs(oracle, host, sample)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        _time_oracle_pairs(oracle, host, sample)
    dt = time.perf_counter() - t0
    ms_per_step = dt / args.steps * 1e3
    value = (per_step_rows / len(pairs)) * kv_bytes(cfg, host.seqlens) / (ms_per_step * 1e-3) / 1e9
    desc = (f"each step: {per_step_rows} of {len(pairs)} (sequence, query head) rows of cfg3 at the full "
            f"32768-token context")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT,
        "n_gpus": int(os.environ.get("WORLD_SIZE", "1")), "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        "config": {"workload": "cfg3: DiffQKV decode batch 4, n_q 32, n_k 4, n_v 8, d 128, KV length 32768, bf16 "
                               "cache [batch, head, seq, dim], one query token per sequence", "sample": desc},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=50)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--quick", action="store_true", help="headline workload only")
    ap.add_argument("--budget-s", type=float, default=150.0,
                    help="--impl reference: seconds of oracle time the whole run may take (sizes the per-step sample)")
    ap.add_argument("--workload", default="decode", choices=["decode", "prefill", "topk", "augq_decode", "fp32", "cfg2"],
                    help="decode = the headline line (default); prefill = only the config 4 timings; "
                         "topk = only selective V fetching on the headline workload; augq_decode = only the projection "
                         "chain at decode row counts; fp32 = only the fp32 mode; cfg2 = only config 2 and its GQA twin")
    ap.add_argument("--tail-reserve", type=int, default=-1,
                    help="tail balance of the TMA decode kernel: -1 automatic (default), 0 off, n tiles per block")
    ap.add_argument("--profile", action="store_true",
                    help="only the timed loop of the headline workload (the command profilers wrap)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
