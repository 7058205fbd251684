#!/usr/bin/env python
"""Benchmark of the BiCache attention hot path.

One "step" is one denoising step's attention: reuse-depth rule, prefix-store lookups (hits), the
per-layer dispatch, and for every layer the shallow-layer call (suffix queries over cached prefix
K/V + own suffix K/V) and/or the deep-layer fallback (full bidirectional attention), all through
the C ABI.  The default workload is the largest single-GPU configuration by FLOPs per step, the
Dream-7B-shaped 28-layer GQA stack with a 16384-token prefix (`config5`); the other configurations
and the small-suffix (bandwidth-bound) shapes are measured in the same run at a few steps each and
reported as the `per_config` list of the same JSON line.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload config5] [--impl reference]

Prints ONE JSON line (rank 0).
"""
import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

METRIC = "prefix_reuse_attention_suffix_tokens_per_s_per_denoising_step"
UNIT = "tokens/s"
DEFAULT_WORKLOAD = "config5"
# what the default run measures besides its own workload: (workload, timed steps)
PER_CONFIG = (("config2", 20), ("config3", 8), ("config4", 4))
SMALL_SUFFIX = ("b1", "b2", "b3", "b4")

# DRAM bytes (read + write) of one launch, from the ncu captures summarised under profiles/ (the file
# is named beside each figure; a capture is of the kernel as it was when the summary was written).
# None: no capture of that launch exists.
NCU_TRAFFIC = {
    "config2": {"full": (652.3e6, "profiles/tc_attention_kernel_config2.md"),
                "attend": (130.4e6, "profiles/tc_attention_kernel_config2.md")},
    "config3": {"attend": (848.6e6, "profiles/tc_attention_kernel_config3_attend.md"),
                "put": (2104.6e6, "profiles/hbm_kernels_config3.md"),
                "similarity": (2147.6e6, "profiles/hbm_kernels_config3.md"),
                "project": (218.0e6, "profiles/project_kv_kernel_config3.md")},
    # captured with 4 of the 32 requests and scaled by the units processed (see the file)
    "config5": {"full": (8848.0e6, "profiles/tc_attention_kernel_config5_traffic.md (4-request capture, scaled)"),
                "attend": (402.0e6, "profiles/tc_attention_kernel_config5_traffic.md (4-request capture, scaled)")},
    "config5s": {"full": (1106.0e6, "profiles/tc_attention_kernel_config5_traffic.md"),
                 "attend": (79.7e6, "profiles/tc_attention_kernel_config5_traffic.md")},
    "b2": {"attend": (274.1e6, "profiles/key_range_kernels_b2.md")},
}


def traffic_of(workload, which):
    t = NCU_TRAFFIC.get(workload, {}).get(which)
    return (None, None) if t is None else t


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"bf16_tflops": p["bf16_tflops"], "bf16_tflops_sustained": p.get("bf16_tflops_sustained") or p["bf16_tflops"],
                "hbm_gbs": p["hbm_gbs"], "source": "measured"}
    return {"bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "hbm_gbs": 6650.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.FIELDS,
                 "--format=csv,noheader,nounits", "-lms", "50"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        time.sleep(0.06)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        for ln in self.lines:
            parts = [x.strip() for x in ln.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"),
                                 parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


class Job:
    """Device state of one workload: context, store, tensors, and the step function."""

    def __init__(self, w, device, delta=0):
        from paper_2606_07571_b200 import binding, workloads
        self.w, self.binding, self.workloads = w, binding, workloads
        torch.cuda.set_device(device)
        self.delta = delta if w.num_layers > 1 else 0
        self.t = 1                                    # 1-based denoising step (Eq. 5)
        npages = w.pages_needed() + 1
        layer_pages = None
        if self.delta > 0:
            # Per-request kept prefix K/V of the deep layers (Eq. 5): request i keeps them from layer
            # depth[i] on, so layer l's pool holds the shared prefixes plus the kept prefixes of the
            # requests whose depth is at most l.
            depth0 = host_reuse_depth(binding, w)
            need = [(w.prefix_lens[g] + 15) // 16 for g in w.req_prefix]
            layer_pages = [npages + sum(nd for nd, d in zip(need, depth0) if d <= l) for l in range(w.num_layers)]
            npages = max(layer_pages)
        order = workloads.shuffled_page_order(npages, 7) if w.shuffle_pages else None
        self.bc = binding.BiCache(w.num_layers, w.num_q_heads, w.num_kv_heads, w.head_dim, npages, w.dtype,
                                  w.total_rows, w.num_requests, device=device, free_order=order,
                                  layer_pages=layer_pages)
        self.pool_bytes = 2 * self.bc.k_pool.numel()
        self.bc.set_depth_table(workloads.standin_depth_table(w.num_layers))
        self.keys = [workloads.prefix_key(w, g) for g in range(len(w.prefix_lens))]
        for g in range(len(w.prefix_lens)):
            kc, vc = workloads.draw_prefix_kv(w, g, "cuda")
            self.bc.put_prefix(self.keys[g], kc, vc)
            del kc, vc
        self.private = [-1] * w.num_requests
        if self.delta > 0:
            self.private = [self.bc.reserve_prefix(0x6000000000000000 + i, w.prefix_lens[g], first_layer=int(d))[0]
                            if d < w.num_layers else -1
                            for i, (g, d) in enumerate(zip(w.req_prefix, depth0))]
        self.q, self.k, self.v = workloads.draw_full_qkv(w, "cuda")
        self.out = torch.empty_like(self.q)
        self.single_layer = w.num_layers == 1
        self.out2 = torch.empty_like(self.q) if self.single_layer else None
        self.depth = self.bc.reuse_depth(w.req_prefix_len(), w.suffix_lens)
        torch.cuda.synchronize()

    def close(self):
        self.bc.close()
        for name in ("q", "k", "v", "out", "out2", "bc"):
            setattr(self, name, None)
        torch.cuda.empty_cache()

    def calls_per_step(self):
        """The layer calls of one step as (layer, kind): kind 'attend' / 'full' when every request of
        the call takes the same path in that layer (one kernel launch of known FLOPs), else 'mixed'."""
        w = self.w
        if self.single_layer:
            return [(0, "attend"), (0, "full")]
        if self.delta > 0:
            return [(l, "mixed") for l in range(w.num_layers)]
        lo, hi = int(min(self.depth)), int(max(self.depth))
        return [(l, "attend" if l < lo else "full" if l >= hi else "mixed") for l in range(w.num_layers)]

    def step(self, q=None, k=None, v=None, out=None, out2=None, events=None):
        """One denoising step's attention through the C ABI.  `events`: a list that receives one
        (start, end) CUDA event pair per layer call, in the order of calls_per_step()."""
        w, bc = self.w, self.bc
        q = self.q if q is None else q
        k = self.k if k is None else k
        v = self.v if v is None else v
        out = self.out if out is None else out
        out2 = self.out2 if out2 is None else out2
        depth = bc.reuse_depth(w.req_prefix_len(), w.suffix_lens)                     # depth rule
        pid = [bc.lookup_prefix(key)[0] for key in self.keys]                         # store hits
        req_pid = [pid[g] for g in w.req_prefix]

        def timed(fn):
            if events is None:
                fn()
                return
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            fn()
            b.record()
            events.append((a, b))

        if self.single_layer:
            # shallow-layer pass (depths from the rule) then deep-layer pass (all recompute)
            timed(lambda: bc.attend_layer(0, depth, req_pid, w.full_row_off, w.full_lens, q, k, v, out, None,
                                          w.softmax_scale))
            timed(lambda: bc.attend_layer(0, [0] * w.num_requests, req_pid, w.full_row_off, w.full_lens, q, k, v,
                                          out2, None, w.softmax_scale))
        elif self.delta > 0:
            # deep layers keep the request's own prefix K/V and recompute them every delta steps
            for l in range(w.num_layers):
                timed(lambda: bc.attend_step(l, self.t, self.delta, depth, req_pid, self.private, w.full_row_off,
                                             w.full_lens, q, k, v, out, None, w.softmax_scale))
            self.t += 1
        else:
            for l in range(w.num_layers):
                timed(lambda: bc.attend_layer(l, depth, req_pid, w.full_row_off, w.full_lens, q, k, v, out, None,
                                              w.softmax_scale))
        return depth

    def step_flops(self):
        w = self.w
        depth = self.depth
        per_req_attend = [4 * w.head_dim * w.num_q_heads * n * (w.prefix_lens[g] + n)
                          for g, n in zip(w.req_prefix, w.suffix_lens)]
        per_req_full = [4 * w.head_dim * w.num_q_heads * N * N for N in w.full_lens]
        if self.single_layer:
            return sum(per_req_attend) + sum(per_req_full)
        tot = 0
        for i in range(w.num_requests):
            tot += int(depth[i]) * per_req_attend[i] + (w.num_layers - int(depth[i])) * per_req_full[i]
        return tot

    def reuse_step_flops(self):
        """A step between two refresh steps: every layer reads a cached prefix (shared or kept)."""
        w = self.w
        return w.num_layers * sum(4 * w.head_dim * w.num_q_heads * n * (w.prefix_lens[g] + n)
                                  for g, n in zip(w.req_prefix, w.suffix_lens))


def host_reuse_depth(binding, w):
    """The depth rule through a host-only context of the library (no device work): needed before the
    device context exists, to size the per-layer pools of the kept deep-layer prefixes."""
    import ctypes as C
    lib = binding.load_library()
    cfg = binding.Config(w.num_layers, w.num_q_heads, w.num_kv_heads, w.head_dim, 16, 1, binding._dtype_code(w.dtype), -1)
    ctx = C.c_void_p()
    assert lib.bicache_create(C.byref(cfg), C.byref(ctx)) == binding.OK
    i32p = C.POINTER(C.c_int32)
    table = np.ascontiguousarray(w_table(w), dtype=np.int32)
    assert lib.bicache_set_depth_table(ctx, table.ctypes.data_as(i32p), 101) == binding.OK
    m = np.ascontiguousarray(w.req_prefix_len(), dtype=np.int32)
    n = np.ascontiguousarray(w.suffix_lens, dtype=np.int32)
    out = np.zeros(len(m), dtype=np.int32)
    assert lib.bicache_reuse_depth(ctx, len(m), m.ctypes.data_as(i32p), n.ctypes.data_as(i32p),
                                   out.ctypes.data_as(i32p)) == binding.OK
    lib.bicache_destroy(ctx)
    return out.tolist()


def w_table(w):
    from paper_2606_07571_b200 import workloads
    return workloads.standin_depth_table(w.num_layers)


def time_call(fn, iters, flush):
    """Average device time of fn() over `iters` runs, each preceded by an L2 flush (untimed): the
    256 MB buffer is written, then read back, so that the timed kernel starts with an L2 full of
    foreign but CLEAN lines and does not pay for writing the flusher's dirty lines back."""
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(iters)]
    for a, b in ev:
        flush.zero_()
        flush.max()
        a.record()
        fn()
        b.record()
    torch.cuda.synchronize()
    return sum(a.elapsed_time(b) for a, b in ev) / iters


def max_over_ranks(value, dist, device):
    """Maximum of a per-rank scalar over all ranks (identity when not distributed)."""
    t = torch.tensor([value], dtype=torch.float64, device=device)
    if dist is not None:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def tensor_roofline(kernel, flops, ms, peaks, sustained, launches, traffic):
    """The roofline record of a tensor-pipe-bound launch.  `sustained`: the launch was timed inside
    a long step (seconds of back-to-back kernels under the power cap), so the denominator is the
    sustained matmul peak; a launch timed alone takes the burst peak."""
    tf = flops / (ms * 1e-3) / 1e12
    peak = peaks["bf16_tflops_sustained"] if sustained else peaks["bf16_tflops"]
    return {"bound": "tensor", "kernel": kernel, "achieved": tf, "peak": peak, "unit": "TFLOP/s", "frac": tf / peak,
            "peak_source": peaks["source"] + (" sustained (launch timed inside a long step)" if sustained
                                              else " burst (launch timed alone or inside a millisecond step)"),
            "frac_of_burst": tf / peaks["bf16_tflops"], "frac_of_sustained": tf / peaks["bf16_tflops_sustained"],
            "traffic": traffic[0], "traffic_source": traffic[1],
            "flops_per_launch": flops, "ms_per_launch": ms, "launches_timed": launches}


def measure_steps(job, name, steps, warmup, flush, peaks, rank, local_rank, world, dist):
    """Warm-up, then `steps` timed steps (each preceded by an untimed L2 flush), with one CUDA event
    pair per layer call so that the launches of the dominant kernels are timed where they run."""
    w = job.w
    for _ in range(warmup):
        flush.zero_()
        job.step()
    assert job.bc.device_status() == 0
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    launches0 = job.bc.launch_count()
    job.t = 1                                         # the timed steps are denoising steps 1 .. K
    ev, per_call = [], []
    for _ in range(steps):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        calls = []
        flush.zero_()
        a.record()
        job.step(events=calls)
        b.record()
        ev.append((a, b))
        per_call.append(calls)
    torch.cuda.synchronize()
    launches = job.bc.launch_count() - launches0
    per_step_ms = [a.elapsed_time(b) for a, b in ev]
    step_ms = sum(per_step_ms) / steps
    if step_ms * steps < 400.0:
        # a short sustained stretch so that the clock sampler sees the kernels under load
        t_end = time.time() + 0.5
        while time.time() < t_end:
            job.step()
            torch.cuda.synchronize()
    clocks = sampler.stop() if rank == 0 else None
    assert job.bc.device_status() == 0
    step_ms_max = max_over_ranks(step_ms, dist, "cuda")
    if dist is not None:
        dist.barrier()

    flops = job.step_flops()
    refresh_info = None
    if job.delta > 0:
        is_ref = [(t - 1) % job.delta == 0 for t in range(1, steps + 1)]
        ref_ms = [m for m, r in zip(per_step_ms, is_ref) if r]
        reu_ms = [m for m, r in zip(per_step_ms, is_ref) if not r]
        flops = (len(ref_ms) * flops + len(reu_ms) * job.reuse_step_flops()) / steps   # mean FLOPs per step
        refresh_info = {"delta": job.delta, "store_bytes": job.pool_bytes,
                        "refresh_steps": len(ref_ms), "reuse_steps": len(reu_ms),
                        "ms_refresh_step": sum(ref_ms) / max(1, len(ref_ms)),
                        "ms_reuse_step": sum(reu_ms) / max(1, len(reu_ms)) if reu_ms else None}

    # launches timed in place: the layer calls in which every request takes the same path
    kinds = job.calls_per_step()
    in_place = {"attend": [], "full": []}
    for calls in per_call:
        for (layer, kind), (a, b) in zip(kinds, calls):
            if kind in in_place:
                in_place[kind].append(a.elapsed_time(b))
    sustained = step_ms >= 50.0          # the stacks: tens of milliseconds to a second of back-to-back kernels
    roofline = roofline_attend = None
    if in_place["full"]:
        roofline = tensor_roofline("tc_attention_kernel (attend_full launch, every request recomputes)",
                                   w.full_flops(), sum(in_place["full"]) / len(in_place["full"]), peaks, sustained,
                                   len(in_place["full"]), traffic_of(name, "full"))
    if in_place["attend"]:
        roofline_attend = tensor_roofline("tc_attention_kernel (attend launch, every request reuses)",
                                          w.attend_flops(), sum(in_place["attend"]) / len(in_place["attend"]), peaks,
                                          sustained, len(in_place["attend"]), traffic_of(name, "attend"))
    depth = job.depth
    return {"value": world * w.suffix_tokens / (step_ms_max * 1e-3), "ms_per_step": step_ms_max, "steps": steps,
            "warmup": warmup, "tflops": flops / (step_ms_max * 1e-3) / 1e12, "step_flops": flops,
            "gpu_launches": int(launches), "clocks": clocks, "roofline": roofline, "roofline_attend": roofline_attend,
            "config": dict(config_keys(w, depth), deep_layer_refresh=refresh_info)}


def measure_calls_alone(job, name, flush, peaks):
    """The `attend` and `attend_full` calls of one layer over all requests, each timed alone after an L2
    flush (CUDA events around the single call): the burst-peak view of the same two launches."""
    w, bc = job.w, job.bc
    pid = [bc.lookup_prefix(key)[0] for key in job.keys]
    req_pid = [pid[g] for g in w.req_prefix]

    def call_attend():
        bc.attend(0, req_pid, w.suffix_row_off, w.suffix_lens, job.q, job.k, job.v, job.out, None, w.softmax_scale)

    def call_full():
        bc.attend_full(0, w.full_row_off, w.full_lens, job.q, job.k, job.v, job.out, None, w.softmax_scale)

    iters = 10 if w.full_flops() < 5e13 else 3
    from paper_2606_07571_b200 import binding as _bind
    bc.set_path(_bind.PATH_AUTO)                       # whatever path the timed steps ran on
    call_attend()
    kernel = bc.last_attention_kernel()
    call_full()
    ms_attend = time_call(call_attend, iters, flush)
    ms_full = time_call(call_full, iters, flush)
    full = tensor_roofline("tc_attention_kernel (attend_full call alone)", w.full_flops(), ms_full, peaks, False,
                           iters, traffic_of(name, "full"))
    # The same call on the variant of the kernel that runs on pairs of SMs (an opt-in path: the measured
    # alternative, not what the steps use).
    pairs = None
    if w.dtype == torch.bfloat16 and w.head_dim == 128:
        bc.set_path(_bind.PATH_TENSOR_PAIRS)
        call_full()
        if bc.last_attention_kernel() == _bind.KERNEL_TENSOR_PAIRS:
            pairs = tensor_roofline("tc_attention_pair_kernel (attend_full call alone, opt-in path)", w.full_flops(),
                                    time_call(call_full, iters, flush), peaks, False, iters, (None, None))
        bc.set_path(_bind.PATH_AUTO)
    if kernel != 3:                                    # not the key-range kernel
        attend = tensor_roofline("tc_attention_kernel (attend call alone)", w.attend_flops(), ms_attend, peaks, False,
                                 iters, traffic_of(name, "attend"))
        return {"attend_full": full, "attend": attend, "attend_full_cta_pairs": pairs}
    # few query rows against a long cached prefix: the call is bound by reading the prefix once
    gbs = w.attend_bytes() / (ms_attend * 1e-3) / 1e9
    # The same call replayed from a CUDA graph (ten calls per replay): what a serving loop that
    # captures its steps sees, without the host time of the Python binding per call.  Only for
    # prefixes larger than L2, where back-to-back calls still read the keys from HBM.
    graph_ms = None
    if w.attend_bytes() > (200 << 20):
        try:
            st = torch.cuda.Stream()
            with torch.cuda.stream(st):
                call_attend()
                torch.cuda.synchronize()
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, stream=st):
                    for _ in range(10):
                        call_attend()
                ts = []
                for _ in range(5):
                    flush.zero_()
                    flush.max()
                    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    a.record(st)
                    g.replay()
                    b.record(st)
                    torch.cuda.synchronize()
                    ts.append(a.elapsed_time(b) / 10)
            graph_ms = sorted(ts)[len(ts) // 2]
        except Exception:                              # capture not available: the figure is left out
            graph_ms = None
    # Host time of one call: through the Python binding (marshalling of the metadata lists every call)
    # and through the C ABI itself with the arguments marshalled once (what a C caller pays).  Enqueue
    # only: 100 calls back to back, then one synchronisation.
    import ctypes as C
    from paper_2606_07571_b200 import binding as _b
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for _ in range(100):
        call_attend()
    host_binding_us = (time.perf_counter() - t0) / 100 * 1e6
    torch.cuda.synchronize()
    pid_a, pid_p = _b._i32(req_pid)
    off_a, off_p = _b._i64(w.suffix_row_off)
    len_a, len_p = _b._i32(w.suffix_lens)
    qp, kp, vp_, qs, ks, op, os_, lp = bc._tensor_args(job.q, job.k, job.v, job.out, None)
    args = (bc.ctx, 0, len(len_a), pid_p, off_p, len_p, qp, kp, vp_, qs, ks, op, os_, lp, C.c_float(w.softmax_scale),
            bc._stream())
    t0 = time.perf_counter()
    for _ in range(100):
        bc.lib.bicache_attend(*args)
    host_c_us = (time.perf_counter() - t0) / 100 * 1e6
    torch.cuda.synchronize()
    assert bc.device_status() == 0
    tr = traffic_of(name, "attend")
    attend = {"bound": "hbm", "kernel": "tc_decode_kernel (+ merge) (attend call alone)",
              "host_us_per_call": {"python_binding": host_binding_us, "c_abi_premarshalled": host_c_us},
              "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": gbs / peaks["hbm_gbs"],
              "peak_source": peaks["source"], "bytes_per_launch": w.attend_bytes(), "ms_per_launch": ms_attend,
              "launches_timed": iters, "tflops": w.attend_flops() / (ms_attend * 1e-3) / 1e12,
              "graph_replay": (None if graph_ms is None else
                               {"ms_per_call": graph_ms, "calls_per_replay": 10,
                                "achieved": w.attend_bytes() / (graph_ms * 1e-3) / 1e9,
                                "frac": w.attend_bytes() / (graph_ms * 1e-3) / 1e9 / peaks["hbm_gbs"]}),
              "traffic": tr[0], "traffic_source": tr[1]}
    return {"attend_full": full, "attend": attend, "attend_full_cta_pairs": pairs}


def pinned_like(t, chunk_bytes=1 << 30):
    """Pinned host buffers for a [rows, ...] tensor, in chunks of at most `chunk_bytes` (a list of
    (first row, buffer)): one allocation per gigabyte instead of one of many."""
    rows = t.shape[0]
    row_bytes = max(1, t[0].numel() * t.element_size())
    step = max(1, chunk_bytes // row_bytes)
    return [(r0, torch.empty((min(step, rows - r0),) + tuple(t.shape[1:]), dtype=t.dtype, pin_memory=True))
            for r0 in range(0, rows, step)]


def measure_e2e(job, steps, world, dist):
    """The same step with HOST inputs and outputs: every step uploads its Q, K, V from pinned host
    memory and downloads its output(s); the copies are inside the timed region."""
    w = job.w
    host_in = []
    for x in (job.q, job.k, job.v):
        chunks = pinned_like(x)
        for r0, c in chunks:
            c.copy_(x[r0:r0 + c.shape[0]])
        host_in.append(chunks)
    n_out = 2 if job.single_layer else 1
    # Two buffer sets and three streams: the upload of step i + 1 and the download of step i - 1
    # run while step i computes (every step still uploads its own inputs and downloads its own
    # outputs; the figure is the steady-state time per step of that pipeline).
    dev = [tuple(torch.empty_like(x) for x in (job.q, job.k, job.v)) +
           tuple(torch.empty_like(job.out) for _ in range(n_out)) for _ in range(2)]
    host_out = [[pinned_like(job.out) for _ in range(n_out)] for _ in range(2)]
    s_c = torch.cuda.current_stream()
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()

    def upload(dst, chunks):
        for r0, c in chunks:
            dst[r0:r0 + c.shape[0]].copy_(c, non_blocking=True)

    def download(chunks, src):
        for r0, c in chunks:
            c.copy_(src[r0:r0 + c.shape[0]], non_blocking=True)

    def run(n):
        ev_in = [torch.cuda.Event() for _ in range(2)]
        ev_done = [torch.cuda.Event() for _ in range(2)]
        ev_out = [torch.cuda.Event() for _ in range(2)]
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        t0.record(s_c)
        s_in.wait_event(t0)
        for i in range(n):
            b = i % 2
            bq, bk, bv = dev[b][:3]
            bo = dev[b][3:]
            with torch.cuda.stream(s_in):
                if i >= 2:
                    s_in.wait_event(ev_done[b])            # step i - 2 no longer reads this buffer set
                upload(bq, host_in[0])
                upload(bk, host_in[1])
                upload(bv, host_in[2])
                ev_in[b].record(s_in)
            s_c.wait_event(ev_in[b])
            if i >= 2:
                s_c.wait_event(ev_out[b])                  # its outputs of step i - 2 are on the host
            job.step(bq, bk, bv, bo[0], bo[1] if n_out == 2 else None)
            ev_done[b].record(s_c)
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev_done[b])
                for j in range(n_out):
                    download(host_out[b][j], bo[j])
                ev_out[b].record(s_out)
        s_c.wait_event(ev_out[0])
        if n > 1:
            s_c.wait_event(ev_out[1])
        t1.record(s_c)
        torch.cuda.synchronize()
        return t0.elapsed_time(t1) / n

    run(2)
    e2e_ms = max_over_ranks(run(steps), dist, "cuda")
    h2d = sum(x.numel() * x.element_size() for x in (job.q, job.k, job.v))
    d2h = job.out.numel() * job.out.element_size() * n_out
    del dev, host_out, host_in
    torch.cuda.empty_cache()
    return {"value": world * w.suffix_tokens / (e2e_ms * 1e-3), "unit": UNIT, "ms_per_step": e2e_ms,
            "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
            "how": "pinned host buffers (1 GiB chunks); upload, compute and download of consecutive steps overlap "
                   "(two device buffer sets, three streams); time of %d steps / %d" % (steps, steps)}


# ---- the oracle as a timed CPU baseline ------------------------------------------------------------

def oracle_sample_plan(w, flop_budget):
    """Which part of a step the oracle is timed on: (request, KV head, query rows of the deep-layer pass)
    units, median-length request first and then spread over the length distribution, until about
    `flop_budget` algorithmic FLOPs are planned.  A unit is the shallow-layer pass (all suffix rows) and the
    deep-layer pass (the first `rows` rows) of the query heads that share one KV head."""
    R, G = w.num_requests, w.num_q_heads // w.num_kv_heads
    order = np.argsort(w.suffix_lens, kind="stable")
    picks = [int(order[R // 2])] + [int(order[(j * 7919) % R]) for j in range(1, R)]
    plan, seen, used = [], set(), 0.0
    for i in picks:
        if i in seen:
            continue
        seen.add(i)
        n, m = w.suffix_lens[i], w.prefix_lens[w.req_prefix[i]]
        N = m + n
        fa = 4.0 * w.head_dim * G * n * N
        left = max(flop_budget - used - fa, 0.25 * flop_budget)
        rows = int(min(N, max(64, left // (4.0 * w.head_dim * G * N))))
        plan.append((i, (7 * i) % w.num_kv_heads, rows))
        used += fa + 4.0 * w.head_dim * G * rows * N
        if used >= flop_budget:
            break
    return plan


def oracle_run_plan(w, workloads, oracle, plan):
    """Runs the oracle on the planned units.  Returns (seconds shallow, seconds deep, FLOPs shallow, FLOPs deep)."""
    G = w.num_q_heads // w.num_kv_heads
    ta = tf = fa = ff = 0.0
    for i, hk, rows in plan:
        g = w.req_prefix[i]
        m, n = w.prefix_lens[g], w.suffix_lens[i]
        sub = workloads.Workload("sample", 1, G, 1, w.head_dim, w.dtype, 16, [m], [0], [n],
                                 softmax_scale=w.softmax_scale, seed=w.seed + 131 * i + hk)
        kc, vc = workloads.draw_prefix_kv(sub, 0, "cpu")
        q, k, v = workloads.draw_full_qkv(sub, "cpu")
        st = oracle.PagedPrefixStore(1, 1, w.head_dim, 16, sub.pages_needed())
        qd, kd, vd = (workloads.to_f64(x) for x in (q, k, v))
        pid, _, _ = st.put(1, workloads.to_f64(kc), workloads.to_f64(vc))
        t0 = time.perf_counter()
        oracle.attend(st, 0, [pid], sub.suffix_row_off, sub.suffix_lens, qd, kd, vd, w.softmax_scale)
        t1 = time.perf_counter()
        # deep-layer pass of the first `rows` query rows over all N keys (Eq. 2 row by row is independent)
        oracle.attention(qd[:rows], kd, vd, w.softmax_scale)
        t2 = time.perf_counter()
        ta, tf = ta + (t1 - t0), tf + (t2 - t1)
        fa += 4.0 * w.head_dim * G * n * (m + n)
        ff += 4.0 * w.head_dim * G * rows * (m + n)
    return ta, tf, fa, ff


def oracle_step_estimate(w, depth, ta, tf, fa, ff):
    """Whole-step time of the oracle: the sampled times scaled by the step's algorithmic FLOPs."""
    tot = 0.0
    for j in range(w.num_requests):
        nj, mj = w.suffix_lens[j], w.prefix_lens[w.req_prefix[j]]
        fa_j = 4.0 * w.head_dim * w.num_q_heads * nj * (mj + nj)
        ff_j = 4.0 * w.head_dim * w.num_q_heads * (mj + nj) ** 2
        if w.num_layers == 1:
            tot += ta * fa_j / fa + tf * ff_j / ff
        else:
            tot += int(depth[j]) * ta * fa_j / fa + (w.num_layers - int(depth[j])) * tf * ff_j / ff
    return tot


def plan_text(w, plan, seconds):
    units = ", ".join("request %d KV head %d (%d of %d deep-layer query rows)"
                      % (i, hk, rows, w.prefix_lens[w.req_prefix[i]] + w.suffix_lens[i]) for i, hk, rows in plan[:3])
    more = "" if len(plan) <= 3 else " and %d more" % (len(plan) - 3)
    return ("%d (request, KV head) unit(s): %s%s; per unit one shallow-layer oracle pass (all suffix rows) and one "
            "deep-layer pass (the stated rows, all keys), %.1f s of oracle work; step time = sampled time scaled "
            "by algorithmic FLOPs" % (len(plan), units, more, seconds))


def host_cores():
    try:
        from threadpoolctl import threadpool_info
        n = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
        return int(n)
    except Exception:
        return len(os.sched_getaffinity(0))


def config_keys(w, depth):
    """The `config` object both arms print."""
    return {"workload": w.name, "note": w.note, "layers": w.num_layers, "requests": w.num_requests,
            "suffix_tokens": w.suffix_tokens,
            "l2": "flushed before every timed step (256 MB write); the tensors of a step exceed L2",
            "step": ("shallow-layer pass + deep-layer pass of the single layer"
                     if w.num_layers == 1 else "all layers, per-request depths from the rule"),
            "depth_min": int(min(depth)), "depth_max": int(max(depth)), "deep_layer_refresh": None}


def run_reference(args, w):
    """The oracle arm: the CPU oracle as it stands, timed on the host cores.  Every step (warm-up steps
    included) runs the same bounded sample of the workload; `ms_per_step` is the measured time of that
    sample, `value` the tokens/s of a whole step at the sampled rate."""
    import oracle
    from paper_2606_07571_b200 import workloads
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    table = workloads.standin_depth_table(w.num_layers)
    depth = oracle.reuse_depth(w.req_prefix_len(), w.suffix_lens, table, w.num_layers)
    plan = oracle_sample_plan(w, args.ref_flops)
    for _ in range(args.warmup):
        oracle_run_plan(w, workloads, oracle, plan)
    times, est = [], []
    for _ in range(args.steps):
        ta, tf, fa, ff = oracle_run_plan(w, workloads, oracle, plan)
        times.append(ta + tf)
        est.append(oracle_step_estimate(w, depth, ta, tf, fa, ff))
    sec_sample, sec_step = float(np.mean(times)), float(np.mean(est))
    value = w.suffix_tokens / sec_step
    desc = plan_text(w, plan, sec_sample) + "; every step repeats this sample"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec_sample * 1e3,
            "ms_per_whole_step_extrapolated": sec_step * 1e3, "sample_fraction_of_step": sec_sample / sec_step,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": config_keys(w, depth),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": host_cores(), "kind": "oracle", "sample": desc},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def measure_extras(job, name, flush, peaks):
    """Off the per-step path: prefix put (scatter into page images), the profiler's similarity
    reduction (Eq. 3) and the K/V projection into the store (Eq. 1), each on prefix 0."""
    w, bc, workloads = job.w, job.bc, job.workloads
    pid = [bc.lookup_prefix(key)[0] for key in job.keys]
    es = 2 if w.dtype == torch.bfloat16 else 4
    put_bytes = 4 * w.num_layers * w.prefix_lens[0] * w.num_kv_heads * w.head_dim * es
    out = {"roofline_put": None, "roofline_similarity": None, "roofline_project": None}
    if w.dtype == torch.bfloat16 and w.head_dim == 128:
        m0, d_model = w.prefix_lens[0], w.num_q_heads * w.head_dim
        hh, wk_, wv_ = workloads.draw_hidden_and_weights(m0, d_model, w.num_kv_heads, w.head_dim, 1, device="cuda")
        ts = []
        for i in range(8):
            flush.zero_()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            bc.project_prefix_layer(pid[0], 0, hh, wk_, wv_)
            b.record()
            torch.cuda.synchronize()
            ts.append(a.elapsed_time(b))
        del hh, wk_, wv_
        ms_proj = sorted(ts[3:])[len(ts[3:]) // 2]
        proj_flops = 2.0 * m0 * d_model * 2 * w.num_kv_heads * w.head_dim
        tf = proj_flops / (ms_proj * 1e-3) / 1e12
        tr = traffic_of(name, "project")
        out["roofline_project"] = {
            "bound": "tensor", "kernel": "project_kv_kernel (project_prefix_layer of prefix 0, one layer)",
            "achieved": tf, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s", "frac": tf / peaks["bf16_tflops"],
            "peak_source": peaks["source"] + " burst", "flops_per_launch": proj_flops, "ms_per_launch": ms_proj,
            "d_model": d_model, "traffic": tr[0], "traffic_source": tr[1]}
    if put_bytes >= (256 << 20):
        # Timed last: every put of a fresh key evicts the oldest prefix (FIFO), the workload's own first.
        kc, vc = workloads.draw_prefix_kv(w, 0, "cuda")
        ts = []
        sim_dev = torch.zeros(w.num_layers, dtype=torch.float32, device="cuda")
        for i in range(5):
            flush.zero_()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            bc.prefix_similarity_async(pid[0], kc, vc, sim_dev)
            b.record()
            torch.cuda.synchronize()
            ts.append(a.elapsed_time(b))
        ms_sim = sorted(ts[1:])[len(ts[1:]) // 2]
        gbs = put_bytes / (ms_sim * 1e-3) / 1e9
        tr = traffic_of(name, "similarity")
        out["roofline_similarity"] = {
            "bound": "hbm", "kernel": "kv_similarity_partial_kernel (prefix_similarity of prefix 0)",
            "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": gbs / peaks["hbm_gbs"],
            "peak_source": peaks["source"], "bytes_per_launch": put_bytes, "ms_per_launch": ms_sim,
            "traffic": tr[0], "traffic_source": tr[1]}
        ts = []
        for i in range(5):
            flush.zero_()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            bc.put_prefix(0x7000000000000000 + i, kc, vc)
            b.record()
            torch.cuda.synchronize()
            ts.append(a.elapsed_time(b))
        del kc, vc
        ms_put = sorted(ts[1:])[len(ts[1:]) // 2]
        gbs = put_bytes / (ms_put * 1e-3) / 1e9
        tr = traffic_of(name, "put")
        out["roofline_put"] = {
            "bound": "hbm", "kernel": "scatter_prefix_kernel (put_prefix of prefix 0, all layers)",
            "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": gbs / peaks["hbm_gbs"],
            "peak_source": peaks["source"], "bytes_per_launch": put_bytes, "ms_per_launch": ms_put,
            "traffic": tr[0], "traffic_source": tr[1]}
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD)
    ap.add_argument("--impl", default="ours")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-extras", action="store_true", help="skip the put / similarity / projection launches")
    ap.add_argument("--per-config", choices=("auto", "on", "off"), default="auto",
                    help="also measure the other configurations and the small-suffix shapes (auto: when the "
                         "default workload runs on one GPU)")
    ap.add_argument("--cpu-flops", type=float, default=1.5e12, help="algorithmic FLOPs of the cpu_baseline sample")
    ap.add_argument("--ref-flops", type=float, default=2.5e11,
                    help="algorithmic FLOPs of the sample one step of --impl reference runs")
    ap.add_argument("--delta", type=int, default=0,
                    help="refresh interval of the deep layers' kept prefix K/V (Eq. 5); 0: recompute every step")
    ap.add_argument("--attend-full-path", choices=("default", "pairs"), default="default",
                    help="pairs: the timed steps run full attention on the CTA-pair variant of the tensor-core "
                         "kernel (an opt-in path of the library; slower, see the design notes)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    args.steps = max(args.steps, 1)

    from paper_2606_07571_b200 import workloads
    w = workloads.CONFIGS[args.workload]()
    if args.impl == "reference":
        run_reference(args, w)
        return

    import __graft_entry__ as entry
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if rank == 0:
        entry.build()
    dist = None
    if world > 1:
        import torch.distributed as dist
        torch.cuda.set_device(local_rank)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
        dist.barrier()
        if rank != 0:
            entry.build()
    peaks = load_peaks()
    job = Job(w, local_rank, args.delta)
    if args.attend_full_path == "pairs":
        job.bc.set_path(job.binding.PATH_TENSOR_PAIRS)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")       # 2x the 126 MB L2

    rec = measure_steps(job, args.workload, args.steps, args.warmup, flush, peaks, rank, local_rank, world, dist)
    if args.attend_full_path == "pairs":
        rec["config"]["attend_full_path"] = "cta pairs (opt-in)"
    alone = measure_calls_alone(job, args.workload, flush, peaks)
    # where no layer has every request on one path, the launch timed alone stands in
    if rec["roofline"] is None:
        rec["roofline"] = alone["attend_full"]
    if rec["roofline_attend"] is None or alone["attend"]["bound"] == "hbm":
        rec["roofline_attend"] = alone["attend"]

    e2e = None
    if not args.no_e2e:
        e2e = measure_e2e(job, max(3, min(args.steps, 6 if rec["ms_per_step"] > 100 else 16)), world, dist)

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        import oracle
        plan = oracle_sample_plan(w, args.cpu_flops)
        ta, tf, fa, ff = oracle_run_plan(w, workloads, oracle, plan)
        sec = oracle_step_estimate(w, job.depth, ta, tf, fa, ff)
        cpu = {"value": w.suffix_tokens / sec, "unit": UNIT, "cores": host_cores(), "kind": "oracle",
               "sample": plan_text(w, plan, ta + tf)}

    extras = {"roofline_put": None, "roofline_similarity": None, "roofline_project": None}
    if not args.no_extras:
        extras = measure_extras(job, args.workload, flush, peaks)
    job.close()

    # ---- the other configurations and the small-suffix shapes, a few steps each ----------------------
    per_config = None
    want_sub = args.per_config == "on" or (args.per_config == "auto" and args.workload == DEFAULT_WORKLOAD
                                           and world == 1 and args.delta == 0)
    if want_sub and rank == 0 and world == 1:
        per_config = []
        for name, steps in PER_CONFIG:
            if name == args.workload:
                continue
            sj = Job(workloads.CONFIGS[name](), local_rank)
            r = measure_steps(sj, name, steps, 3, flush, peaks, 0, local_rank, 1, None)
            a = measure_calls_alone(sj, name, flush, peaks)
            sj.close()
            per_config.append({"workload": sj.w.name, "value": r["value"], "unit": UNIT, "ms_per_step": r["ms_per_step"],
                               "steps": steps, "warmup": 3, "tflops": r["tflops"], "gpu_launches": r["gpu_launches"],
                               "roofline": r["roofline"] or a["attend_full"],
                               "roofline_attend": r["roofline_attend"] or a["attend"],
                               "calls_alone": a, "clocks": r["clocks"], "config": r["config"]})
        for name in SMALL_SUFFIX:
            sw = workloads.CONFIGS[name]()
            sj = Job(sw, local_rank)
            sampler = ClockSampler(local_rank)
            sampler.start()
            a = measure_calls_alone(sj, name, flush, peaks)
            clocks = sampler.stop()
            sj.close()
            per_config.append({"workload": sw.name, "note": sw.note, "roofline_attend": a["attend"], "clocks": clocks})

    if rank == 0:
        line = {"metric": METRIC, "value": rec["value"], "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": rec["ms_per_step"], "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": "bf16" if w.dtype == torch.bfloat16 else "f32", "data": "synthetic",
                "config": rec["config"], "tflops": rec["tflops"], "step_flops": rec["step_flops"],
                "clocks": rec["clocks"], "e2e": e2e, "gpu_launches": rec["gpu_launches"],
                "roofline": rec["roofline"], "roofline_attend": rec["roofline_attend"], "calls_alone": alone,
                "roofline_put": extras["roofline_put"], "roofline_similarity": extras["roofline_similarity"],
                "roofline_project": extras["roofline_project"], "cpu_baseline": cpu, "per_config": per_config}
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
