#!/usr/bin/env python
"""Benchmark of the BiCache attention hot path.

One "step" is one denoising step's attention: reuse-depth rule, prefix-store lookups (hits), the
per-layer dispatch, and for every layer the shallow-layer call (suffix queries over cached prefix
K/V + own suffix K/V) and/or the deep-layer fallback (full bidirectional attention), all through
the C ABI.  The default workload is the LLaDA-8B-shaped single layer (prefix 1024, 16 requests x
256 suffix tokens, bf16): being one layer, its step runs the layer once as a shallow layer (every
request reuses, as the depth rule says) and once as a deep layer (every request recomputes), so
that every stage of the path is inside the timed region.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload config2] [--impl reference]

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

# DRAM bytes (read + write) of one launch of the dominant kernel, from ncu captures summarised
# under profiles/ (None until a capture of that workload exists).
NCU_TRAFFIC_BYTES = {"config2": {"full": 647.9e6, "attend": 135.3e6},     # profiles/tc_attention_kernel_config2.md
                     "config3": {"put": 2104.6e6, "similarity": 2147.6e6,    # profiles/hbm_kernels_config3.md
                                 "project": 218.0e6},                         # profiles/project_kv_kernel_config3.md
                     "b2": {"attend": 274.1e6}}                               # profiles/key_range_kernels_b2.md


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"bf16_tflops": p["bf16_tflops"], "bf16_tflops_sustained": p.get("bf16_tflops_sustained"),
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
        if self.delta > 0:                            # per-request kept prefix K/V of the deep layers
            npages += sum((w.prefix_lens[g] + 15) // 16 for g in w.req_prefix)
        order = workloads.shuffled_page_order(npages, 7) if w.shuffle_pages else None
        self.bc = binding.BiCache(w.num_layers, w.num_q_heads, w.num_kv_heads, w.head_dim, npages, w.dtype,
                                  w.total_rows, w.num_requests, device=device, free_order=order)
        self.bc.set_depth_table(workloads.standin_depth_table(w.num_layers))
        self.keys = [workloads.prefix_key(w, g) for g in range(len(w.prefix_lens))]
        for g in range(len(w.prefix_lens)):
            kc, vc = workloads.draw_prefix_kv(w, g, "cuda")
            self.bc.put_prefix(self.keys[g], kc, vc)
            del kc, vc
        self.private = [-1] * w.num_requests
        if self.delta > 0:
            self.private = [self.bc.reserve_prefix(0x6000000000000000 + i, w.prefix_lens[g])[0]
                            for i, g in enumerate(w.req_prefix)]
        self.q, self.k, self.v = workloads.draw_full_qkv(w, "cuda")
        self.out = torch.empty_like(self.q)
        self.single_layer = w.num_layers == 1
        self.out2 = torch.empty_like(self.q) if self.single_layer else None
        torch.cuda.synchronize()

    def step(self, q=None, k=None, v=None, out=None, out2=None):
        """One denoising step's attention through the C ABI."""
        w, bc = self.w, self.bc
        q = self.q if q is None else q
        k = self.k if k is None else k
        v = self.v if v is None else v
        out = self.out if out is None else out
        out2 = self.out2 if out2 is None else out2
        depth = bc.reuse_depth(w.req_prefix_len(), w.suffix_lens)                     # depth rule
        pid = [bc.lookup_prefix(key)[0] for key in self.keys]                         # store hits
        req_pid = [pid[g] for g in w.req_prefix]
        if self.single_layer:
            # shallow-layer pass (depths from the rule) then deep-layer pass (all recompute)
            bc.attend_layer(0, depth, req_pid, w.full_row_off, w.full_lens, q, k, v, out, None, w.softmax_scale)
            bc.attend_layer(0, [0] * w.num_requests, req_pid, w.full_row_off, w.full_lens, q, k, v, out2, None,
                            w.softmax_scale)
        elif self.delta > 0:
            # deep layers keep the request's own prefix K/V and recompute them every delta steps
            for l in range(w.num_layers):
                bc.attend_step(l, self.t, self.delta, depth, req_pid, self.private, w.full_row_off, w.full_lens,
                               q, k, v, out, None, w.softmax_scale)
            self.t += 1
        else:
            for l in range(w.num_layers):
                bc.attend_layer(l, depth, req_pid, w.full_row_off, w.full_lens, q, k, v, out, None,
                                w.softmax_scale)
        return depth

    def step_flops(self):
        w = self.w
        depth = self.bc.reuse_depth(w.req_prefix_len(), w.suffix_lens)
        per_req_attend = [4 * w.head_dim * w.num_q_heads * n * (w.prefix_lens[g] + n)
                          for g, n in zip(w.req_prefix, w.suffix_lens)]
        per_req_full = [4 * w.head_dim * w.num_q_heads * N * N for N in w.full_lens]
        if self.single_layer:
            return sum(per_req_attend) + sum(per_req_full), depth
        tot = 0
        for i in range(w.num_requests):
            tot += int(depth[i]) * per_req_attend[i] + (w.num_layers - int(depth[i])) * per_req_full[i]
        return tot, depth

    def reuse_step_flops(self):
        """A step between two refresh steps: every layer reads a cached prefix (shared or kept)."""
        w = self.w
        return w.num_layers * sum(4 * w.head_dim * w.num_q_heads * n * (w.prefix_lens[g] + n)
                                  for g, n in zip(w.req_prefix, w.suffix_lens))


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


def oracle_one_request(w, workloads, oracle, i):
    """The oracle on request i of the workload: one shallow-layer and one deep-layer pass (all heads).
    Returns (seconds of the shallow pass, seconds of the deep pass)."""
    g = w.req_prefix[i]
    m, n = w.prefix_lens[g], w.suffix_lens[i]
    sub = workloads.Workload("sample", 1, w.num_q_heads, w.num_kv_heads, w.head_dim, w.dtype, 16, [m], [0], [n],
                             softmax_scale=w.softmax_scale, seed=w.seed + i)
    kc, vc = workloads.draw_prefix_kv(sub, 0, "cpu")
    q, k, v = workloads.draw_full_qkv(sub, "cpu")
    st = oracle.PagedPrefixStore(1, w.num_kv_heads, w.head_dim, 16, sub.pages_needed())
    qd, kd, vd = (workloads.to_f64(x) for x in (q, k, v))
    pid, _, _ = st.put(1, workloads.to_f64(kc), workloads.to_f64(vc))
    t0 = time.perf_counter()
    oracle.attend(st, 0, [pid], sub.suffix_row_off, sub.suffix_lens, qd, kd, vd, w.softmax_scale)
    t1 = time.perf_counter()
    oracle.attend_full(sub.full_row_off, sub.full_lens, qd, kd, vd, w.softmax_scale)
    t2 = time.perf_counter()
    return (t1 - t0), (t2 - t1)


def oracle_step_seconds(w, workloads, oracle, depth, budget_s=12.0):
    """Time of one whole step for the oracle.  Requests are sampled (median length first, then
    spread over the length distribution) until about `budget_s` seconds of oracle work are done;
    the step time is the sampled time scaled by the step's algorithmic FLOPs over the sample's."""
    order = np.argsort(w.suffix_lens)
    R = w.num_requests
    picks = [int(order[R // 2])] + [int(order[(j * 7919) % R]) for j in range(1, R)]
    seen, ta, tf, fa, ff = [], 0.0, 0.0, 0.0, 0.0
    for i in picks:
        if i in seen:
            continue
        a, f = oracle_one_request(w, workloads, oracle, i)
        n, m = w.suffix_lens[i], w.prefix_lens[w.req_prefix[i]]
        seen.append(i)
        ta, tf = ta + a, tf + f
        fa += 4.0 * w.head_dim * w.num_q_heads * n * (m + n)
        ff += 4.0 * w.head_dim * w.num_q_heads * (m + n) ** 2
        if ta + tf >= budget_s:
            break
    tot = 0.0
    for j in range(R):
        nj, mj = w.suffix_lens[j], w.prefix_lens[w.req_prefix[j]]
        fa_j = 4.0 * w.head_dim * w.num_q_heads * nj * (mj + nj)
        ff_j = 4.0 * w.head_dim * w.num_q_heads * (mj + nj) ** 2
        if w.num_layers == 1:
            tot += ta * fa_j / fa + tf * ff_j / ff
        else:
            tot += int(depth[j]) * ta * fa_j / fa + (w.num_layers - int(depth[j])) * tf * ff_j / ff
    desc = ("%d of %d requests (all heads), one shallow-layer and one deep-layer oracle pass each, %.1f s of "
            "oracle work; step time = sampled time scaled by algorithmic FLOPs" % (len(seen), R, ta + tf))
    return tot, desc, ta + tf


def host_cores():
    try:
        from threadpoolctl import threadpool_info
        n = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
        return int(n)
    except Exception:
        return len(os.sched_getaffinity(0))


def run_reference(args, w):
    """The oracle arm: the CPU oracle as it stands, timed on the host cores."""
    import oracle
    from paper_2606_07571_b200 import workloads
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    table = workloads.standin_depth_table(w.num_layers)
    depth = oracle.reuse_depth(w.req_prefix_len(), w.suffix_lens, table, w.num_layers)
    for _ in range(min(args.warmup, 1)):
        oracle_step_seconds(w, workloads, oracle, depth)
    times, desc = [], ""
    for _ in range(max(1, min(args.steps, 3))):
        t, desc, _ = oracle_step_seconds(w, workloads, oracle, depth)
        times.append(t)
    sec = float(np.mean(times))
    value = w.suffix_tokens / sec
    cores = host_cores()
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": w.name, "note": w.note},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="config2")
    ap.add_argument("--impl", default="ours")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--delta", type=int, default=0,
                    help="refresh interval of the deep layers' kept prefix K/V (Eq. 5); 0: recompute every step")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)

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
    flops, depth = job.step_flops()
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")       # 2x the 126 MB L2

    # ---- device-resident timing: K steps, each preceded by an (untimed) L2 flush -------------
    for _ in range(args.warmup):
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
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    job.t = 1                                         # the timed steps are denoising steps 1 .. K
    for a, b in ev:
        flush.zero_()
        a.record()
        job.step()
        b.record()
    torch.cuda.synchronize()
    launches = job.bc.launch_count() - launches0
    per_step_ms = [a.elapsed_time(b) for a, b in ev]
    step_ms = sum(per_step_ms) / args.steps
    refresh_info = None
    if job.delta > 0:
        is_ref = [(t - 1) % job.delta == 0 for t in range(1, args.steps + 1)]
        ref_ms = [m for m, r in zip(per_step_ms, is_ref) if r]
        reu_ms = [m for m, r in zip(per_step_ms, is_ref) if not r]
        flops = (len(ref_ms) * flops + len(reu_ms) * job.reuse_step_flops()) / args.steps   # mean FLOPs per step
        refresh_info = {"delta": job.delta, "refresh_steps": len(ref_ms), "reuse_steps": len(reu_ms),
                        "ms_refresh_step": sum(ref_ms) / max(1, len(ref_ms)),
                        "ms_reuse_step": sum(reu_ms) / max(1, len(reu_ms)) if reu_ms else None}
    # a short sustained stretch so that the clock sampler sees the kernels under load
    t_end = time.time() + 0.6
    while time.time() < t_end:
        job.step()
        torch.cuda.synchronize()
    clocks = sampler.stop() if rank == 0 else None
    assert job.bc.device_status() == 0
    step_ms_max = max_over_ranks(step_ms, dist, "cuda")
    if dist is not None:
        dist.barrier()
    value = world * w.suffix_tokens / (step_ms_max * 1e-3)

    # ---- per-call timing for the roofline (CUDA events around the single kernel launch) ------
    bc = job.bc
    pid = [bc.lookup_prefix(key)[0] for key in job.keys]
    req_pid = [pid[g] for g in w.req_prefix]
    layer_mid = 0

    def call_attend():
        bc.attend(layer_mid, req_pid, w.suffix_row_off, w.suffix_lens, job.q, job.k, job.v, job.out, None,
                  w.softmax_scale)

    def call_full():
        bc.attend_full(layer_mid, w.full_row_off, w.full_lens, job.q, job.k, job.v, job.out, None, w.softmax_scale)

    iters = 10 if w.full_flops() < 5e13 else 3
    call_attend(); call_full()
    ms_attend = time_call(call_attend, iters, flush)
    ms_full = time_call(call_full, iters, flush)
    tf_attend = w.attend_flops() / (ms_attend * 1e-3) / 1e12
    tf_full = w.full_flops() / (ms_full * 1e-3) / 1e12
    peak = peaks["bf16_tflops"]
    roofline = {"bound": "tensor", "kernel": "tc_attention_kernel (attend_full launch)", "achieved": tf_full,
                "peak": peak, "unit": "TFLOP/s", "frac": tf_full / peak, "peak_source": peaks["source"] + " burst",
                "traffic": NCU_TRAFFIC_BYTES.get(args.workload, {}).get("full"),
                "flops_per_launch": w.full_flops(), "ms_per_launch": ms_full}
    roofline_attend = {"bound": "tensor", "kernel": "tc_attention_kernel (attend launch)", "achieved": tf_attend,
                       "peak": peak, "unit": "TFLOP/s", "frac": tf_attend / peak,
                       "traffic": NCU_TRAFFIC_BYTES.get(args.workload, {}).get("attend"),
                       "flops_per_launch": w.attend_flops(), "ms_per_launch": ms_attend}
    call_attend()
    if bc.last_attention_kernel() == 3:                    # the key-range kernel (BICACHE_KERNEL_KEY_RANGES)
        # few query rows against a long cached prefix: the launch is bound by reading the prefix once
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
        roofline_attend = {"bound": "hbm", "kernel": "tc_decode_kernel + merge_ranges_kernel (attend call)",
                           "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": gbs / peaks["hbm_gbs"],
                           "peak_source": peaks["source"], "bytes_per_launch": w.attend_bytes(),
                           "ms_per_launch": ms_attend, "tflops": tf_attend,
                           "graph_replay": (None if graph_ms is None else
                                            {"ms_per_call": graph_ms, "calls_per_replay": 10,
                                             "achieved": w.attend_bytes() / (graph_ms * 1e-3) / 1e9,
                                             "frac": w.attend_bytes() / (graph_ms * 1e-3) / 1e9 / peaks["hbm_gbs"]}),
                           "traffic": NCU_TRAFFIC_BYTES.get(args.workload, {}).get("attend")}

    # ---- end to end: host buffers, copies inside the timed region ------------------------------
    e2e = None
    if not args.no_e2e and w.total_rows * w.num_q_heads * w.head_dim * 2 < (4 << 30):
        hq, hk, hv = (x.to("cpu").pin_memory() for x in (job.q, job.k, job.v))
        ho = torch.empty_like(hq).pin_memory()
        ho2 = torch.empty_like(hq).pin_memory() if job.single_layer else None
        dq, dk, dv = (torch.empty_like(x) for x in (job.q, job.k, job.v))

        # Two buffer sets and three streams: the upload of step i + 1 and the download of step i - 1
        # run while step i computes (every step still uploads its own inputs and downloads its own
        # outputs; the figure is the steady-state time per step of that pipeline).
        dev = [(dq, dk, dv, torch.empty_like(job.out), torch.empty_like(job.out) if ho2 is not None else None),
               (torch.empty_like(dq), torch.empty_like(dk), torch.empty_like(dv), torch.empty_like(job.out),
                torch.empty_like(job.out) if ho2 is not None else None)]
        host_out = [(ho, ho2), (torch.empty_like(ho).pin_memory(), torch.empty_like(ho).pin_memory() if ho2 is not None else None)]
        s_c = torch.cuda.current_stream()
        s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()

        def e2e_run(n):
            ev_in = [torch.cuda.Event() for _ in range(2)]
            ev_done = [torch.cuda.Event() for _ in range(2)]
            ev_out = [torch.cuda.Event() for _ in range(2)]
            t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            t0.record(s_c)
            s_in.wait_event(t0)
            for i in range(n):
                b = i % 2
                bq, bk, bv, bo, bo2 = dev[b]
                with torch.cuda.stream(s_in):
                    if i >= 2:
                        s_in.wait_event(ev_done[b])            # step i - 2 no longer reads this buffer set
                    bq.copy_(hq, non_blocking=True)
                    bk.copy_(hk, non_blocking=True)
                    bv.copy_(hv, non_blocking=True)
                    ev_in[b].record(s_in)
                s_c.wait_event(ev_in[b])
                if i >= 2:
                    s_c.wait_event(ev_out[b])                  # its outputs of step i - 2 are on the host
                job.step(bq, bk, bv, bo, bo2)
                ev_done[b].record(s_c)
                with torch.cuda.stream(s_out):
                    s_out.wait_event(ev_done[b])
                    host_out[b][0].copy_(bo, non_blocking=True)
                    if bo2 is not None:
                        host_out[b][1].copy_(bo2, non_blocking=True)
                    ev_out[b].record(s_out)
            s_c.wait_event(ev_out[0])
            s_c.wait_event(ev_out[1])
            t1.record(s_c)
            torch.cuda.synchronize()
            return t0.elapsed_time(t1) / n

        e2e_run(3)
        n_e2e = max(4, min(args.steps, 16))
        e2e_ms = e2e_run(n_e2e)
        e2e_ms = max_over_ranks(e2e_ms, dist, "cuda")
        h2d = sum(x.numel() * x.element_size() for x in (hq, hk, hv))
        d2h = ho.numel() * ho.element_size() * (2 if ho2 is not None else 1)
        e2e = {"value": world * w.suffix_tokens / (e2e_ms * 1e-3), "unit": UNIT, "ms_per_step": e2e_ms,
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
               "how": "pinned host buffers; upload, compute and download of consecutive steps overlap "
                      "(two buffer sets, three streams); time of %d steps / %d" % (n_e2e, n_e2e)}

    # ---- CPU baseline: the oracle on a bounded sample (rank 0, N = 1 only) ---------------------
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        import oracle
        sec, desc, _ = oracle_step_seconds(w, workloads, oracle, depth)
        cpu = {"value": w.suffix_tokens / sec, "unit": UNIT, "cores": host_cores(), "kind": "oracle", "sample": desc}

    # ---- prefix store put (bandwidth-bound scatter into page images), off the per-step path ----
    # Timed last: every put of a fresh key evicts the oldest prefix (FIFO), the workload's own first.
    roofline_put = None
    put_bytes = 4 * w.num_layers * w.prefix_lens[0] * w.num_kv_heads * w.head_dim * (2 if w.dtype == torch.bfloat16 else 4)
    roofline_sim = None
    # ---- prefix K/V projection into the store (Eq. 1), one layer of prefix 0, off the per-step path ----
    roofline_proj = None
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
        roofline_proj = {"bound": "tensor", "kernel": "project_kv_kernel (project_prefix_layer of prefix 0, one layer)",
                         "achieved": tf, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s", "frac": tf / peaks["bf16_tflops"],
                         "peak_source": peaks["source"], "flops_per_launch": proj_flops, "ms_per_launch": ms_proj,
                         "d_model": d_model, "traffic": NCU_TRAFFIC_BYTES.get(args.workload, {}).get("project")}
    if put_bytes >= (256 << 20):
        kc, vc = workloads.draw_prefix_kv(w, 0, "cuda")
        # profiler reduction (Eq. 3): cached prefix 0 against a reference K/V of the same shape; reads both once
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
        roofline_sim = {"bound": "hbm", "kernel": "kv_similarity_partial_kernel (prefix_similarity of prefix 0)",
                        "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": gbs / peaks["hbm_gbs"],
                        "peak_source": peaks["source"], "bytes_per_launch": put_bytes, "ms_per_launch": ms_sim,
                        "traffic": NCU_TRAFFIC_BYTES.get(args.workload, {}).get("similarity")}
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
        roofline_put = {"bound": "hbm", "kernel": "scatter_prefix_kernel (put_prefix of prefix 0, all layers)",
                        "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": gbs / peaks["hbm_gbs"],
                        "peak_source": peaks["source"], "bytes_per_launch": put_bytes, "ms_per_launch": ms_put,
                        "traffic": NCU_TRAFFIC_BYTES.get(args.workload, {}).get("put")}

    if rank == 0:
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": step_ms_max, "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": "bf16" if w.dtype == torch.bfloat16 else "f32", "data": "synthetic",
                "config": {"workload": w.name, "note": w.note, "layers": w.num_layers, "requests": w.num_requests,
                           "suffix_tokens": w.suffix_tokens, "l2": "flushed between timed steps (256 MB write)",
                           "step": ("shallow-layer pass + deep-layer pass of the single layer"
                                    if job.single_layer else "all layers, per-request depths from the rule"),
                           "depth_min": int(min(depth)), "depth_max": int(max(depth)),
                           "deep_layer_refresh": refresh_info},
                "tflops": flops / (step_ms_max * 1e-3) / 1e12, "step_flops": flops,
                "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches),
                "roofline": roofline, "roofline_attend": roofline_attend, "roofline_put": roofline_put,
                "roofline_similarity": roofline_sim, "roofline_project": roofline_proj,
                "cpu_baseline": cpu}
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
