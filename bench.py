#!/usr/bin/env python
"""Benchmark of the batch-invariant paged-attention hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

One step = one pass of the whole path over one decode-heavy batch:
vosti_kv_append of the batch's 64 new tokens, then vosti_paged_attention
(work planning, page gathers, QK^T, online softmax, PV, split partials,
cross-split combine).  The workload is the decode-heavy recipe: 32 query /
8 KV heads, head_dim 128, page size 16, batch 64, one query token each,
contexts uniform in [512, 4096], pages scattered over a 200k-page pool.

Prints ONE JSON line (rank 0).  `value` is KV GB/s with inputs resident in
HBM; `e2e` is the same metric through vosti_step_host_async with pinned host
buffers (every step copies its inputs up and its output down; a few steps are
in flight, as in a serving loop), with the one-step-at-a-time figure beside it; `roofline` is the split-parallel attention kernel against the
measured HBM copy peak; `cpu_baseline` is the fp64 oracle on the host cores.
With N > 1 every rank runs its own batch (different seed) on its own GPU:
no collective on the data path, weak scaling.
"""
from __future__ import annotations

import argparse
import json
import os
import re
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "decode paged-attn KV GB/s"
UNIT = "GB/s"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="vosti", choices=["vosti", "reference"])
    ap.add_argument("--workload", default="decode_heavy",
                    choices=["decode_heavy", "prefix_sharing", "long_context_speculative",
                             "mixed_chunked_prefill", "linear"])
    ap.add_argument("--e2e-steps", type=int, default=200)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-kernel-events", action="store_true",
                    help="experiment: do not record per-kernel events in the timed region")
    ap.add_argument("--batch", type=int, default=0, help="override the batch size (experiments only)")
    ap.add_argument("--pack-shared-splits", action="store_true",
                    help="create the context with VOSTI_FLAG_PACK_SHARED_SPLITS (same bits, fewer tiles "
                         "when requests share prefix pages)")
    ap.add_argument("--pack-through-tiles", action="store_true",
                    help="with --pack-shared-splits: VOSTI_FLAG_PACK_THROUGH_TILES (large sharing groups always "
                         "go through the tile kernel)")
    ap.add_argument("--shared-prefix", type=int, default=0,
                    help="prefix_sharing workload: length of the common prefix (experiments; default 2048)")
    ap.add_argument("--device-plan", action="store_true",
                    help="time the step as a CUDA-graph replay of vosti_plan_device + vosti_kv_append_planned + "
                         "vosti_paged_attention_planned (metadata in device memory); same bits")
    ap.add_argument("--window", type=int, default=0,
                    help="sliding window (keys); experiments with vosti_paged_attention_ex, the e2e and "
                         "cpu_baseline legs stay unwindowed")
    ap.add_argument("--pool-pages", type=int, default=0,
                    help="override the pool size (small pools keep profiler captures short)")
    return ap.parse_args()


def make_workload(name: str, rank: int, pool_pages: int = 0, batch: int = 0, shared_prefix: int = 0):
    from paper_2609_38981_b200 import inputs
    fn = getattr(inputs, name)
    base = {"decode_heavy": 2, "mixed_chunked_prefill": 3, "prefix_sharing": 4,
            "long_context_speculative": 5}[name]
    kw = {"num_pages": pool_pages} if pool_pages else {}
    if batch:
        kw["batch"] = batch
    if shared_prefix:
        kw["prefix"] = shared_prefix
    return fn(seed=inputs.BASE_SEED * 10 + base + 1000 * rank, **kw)


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback (6.65 TB/s, earlier measurement on this pool)"


def ncu_traffic_per_launch(workload: str):
    """dram bytes per launch of the dominant kernel from the committed ncu summary, if any."""
    path = os.path.join(ROOT, "profiles", f"attn_split_kernel_{workload}.md")
    try:
        m = re.search(r"dram_bytes_per_launch:\s*([0-9.eE+]+)", open(path).read())
        return float(m.group(1)) if m else None
    except Exception:
        return None


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, index: int):
        super().__init__(daemon=True)
        self.index, self.samples, self.reasons, self.max_mhz = index, [], set(), None
        self._halt = threading.Event()
        self.ok = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            self.ok = True
        except Exception:
            self.ok = False

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        names = {
            getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4): "sw_power_cap",
            getattr(nv, "nvmlClocksThrottleReasonHwSlowdown", 0x8): "hw_slowdown",
            getattr(nv, "nvmlClocksThrottleReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
            getattr(nv, "nvmlClocksThrottleReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
            getattr(nv, "nvmlClocksThrottleReasonHwPowerBrakeSlowdown", 0x80): "hw_power_brake",
        }
        while not self._halt.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                try:
                    mask = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for bit, nm in names.items():
                    if mask & bit:
                        self.reasons.add(nm)
            except Exception:
                pass
            time.sleep(0.01)

    def stop(self):
        self._halt.set()
        self.join(timeout=2)
        med = sorted(self.samples)[len(self.samples) // 2] if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


def oracle_step_factory(w):
    """Builds the oracle's view of the workload (a compact host pool holding only
    the used pages, page ids renumbered) and returns a function running one step."""
    import numpy as np
    import torch
    from oracle import oracle
    from paper_2609_38981_b200 import inputs
    geo = w.geo
    seen, tables = {}, []
    for tb in w.tables:
        tables.append([seen.setdefault(p, len(seen)) for p in tb])
    pool = np.zeros((len(seen), geo.n_kv_heads, 2, geo.page_size, geo.head_dim), dtype=np.uint16)
    bt = inputs.block_table_array(tables)
    for r, tb, s in zip(w.requests, tables, w.start_pos):   # cached context, shared pages once
        oracle.kv_append(pool, inputs.bits(r.k[:s]), inputs.bits(r.v[:s]), [s], [0],
                         inputs.block_table_array([tb]))
    q = inputs.bits(w.packed_q())
    kn, vn = w.packed_new_kv()
    kn, vn = inputs.bits(kn), inputs.bits(vn)
    scale = geo.head_dim ** -0.5

    def step():
        oracle.kv_append(pool, kn, vn, w.q_lens, w.start_pos, bt)
        return oracle.paged_attention(q, pool, w.q_lens, w.start_pos, w.seq_lens, bt,
                                      n_kv_heads=geo.n_kv_heads, page_size=geo.page_size,
                                      scale=scale)
    return step, oracle.num_threads()


def run_reference(args):
    """The reference arm: the fp64 oracle, as it stands, on the host cores."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w = make_workload(args.workload, 0, args.pool_pages)
    step, cores = oracle_step_factory(w)
    # one step is the whole batch through the oracle (about 70 ms on 16 cores): K steps as asked,
    # fewer only where K of them would take more than about two minutes
    t0 = time.perf_counter()
    step()
    first = time.perf_counter() - t0
    steps = max(1, min(args.steps, int(120.0 / max(first, 1e-3))))
    warm = max(0, min(args.warmup, 3))
    for _ in range(warm):
        step()
    t0 = time.perf_counter()
    for _ in range(steps):
        step()
    dt = (time.perf_counter() - t0) / steps
    val = w.kv_bytes() / dt / 1e9
    sample = f"full {w.name} step (batch {w.batch}, {sum(w.seq_lens)} cached tokens), {steps} timed steps"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
        "steps": steps, "warmup": warm, "ms_per_step": dt * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "batch": w.batch, "geometry": "32q/8kv/d128/page16"},
        "tokens_per_s": w.total_q / dt,
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def run_linear(args):
    """Side benchmark (not the headline metric): the batch-invariant linear layer on the four
    weight shapes of a Llama-3.1-8B decoder layer at a prefill batch of 8192 token rows, with the
    library GEMM (torch.matmul) timed beside it for context, and the decode batch of 64 rows."""
    import torch
    from paper_2609_38981_b200 import linear as vl
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    try:
        peak = float(json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))["bf16_tflops"])
        src = "measured (MEASURED_PEAKS.json bf16_tflops, burst)"
    except Exception:
        peak, src = 1590.0, "fallback"
    sampler = ClockSampler(torch.cuda.current_device())
    sampler.start()

    def timed(fn, n):
        for _ in range(max(3, args.warmup)):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(n):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / n

    shapes = {"qkv": (6144, 4096), "o": (4096, 4096), "gate_up": (28672, 4096), "down": (4096, 14336)}
    g = torch.Generator(device="cuda")
    g.manual_seed(1)
    rows, flops_all, ms_all, launches = {}, 0.0, 0.0, 0
    n = max(10, min(args.steps, 100))
    for M in (8192, 64):
        for name, (N, K) in shapes.items():
            x = torch.randn(M, K, device="cuda", generator=g).bfloat16()
            w = (torch.randn(N, K, device="cuda", generator=g) * K ** -0.5).bfloat16()
            y = torch.empty(M, N, device="cuda", dtype=torch.bfloat16)
            ws = torch.empty(max(vl.vosti_linear_workspace_bytes(M, N, K), 16), dtype=torch.uint8, device="cuda")
            ms = timed(lambda: vl.vosti_linear(x, w, y, workspace=ws), n)
            ms_lib = timed(lambda: torch.matmul(x, w.t(), out=y), n)
            launches += n + max(3, args.warmup)
            fl = 2.0 * M * N * K
            rows[f"{name}_M{M}"] = {"N": N, "K": K, "us": ms * 1e3, "tflops": fl / ms / 1e9,
                                    "weight_gbs": N * K * 2 / ms / 1e6, "library_gemm_us": ms_lib * 1e3,
                                    "tile": list(vl.vosti_linear_tile_shape(N, K)),
                                    "k_segments": vl.vosti_linear_segments(N, K)}
            if M == 8192:
                flops_all += fl
                ms_all += ms
    clocks = sampler.stop()
    assert vl.vosti_linear_poll_status() == 0
    ach = flops_all / ms_all / 1e9
    print(json.dumps({
        "metric": "batch-invariant linear TFLOP/s (Llama-3.1-8B layer weights, 8192 token rows)", "value": ach,
        "unit": "TFLOP/s", "n_gpus": 1, "steps": n, "warmup": max(3, args.warmup), "ms_per_step": ms_all,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": "linear", "shapes": shapes, "l2": "operands of a layer exceed L2; no flush"},
        "gpu_launches": launches, "clocks": clocks, "per_shape": rows,
        "roofline": {"bound": "tensor", "kernel": "linear_kernel<256>", "achieved": ach, "peak": peak,
                     "unit": "TFLOP/s", "frac": ach / peak, "peak_source": src, "traffic": None},
    }))


def main():
    args = parse_args()
    if args.impl == "reference":
        return run_reference(args)
    if args.workload == "linear":
        return run_linear(args)

    import numpy as np
    import torch
    from paper_2609_38981_b200 import binding as vb
    from paper_2609_38981_b200 import inputs
    from paper_2609_38981_b200.harness import DeviceCache

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the path has no CPU fallback")
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    w = make_workload(args.workload, rank, args.pool_pages, args.batch, args.shared_prefix)
    geo = w.geo
    scale = geo.head_dim ** -0.5
    max_seq = max(w.seq_lens)
    cache = DeviceCache(geo, w.num_pages, max_batch=w.batch, max_total_q=max(8192, w.total_q),
                        max_seq_len=max_seq, device=f"cuda:{local}",
                        flags=(vb.VOSTI_FLAG_PACK_SHARED_SPLITS if args.pack_shared_splits else 0) |
                        (vb.VOSTI_FLAG_PACK_THROUGH_TILES if args.pack_through_tiles else 0))
    cache.upload(w.requests, w.tables, upto=w.start_pos)      # cached context before the step
    bt = inputs.block_table_array(w.tables)
    ql, st, sl = (np.asarray(x, dtype=np.int32) for x in (w.q_lens, w.start_pos, w.seq_lens))
    q_cpu = w.packed_q().contiguous()
    kn_cpu, vn_cpu = (t.contiguous() for t in w.packed_new_kv())
    dev = cache.device
    q, kn, vn = q_cpu.to(dev), kn_cpu.to(dev), vn_cpu.to(dev)
    out = torch.empty_like(q)
    stream = torch.cuda.current_stream()

    def step():
        vb.vosti_kv_append(cache.ctx, kn, vn, ql, st, bt, stream=stream)
        if args.window:
            vb.vosti_paged_attention_ex(cache.ctx, q, out, None, ql, st, sl, bt, scale, window=args.window,
                                        stream=stream)
        else:
            vb.vosti_paged_attention(cache.ctx, q, out, ql, st, sl, bt, scale, stream=stream)

    host_step = step
    if args.device_plan:
        # The same step with its metadata in device memory, planned by a kernel, captured once in a
        # CUDA graph: the host's share of a step is one graph launch.
        if max(w.q_lens) * (geo.n_q_heads // geo.n_kv_heads) > 32:
            raise SystemExit("--device-plan covers split-parallel batches (decode, speculative)")
        plan = torch.empty(vb.vosti_device_plan_bytes(cache.ctx), dtype=torch.uint8, device=dev)
        ql_d, st_d, bt_d = (torch.from_numpy(np.ascontiguousarray(x)).to(dev) for x in (ql, st, bt))
        max_q = int(max(w.q_lens))

        def planned_step():
            vb.vosti_plan_device(cache.ctx, plan, ql_d, st_d, bt_d, max_q, window=args.window)
            vb.vosti_kv_append_planned(cache.ctx, plan, kn, vn, bt_d, max_q)
            vb.vosti_paged_attention_planned(cache.ctx, plan, q, out, None, bt_d, max_q, scale, window=args.window)

        side = torch.cuda.Stream()
        side.wait_stream(stream)
        with torch.cuda.stream(side):
            planned_step()
        stream.wait_stream(side)
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            planned_step()
        step = graph.replay

    def sync_all():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    warm = max(args.warmup, 3)
    for _ in range(warm):
        step()
    sync_all()
    assert vb.vosti_poll_device_status(cache.ctx) == vb.VOSTI_OK

    # host cost of enqueuing a step, measured on an idle queue (nothing to wait for)
    h_us = []
    for _ in range(5):
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        step()
        step()
        h_us.append((time.perf_counter() - t0) * 1e6 / 2)
    torch.cuda.synchronize()

    def timed_pass(profile_mode, step=step):
        """K steps bracketed by barrier + synchronize, timed with CUDA events on the stream."""
        vb.vosti_profile_enable(cache.ctx, profile_mode)
        l0 = vb.vosti_launch_count(cache.ctx)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        sync_all()
        a.record(stream)
        for _ in range(args.steps):
            step()
        b.record(stream)
        sync_all()
        ms = a.elapsed_time(b)
        k_ms_, k_n_ = vb.vosti_profile_read(cache.ctx) if profile_mode else (0.0, 0)
        vb.vosti_profile_enable(cache.ctx, 0)
        return ms, vb.vosti_launch_count(cache.ctx) - l0, k_ms_, k_n_

    tile_bound = w.name == "mixed_chunked_prefill"     # dominant kernel: tcgen05 tile kernel
    sampler = ClockSampler(local)
    sampler.start()
    # Pass 1 gives `value`: the step as a caller runs it, nothing recorded between its kernels.
    elapsed_ms, launches, _, _ = timed_pass(0)
    clocks = sampler.stop()
    # Pass 2, same K steps, records a CUDA event pair around every launch of the dominant kernel
    # (on the launching stream) for the roofline.  The event nodes sit between the step's kernels
    # and defeat their dependent launch, which is why they are kept out of pass 1.
    # (Always the host-planned step: the library records its events around its own launches.)
    roof_ms, _, kernel_ms, kernels_timed = timed_pass(0 if args.no_kernel_events else (2 if tile_bound else 1),
                                                      step=host_step)
    if args.device_plan:
        launches = 4 * args.steps        # plan, append, attention, combine per replay
        out_graph = out.clone()
        host_step()
        torch.cuda.synchronize()
        assert torch.equal(out_graph.view(torch.int16), out.view(torch.int16)), "device-planned output differs"
    assert vb.vosti_poll_device_status(cache.ctx) == vb.VOSTI_OK

    # end to end: host buffers in, host buffer out, every step
    pin = lambda t: t.pin_memory()
    qh, knh, vnh = pin(q_cpu), pin(kn_cpu), pin(vn_cpu)
    outh = torch.empty_like(q_cpu).pin_memory()

    def e2e_pass(step_fn, drain):
        for _ in range(3):
            step_fn()
        drain()
        sync_all()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0 = time.perf_counter()
        e0.record(stream)
        for _ in range(args.e2e_steps):
            step_fn()
        drain()                      # the last outputs are on the host before the clock stops
        e1.record(stream)
        torch.cuda.synchronize()
        return max(e0.elapsed_time(e1), (time.perf_counter() - t0) * 1e3) / args.e2e_steps

    # (a) the waiting call: one step at a time, the host idle while the GPU works and the reverse
    e2e_wait_ms = e2e_pass(lambda: vb.vosti_step_host(cache.ctx, qh, outh, knh, vnh, ql, st, sl, bt, scale,
                                                      stream=stream), lambda: None)
    out_match = bool(torch.equal(outh.view(torch.int16), out.cpu().view(torch.int16)))
    # (b) the pipelined call, as a serving loop uses it: every step still copies its own inputs up
    # and its own output down (to its own host buffer), but the copies and the host's planning of
    # one step run under the kernels of its neighbours.
    depth = vb.VOSTI_HOST_STEPS_IN_FLIGHT
    outs_h = [torch.empty_like(q_cpu).pin_memory() for _ in range(depth)]
    tickets = []
    issued = [0]

    def pipelined_step():
        if len(tickets) == depth:
            vb.vosti_step_host_wait(cache.ctx, tickets.pop(0))
        issued[0] += 1
        tickets.append(vb.vosti_step_host_async(cache.ctx, qh, outs_h[issued[0] % depth], knh, vnh, ql, st, sl,
                                                bt, scale, stream=stream))

    def drain():
        while tickets:
            vb.vosti_step_host_wait(cache.ctx, tickets.pop(0))

    e2e_ms = e2e_pass(pipelined_step, drain)
    out_match = out_match and all(bool(torch.equal(o.view(torch.int16), outh.view(torch.int16))) for o in outs_h)

    kv_bytes = float(w.kv_bytes())
    if args.window:  # keys some row of the request sees: from the first row's window start to the last position
        kv_bytes = float(sum(min(s + n, args.window + n - 1) for s, n in zip(w.start_pos, w.q_lens) if n > 0)
                         * geo.kv_bytes_per_token)
    t_max, e2e_max, bytes_all, tok_all = elapsed_ms, e2e_ms, kv_bytes, float(w.total_q)
    e2e_wait_max = e2e_wait_ms
    if dist is not None:
        t = torch.tensor([elapsed_ms, e2e_ms, e2e_wait_ms], device=dev, dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        s = torch.tensor([kv_bytes, float(w.total_q)], device=dev, dtype=torch.float64)
        dist.all_reduce(s, op=dist.ReduceOp.SUM)
        t_max, e2e_max, e2e_wait_max = float(t[0]), float(t[1]), float(t[2])
        bytes_all, tok_all = float(s[0]), float(s[1])
    ms_per_step = t_max / args.steps
    value = bytes_all / (ms_per_step * 1e-3) / 1e9

    if rank == 0:
        peak, peak_src = measured_peak()
        k_ms = kernel_ms / max(kernels_timed, 1)
        achieved = kv_bytes / (k_ms * 1e-3) / 1e9 if kernels_timed else None
        if tile_bound:
            # useful work of the tile kernel: visible (query, key) pairs of the long-query requests,
            # 2*d flops each for QK^T and for PV, per query head
            pairs = sum(q * s_ + q * (q + 1) // 2 for q, s_ in zip(w.q_lens, w.start_pos)
                        if q * geo.group > 32)
            flops = 4.0 * geo.head_dim * geo.n_q_heads * pairs
            try:
                peaks = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))
                tpeak, tsrc = float(peaks["bf16_tflops"]), "measured (MEASURED_PEAKS.json bf16_tflops, burst)"
            except Exception:
                tpeak, tsrc = 1590.0, "fallback (1.59 PFLOP/s, earlier measurement on this pool)"
            t_ach = flops / (k_ms * 1e-3) / 1e12 if kernels_timed else None
            roof = {"bound": "tensor", "kernel": "attn_tile_kernel<128>", "achieved": t_ach, "peak": tpeak,
                    "unit": "TFLOP/s", "frac": (t_ach / tpeak) if t_ach else None, "peak_source": tsrc,
                    "frac_of_nominal_2250": (t_ach / 2250.0) if t_ach else None,
                    "useful_flops_per_launch": flops, "kernel_us": k_ms * 1e3,
                    "launches_timed": int(kernels_timed), "traffic": None}
        else:
            roof = {"bound": "hbm", "kernel": "attn_split_kernel<128, 8>",
                    "achieved": achieved, "peak": peak, "unit": "GB/s",
                    "frac": (achieved / peak) if achieved else None,
                    "frac_of_8TBs": (achieved / NOMINAL_HBM_GBS) if achieved else None,
                    "peak_source": peak_src, "kernel_us": k_ms * 1e3,
                    "launches_timed": int(kernels_timed),
                    "traffic": ncu_traffic_per_launch(w.name)}
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": warm, "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {
                "workload": w.name, "batch": w.batch, "geometry":
                    f"{geo.n_q_heads}q/{geo.n_kv_heads}kv/d{geo.head_dim}/page{geo.page_size}",
                "cached_tokens": int(sum(w.seq_lens)), "pool_pages": w.num_pages,
                "kv_bytes_per_step": int(kv_bytes),
                "l2": "inputs larger than L2 (KV read per step exceeds 126 MB), no flush",
                "step": "vosti_kv_append + vosti_paged_attention",
                "timing": "value: K steps with nothing recorded between kernels; roofline: a second pass of "
                          "K steps with a CUDA event pair around each launch of the dominant kernel",
                "ms_per_step_with_kernel_events": roof_ms / args.steps,
                "pack_shared_splits": bool(args.pack_shared_splits),
                "pack_through_tiles": bool(args.pack_through_tiles),
                "shared_prefix": int(args.shared_prefix) or None,
                "device_plan": bool(args.device_plan),
                "window": int(args.window),
                "schedule": dict(zip(("split_items", "packed_items", "tile_items"),
                                     vb.vosti_last_schedule(cache.ctx))),
            },
            "tokens_per_s": tok_all / (ms_per_step * 1e-3),
            "pct_of_8TBs": 100.0 * value / world / NOMINAL_HBM_GBS,
            "host_enqueue_us_per_step": min(h_us),
            "gpu_launches": int(launches),
            "clocks": clocks,
            "e2e": {"value": bytes_all / (e2e_max * 1e-3) / 1e9, "unit": UNIT,
                    "h2d_bytes_per_step": int(qh.nbytes + knh.nbytes + vnh.nbytes + bt.nbytes
                                              + ql.nbytes + st.nbytes + sl.nbytes),
                    "d2h_bytes_per_step": int(outh.nbytes), "ms_per_step": e2e_max,
                    "call": f"vosti_step_host_async, {depth} steps in flight",
                    "one_step_at_a_time": {"call": "vosti_step_host", "ms_per_step": e2e_wait_max,
                                           "value": bytes_all / (e2e_wait_max * 1e-3) / 1e9},
                    "output_equals_device_path": out_match},
            "roofline": roof,
        }
        if world == 1 and not args.no_cpu_baseline:
            ostep, cores = oracle_step_factory(w)
            c0 = time.perf_counter()
            ostep()
            # about ten seconds of host work: enough repetitions to average out the box's other tenants
            reps = int(min(400, max(8, 10.0 / max(time.perf_counter() - c0, 1e-3))))
            c0 = time.perf_counter()
            for _ in range(reps):
                ref = ostep()
            cdt = (time.perf_counter() - c0) / reps
            got = out.cpu().to(torch.float64).numpy()
            err = np.abs(got - ref)
            line["cpu_baseline"] = {
                "value": kv_bytes / cdt / 1e9, "unit": UNIT, "cores": cores, "kind": "oracle",
                "sample": f"the full {w.name} step, {reps} repetitions ({cdt * 1e3:.0f} ms each)"}
            line["parity"] = {"max_abs_err": float(err.max()), "mean_abs_err": float(err.mean()),
                              "rows": int(got.shape[0] * got.shape[1])}
        print(json.dumps(line))
    cache.close()
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
