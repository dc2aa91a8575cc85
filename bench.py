#!/usr/bin/env python
"""Benchmark of the H2O hot path on B200: prefill-select + the fused decode steps.

One *step* is one pass of the whole path over one batch of synthetic prompts:
for each of ``--layers`` independent layer caches, reset + prefill-select over the
prompts, then ``decode_steps`` decode steps through all layers in model order
(step s of layer 0, 1, ... L-1, then step s+1, ...).  The layer caches together
are larger than the L2 cache, so every decode launch streams its cache from HBM.

Prints ONE JSON line (see the keys at the bottom of main()).
  value     : (sequence, head) decode steps per second over the whole timed region
              (prefill-select included), inputs resident in HBM
  e2e       : the same through the host-buffer C calls (pinned host tensors, H2D/D2H inside)
  roofline  : fused decode kernel, algorithmic bytes / average launch duration vs measured HBM peak
  cpu_baseline : the fp64 oracle on this machine's host cores, on a bounded sample
``--impl reference`` times the oracle alone (a deliberately slow CPU program).
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

from workloads import CONFIGS, make_prompt_inputs
from workloads.synth import _draw  # bulk decode inputs: one draw per layer and tensor

METRIC = "h2o_decode_seq_head_steps_per_s"
UNIT = "seq-heads/s"


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return float(p["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def decode_bytes_per_unit_step(cnt: int, d: int, esize: int) -> int:
    """Algorithmic bytes of one unit-step: K and V slots read once, accumulated score (f64)
    read + written, positions read, q/k_new/v_new read, out written, new K/V row written."""
    return 2 * cnt * d * esize + 16 * cnt + 4 * cnt + 6 * d * esize


def decode_bytes_per_unit_step_kv4(cnt: int, d: int) -> int:
    """The same with 4-bit group-quantised slots (80-byte rows for d = 128), bf16 q/k/v/out."""
    row = d // 2 + (d // 32) * 4
    return 2 * cnt * row + 16 * cnt + 4 * cnt + 4 * d * 2 + 2 * row


# DRAM bytes of one decode launch, dram__bytes_read.sum + dram__bytes_write.sum of an ncu capture (the
# summaries are committed with the profiles): 55.26 MB read + 0.07 MB written for config 2, captured at
# full size; c3 on the first 32 of 64 sequences (102.5 MB) and scaled by the units, which the traffic is
# proportional to (every unit's slots are read once).
NCU_DECODE_TRAFFIC_PER_LAUNCH = {"c2_opt6p7b": 55.33e6, "c3_opt30b": 2 * 102.5e6}


def aggregate_over_ranks(values, world: int, device, dist=None):
    """Max over ranks of per-rank timings (the job is as slow as its slowest replica)."""
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t.cpu()]


def whole_job_value(units_per_rank: int, layers: int, decode_steps: int, bench_steps: int, world: int, total_ms: float):
    """(sequence, head) decode steps per second over all replicas."""
    return units_per_rank * layers * world * decode_steps * bench_steps / (total_ms * 1e-3)


def prefill_flops(n: int, d: int) -> float:
    """Algorithmic flops of one unit's prompt attention: QK^T and PV over the causal triangle."""
    return 4.0 * d * n * (n + 1) / 2.0


class ClockSampler(threading.Thread):
    def __init__(self, index: int, period: float = 0.05):
        super().__init__(daemon=True)
        self.index, self.period = index, period
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop_evt = threading.Event()
        try:
            import pynvml

            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.nv = None

    def run(self):
        if self.nv is None:
            return
        nv = self.nv
        names = {
            nv.nvmlClocksThrottleReasonHwSlowdown: "hw_slowdown",
            nv.nvmlClocksThrottleReasonHwThermalSlowdown: "hw_thermal_slowdown",
            nv.nvmlClocksThrottleReasonSwThermalSlowdown: "sw_thermal_slowdown",
            nv.nvmlClocksThrottleReasonSwPowerCap: "sw_power_cap",
            nv.nvmlClocksThrottleReasonHwPowerBrakeSlowdown: "hw_power_brake",
        }
        while not self._stop_evt.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                mask = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                for bit, name in names.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            self._stop_evt.wait(self.period)

    def stop(self):
        self._stop_evt.set()
        self.join(timeout=2)
        return {
            "sm_mhz": int(np.median(self.samples)) if self.samples else None,
            "sm_max_mhz": self.max_mhz,
            "reasons": sorted(self.reasons),
        }


def _physical_gpu_index(local: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local])
        except Exception:
            return local
    return local


# ---------------------------------------------------------------------------
# oracle legs (CPU)
# ---------------------------------------------------------------------------
def oracle_sample_run(wl, n_units: int, steps: int, layer: int = 0):
    """Prefill-select + `steps` decode steps of the first `n_units` units on the host cores."""
    from oracle import h2o_oracle

    q, k, v, cu = make_prompt_inputs(wl, layer=layer, device="cpu")
    units = list(range(n_units))
    dq = [_draw(wl, layer, kind, 1, steps * wl.batch, "cpu").to(wl.torch_dtype).float().numpy().reshape(
        steps, wl.batch, wl.n_heads, wl.head_dim) for kind in ("q", "k", "v")]
    qf, kf, vf = (x.float().numpy() for x in (q, k, v))
    cache = h2o_oracle.OracleCache(wl.batch, wl.n_heads, wl.head_dim, wl.heavy, wl.recent)
    t0 = time.perf_counter()
    cache.prefill(qf, kf, vf, cu, units=units)
    t1 = time.perf_counter()
    for s in range(steps):
        cache.decode_step(dq[0][s], dq[1][s], dq[2][s], units=units)
    t2 = time.perf_counter()
    return dict(prefill_s=t1 - t0, decode_s=t2 - t1, total_s=t2 - t0, cores=h2o_oracle.num_threads())


def cpu_baseline(wl, budget_s: float = 15.0):
    probe = oracle_sample_run(wl, 1, min(4, wl.decode_steps))
    per_unit = probe["prefill_s"] + probe["decode_s"] / min(4, wl.decode_steps) * wl.decode_steps
    n_units = int(max(1, min(wl.units, budget_s / max(per_unit, 1e-3))))
    r = oracle_sample_run(wl, n_units, wl.decode_steps)
    return {
        "value": n_units * wl.decode_steps / r["total_s"],
        "unit": UNIT,
        "cores": r["cores"],
        "kind": "oracle",
        "sample": "%d of %d units of %s (layer 0): prefill-select + %d decode steps in %.1f s (prefill %.1f s)" % (
            n_units, wl.units, wl.name, wl.decode_steps, r["total_s"], r["prefill_s"]),
    }


def run_reference(args, wl):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    n_units = args.ref_units
    times = []
    cores = None
    for i in range(args.warmup + args.steps):
        r = oracle_sample_run(wl, n_units, wl.decode_steps)
        cores = r["cores"]
        if i >= args.warmup:
            times.append(r["total_s"])
    total = float(sum(times))
    value = n_units * wl.decode_steps * len(times) / total
    sample = "%d of %d units per step, prefill-select + %d decode steps each" % (n_units, wl.units, wl.decode_steps)
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * total / len(times), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": "%s x %d layer caches" % (wl.name, args.layers), "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


# ---------------------------------------------------------------------------
# CUDA arm
# ---------------------------------------------------------------------------
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="c2_opt6p7b", choices=sorted(CONFIGS))
    ap.add_argument("--layers", type=int, default=8, help="independent layer caches rotated per decode step")
    ap.add_argument("--decode-steps", type=int, default=0, help="override the config's decode step count")
    ap.add_argument("--batch-limit", type=int, default=0,
                    help="keep only the first N sequences of the configuration (for small profiler captures)")
    ap.add_argument("--ref-units", type=int, default=4)
    ap.add_argument("--split", type=int, default=0, help="decode thread blocks per unit (0 = library default)")
    ap.add_argument("--stages", type=int, default=0, help="decode ring depth (0 = library default)")
    ap.add_argument("--no-graph", dest="graph", action="store_false",
                    help="launch every decode step from the host instead of replaying a CUDA graph of the decode loop")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()

    wl = CONFIGS[args.config]
    if args.decode_steps:
        wl = wl.scaled(decode_steps=args.decode_steps)
    if args.batch_limit and args.batch_limit < wl.batch:
        n = args.batch_limit
        wl = wl.scaled(name="%s[:%d]" % (wl.name, n), batch=n, prompt_lens=wl.prompt_lens[:n], heavy=wl.heavy[:n],
                       recent=wl.recent[:n])
    if args.impl == "reference":
        run_reference(args, wl)
        return

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        import torch.distributed as dist

        dist.init_process_group("nccl", device_id=dev)

    import __graft_entry__

    if rank == 0:
        __graft_entry__.build()
    if world > 1:
        dist.barrier()
    import paper_2306_14048_b200 as pkg

    L, S = args.layers, wl.decode_steps
    H, d = wl.n_heads, wl.head_dim
    esize = 4 if wl.dtype == "f32" else 2
    stream = torch.cuda.Stream(device=dev)
    caches = [pkg.H2OCache(wl.batch, H, d, wl.dtype, wl.heavy, wl.recent, device=local) for _ in range(L)]
    for cch in caches:
        cch.set_decode_shape(args.split, args.stages)
    cu = wl.cu_seqlens()
    prompts, dec = [], []
    for l in range(L):  # each rank draws its own data: the units are independent, nothing is exchanged
        q, k, v, _ = make_prompt_inputs(wl.scaled(seed=wl.seed + 1000 * rank), layer=l, device=dev)
        prompts.append((q, k, v, torch.empty_like(q)))
        dq = [_draw(wl.scaled(seed=wl.seed + 1000 * rank), l, kind, 1, S * wl.batch, dev).to(wl.torch_dtype).view(S, wl.batch, H, d)
              for kind in ("q", "k", "v")]
        dec.append((dq[0], dq[1], dq[2], torch.empty(S, wl.batch, H, d, dtype=wl.torch_dtype, device=dev),
                    torch.empty(S, wl.batch, H, dtype=torch.int32, device=dev)))
    torch.cuda.synchronize()

    # raw pointers once, so that the host loop is a bare C call per launch
    sp = int(stream.cuda_stream)
    dec_args = [[(caches[l]._h, dec[l][0][s].data_ptr(), dec[l][1][s].data_ptr(), dec[l][2][s].data_ptr(),
                  dec[l][3][s].data_ptr(), dec[l][4][s].data_ptr(), sp) for l in range(L)] for s in range(S)]
    c_decode = pkg.lib.h2o_decode_step

    def decode_loop():
        for s in range(S):
            for a in dec_args[s]:
                rc = c_decode(*a)
                if rc != 0:
                    raise pkg.H2OError(rc, "h2o_decode_step")

    graph = None
    if args.graph:
        # the decode loop of one step (S x L launches of h2o_decode_step) as one CUDA graph
        for l in range(L):
            q, k, v, o = prompts[l]
            caches[l].reset(stream)
            caches[l].prefill_select(q, k, v, cu, o, stream)
        decode_loop()
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            decode_loop()
        torch.cuda.synchronize()

    def one_step(ev=None):
        if ev:
            ev[0].record(stream)
        for l in range(L):
            q, k, v, o = prompts[l]
            caches[l].reset(stream)
            caches[l].prefill_select(q, k, v, cu, o, stream)
        if ev:
            ev[1].record(stream)
        if graph is not None:
            with torch.cuda.stream(stream):
                graph.replay()
        else:
            decode_loop()
        if ev:
            ev[2].record(stream)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    for _ in range(args.warmup):
        one_step()
    barrier()
    sampler = ClockSampler(_physical_gpu_index(local))
    sampler.start()
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
    t_start, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t_start.record(stream)
    for i in range(args.steps):
        one_step(evs[i])
    t_end.record(stream)
    barrier()
    clocks = sampler.stop()
    total_ms = t_start.elapsed_time(t_end)
    prefill_ms = float(np.mean([e[0].elapsed_time(e[1]) for e in evs]))
    decode_ms = float(np.mean([e[1].elapsed_time(e[2]) for e in evs]))
    for c in caches:
        assert c.status() == 0, "device status word set"

    # context figure: the same decode launches on ONE layer cache back to back, so that the cache
    # (smaller than L2 for this workload) is served from L2 instead of HBM
    warm_us = None
    if rank == 0:
        n_warm = min(64, S)
        one_layer = [dec_args[s][0] for s in range(n_warm)]

        def warm_loop():
            for a in one_layer:
                rc = c_decode(*a)
                if rc != 0:
                    raise pkg.H2OError(rc, "h2o_decode_step")

        warm_loop()
        torch.cuda.synchronize()
        wgraph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(wgraph, stream=stream):
            warm_loop()
        w0, w1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        with torch.cuda.stream(stream):
            wgraph.replay()
            w0.record(stream)
            wgraph.replay()
            w1.record(stream)
        torch.cuda.synchronize()
        warm_us = w0.elapsed_time(w1) * 1e3 / n_warm

    # context figure: the same decode steps of layer 0 through h2o_decode_chunk (several tokens per
    # launch, the token-by-token mode of Algorithm 1), from a freshly prefilled cache
    chunk_fig = None
    if rank == 0:
        n_tok = min(256, S)
        q, k, v, o = prompts[0]
        ms = []
        for _ in range(3):
            caches[0].reset(stream)
            caches[0].prefill_select(q, k, v, cu, o, stream)
            c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            c0.record(stream)
            caches[0].decode_chunk(dec[0][0][:n_tok], dec[0][1][:n_tok], dec[0][2][:n_tok], dec[0][3][:n_tok],
                                   dec[0][4][:n_tok], stream)
            c1.record(stream)
            torch.cuda.synchronize()
            ms.append(c0.elapsed_time(c1))
        assert caches[0].status() == 0, "device status word set"
        chunk_fig = {"tokens": n_tok, "ms": float(np.median(ms)), "us_per_token_step": float(np.median(ms)) * 1e3 / n_tok,
                     "seq_heads_per_s": wl.units * n_tok / (float(np.median(ms)) * 1e-3)}

    # context figure: the same decode steps with 4-bit group-quantised K/V slots (dtype bf16_kv4), rotating
    # over the layer caches like the main loop
    kv4_fig = None
    if rank == 0 and wl.dtype == "bf16" and d == 128 and max(k_ + r_ for k_, r_ in zip(wl.heavy, wl.recent)) <= 8192:
        kcaches = [pkg.H2OCache(wl.batch, H, d, "bf16_kv4", wl.heavy, wl.recent, device=local) for _ in range(L)]
        for l in range(L):
            q, k, v, o = prompts[l]
            kcaches[l].prefill_select(q, k, v, cu, o, stream)
        n_k = min(64, S)

        def kv4_loop():
            for s_ in range(n_k):
                for l in range(L):
                    kcaches[l].decode_step(dec[l][0][s_], dec[l][1][s_], dec[l][2][s_], dec[l][3][s_], dec[l][4][s_], stream)

        kv4_loop()
        torch.cuda.synchronize()
        kgraph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(kgraph, stream=stream):
            kv4_loop()
        k0, k1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        with torch.cuda.stream(stream):
            kgraph.replay()
            k0.record(stream)
            kgraph.replay()
            k1.record(stream)
        torch.cuda.synchronize()
        for c_ in kcaches:
            assert c_.status() == 0, "device status word set"
        k_us = k0.elapsed_time(k1) * 1e3 / (n_k * L)
        k_cnt = [min(n, kk + rr) for n, kk, rr in zip(wl.prompt_lens, wl.heavy, wl.recent)]
        k_bytes = sum(decode_bytes_per_unit_step_kv4(c_, d) for c_ in k_cnt) * H
        kv4_fig = {"us_per_launch": k_us, "bytes_per_launch": k_bytes, "achieved_gbs": k_bytes / (k_us * 1e-6) / 1e9,
                   "speedup_vs_bf16_slots": None}
        for c_ in kcaches:
            c_.close()
        del kcaches

    # ---- end to end: pinned host tensors through the host-buffer C calls -----------------
    e2e = None
    if not args.no_e2e:
        hp = [tuple(x.cpu().pin_memory() for x in p) for p in prompts]
        hd = [tuple(x.cpu().pin_memory() for x in t) for t in dec]
        h2d = L * 3 * prompts[0][0].numel() * esize + S * L * 3 * wl.batch * H * d * esize
        d2h = L * prompts[0][0].numel() * esize + S * L * (wl.batch * H * d * esize + wl.batch * H * 4)

        # one stream per layer cache for the prompt phase: the device-to-host copy of one layer's output
        # overlaps the host-to-device copies of the next layer's prompt
        lstreams = [torch.cuda.Stream(device=dev) for _ in range(L)]

        def one_step_host():
            start = torch.cuda.Event()
            start.record(stream)
            for l in range(L):
                q, k, v, o = hp[l]
                lstreams[l].wait_event(start)
                caches[l].reset(lstreams[l])
                caches[l].prefill_select_host(q, k, v, cu, o, lstreams[l])
                done = torch.cuda.Event()
                done.record(lstreams[l])
                stream.wait_event(done)
            for s in range(S):
                for l in range(L):
                    dq, dk, dv, do, de = hd[l]
                    caches[l].decode_step_host(dq[s], dk[s], dv[s], do[s], de[s], stream)

        one_step_host()
        barrier()
        n_e2e = max(1, min(args.steps, 3))
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for _ in range(n_e2e):
            one_step_host()
        b.record(stream)
        barrier()
        e2e_ms = a.elapsed_time(b) / n_e2e
        e2e = {"ms_per_step": e2e_ms, "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h), "steps": n_e2e}
        del hp, hd

    total_ms, prefill_ms, decode_ms, e2e_ms = aggregate_over_ranks(
        [total_ms, prefill_ms, decode_ms, e2e["ms_per_step"] if e2e else 0.0], world, dev, dist if world > 1 else None)

    if rank == 0:
        units_all = wl.units * L * world
        unit_steps = units_all * S
        value = whole_job_value(wl.units, L, S, args.steps, world, total_ms)
        hbm_peak, peak_kind = _peaks()
        cnt = [min(n, kk + rr) for n, kk, rr in zip(wl.prompt_lens, wl.heavy, wl.recent)]
        bytes_launch = sum(decode_bytes_per_unit_step(c, d, esize) for c in cnt) * H
        launch_us = decode_ms * 1e3 / (S * L)
        if kv4_fig:
            kv4_fig["speedup_vs_bf16_slots"] = launch_us / kv4_fig["us_per_launch"]
        achieved = bytes_launch / (launch_us * 1e-6) / 1e9
        flops = sum(prefill_flops(n, d) for n in wl.prompt_lens) * H * L
        out = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": total_ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": wl.dtype, "data": "synthetic",
            "config": {
                "workload": "%s x %d layer caches" % (wl.name, L), "batch": wl.batch, "n_heads": H, "head_dim": d,
                "prompt_len": int(np.mean(wl.prompt_lens)), "decode_steps": S, "heavy": int(np.mean(wl.heavy)),
                "recent": int(np.mean(wl.recent)), "layers": L,
                "decode_launch": "cuda graph of the decode loop" if graph is not None else "one host call per launch",
                "l2": "inputs larger than L2: %d layer caches of %.0f MB rotated every decode launch" % (
                    L, bytes_launch / 1e6),
            },
            "prefill_ms": prefill_ms, "decode_ms": decode_ms,
            "decode_only_seq_heads_per_s": wl.units * L * S / (decode_ms * 1e-3),
            "prefill_tflops_algorithmic": flops / (prefill_ms * 1e-3) / 1e12,
            # tensor-core work actually issued: S, P_hi V, P_lo V and S^T (four triangle products for two)
            "prefill_tflops_executed_mma": 2.0 * flops / (prefill_ms * 1e-3) / 1e12,
            "gpu_launches": args.steps * L * (3 + S),
            "decode_one_layer_back_to_back_us": warm_us,
            "decode_chunk_one_layer": chunk_fig,
            "decode_kv4_slots": kv4_fig,
            "clocks": clocks,
            "roofline": {
                "kernel": "decode_kernel", "bound": "hbm", "achieved": achieved, "peak": hbm_peak, "unit": "GB/s",
                "frac": achieved / hbm_peak, "peak_source": peak_kind,
                "traffic": NCU_DECODE_TRAFFIC_PER_LAUNCH.get(wl.name),
                "bytes_per_launch": bytes_launch, "avg_launch_us": launch_us,
                "frac_of_nominal_8TBs": achieved / 8000.0,
            },
        }
        if e2e:
            out["e2e"] = {"value": unit_steps / (e2e_ms * 1e-3), "unit": UNIT,
                          "h2d_bytes_per_step": e2e["h2d_bytes_per_step"], "d2h_bytes_per_step": e2e["d2h_bytes_per_step"],
                          "ms_per_step": e2e_ms}
        if world == 1 and not args.no_cpu_baseline:
            out["cpu_baseline"] = cpu_baseline(wl)
        print(json.dumps(out))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
