#!/usr/bin/env python
"""Benchmark of the H2O hot path on B200: prefill-select + the fused decode steps.

One *step* is one pass of the whole path over one batch of synthetic prompts: for each of the
workload's independent layer caches, reset + prefill-select over that layer's prompts, then
``decode_steps`` decode steps through all layers in model order (step s of layer 0, 1, ... L-1,
then step s+1, ...).  The layer caches together are larger than the L2 cache, so every decode
launch streams its cache from HBM.

The headline workload is the largest configuration that fits one GPU: the 32-layer ragged batch
(config 5) at full size — 32 layer caches resident (28 GB), 128 decode steps replayed as one CUDA
graph of 4096 launches, prefill-select timed layer by layer with the prompt tensors of one layer
resident at a time (the next layer's prompts are drawn between the timed regions).  The other
configurations follow in ``per_config`` at their own sizes.

Prints ONE JSON line:
  value            (sequence, head) decode steps per second over the timed regions of the step
                   (all prefill-selects + the decode loop), inputs resident in HBM
  e2e              the same through the host-buffer C calls (pinned host tensors, H2D/D2H inside)
  roofline         fused decode kernel: algorithmic bytes / average launch duration vs measured HBM peak
  roofline_prefill column-sum kernel (and the attention kernel) against the measured bf16 tensor peak
  per_config       the same figures for the other configurations
  cpu_baseline     the fp64 oracle on this machine's host cores, on a bounded sample
``--impl reference`` times the oracle alone (a deliberately slow CPU program).
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
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

from workloads import CONFIGS, make_decode_inputs, make_prompt_inputs

METRIC = "h2o_decode_seq_head_steps_per_s"
UNIT = "seq-heads/s"
HEADLINE = "c5_ragged_32layer"
# layer caches per configuration: the stated layer count for the 32-layer stack; for the single-layer
# configurations enough independent copies that the rotation exceeds the L2 cache
DEFAULT_LAYERS = {"c1_tiny": 8, "c2_opt6p7b": 8, "c3_opt30b": 2, "c4_longctx": 8, "c5_ragged_32layer": 32}
PER_CONFIG = ("c1_tiny", "c2_opt6p7b", "c3_opt30b", "c4_longctx")
NOMINAL_HBM_GBS = 8000.0
RESIDENT_PROMPT_BYTES = 24e9  # keep all layers' prompt tensors on the device when they fit in this


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p["bf16_tflops_sustained"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


def decode_bytes_per_unit_step(cnt: int, d: int, esize: int) -> int:
    """Algorithmic bytes of one unit-step: K and V slots read once, accumulated score (f64)
    read + written, positions read, q/k_new/v_new read, out written, new K/V row written."""
    return 2 * cnt * d * esize + 16 * cnt + 4 * cnt + 6 * d * esize


def decode_bytes_per_unit_step_kv4(cnt: int, d: int) -> int:
    """The same with 4-bit group-quantised slots (80-byte rows for d = 128), bf16 q/k/v/out."""
    row = d // 2 + (d // 32) * 4
    return 2 * cnt * row + 16 * cnt + 4 * cnt + 4 * d * 2 + 2 * row


def slot_counts(wl):
    return [min(n, kk + rr) for n, kk, rr in zip(wl.prompt_lens, wl.heavy, wl.recent)]


def decode_bytes_per_launch(wl, kv4: bool = False) -> int:
    esize = 4 if wl.dtype == "f32" else 2
    if kv4:
        return sum(decode_bytes_per_unit_step_kv4(c, wl.head_dim) for c in slot_counts(wl)) * wl.n_heads
    return sum(decode_bytes_per_unit_step(c, wl.head_dim, esize) for c in slot_counts(wl)) * wl.n_heads


def profile_table(name: str):
    """Rows of the first markdown table of profiles/<name> as dicts keyed by the header cells (figures read
    from ncu captures live there as text; nothing under profiles/ runs)."""
    path = os.path.join(ROOT, "profiles", name)
    rows, header = [], None
    if not os.path.exists(path):
        return rows
    for line in open(path):
        if not line.startswith("|"):
            if header and rows:
                break
            continue
        cells = [c.strip() for c in line.strip().strip("|").split("|")]
        if header is None:
            header = cells
        elif not all(re.fullmatch(r":?-+:?", c) for c in cells):
            rows.append(dict(zip(header, cells)))
    return rows


def ncu_decode_traffic(wl):
    """dram__bytes_read.sum + dram__bytes_write.sum of one decode launch of this workload, from the committed
    ncu summary: bytes per unit-slot of the captured case x this workload's unit-slots (the traffic is
    proportional to the slots streamed)."""
    for row in profile_table("decode_kernel__dram_traffic.md"):
        if row.get("workload") == wl.name.split("[")[0]:
            try:
                per_slot = float(row["dram bytes per launch"]) / float(row["unit-slots in the capture"])
            except (KeyError, ValueError, ZeroDivisionError):
                return None
            return per_slot * sum(slot_counts(wl)) * wl.n_heads
    return None


def ncu_tensor_pipe(kernel: str, wl_name: str):
    for row in profile_table("prefill_kernels__tensor_pipe.md"):
        if row.get("kernel") == kernel and row.get("workload") == wl_name.split("[")[0]:
            try:
                return float(row["sm__pipe_tensor_cycles_active (%)"]), row.get("profile")
            except (KeyError, ValueError):
                return None, None
    return None, None


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


def _med_min(xs):
    return {"median": float(np.median(xs)), "min": float(np.min(xs))}


# ---------------------------------------------------------------------------
# oracle legs (CPU)
# ---------------------------------------------------------------------------
def _sample_units(wl, count: int, seed: int = 77):
    rng = np.random.default_rng(seed)
    return sorted(int(u) for u in rng.choice(wl.units, size=min(count, wl.units), replace=False))


def oracle_sample_run(wl, units, steps: int, layer: int = 0):
    """Prefill-select + ``steps`` decode steps of the sampled units on the host cores.

    The inputs come from the same seeded generator as the CUDA arm's (drawn on the GPU when there is one:
    only drawing; the rows of the sampled units are then copied to the host); the timed part is the oracle alone."""
    from oracle import h2o_oracle

    gen_dev = "cuda" if torch.cuda.is_available() else "cpu"
    H, d = wl.n_heads, wl.head_dim
    q, k, v, cu = make_prompt_inputs(wl, layer=layer, device=gen_dev)

    def rows(x):  # the sampled units as a batch of single-head sequences [sum n_u, 1, d]
        parts = [x[int(cu[u // H]):int(cu[u // H + 1]), u % H] for u in units]
        return np.ascontiguousarray(torch.cat(parts, 0).float().cpu().numpy()[:, None, :])

    qf, kf, vf = rows(q), rows(k), rows(v)
    del q, k, v
    lens = [int(cu[u // H + 1] - cu[u // H]) for u in units]
    ocu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    uidx = torch.as_tensor(units, dtype=torch.long)
    dec = []
    for s in range(steps):
        dq, dk, dv = make_decode_inputs(wl, s, layer=layer, device=gen_dev)
        dec.append(tuple(x.reshape(wl.units, d).cpu()[uidx].float().numpy()[:, None, :] for x in (dq, dk, dv)))
    cache = h2o_oracle.OracleCache(len(units), 1, d, [wl.heavy[u // H] for u in units], [wl.recent[u // H] for u in units])
    t0 = time.perf_counter()
    cache.prefill(qf, kf, vf, ocu)
    t1 = time.perf_counter()
    for s in range(steps):
        cache.decode_step(*dec[s])
    t2 = time.perf_counter()
    return dict(prefill_s=t1 - t0, decode_s=t2 - t1, total_s=t2 - t0, cores=h2o_oracle.num_threads())


def cpu_baseline(wl, budget_s: float = 12.0):
    """The oracle as it stands on a bounded sample: as many seeded random units as fit ~budget_s."""
    # rough cost of one unit (fp64 flops of the prompt attention twice over, decode steps over the slots) at ~4 GFLOP/s
    # per core, only to size the sample; what is reported is the measured time of the sample itself
    from oracle import h2o_oracle

    n_mean = float(np.mean([n * n for n in wl.prompt_lens]))
    slots = float(np.mean(slot_counts(wl)))
    per_unit = (3.0 * wl.head_dim * n_mean + 6.0 * wl.head_dim * slots * wl.decode_steps) / (4.0e9 * h2o_oracle.num_threads())
    n_units = int(max(1, min(wl.units, 1024, budget_s / max(per_unit, 1e-3))))
    units = _sample_units(wl, n_units)
    r = oracle_sample_run(wl, units, wl.decode_steps)
    return {
        "value": n_units * wl.decode_steps / r["total_s"],
        "unit": UNIT,
        "cores": r["cores"],
        "kind": "oracle",
        "sample": "%d of %d units of %s (layer 0, seeded random pick): prefill-select + %d decode steps in %.1f s "
                  "(prefill %.1f s)" % (n_units, wl.units, wl.name, wl.decode_steps, r["total_s"], r["prefill_s"]),
    }


def run_reference(args, wl, layers):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    units = _sample_units(wl, args.ref_units)
    times = []
    cores = None
    for i in range(args.warmup + args.steps):
        r = oracle_sample_run(wl, units, wl.decode_steps)
        cores = r["cores"]
        if i >= args.warmup:
            times.append(r["total_s"])
    total = float(sum(times))
    value = len(units) * wl.decode_steps * len(times) / total
    sample = "%d of %d units of layer 0 per step (seeded random pick), prefill-select + %d decode steps each" % (
        len(units), wl.units, wl.decode_steps)
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * total / len(times), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": workload_label(wl, layers), "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def workload_label(wl, layers):
    return "%s: %d layer caches x %d decode steps" % (wl.name, layers, wl.decode_steps)


# ---------------------------------------------------------------------------
# CUDA arm
# ---------------------------------------------------------------------------
class ConfigRun:
    """One configuration on one GPU: layer caches, decode inputs, the CUDA graph of the decode loop."""

    def __init__(self, pkg, wl, layers, dev, local, rank, args):
        self.pkg, self.wl, self.L, self.S = pkg, wl, layers, wl.decode_steps
        self.dev, self.local, self.rank, self.args = dev, local, rank, args
        self.H, self.d = wl.n_heads, wl.head_dim
        self.esize = 4 if wl.dtype == "f32" else 2
        self.wl_rank = wl.scaled(seed=wl.seed + 1000 * rank)  # every rank draws its own data: nothing is exchanged
        self.stream = torch.cuda.Stream(device=dev)
        self.cu = wl.cu_seqlens()
        L, S, H, d = self.L, self.S, self.H, self.d
        self.caches = [pkg.H2OCache(wl.batch, H, d, wl.dtype, wl.heavy, wl.recent, device=local) for _ in range(L)]
        for c in self.caches:
            c.set_decode_shape(args.split, args.stages)
        prompt_bytes = 4 * wl.total_tokens * H * d * self.esize
        self.resident = L * prompt_bytes <= RESIDENT_PROMPT_BYTES
        self.prompts = [self._draw_prompt(l) for l in range(L)] if self.resident else None
        self.outs = [torch.empty(wl.total_tokens, H, d, dtype=wl.torch_dtype, device=dev) for _ in range(L if self.resident else 1)]
        # decode inputs of every (layer, step) through the recipe's generator, stacked per layer
        self.dec = []
        for l in range(L):
            qs, ks, vs = zip(*[make_decode_inputs(self.wl_rank, s, layer=l, device=dev) for s in range(S)])
            self.dec.append((torch.stack(qs), torch.stack(ks), torch.stack(vs),
                             torch.empty(S, wl.batch, H, d, dtype=wl.torch_dtype, device=dev),
                             torch.empty(S, wl.batch, H, dtype=torch.int32, device=dev)))
        torch.cuda.synchronize(dev)
        sp = int(self.stream.cuda_stream)
        self.dec_args = [[(self.caches[l]._h, self.dec[l][0][s].data_ptr(), self.dec[l][1][s].data_ptr(),
                           self.dec[l][2][s].data_ptr(), self.dec[l][3][s].data_ptr(), self.dec[l][4][s].data_ptr(), sp)
                          for l in range(L)] for s in range(S)]
        self.graph = None
        self.launches = 0  # kernels of this library launched by the last one_step

    def _draw_prompt(self, l):
        with torch.cuda.stream(self.stream):
            q, k, v, _ = make_prompt_inputs(self.wl_rank, layer=l, device=self.dev)
        return q, k, v

    def decode_loop(self, args_rows=None):
        c_decode = self.pkg.lib.h2o_decode_step
        for row in (self.dec_args if args_rows is None else args_rows):
            for a in row:
                rc = c_decode(*a)
                if rc != 0:
                    raise self.pkg.H2OError(rc, "h2o_decode_step")

    def prefill_layer(self, l, ev=None):
        """reset + prefill-select of layer l; the prompt tensors are drawn first (untimed) unless resident."""
        q, k, v = self.prompts[l] if self.resident else self._draw_prompt(l)
        out = self.outs[l if self.resident else 0]
        if ev:
            ev[0].record(self.stream)
        self.caches[l].reset(self.stream)
        self.caches[l].prefill_select(q, k, v, self.cu, out, self.stream)
        if ev:
            ev[1].record(self.stream)

    def build_graph(self):
        for l in range(self.L):
            self.prefill_layer(l)
        self.decode_loop()
        torch.cuda.synchronize(self.dev)
        if self.args.graph:
            self.graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(self.graph, stream=self.stream):
                self.decode_loop()
            torch.cuda.synchronize(self.dev)

    def one_step(self, timed=False):
        """Returns (prefill ms summed over the layers, decode-loop ms) when timed."""
        L = self.L
        pev = [[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(L)] if timed else [None] * L
        for l in range(L):
            self.prefill_layer(l, pev[l])
        dev0, dev1 = (torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) if timed else (None, None)
        if timed:
            dev0.record(self.stream)
        if self.graph is not None:
            with torch.cuda.stream(self.stream):
                self.graph.replay()
        else:
            self.decode_loop()
        if timed:
            dev1.record(self.stream)
        self.launches = L * 3 + L * self.S  # attention, column sums, select+gather per layer; one kernel per decode step
        if not timed:
            return None
        torch.cuda.synchronize(self.dev)
        return sum(a.elapsed_time(b) for a, b in pev), dev0.elapsed_time(dev1)

    # -- context figures ---------------------------------------------------------------------------
    def graph_replay_us(self, loop, launches):
        """Average launch period of `loop` (a callable enqueuing `launches` launches) in CUDA-graph replay."""
        loop()
        torch.cuda.synchronize(self.dev)
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=self.stream):
            loop()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        with torch.cuda.stream(self.stream):
            g.replay()
            a.record(self.stream)
            g.replay()
            b.record(self.stream)
        torch.cuda.synchronize(self.dev)
        return a.elapsed_time(b) * 1e3 / launches

    def l2_warm_us(self):
        """The same decode launches on ONE layer cache back to back: served from L2 when the cache fits in it."""
        n = min(64, self.S)
        rows = [[self.dec_args[s][0]] for s in range(n)]
        return self.graph_replay_us(lambda: self.decode_loop(rows), n)

    def prefill_breakdown(self, reps=3):
        """Per-kernel times of prefill-select on layer 0 (events recorded between the kernels by the library)."""
        times = []
        for _ in range(reps):
            evs = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
            for e in evs:
                e.record(self.stream)  # torch creates the CUDA event handle on first record
            q, k, v = self.prompts[0] if self.resident else self._draw_prompt(0)
            out = self.outs[0]
            self.caches[0].reset(self.stream)
            self.caches[0].set_prefill_events(evs)
            self.caches[0].prefill_select(q, k, v, self.cu, out, self.stream)
            torch.cuda.synchronize(self.dev)
            times.append([evs[i].elapsed_time(evs[i + 1]) for i in range(3)])
        t = np.median(np.asarray(times), axis=0)
        return {"attention_ms": float(t[0]), "column_sums_ms": float(t[1]), "select_gather_ms": float(t[2])}

    def chunk_figure(self):
        """Layer 0's decode steps through h2o_decode_chunk (several tokens per launch), from a fresh prefill."""
        n_tok = min(256, self.S)
        ms = []
        for _ in range(3):
            self.prefill_layer(0)
            c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            c0.record(self.stream)
            d0 = self.dec[0]
            self.caches[0].decode_chunk(d0[0][:n_tok], d0[1][:n_tok], d0[2][:n_tok], d0[3][:n_tok], d0[4][:n_tok], self.stream)
            c1.record(self.stream)
            torch.cuda.synchronize(self.dev)
            ms.append(c0.elapsed_time(c1))
        assert self.caches[0].status() == 0, "device status word set"
        m = float(np.median(ms))
        return {"tokens": n_tok, "ms": m, "us_per_token_step": m * 1e3 / n_tok, "seq_heads_per_s": self.wl.units * n_tok / (m * 1e-3)}

    def kv4_figure(self, bf16_launch_us):
        """The same decode steps with 4-bit group-quantised slots, rotating over (up to 8) layer caches."""
        wl, pkg = self.wl, self.pkg
        if not (wl.dtype == "bf16" and self.d == 128 and max(k + r for k, r in zip(wl.heavy, wl.recent)) <= 8192):
            return None
        Lk = min(self.L, 8)
        kc = [pkg.H2OCache(wl.batch, self.H, self.d, "bf16_kv4", wl.heavy, wl.recent, device=self.local) for _ in range(Lk)]
        for l in range(Lk):
            q, k, v = self.prompts[l] if self.resident else self._draw_prompt(l)
            out = self.outs[l if self.resident else 0]
            kc[l].prefill_select(q, k, v, self.cu, out, self.stream)
        n_k = min(32, self.S)

        def loop():
            for s in range(n_k):
                for l in range(Lk):
                    d_ = self.dec[l]
                    kc[l].decode_step(d_[0][s], d_[1][s], d_[2][s], d_[3][s], d_[4][s], self.stream)

        us = self.graph_replay_us(loop, n_k * Lk)
        for c in kc:
            assert c.status() == 0, "device status word set"
            c.close()
        nbytes = decode_bytes_per_launch(wl, kv4=True)
        return {"us_per_launch": us, "bytes_per_launch": nbytes, "achieved_gbs": nbytes / (us * 1e-6) / 1e9,
                "speedup_vs_bf16_slots": bf16_launch_us / us, "layer_caches": Lk}

    def gqa_figure(self, G=4):
        """Grouped-query attention on the same tensors: the workload's heads are the query heads, every G of them
        share one K/V head (the first H / G heads of the K and V inputs), i.e. units = batch x H / G.  One layer's
        prefill-select and the decode steps, rotating over (up to 8) layer caches."""
        wl, pkg = self.wl, self.pkg
        if not (wl.dtype == "bf16" and self.d == 128 and self.H % G == 0):
            return None
        Hk = self.H // G
        Lk = min(self.L, 8)
        kc = [pkg.H2OCache(wl.batch, Hk, self.d, "bf16", wl.heavy, wl.recent, device=self.local, query_group=G) for _ in range(Lk)]
        pre_ms = []
        for l in range(Lk):
            q, k, v = self.prompts[l] if self.resident else self._draw_prompt(l)
            kk, vv = k[:, :Hk].contiguous(), v[:, :Hk].contiguous()
            out = self.outs[l if self.resident else 0]
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(self.stream)
            kc[l].prefill_select(q, kk, vv, self.cu, out, self.stream)
            b.record(self.stream)
            torch.cuda.synchronize(self.dev)
            pre_ms.append(a.elapsed_time(b))
            del kk, vv
        n_k = min(32, self.S)
        dk = [[self.dec[l][1][s][:, :Hk].contiguous() for s in range(n_k)] for l in range(Lk)]
        dv = [[self.dec[l][2][s][:, :Hk].contiguous() for s in range(n_k)] for l in range(Lk)]
        ev = torch.empty(wl.batch, Hk, dtype=torch.int32, device=self.dev)

        def loop():
            for s in range(n_k):
                for l in range(Lk):
                    d_ = self.dec[l]
                    kc[l].decode_step(d_[0][s], dk[l][s], dv[l][s], d_[3][s], ev, self.stream)

        us = self.graph_replay_us(loop, n_k * Lk)
        for c in kc:
            assert c.status() == 0, "device status word set"
            c.close()
        nbytes = sum(decode_bytes_per_unit_step(c_, self.d, self.esize) + 2 * (G - 1) * self.d * self.esize for c_ in slot_counts(wl)) * Hk
        return {"query_group": G, "kv_heads": Hk, "units": wl.batch * Hk, "us_per_launch": us, "bytes_per_launch": nbytes,
                "achieved_gbs": nbytes / (us * 1e-6) / 1e9, "frac_of_measured_hbm": nbytes / (us * 1e-6) / 1e9 / _peaks()["hbm_gbs"],
                "prefill_select_ms_per_layer": float(np.median(pre_ms)), "layer_caches": Lk}

    def topk_figure(self, m=64):
        """The same decode steps with "Top-K" attention (each query attends its m largest logits): the kernel streams
        the keys only and reads m value rows per unit; rotating over (up to 8) layer caches."""
        wl, pkg = self.wl, self.pkg
        if max(k + r for k, r in zip(wl.heavy, wl.recent)) > 8192:
            return None
        Lk = min(self.L, 8)
        kc = [pkg.H2OCache(wl.batch, self.H, self.d, wl.dtype, wl.heavy, wl.recent, device=self.local) for _ in range(Lk)]
        for l in range(Lk):
            kc[l].set_topk(m)
            q, k, v = self.prompts[l] if self.resident else self._draw_prompt(l)
            kc[l].prefill_select(q, k, v, self.cu, self.outs[l if self.resident else 0], self.stream)
        n_k = min(32, self.S)

        def loop():
            for s in range(n_k):
                for l in range(Lk):
                    d_ = self.dec[l]
                    kc[l].decode_step(d_[0][s], d_[1][s], d_[2][s], d_[3][s], d_[4][s], self.stream)

        us = self.graph_replay_us(loop, n_k * Lk)
        for c in kc:
            assert c.status() == 0, "device status word set"
            c.close()
        cnt = slot_counts(wl)
        nbytes = sum(c_ * self.d * self.esize + min(m, c_) * self.d * self.esize + 20 * c_ + 6 * self.d * self.esize for c_ in cnt) * self.H
        return {"m": m, "us_per_launch": us, "bytes_per_launch": nbytes, "achieved_gbs": nbytes / (us * 1e-6) / 1e9,
                "layer_caches": Lk}

    def e2e(self, n_steps):
        """The same step through the host-buffer C calls, pinned host tensors; on at most `e2e_layers` layers."""
        wl, L, S = self.wl, self.L, self.S
        prompt_bytes = 4 * wl.total_tokens * self.H * self.d * self.esize
        Le = max(1, min(L, int(self.args.e2e_pinned_gb * 1e9 // prompt_bytes)))
        hp = []
        for l in range(Le):
            q, k, v = self.prompts[l] if self.resident else self._draw_prompt(l)
            torch.cuda.synchronize(self.dev)
            hp.append(tuple(torch.empty(x.shape, dtype=x.dtype, pin_memory=True).copy_(x) for x in (q, k, v)) +
                      (torch.empty(q.shape, dtype=q.dtype, pin_memory=True),))
            del q, k, v
        hd = [tuple(torch.empty(x.shape, dtype=x.dtype, pin_memory=True).copy_(x) for x in self.dec[l]) for l in range(Le)]
        h2d = Le * 3 * wl.total_tokens * self.H * self.d * self.esize + S * Le * 3 * wl.units * self.d * self.esize
        d2h = Le * wl.total_tokens * self.H * self.d * self.esize + S * Le * (wl.units * self.d * self.esize + wl.units * 4)
        lstreams = [torch.cuda.Stream(device=self.dev) for _ in range(Le)]
        stream = self.stream

        def one_step_host():
            # one stream per layer for the prompt phase: the device-to-host copy of one layer's output overlaps
            # the host-to-device copies of the next layer's prompt
            start = torch.cuda.Event()
            start.record(stream)
            for l in range(Le):
                q, k, v, o = hp[l]
                lstreams[l].wait_event(start)
                self.caches[l].reset(lstreams[l])
                self.caches[l].prefill_select_host(q, k, v, self.cu, o, lstreams[l])
                done = torch.cuda.Event()
                done.record(lstreams[l])
                stream.wait_event(done)
            for s in range(S):
                for l in range(Le):
                    dq, dk, dv, do, de = hd[l]
                    self.caches[l].decode_step_host(dq[s], dk[s], dv[s], do[s], de[s], stream)

        one_step_host()
        torch.cuda.synchronize(self.dev)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for _ in range(n_steps):
            one_step_host()
        b.record(stream)
        torch.cuda.synchronize(self.dev)
        ms = a.elapsed_time(b) / n_steps
        for l in range(Le):
            assert self.caches[l].status() == 0, "device status word set"
        return {"ms_per_step": ms, "layers": Le, "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h), "steps": n_steps}

    def close(self):
        for c in self.caches:
            c.close()
        self.caches, self.prompts, self.dec, self.graph, self.outs = [], None, None, None, None
        torch.cuda.empty_cache()


def measure_config(pkg, wl, layers, dev, local, rank, world, dist, args, steps, warmup, headline):
    """Runs one configuration; returns (record for the JSON line, per-rank aggregated timings)."""
    run = ConfigRun(pkg, wl, layers, dev, local, rank, args)
    run.build_graph()

    def barrier():
        torch.cuda.synchronize(dev)
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize(dev)

    for _ in range(warmup):
        run.one_step()
    barrier()
    sampler = ClockSampler(_physical_gpu_index(local))
    sampler.start()
    wall0 = time.perf_counter()
    timed = [run.one_step(timed=True) for _ in range(steps)]
    barrier()
    wall_ms = (time.perf_counter() - wall0) * 1e3
    clocks = sampler.stop()
    for c in run.caches:
        assert c.status() == 0, "device status word set"
    pre = [t[0] for t in timed]
    decm = [t[1] for t in timed]
    total_ms = float(sum(pre) + sum(decm))
    # slowest replica decides: max over ranks of every figure that is reported
    agg = aggregate_over_ranks([total_ms, float(np.median(pre)), float(np.min(pre)), float(np.median(decm)), float(np.min(decm))],
                               world, dev, dist)
    total_ms, pre_med, pre_min, dec_med, dec_min = agg
    L, S, d, H = run.L, run.S, run.d, run.H
    peaks = _peaks()
    bytes_launch = decode_bytes_per_launch(wl)
    launch_us = dec_med * 1e3 / (S * L)
    achieved = bytes_launch / (launch_us * 1e-6) / 1e9
    flops_layer = sum(prefill_flops(n, d) for n in wl.prompt_lens) * H
    rec = {
        "workload": workload_label(wl, L),
        "value": whole_job_value(wl.units, L, S, steps, world, total_ms), "unit": UNIT,
        "ms_per_step": total_ms / steps,
        "prefill_ms": {"median": pre_med, "min": pre_min, "per_layer_median": pre_med / L},
        "decode_ms": {"median": dec_med, "min": dec_min},
        "decode_only_seq_heads_per_s": wl.units * L * S / (dec_med * 1e-3),
        "prefill_tflops_algorithmic": flops_layer * L / (pre_med * 1e-3) / 1e12,
        "prompts": "resident" if run.resident else "one layer resident at a time, drawn between the timed regions",
        "decode_launch": "cuda graph of the decode loop (%d launches)" % (S * L) if run.graph is not None else "one host call per launch",
        "l2": ("inputs larger than L2: %d layer caches of %.0f MB rotated every decode launch" % (L, bytes_launch / 1e6))
        if L * bytes_launch > 126e6 else "working set fits in L2 (correctness vehicle: no HBM roofline claim)",
        "wall_ms_per_step_with_input_generation": wall_ms / steps,
        "clocks": clocks,
        "roofline": {
            "kernel": "decode_two_pass_kernel" if run.caches[0].decode_path() == 2 else "decode_kernel", "bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
            "frac": achieved / peaks["hbm_gbs"], "peak_source": peaks["source"], "traffic": ncu_decode_traffic(wl),
            "bytes_per_launch": bytes_launch, "avg_launch_us": launch_us, "min_launch_us": dec_min * 1e3 / (S * L),
            "frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS,
        },
    }
    gpu_launches = steps * run.launches
    if rank == 0:
        rec["roofline"]["l2_warm_launch_us"] = run.l2_warm_us()
        if wl.dtype == "bf16" and d == 128:
            bd = run.prefill_breakdown()
            cs_flops = flops_layer / 2.0  # S^T = K Q^T over the triangle: 2 d n(n+1)/2 per unit
            cs_tf = cs_flops / (bd["column_sums_ms"] * 1e-3) / 1e12
            at_tf = flops_layer / (bd["attention_ms"] * 1e-3) / 1e12
            whole_ms = bd["attention_ms"] + bd["column_sums_ms"] + bd["select_gather_ms"]
            pipe_cs, prof_cs = ncu_tensor_pipe("colsum_tc_kernel", wl.name)
            pipe_at, prof_at = ncu_tensor_pipe("fwd_tc_short_kernel" if max(wl.prompt_lens) <= 4096 else "fwd_tc_kernel", wl.name)
            rec["roofline_prefill"] = {
                "kernel": "colsum_tc_kernel", "bound": "tensor", "unit": "TFLOP/s",
                "achieved": cs_tf, "peak": peaks["bf16_tflops"], "frac": cs_tf / peaks["bf16_tflops"],
                "frac_of_sustained": cs_tf / peaks["bf16_tflops_sustained"], "peak_source": peaks["source"],
                "flops_per_launch": cs_flops, "launch_ms": bd["column_sums_ms"],
                "tensor_pipe_pct_ncu": pipe_cs, "tensor_pipe_profile": prof_cs,
                "attention_kernel": {
                    "launch_ms": bd["attention_ms"], "tflops_algorithmic": at_tf,
                    "frac": at_tf / peaks["bf16_tflops"],
                    "tflops_issued_incl_hi_lo_split_of_P": 1.5 * at_tf,
                    "tensor_pipe_pct_ncu": pipe_at, "tensor_pipe_profile": prof_at},
                "select_gather_ms": bd["select_gather_ms"],
                "whole_prefill_select": {
                    "ms_per_layer": whole_ms,
                    "tflops_algorithmic": flops_layer / (whole_ms * 1e-3) / 1e12,
                    "tflops_executed_with_score_recompute": 1.5 * flops_layer / (whole_ms * 1e-3) / 1e12,
                    "frac_executed_of_burst": 1.5 * flops_layer / (whole_ms * 1e-3) / 1e12 / peaks["bf16_tflops"],
                    "frac_executed_of_sustained": 1.5 * flops_layer / (whole_ms * 1e-3) / 1e12 / peaks["bf16_tflops_sustained"]},
            }
        if headline or args.context:
            rec["decode_chunk_one_layer"] = run.chunk_figure()
        rec["decode_kv4_slots"] = run.kv4_figure(launch_us)
        if headline or args.context:
            rec["decode_topk_attention"] = run.topk_figure()
            rec["grouped_query_attention"] = run.gqa_figure()
    e2e = None
    if not args.no_e2e and (headline or args.e2e_all):
        e = run.e2e(max(1, min(steps, 2)))
        (e_ms,) = aggregate_over_ranks([e["ms_per_step"]], world, dev, dist)
        e2e = {"value": wl.units * e["layers"] * S * world / (e_ms * 1e-3), "unit": UNIT,
               "h2d_bytes_per_step": e["h2d_bytes_per_step"], "d2h_bytes_per_step": e["d2h_bytes_per_step"],
               "ms_per_step": e_ms,
               "layers": "%d of %d layer caches (pinned host copies of every layer's prompts would not fit; the layers "
                         "are independent and equally sized, so the rate is that of the whole stack)" % (e["layers"], L)
               if e["layers"] < L else "all %d" % L}
        rec["e2e"] = e2e
    run.close()
    return rec, gpu_launches


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default=HEADLINE, choices=sorted(CONFIGS))
    ap.add_argument("--layers", type=int, default=0, help="independent layer caches rotated per decode step (0 = the configuration's own)")
    ap.add_argument("--decode-steps", type=int, default=0, help="override the config's decode step count")
    ap.add_argument("--batch-limit", type=int, default=0,
                    help="keep only the first N sequences of the configuration (for small profiler captures)")
    ap.add_argument("--ref-units", type=int, default=64, help="units per step of the reference arm (the oracle on a sample)")
    ap.add_argument("--split", type=int, default=0, help="decode thread blocks per unit (0 = library default)")
    ap.add_argument("--stages", type=int, default=0, help="decode ring depth (0 = library default)")
    ap.add_argument("--no-graph", dest="graph", action="store_false",
                    help="launch every decode step from the host instead of replaying a CUDA graph of the decode loop")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--e2e-all", action="store_true", help="end-to-end figure for the per_config workloads too")
    ap.add_argument("--e2e-pinned-gb", type=float, default=28.0, help="pinned host memory the end-to-end leg may use for prompts")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-per-config", action="store_true", help="only the selected configuration")
    ap.add_argument("--context", action="store_true", help="chunk-call context figure for every configuration")
    args = ap.parse_args()

    wl = CONFIGS[args.config]
    if args.decode_steps:
        wl = wl.scaled(decode_steps=args.decode_steps)
    if args.batch_limit and args.batch_limit < wl.batch:
        n = args.batch_limit
        wl = wl.scaled(name="%s[:%d]" % (wl.name, n), batch=n, prompt_lens=wl.prompt_lens[:n], heavy=wl.heavy[:n],
                       recent=wl.recent[:n])
    layers = args.layers or DEFAULT_LAYERS[args.config]
    if args.impl == "reference":
        run_reference(args, wl, layers)
        return

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist

        dist.init_process_group("nccl", device_id=dev)

    import __graft_entry__

    if rank == 0:
        __graft_entry__.build()
    if world > 1:
        dist.barrier()
    import paper_2306_14048_b200 as pkg

    rec, gpu_launches = measure_config(pkg, wl, layers, dev, local, rank, world, dist, args, args.steps, args.warmup, True)
    per_config = []
    full_default = args.config == HEADLINE and not args.batch_limit and not args.decode_steps and not args.layers
    if world == 1 and not args.no_per_config and full_default:
        for name in PER_CONFIG:
            r, _ = measure_config(pkg, CONFIGS[name], DEFAULT_LAYERS[name], dev, local, rank, world, dist, args,
                                  max(5, args.steps), 3, False)
            per_config.append(r)

    if rank == 0:
        out = {
            "metric": METRIC, "value": rec["value"], "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": rec["ms_per_step"], "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": wl.dtype, "data": "synthetic",
            "config": {
                "workload": rec["workload"], "batch": wl.batch, "n_heads": wl.n_heads, "head_dim": wl.head_dim,
                "prompt_len_mean": int(np.mean(wl.prompt_lens)), "prompt_len_max": int(max(wl.prompt_lens)),
                "decode_steps": wl.decode_steps, "heavy_mean": int(np.mean(wl.heavy)), "recent_mean": int(np.mean(wl.recent)),
                "layers": layers, "decode_launch": rec["decode_launch"], "l2": rec["l2"], "prompts": rec["prompts"],
                "timed": "per step: one CUDA-event pair per layer around reset + prefill-select, one around the decode loop; "
                         "value = unit-steps / their sum over the steps",
            },
            "gpu_launches": gpu_launches,
        }
        for key in ("prefill_ms", "decode_ms", "decode_only_seq_heads_per_s", "prefill_tflops_algorithmic",
                    "wall_ms_per_step_with_input_generation", "clocks", "roofline", "roofline_prefill",
                    "decode_chunk_one_layer", "decode_kv4_slots", "decode_topk_attention", "grouped_query_attention", "e2e"):
            if key in rec:
                out[key] = rec[key]
        if per_config:
            out["per_config"] = per_config
        if world == 1 and not args.no_cpu_baseline:
            out["cpu_baseline"] = cpu_baseline(wl)
            if per_config:
                out["cpu_baseline_per_config"] = [dict(cpu_baseline(CONFIGS[name], budget_s=6.0), workload=name) for name in PER_CONFIG]
        print(json.dumps(out))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
