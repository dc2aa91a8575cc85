"""Lock-step comparison of the CUDA path (through the C ABI) with the fp64 oracle.

Both sides consume the same input bytes: tensors are produced once by the seeded
generators, the CUDA path reads them on the device and the oracle reads a host
copy.  Decisions (kept sets, evicted positions) must agree exactly; a disagreement
is excused, counted and re-synchronised only when the oracle's own fp64 scores of
the two choices differ by less than ``TIE_REL`` relative.  Outputs and accumulated
scores must agree within the stated tolerance.
"""
from __future__ import annotations

import dataclasses
import json
import os
from typing import Optional, Sequence

import numpy as np
import torch

from oracle import h2o_oracle
from workloads import Workload, make_decode_inputs, make_prompt_inputs

TIE_REL = 1e-6
TOPK_TIE_REL = 1e-5  # "Top-K" attention: the weakest kept and the strongest dropped logit closer than this (relative)
                     # are a floating-point toss-up between fp32 and fp64; the unit is left out from then on
TOL = {"bf16": (2e-3, 1e-2), "f32": (1e-5, 1e-4), "bf16_kv4": (2e-3, 1e-2)}  # |gpu - oracle| <= abs + rel * |oracle|


@dataclasses.dataclass
class ParityStats:
    units_checked: int = 0
    steps: int = 0
    decisions: int = 0
    near_ties_decode: int = 0
    near_ties_prefill: int = 0
    near_ties_topk: int = 0
    max_out_err: float = 0.0
    max_acc_err: float = 0.0


def record(stats: ParityStats, case: str) -> None:
    """One JSON line per parity case: printed, and appended to the file named by H2O_PARITY_LOG when that is set."""
    line = json.dumps({"case": case, **dataclasses.asdict(stats)})
    print(line)
    path = os.environ.get("H2O_PARITY_LOG")
    if path:
        with open(path, "a") as f:
            f.write(line + "\n")


def assert_close(got, want, dtype: str, what: str):
    a, r = TOL[dtype]
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    err = np.abs(got - want)
    bound = a + r * np.abs(want)
    if not np.all(err <= bound):
        i = int(np.argmax(err - bound))
        raise AssertionError("%s: |%g - %g| = %g exceeds %g (flat index %d)" % (
            what, got.flat[i], want.flat[i], err.flat[i], bound.flat[i], i))
    return float(err.max()) if err.size else 0.0


def _rel(a, b):
    m = max(abs(a), abs(b))
    return abs(a - b) / m if m > 0 else 0.0


def compare_state(gpu_cache, ora, units, dtype, stats: ParityStats, where: str, skip=()):
    pos, acc, count, t = gpu_cache.export()
    for x, u in enumerate(units):  # oracle unit x mirrors GPU unit u
        if x in skip:
            continue
        opos, oacc = ora.export(x)
        m = int(count[u])
        assert m == len(opos), "%s unit %d: count %d vs oracle %d" % (where, u, m, len(opos))
        assert int(t[u]) == int(ora.t[x]), "%s unit %d: t" % (where, u)
        order = np.argsort(pos[u, :m], kind="stable")
        gpos = pos[u, :m][order]
        assert np.array_equal(gpos, opos), "%s unit %d: kept positions differ" % (where, u)
        stats.max_acc_err = max(stats.max_acc_err, assert_close(acc[u, :m][order], oacc, dtype, "%s unit %d acc" % (where, u)))


def _gather_units(x, cu, units, H, G=1):
    """Rows of the sampled units, packed as [sum n_u, G, d] float32 on the host (G = 1 for keys and values; the
    query heads of a unit's group are heads h * G .. h * G + G - 1), plus their cu_seqlens."""
    parts, lens = [], []
    for u in units:
        s, h = divmod(u, H)
        parts.append(x[int(cu[s]):int(cu[s + 1]), h * G:(h + 1) * G])
        lens.append(int(cu[s + 1] - cu[s]))
    packed = torch.cat(parts, dim=0).float().cpu().numpy()
    return np.ascontiguousarray(packed), np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)


def run_parity(wl: Workload, gpu_cache_cls, units: Optional[Sequence[int]] = None, steps: Optional[int] = None,
               export_every: int = 32, layer: int = 0, prefill: bool = True, scale: float = 0.0,
               device: str = "cuda", prefill_path: int = 0, chunk: int = 0, chunk_path: int = 0,
               pattern: Optional[Sequence[int]] = None, score_mode: int = 0, static_scratch: bool = False,
               mask: Optional[Sequence[int]] = None, split: int = 0, topk: int = 0, group: int = 1,
               decode_path: int = 0) -> ParityStats:
    """Run prefill-select (optional) and ``steps`` decode steps on both sides, comparing as it goes.

    The CUDA path always processes the whole workload; the oracle mirrors only the sampled ``units``
    (all of them by default) as a batch of single-head sequences, which is exact because units never
    interact.  With ``chunk`` > 0 the CUDA path advances ``chunk`` tokens per call (h2o_decode_chunk)
    while the oracle still takes them one decode step at a time.  ``pattern`` cycles through call
    sizes instead: 0 = one h2o_decode_step call, n > 0 = one h2o_decode_chunk call of n tokens.
    ``split``: thread blocks (one cluster) per unit in the decode kernel, 0 = the library's choice.
    ``decode_path``: h2o_cache_set_decode_path (0 automatic, 1 online-softmax kernel, 2 two-pass streaming kernel).
    ``group`` > 1: grouped-query attention: wl.n_heads counts the K/V heads, q and out carry n_heads * group query heads
    (drawn from the same recipe with that many heads).
    ``topk`` > 0: "Top-K" attention in decode steps on both sides (h2o_cache_set_topk); a unit whose weakest kept and
    strongest dropped logit come closer than TOPK_TIE_REL is counted and left out of every later comparison.
    ``mask`` = (kind, a, b): sparse pattern inside the recent window (h2o_cache_set_mask) on both sides.
    ``scale`` > 0 replaces the default softmax scale 1/sqrt(d) (4/sqrt(d) is the peaky-softmax stress run).
    """
    if topk > 0:  # the oracle's attention rule is process-wide: always put it back
        h2o_oracle.set_topk(topk)
        try:
            return run_parity(wl, gpu_cache_cls, units, steps, export_every, layer, prefill, scale, device, prefill_path,
                              chunk, chunk_path, pattern, score_mode, static_scratch, mask, split, topk=-topk, group=group, decode_path=decode_path)
        finally:
            h2o_oracle.set_topk(0)
    topk = -topk  # (negative: the oracle already has it)
    if mask is not None and len(mask) == 3 and mask[0] == 0:
        mask = None
    if mask is not None and mask[0] != 0:  # the oracle's attention pattern is process-wide as well
        h2o_oracle.set_mask(*mask)
        try:
            return run_parity(wl, gpu_cache_cls, units, steps, export_every, layer, prefill, scale, device, prefill_path,
                              chunk, chunk_path, pattern, score_mode, static_scratch, mask=(0,) + tuple(mask), split=split,
                              topk=-topk, group=group, decode_path=decode_path)
        finally:
            h2o_oracle.set_mask(0)
    if score_mode > 0:  # the oracle's ranking rule is process-wide: always put it back
        h2o_oracle.set_score_mode(score_mode)
        try:
            return run_parity(wl, gpu_cache_cls, units, steps, export_every, layer, prefill, scale, device, prefill_path,
                              chunk, chunk_path, pattern, score_mode=0 - score_mode, static_scratch=static_scratch, mask=mask,
                              split=split, topk=-topk, group=group, decode_path=decode_path)
        finally:
            h2o_oracle.set_score_mode(0)
    score_mode = -score_mode  # (negative: the oracle is already in that mode)
    stats = ParityStats()
    H, d = wl.n_heads, wl.head_dim
    units = list(range(wl.units)) if units is None else sorted(set(int(u) for u in units))
    stats.units_checked = len(units)
    steps = wl.decode_steps if steps is None else steps
    # the C ABI takes the softmax scale as a float: both sides get that same fp32 value
    scale = float(np.float32(scale if scale > 0 else 1.0 / np.sqrt(float(d))))
    G = int(group)
    wl_q = wl.scaled(n_heads=H * G) if G > 1 else wl  # the query side has H * G heads
    gpu = gpu_cache_cls(wl.batch, H, d, wl.dtype, wl.heavy, wl.recent, softmax_scale=scale, device=0, query_group=G) \
        if G > 1 else gpu_cache_cls(wl.batch, H, d, wl.dtype, wl.heavy, wl.recent, softmax_scale=scale, device=0)
    gpu.set_prefill_path(prefill_path)
    gpu.set_decode_shape(split, 0)
    if decode_path:
        gpu.set_decode_path(decode_path)
    if topk > 0:
        gpu.set_topk(topk)
    gpu.set_score_mode(score_mode)
    if mask is not None:  # (0, kind, a, b): the oracle already has it
        gpu.set_mask(*mask[1:])
    ora = h2o_oracle.OracleCache(len(units), 1, d, [wl.heavy[u // H] for u in units], [wl.recent[u // H] for u in units],
                                 scale=scale, kv4=(wl.dtype == "bf16_kv4"), group=G)
    uidx = torch.as_tensor(units, dtype=torch.long, device=device)
    if prefill:
        q, k, v, cu = make_prompt_inputs(wl, layer=layer, device=device)
        if G > 1:
            q = make_prompt_inputs(wl_q, layer=layer, device=device)[0]
        out = torch.empty_like(q)
        if static_scratch:  # the entry point that takes no scratch buffer
            gpu.prefill_select_static(q, k, v, cu, out)
        else:
            gpu.prefill_select(q, k, v, cu, out)
        assert gpu.status() == 0
        qh, ocu = _gather_units(q, cu, units, H, G)
        kh, _ = _gather_units(k, cu, units, H)
        vh, _ = _gather_units(v, cu, units, H)
        out_h, _ = _gather_units(out, cu, units, H, G)
        o_out, o_kept = ora.prefill(qh, kh, vh, ocu)
        pos, acc, count, t = gpu.export()
        for x, u in enumerate(units):
            lo, hi = int(ocu[x]), int(ocu[x + 1])
            stats.max_out_err = max(stats.max_out_err, assert_close(out_h[lo:hi], o_out[lo:hi], wl.dtype,
                                                                    "prefill out unit %d" % u))
            m = int(count[u])
            gkept = np.sort(pos[u, :m])
            if not np.array_equal(gkept, o_kept[x]):
                acc0, (b_keep, b_drop) = ora.last_acc0[x], ora.last_boundary[x]
                diff = set(gkept.tolist()) ^ set(o_kept[x].tolist())
                assert len(gkept) == len(o_kept[x]), "prefill unit %d: kept count" % u
                rank = (lambda j: acc0[j] / (hi - lo - j)) if score_mode == 1 else (lambda j: acc0[j])
                for j in diff:  # every disputed position must sit on the k-th / (k+1)-th boundary
                    assert _rel(rank(j), b_keep) < TIE_REL and _rel(rank(j), b_drop) < TIE_REL, (
                        "prefill unit %d: position %d (score %.17g) kept/dropped against the oracle "
                        "(boundary %.17g / %.17g)" % (u, j, acc0[j], b_keep, b_drop))
                stats.near_ties_prefill += 1
                ora.load_unit(x, gkept, acc0[gkept], kh[lo:hi, 0][gkept], vh[lo:hi, 0][gkept], hi - lo)
            stats.decisions += 1
        compare_state(gpu, ora, units, wl.dtype, stats, "after prefill")
        del q, k, v, out, qh, kh, vh, out_h
    ev = torch.empty(wl.batch, H, dtype=torch.int32, device=device)

    def pick(x, g=1):  # [batch, H * g, d] -> the sampled units as [len(units), g, d] float32 on the host
        return x.reshape(wl.units, g, d)[uidx].float().cpu().numpy()

    dead = set()  # oracle units left out after a "Top-K" toss-up
    step, call = 0, 0
    while step < steps:
        if pattern:
            chunk = int(pattern[call % len(pattern)])
            call += 1
        nt = min(chunk, steps - step) if chunk > 0 else 1
        qs, ks, vs = zip(*[make_decode_inputs(wl, step + i, layer=layer, device=device) for i in range(nt)])
        if G > 1:
            qs = tuple(make_decode_inputs(wl_q, step + i, layer=layer, device=device)[0] for i in range(nt))
        if chunk > 0:
            q, k, v = (torch.stack(x).contiguous() for x in (qs, ks, vs))  # [nt, batch, H, d]
            out = torch.empty_like(q)
            evs = torch.full((nt, wl.batch, H), -7, dtype=torch.int32, device=device)
            gpu.set_chunk_path(chunk_path)
            gpu.decode_chunk(q, k, v, out, evs)
        else:
            out = torch.empty_like(qs[0])[None]
            ev.fill_(-7)
            gpu.decode_step(qs[0], ks[0], vs[0], out[0], ev)
            evs = ev[None]
        for i in range(nt):
            g_ev = evs[i].reshape(-1)[uidx].cpu().numpy()
            g_out = out[i].reshape(wl.units, G * d)[uidx].float().cpu().numpy()
            res = ora.decode_step(pick(qs[i], G), pick(ks[i]), pick(vs[i]), hint=g_ev, tie_rel=TIE_REL)
            if topk > 0:
                for x in range(len(units)):
                    if x not in dead and res["topk_gap"][x] < TOPK_TIE_REL:
                        dead.add(x)
                        stats.near_ties_topk += 1
            live = [x for x in range(len(units)) if x not in dead]
            for x in live:
                st = int(res["status"][x])
                if st == 2:
                    raise AssertionError("step %d unit %d: evicted %d, oracle %d (gap %.3g)" % (
                        step + i, units[x], g_ev[x], res["evicted"][x], res["gap"][x]))
                stats.near_ties_decode += st == 1
            stats.decisions += len(live)
            stats.max_out_err = max(stats.max_out_err,
                                    assert_close(g_out[live], res["out"][live], wl.dtype, "decode out step %d" % (step + i)))
        last = step + nt - 1
        if (last + 1) % export_every < nt or last == steps - 1:
            compare_state(gpu, ora, units, wl.dtype, stats, "after step %d" % last, skip=dead)
        step += nt
    assert gpu.status() == 0
    stats.steps = steps
    gpu.close()
    return stats
