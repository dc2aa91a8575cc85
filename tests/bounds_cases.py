"""Parity cases run against the checked build of the library (every slot / unit / row index verified before use).

Executed as a script by tests/test_gpu_bounds_build.py in a process of its own, with H2O_B200_LIB naming
libh2o_b200_bounds.so: the binding loads one library per process.  Every case must pass parity AND leave the status
word clear (a check that fired would have recorded H2O_ERR_STATE); the last case plants an out-of-range counter
that stays inside the allocation and expects exactly that code.
"""
import os
import sys

import numpy as np
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
sys.path.insert(0, os.path.join(ROOT, "tests"))


def main():
    import paper_2306_14048_b200 as pkg
    from oracle import h2o_oracle
    from parity_harness import run_parity
    from workloads import CONFIGS, Workload, make_decode_inputs

    h2o_oracle.build()
    assert pkg.lib.h2o_debug_bounds_checked() == 1, "this script must run against the checked build"

    def wl(name, batch, heads, d, dtype, lens, steps, heavy, recent, seed):
        return Workload(name, batch, heads, d, dtype, tuple(lens), steps, tuple(heavy), tuple(recent), 1, seed)

    cases = [
        ("tiny fp32 config", CONFIGS["c1_tiny"], {}),
        ("ragged bf16, tensor-core prefill", wl("b1", 4, 3, 128, "bf16", [300, 77, 513, 40], 24, [20, 9, 33, 30], [24, 5, 31, 30], 801), {}),
        ("ragged f32 d64", wl("b2", 4, 3, 64, "f32", [300, 77, 513, 40], 24, [20, 9, 33, 30], [24, 5, 31, 30], 802), {}),
        ("k = 0", wl("b3", 2, 2, 64, "f32", [37, 21], 30, [0, 0], [7, 16], 803), {}),
        ("r = 0", wl("b4", 2, 2, 64, "f32", [37, 21], 30, [5, 12], [0, 0], 804), {}),
        ("single slots", wl("b5", 2, 2, 64, "f32", [37, 21], 30, [1, 0], [0, 1], 805), {}),
        ("fill phase from empty", wl("b6", 2, 2, 128, "bf16", [1, 1], 60, [10, 4], [6, 20], 806), dict(prefill=False)),
        ("units split over a cluster", wl("b7", 2, 2, 128, "bf16", [1500, 1300], 16, [150, 30], [150, 40], 807), {}),
        ("4-bit slots", wl("b8", 3, 2, 128, "bf16_kv4", [300, 77, 513], 24, [20, 9, 33], [24, 5, 31], 808), {}),
        ("chunk call", wl("b9", 2, 3, 128, "bf16", [400, 300], 40, [20, 30], [24, 16], 809), dict(chunk=16)),
        ("sparse pattern", wl("b10", 2, 3, 128, "bf16", [400, 300], 24, [20, 30], [24, 16], 810), dict(mask=(1, 8, 3))),
        ("top-k attention", wl("b12", 2, 3, 128, "bf16", [400, 300], 24, [20, 30], [24, 16], 812), dict(topk=9)),
        ("grouped-query attention", wl("b13", 2, 2, 128, "bf16", [300, 200], 24, [20, 30], [24, 16], 813), dict(group=4)),
        ("4-bit slots split over a cluster", wl("b15", 1, 2, 128, "bf16_kv4", [1500], 12, [300], [260], 815), dict(split=4)),
        ("two-pass step kernel split over a cluster", wl("b16", 1, 2, 128, "bf16", [1500], 12, [300], [260], 816), dict(split=4, decode_path=2)),
        ("two-pass step kernel, fill phase", wl("b14", 3, 2, 128, "bf16", [300, 20, 513], 24, [20, 30, 33], [24, 16, 31], 814), dict(decode_path=2)),
    ]
    for name, w, kw in cases:
        st = run_parity(w, pkg.H2OCache, export_every=8, **kw)  # asserts status == 0 at the end
        print("ok:", name, st)

    # a counter beyond the budget (it stays inside the allocation: the next unit's slots follow): the checked build
    # records H2O_ERR_STATE and skips the unit's rows instead of reading past the unit
    w = wl("b11", 1, 4, 128, "bf16", [64], 1, [8], [8], 811)
    cache = pkg.H2OCache(w.batch, w.n_heads, w.head_dim, w.dtype, w.heavy, w.recent)
    dq, dk, dv = make_decode_inputs(w, 0, device="cuda")
    out = torch.empty_like(dq)
    for _ in range(20):
        cache.decode_step(dq, dk, dv, out)
    assert cache.status() == 0
    slots, align = 4 * 16, 256
    up = lambda x: (x + align - 1) // align * align
    off_count = up(slots * 256) * 2 + up(slots * 8) + up(slots * 4)  # K, V, accumulated scores, positions, then the counters
    base = cache._ws_ptr - cache.workspace.data_ptr()
    counters = cache.workspace[base + off_count: base + off_count + 16].view(torch.int32)
    assert counters.tolist() == [16, 16, 16, 16], counters.tolist()
    counters[1] = 19  # unit 1 claims three entries more than its budget
    torch.cuda.synchronize()
    cache.decode_step(dq, dk, dv, out)
    assert cache.status() == pkg.H2O_ERR_STATE
    cache.close()
    print("ok: planted counter caught")
    print("BOUNDS_CASES_PASSED")


if __name__ == "__main__":
    main()
