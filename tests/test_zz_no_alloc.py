"""The allocation-free prefill entry point against the ordinary one (needs a B200).

h2o_prefill_select_static exists for callers that may not allocate device memory (no
cudaMalloc in their position: a plugin inside someone else's memory pool, a loop that
must stay clear of the allocator).  Its scratch is an array inside the library, so the
interesting failure modes are a wrong device address for that array and state left over
from one call leaking into the next.  Hence: two calls in a row on different prompts,
each compared with the caller-scratch entry point on the same inputs, through the C ABI.

This file sorts last on purpose: a run that stops at the first failure has then already
executed every other test.
"""
import ctypes

import numpy as np
import pytest
import torch

from workloads import Workload, make_decode_inputs, make_prompt_inputs

pytestmark = pytest.mark.gpu


def _run(pkg, wl, use_static):
    """Prefill-select + two decode steps; returns everything observable."""
    cache = pkg.H2OCache(wl.batch, wl.n_heads, wl.head_dim, wl.dtype, wl.heavy, wl.recent)
    q, k, v, cu = make_prompt_inputs(wl, device="cuda")
    out = torch.zeros_like(q)
    if use_static:
        cache.prefill_select_static(q, k, v, cu, out)
    else:
        cache.prefill_select(q, k, v, cu, out)
    assert cache.status() == 0
    state0 = cache.export()
    dec = []
    ev = torch.empty(wl.batch, wl.n_heads, dtype=torch.int32, device="cuda")
    for step in range(2):
        dq, dk, dv = make_decode_inputs(wl, step, device="cuda")
        do = torch.empty_like(dq)
        cache.decode_step(dq, dk, dv, do, ev)
        dec.append((do.float().cpu().numpy(), ev.cpu().numpy().copy()))
    state1 = cache.export()
    assert cache.status() == 0
    cache.close()
    return out.float().cpu().numpy(), state0, dec, state1


def _same(a, b):
    """Both entry points run the same deterministic kernels, so everything observable must be bit-identical:
    a tolerance would let a stale or misplaced scratch that only perturbs low bits through."""
    out_a, s0a, dec_a, s1a = a
    out_b, s0b, dec_b, s1b = b
    assert np.array_equal(out_a, out_b), "prefill out"
    for (pa, aa, ca, ta), (pb, ab, cb, tb) in ((s0a, s0b), (s1a, s1b)):
        assert np.array_equal(pa, pb) and np.array_equal(ca, cb) and np.array_equal(ta, tb)  # kept sets
        assert np.array_equal(aa, ab), "accumulated scores"
    for (oa, ea), (ob, eb) in zip(dec_a, dec_b):
        assert np.array_equal(ea, eb)  # eviction decisions
        assert np.array_equal(oa, ob), "decode out"


def test_static_scratch_entry_point_matches_caller_scratch_twice_in_a_row():
    import paper_2306_14048_b200 as pkg

    assert torch.cuda.is_available(), "needs a CUDA device; there is no CPU fallback"
    limit = int(pkg.lib.h2o_prefill_static_scratch_bytes())
    assert limit == 16 << 20
    # first call: tensor-core path, ragged, several tiles; second call: different shape and dtype,
    # so anything the first call left in the shared array would be in the way
    first = Workload("noalloc_a", 3, 4, 128, "bf16", (700, 257, 64), 2, (24, 16, 8), (24, 16, 8), 1, 515)
    second = Workload("noalloc_b", 2, 3, 64, "f32", (190, 333), 2, (12, 20), (10, 20), 1, 516)
    for wl in (first, second):
        _same(_run(pkg, wl, use_static=True), _run(pkg, wl, use_static=False))


def test_static_scratch_entry_point_against_the_oracle(oracle):
    """The same entry point checked against the fp64 oracle (prefill outputs, kept sets, scores, then decode steps)."""
    import paper_2306_14048_b200 as pkg
    from parity_harness import run_parity

    assert torch.cuda.is_available(), "needs a CUDA device; there is no CPU fallback"
    wl = Workload("noalloc_c", 3, 4, 128, "bf16", (700, 257, 64), 12, (24, 16, 8), (24, 16, 8), 1, 518)
    st = run_parity(wl, pkg.H2OCache, export_every=6, static_scratch=True)
    assert st.units_checked == wl.units and st.decisions > 0


def test_static_scratch_entry_point_refuses_oversized_prompts():
    import paper_2306_14048_b200 as pkg

    assert torch.cuda.is_available(), "needs a CUDA device; there is no CPU fallback"
    # 40 heads x 32768 tokens needs ~21 MB of scratch: more than the built-in 16 MiB
    wl = Workload("noalloc_big", 1, 40, 64, "bf16", (32768,), 1, (8,), (8,), 1, 517)
    cache = pkg.H2OCache(wl.batch, wl.n_heads, wl.head_dim, wl.dtype, wl.heavy, wl.recent)
    assert pkg.h2o_prefill_scratch_bytes(cache.cfg, 32768) > int(pkg.lib.h2o_prefill_static_scratch_bytes())
    q = torch.zeros(32768, 40, 64, dtype=torch.bfloat16, device="cuda")
    out = torch.empty_like(q)
    cu = np.array([0, 32768], dtype=np.int32)
    rc = pkg.lib.h2o_prefill_select_static(cache._h, q.data_ptr(), q.data_ptr(), q.data_ptr(),
                                           cu.ctypes.data_as(ctypes.POINTER(ctypes.c_int32)), out.data_ptr(), None)
    assert rc == pkg.H2O_ERR_WORKSPACE
    _, _, count, t = cache.export()
    assert not count.any() and not t.any()  # nothing was launched: the cache is still empty
    cache.close()
