"""Behaviour of the C ABI on a device: call order, host-buffer variants, reset, determinism."""
import ctypes

import numpy as np
import pytest
import torch

from workloads import Workload, make_decode_inputs, make_prompt_inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def pkg():
    import paper_2306_14048_b200 as p

    assert torch.cuda.is_available(), "these tests need a CUDA device; there is no CPU fallback"
    return p


WL = Workload("api", 3, 4, 128, "bf16", (260, 97, 513), 6, (16, 8, 20), (16, 8, 20), 1, 909)


def _full_run(pkg, wl, host=False, reset_first=False, group=1):
    cache = pkg.H2OCache(wl.batch, wl.n_heads, wl.head_dim, wl.dtype, wl.heavy, wl.recent, query_group=group)
    wlq = wl.scaled(n_heads=wl.n_heads * group)  # the query side carries n_heads * group heads
    q, k, v, cu = make_prompt_inputs(wl, device="cuda")
    if group > 1:
        q = make_prompt_inputs(wlq, device="cuda")[0]
        reset_first = False
    if reset_first:  # dirty the cache with another prompt, then reset it
        cache.prefill_select(v, q, k, cu, torch.empty_like(q))
        cache.reset()
    outs = []
    if host:
        hq, hk, hv = (x.cpu().pin_memory() for x in (q, k, v))
        ho = torch.empty_like(hq).pin_memory()
        cache.prefill_select_host(hq, hk, hv, cu, ho)  # (staging sized for the larger q / out of a grouped cache)
        torch.cuda.synchronize()
        outs.append(ho.float().numpy().copy())
    else:
        o = torch.empty_like(q)
        cache.prefill_select(q, k, v, cu, o)
        outs.append(o.float().cpu().numpy())
    evs = []
    for step in range(wl.decode_steps):
        dq, dk, dv = make_decode_inputs(wl, step, device="cuda")
        if group > 1:
            dq = make_decode_inputs(wlq, step, device="cuda")[0]
        if host:
            # pinned buffers are read and written by the kernel directly; pageable ones go through the staging copies
            pin = (lambda x: x.pin_memory()) if host != "pageable" else (lambda x: x)
            hq, hk, hv = (pin(x.cpu()) for x in (dq, dk, dv))
            ho = pin(torch.empty_like(hq))
            he = pin(torch.empty(wl.batch, wl.n_heads, dtype=torch.int32))
            cache.decode_step_host(hq, hk, hv, ho, he)
            torch.cuda.synchronize()
            outs.append(ho.float().numpy().copy())
            evs.append(he.numpy().copy())
        else:
            do = torch.empty_like(dq)
            de = torch.empty(wl.batch, wl.n_heads, dtype=torch.int32, device="cuda")
            cache.decode_step(dq, dk, dv, do, de)
            outs.append(do.float().cpu().numpy())
            evs.append(de.cpu().numpy())
    state = cache.export()
    assert cache.status() == 0
    cache.close()
    return outs, evs, state


def _identical(a, b):
    for x, y in zip(a[0], b[0]):
        assert np.array_equal(x, y)
    for x, y in zip(a[1], b[1]):
        assert np.array_equal(x, y)
    for x, y in zip(a[2], b[2]):
        assert np.array_equal(x, y)


def test_two_runs_are_bit_identical(pkg):
    """No float atomics anywhere on the path: the same inputs give the same bits."""
    _identical(_full_run(pkg, WL), _full_run(pkg, WL))


@pytest.mark.parametrize("mode", ["pinned", "pageable"])
def test_host_buffer_calls_equal_device_calls(pkg, mode):
    _identical(_full_run(pkg, WL, host=mode), _full_run(pkg, WL))


@pytest.mark.parametrize("mode", ["pinned", "pageable"])
def test_host_buffer_calls_with_grouped_query_heads(pkg, mode):
    """q and out carry n_heads * group heads, k / v / evicted positions n_heads: the staging is laid out for that."""
    _identical(_full_run(pkg, WL, host=mode, group=4), _full_run(pkg, WL, group=4))


def test_kv4_slots_host_calls_snapshots_and_reproducibility(pkg):
    """The 4-bit slot format through the same API surface: host-buffer calls equal device calls, two runs are
    bit-identical, and a snapshot of its (smaller) workspace resumes exactly."""
    wl = Workload("kv4api", 3, 4, 128, "bf16_kv4", (260, 97, 513), 6, (16, 8, 20), (16, 8, 20), 1, 909)
    _identical(_full_run(pkg, wl), _full_run(pkg, wl))
    _identical(_full_run(pkg, wl, host="pinned"), _full_run(pkg, wl))
    q, k, v, cu = make_prompt_inputs(wl, device="cuda")
    a = pkg.H2OCache(wl.batch, wl.n_heads, wl.head_dim, wl.dtype, wl.heavy, wl.recent)
    full = pkg.H2OCache(wl.batch, wl.n_heads, wl.head_dim, "bf16", wl.heavy, wl.recent)
    assert a.workspace_bytes < 0.5 * full.workspace_bytes
    full.close()
    a.prefill_select(q, k, v, cu, torch.empty_like(q))
    steps = [make_decode_inputs(wl, s, device="cuda") for s in range(wl.decode_steps)]

    def step(c, s):
        dq, dk, dv = steps[s]
        o = torch.empty_like(dq)
        e = torch.empty(wl.batch, wl.n_heads, dtype=torch.int32, device="cuda")
        c.decode_step(dq, dk, dv, o, e)
        return o.float().cpu().numpy(), e.cpu().numpy()

    for s in range(3):
        step(a, s)
    b = pkg.H2OCache(wl.batch, wl.n_heads, wl.head_dim, wl.dtype, wl.heavy, wl.recent, snapshot=a.snapshot().cpu())
    for s in range(3, wl.decode_steps):
        oa, ea = step(a, s)
        ob, eb = step(b, s)
        assert np.array_equal(oa, ob) and np.array_equal(ea, eb)
    assert a.status() == 0 and b.status() == 0
    a.close()
    b.close()


def test_reset_returns_the_cache_to_empty(pkg):
    _identical(_full_run(pkg, WL, reset_first=True), _full_run(pkg, WL))


def test_call_order_and_argument_errors(pkg):
    wl = WL
    cache = pkg.H2OCache(wl.batch, wl.n_heads, wl.head_dim, wl.dtype, wl.heavy, wl.recent)
    q, k, v, cu = make_prompt_inputs(wl, device="cuda")
    o = torch.empty_like(q)
    with pytest.raises(pkg.H2OError) as e:  # out aliases an input
        cache.prefill_select(q, k, v, cu, q)
    assert e.value.code == pkg.H2O_ERR_INVALID_ARG
    bad_cu = np.array(cu)
    bad_cu[1] = 0  # an empty sequence
    with pytest.raises(pkg.H2OError) as e:
        cache.prefill_select(q, k, v, bad_cu, o)
    assert e.value.code == pkg.H2O_ERR_INVALID_ARG
    cache.prefill_select(q, k, v, cu, o)
    with pytest.raises(pkg.H2OError) as e:  # only once per cache
        cache.prefill_select(q, k, v, cu, o)
    assert e.value.code == pkg.H2O_ERR_STATE
    dq, dk, dv = make_decode_inputs(wl, 0, device="cuda")
    cache.decode_step(dq, dk, dv, torch.empty_like(dq), None)  # evicted_pos is optional
    with pytest.raises(pkg.H2OError) as e:  # and not after decoding has started
        cache.prefill_select(q, k, v, cu, o)
    assert e.value.code == pkg.H2O_ERR_STATE
    # undersized scratch
    need = pkg.h2o_prefill_scratch_bytes(cache.cfg, int(cu[-1]))
    cache.reset()
    small = torch.empty(need // 2 + 256, dtype=torch.uint8, device="cuda")
    sp = (small.data_ptr() + 255) // 256 * 256
    rc = pkg.lib.h2o_prefill_select(cache._h, q.data_ptr(), k.data_ptr(), v.data_ptr(),
                                    np.ascontiguousarray(cu, dtype=np.int32).ctypes.data_as(ctypes.POINTER(ctypes.c_int32)),
                                    o.data_ptr(), sp, need // 2, None)
    assert rc == pkg.H2O_ERR_WORKSPACE
    assert cache.status() == 0
    _, _, count, t = cache.export()
    assert not count.any() and not t.any()  # refused calls launch nothing
    cache.close()


def test_caches_on_different_streams(pkg):
    """Two caches driven from two streams at once give the same results as one after the other."""
    wl = WL
    ref = _full_run(pkg, wl)
    streams = [torch.cuda.Stream() for _ in range(2)]
    caches = [pkg.H2OCache(wl.batch, wl.n_heads, wl.head_dim, wl.dtype, wl.heavy, wl.recent) for _ in range(2)]
    q, k, v, cu = make_prompt_inputs(wl, device="cuda")
    outs = [[], []]
    torch.cuda.synchronize()
    for i, (c, st) in enumerate(zip(caches, streams)):
        o = torch.empty_like(q)
        c.prefill_select(q, k, v, cu, o, st)
        outs[i].append(o)
    ins = [make_decode_inputs(wl, s, device="cuda") for s in range(wl.decode_steps)]
    torch.cuda.synchronize()
    for s in range(wl.decode_steps):
        for i, (c, st) in enumerate(zip(caches, streams)):
            dq, dk, dv = ins[s]
            do = torch.empty_like(dq)
            c.decode_step(dq, dk, dv, do, None, st)
            outs[i].append(do)
    torch.cuda.synchronize()
    for i, c in enumerate(caches):
        for got, want in zip(outs[i], ref[0]):
            assert np.array_equal(got.float().cpu().numpy(), want)
        for x, y in zip(c.export(), ref[2]):
            assert np.array_equal(x, y)
        c.close()


def test_create_then_decode_at_once_on_a_non_blocking_stream(pkg):
    """h2o_cache_create returns with its tables on the device: a stream that is not ordered behind the legacy
    default stream (every torch side stream is non-blocking) may be used right away, with no synchronisation
    between create and the first call."""
    wl = Workload("fresh", 4, 8, 128, "bf16", (1, 1, 1, 1), 24, (6, 8, 4, 10), (6, 8, 4, 10), 1, 910)
    ins = [make_decode_inputs(wl, s, device="cuda") for s in range(wl.decode_steps)]
    side = torch.cuda.Stream()
    torch.cuda.synchronize()
    runs = []
    for rep in range(6):
        # dirty a block of memory the allocator will hand to the next workspace
        junk = torch.full((pkg.h2o_cache_workspace_bytes(pkg.make_config(
            wl.batch, wl.n_heads, wl.head_dim, wl.dtype, wl.heavy, wl.recent)[0]) + 256,), 0x5A, dtype=torch.uint8, device="cuda")
        torch.cuda.synchronize()
        del junk
        cache = pkg.H2OCache(wl.batch, wl.n_heads, wl.head_dim, wl.dtype, wl.heavy, wl.recent)
        outs, evs = [], []
        for dq, dk, dv in ins:  # token-by-token from the empty cache, nothing in between
            do = torch.empty_like(dq)
            de = torch.empty(wl.batch, wl.n_heads, dtype=torch.int32, device="cuda")
            cache.decode_step(dq, dk, dv, do, de, side)
            outs.append(do)
            evs.append(de)
        side.synchronize()
        assert cache.status(side) == 0
        runs.append(([o.float().cpu().numpy() for o in outs], [e.cpu().numpy() for e in evs], cache.export(side)))
        cache.close()
    for r in runs[1:]:
        _identical(runs[0], r)
    assert (runs[0][2][3] == wl.decode_steps).all()  # every unit advanced from t = 0


def test_snapshot_and_attach_resume_bit_identically(pkg):
    """The workspace bytes are the whole state: a handle attached to a copy continues exactly like the original,
    also through a file-like round trip on the host; a different configuration is refused."""
    wl = WL
    q, k, v, cu = make_prompt_inputs(wl, device="cuda")
    a = pkg.H2OCache(wl.batch, wl.n_heads, wl.head_dim, wl.dtype, wl.heavy, wl.recent)
    a.prefill_select(q, k, v, cu, torch.empty_like(q))
    steps = [make_decode_inputs(wl, s, device="cuda") for s in range(wl.decode_steps)]

    def step(c, s):
        dq, dk, dv = steps[s]
        o = torch.empty_like(dq)
        e = torch.empty(wl.batch, wl.n_heads, dtype=torch.int32, device="cuda")
        c.decode_step(dq, dk, dv, o, e)
        return o.float().cpu().numpy(), e.cpu().numpy()

    for s in range(2):
        step(a, s)
    snap = a.snapshot().cpu()  # as if written to and read back from a file
    b = pkg.H2OCache(wl.batch, wl.n_heads, wl.head_dim, wl.dtype, wl.heavy, wl.recent, snapshot=snap)
    for s in range(2, wl.decode_steps):
        oa, ea = step(a, s)
        ob, eb = step(b, s)
        assert np.array_equal(oa, ob) and np.array_equal(ea, eb)
    for x, y in zip(a.export(), b.export()):
        assert np.array_equal(x, y)
    assert a.status() == 0 and b.status() == 0
    # an attached cache is not prefilled again
    with pytest.raises(pkg.H2OError) as err:
        b.prefill_select(q, k, v, cu, torch.empty_like(q))
    assert err.value.code == pkg.H2O_ERR_STATE
    # the unit table of another configuration does not match
    heavy2 = tuple(x + 4 for x in wl.heavy)
    snap2 = pkg.H2OCache(wl.batch, wl.n_heads, wl.head_dim, wl.dtype, heavy2, wl.recent).snapshot()
    with pytest.raises(pkg.H2OError) as err:
        pkg.H2OCache(wl.batch, wl.n_heads, wl.head_dim, wl.dtype, wl.heavy, wl.recent, snapshot=snap2[:a.workspace_bytes])
    assert err.value.code == pkg.H2O_ERR_STATE
    a.close()
    b.close()


def test_a_wait_that_gives_up_costs_a_status_code_not_the_context(pkg):
    """A bounded wait that runs out records H2O_ERR_TIMEOUT; the kernel returns, reset clears the word and
    the cache works as before."""
    wl = WL
    c = pkg.H2OCache(wl.batch, wl.n_heads, wl.head_dim, wl.dtype, wl.heavy, wl.recent)
    assert c.status() == 0
    assert pkg.lib.h2o_debug_wait_probe(c._h, 2000, None) == 0
    assert c.status() == pkg.H2O_ERR_TIMEOUT
    assert pkg.lib.h2o_debug_wait_probe(c._h, 0, None) == pkg.H2O_ERR_INVALID_ARG
    c.reset()
    assert c.status() == 0
    c.close()
    _identical(_full_run(pkg, wl), _full_run(pkg, wl))  # the device is as usable as before
