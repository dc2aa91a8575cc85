"""h2o_decode_chunk (several decode steps per call) vs the oracle's single steps, through the C ABI."""
import numpy as np
import pytest
import torch

from workloads import CONFIGS, Workload

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def H2OCache():
    import paper_2306_14048_b200 as pkg

    assert torch.cuda.is_available(), "these tests need a CUDA device; there is no CPU fallback"
    return pkg.H2OCache


@pytest.fixture(scope="module", autouse=True)
def _oracle_built(oracle):
    return oracle


def _wl(name, batch, heads, d, dtype, lens, steps, heavy, recent, seed=1234):
    return Workload(name, batch, heads, d, dtype, tuple(lens), steps, tuple(heavy), tuple(recent), 1, seed)


@pytest.mark.parametrize("chunk", [32, 7, 50])
def test_chunk_after_prefill_ragged(H2OCache, chunk):
    """Chunk kernel after a prefill: whole chunks, a chunk shorter than the kernel's 32 tokens, and a
    call that spans two launches with a ragged second one."""
    from parity_harness import run_parity

    wl = _wl("chunk", 3, 3, 128, "bf16", [300, 77, 513], 100, [20, 9, 33], [24, 5, 31], seed=101)
    st = run_parity(wl, H2OCache, chunk=chunk, export_every=chunk)
    assert st.decisions == 9 + 9 * 100
    print(st)


def test_chunk_from_empty_cache_is_algorithm_1(H2OCache):
    """No prefill: Algorithm 1 token by token over the whole text — fill phase, then steady-state
    eviction, including chunks in which the cache becomes full half-way."""
    from parity_harness import run_parity

    wl = _wl("chunkseq", 2, 2, 128, "bf16", [1, 1], 150, [10, 40], [6, 50], seed=102)
    st = run_parity(wl, H2OCache, prefill=False, chunk=32, export_every=32)
    print(st)


@pytest.mark.parametrize("heavy,recent", [([0, 0], [7, 16]), ([5, 12], [0, 0]), ([1, 0], [0, 1]), ([3, 2], [1, 2])])
def test_chunk_edge_budgets(H2OCache, heavy, recent):
    """k = 0, r = 0 (the new token may be the one dropped, also several times within one chunk), one-slot caches."""
    from parity_harness import run_parity

    wl = _wl("chunkedge", 2, 2, 128, "bf16", [37, 21], 70, heavy, recent, seed=103)
    st = run_parity(wl, H2OCache, chunk=32, export_every=32)
    print(st)


def test_chunk_four_tiles_and_peaky_softmax(H2OCache):
    """Budget 480 (four keys per thread, all four key tiles in use); four times the default scale."""
    from parity_harness import run_parity

    wl = _wl("chunkmax", 2, 2, 128, "bf16", [700, 600], 64, [240, 200], [240, 200], seed=104)
    st = run_parity(wl, H2OCache, chunk=32, export_every=32, scale=4.0 / np.sqrt(128.0))
    print(st)


def test_chunk_largest_supported_budget(H2OCache):
    """Budget 992 (= 1024 keys - 32 tokens): eight keys per thread, four batches of tiles; the short
    sequence of the batch uses a single tile of the same kernel."""
    from parity_harness import run_parity

    wl = _wl("chunk8", 2, 2, 128, "bf16", [1500, 90], 64, [496, 20], [496, 30], seed=107)
    st = run_parity(wl, H2OCache, chunk=32, export_every=32)
    print(st)


def test_chunk_one_tile_budgets(H2OCache):
    """Small budgets (two keys per thread, one tile resident at a time), several blocks per SM."""
    from parity_harness import run_parity

    wl = _wl("chunk2", 6, 8, 128, "bf16", [200, 90, 150, 300, 64, 222], 64, [20, 10, 50, 100, 6, 60], [20, 20, 46, 100, 6, 64], seed=108)
    st = run_parity(wl, H2OCache, chunk=32, export_every=32)
    print(st)


def test_chunk_and_single_step_calls_interleaved(H2OCache):
    """The two kernels hand the cache to one another: chunk calls of several sizes mixed with single steps."""
    from parity_harness import run_parity

    wl = _wl("chunkmix", 3, 4, 128, "bf16", [200, 64, 333], 120, [30, 8, 60], [30, 8, 40], seed=109)
    st = run_parity(wl, H2OCache, pattern=[32, 0, 0, 5, 1, 0, 40, 3], export_every=1)
    assert st.decisions == 12 + 12 * 120
    print(st)


@pytest.mark.parametrize("dtype,d,heavy,recent", [
    ("f32", 64, [20, 9], [24, 5]),          # no tensor-core path for this dtype
    ("bf16", 128, [600, 100], [600, 100]),  # budget too large for the chunk kernel
])
def test_chunk_served_by_single_step_kernels(H2OCache, dtype, d, heavy, recent):
    """Configurations outside the chunk kernel's range take one decode-step kernel per token, same results."""
    from parity_harness import run_parity

    wl = _wl("chunkfb", 2, 2, d, dtype, [1500, 400], 40, heavy, recent, seed=105)
    st = run_parity(wl, H2OCache, chunk=20, export_every=20)
    print(st)


def test_chunk_kernel_and_single_steps_leave_the_same_cache(H2OCache):
    """The same 96 tokens through h2o_decode_chunk and through h2o_decode_step: same evictions, same kept
    positions; scores and outputs agree to rounding."""
    from workloads import make_decode_inputs, make_prompt_inputs

    wl = _wl("chunkeq", 4, 4, 128, "bf16", [256, 300, 200, 411], 96, [26, 30, 20, 42], [26, 30, 20, 42], seed=106)
    q, k, v, cu = make_prompt_inputs(wl, layer=0, device="cuda")
    steps = [make_decode_inputs(wl, s, layer=0, device="cuda") for s in range(96)]
    qs, ks, vs = (torch.stack(x).contiguous() for x in zip(*steps))
    res = []
    for mode in ("chunk", "steps"):
        c = H2OCache(wl.batch, wl.n_heads, wl.head_dim, wl.dtype, wl.heavy, wl.recent)
        c.prefill_select(q, k, v, cu, torch.empty_like(q))
        out = torch.empty_like(qs)
        ev = torch.full((96, wl.batch, wl.n_heads), -7, dtype=torch.int32, device="cuda")
        if mode == "chunk":
            c.decode_chunk(qs, ks, vs, out, ev)
        else:
            for s in range(96):
                c.decode_step(qs[s], ks[s], vs[s], out[s], ev[s])
        assert c.status() == 0
        res.append((out.float().cpu().numpy(), ev.cpu().numpy(), c.export()))
        c.close()
    (o1, e1, (p1, a1, c1, t1)), (o2, e2, (p2, a2, c2, t2)) = res
    assert np.array_equal(e1, e2)
    assert np.array_equal(c1, c2) and np.array_equal(t1, t2)
    for u in range(wl.units):
        m = int(c1[u])
        i1, i2 = np.argsort(p1[u, :m]), np.argsort(p2[u, :m])
        assert np.array_equal(p1[u, :m][i1], p2[u, :m][i2])
        np.testing.assert_allclose(a1[u, :m][i1], a2[u, :m][i2], rtol=1e-5, atol=1e-6)
    np.testing.assert_allclose(o1, o2, rtol=1e-2, atol=2e-3)


@pytest.mark.parametrize("name,units", [("c2_opt6p7b", [0, 77, 255]), ("c3_opt30b", [5, 2000, 3583]),
                                        ("c5_ragged_32layer", [3, 1234, 4095])])
def test_chunk_full_size_sampled(H2OCache, name, units):
    """Configs 2, 3 and 5 (one layer) at full size: 64 tokens in two chunk launches, sampled units against the oracle."""
    from parity_harness import run_parity

    wl = CONFIGS[name]
    st = run_parity(wl, H2OCache, units=units, steps=64, chunk=64, export_every=64)
    print(st)


def test_chunk_dead_key_towers_over_the_live_ones(H2OCache):
    """A key that is evicted early in a chunk and would dominate the later rows by ~100 nats: the
    kernel's per-row reference maximum includes it, so the live exponentials underflow and the row has
    to fall back to the live maximum.  Outputs and evictions must still match the oracle's single steps."""
    from oracle import h2o_oracle
    from parity_harness import assert_close

    d, nt, heads = 128, 32, 2
    g = torch.Generator().manual_seed(4321)
    a = torch.zeros(d); a[0] = 1.0
    b = torch.zeros(d); b[1] = 1.0
    q = 0.3 * torch.randn(nt, 1, heads, d, generator=g)
    k = 0.3 * torch.randn(nt, 1, heads, d, generator=g)
    v = torch.randn(nt, 1, heads, d, generator=g)
    q[:16] += 3.0 * a
    q[16:] += 3.0 * b
    k[1] = 384.0 * (b - a)  # score about -100 under the first queries (never attended, evicted), +100 under the later ones
    q, k, v = (x.to(torch.bfloat16).cuda().contiguous() for x in (q, k, v))
    scale = float(np.float32(1.0 / np.sqrt(d)))
    heavy, recent = [2], [2]
    gpu = H2OCache(1, heads, d, "bf16", heavy, recent, softmax_scale=scale)
    out = torch.empty_like(q)
    ev = torch.full((nt, 1, heads), -7, dtype=torch.int32, device="cuda")
    gpu.decode_chunk(q, k, v, out, ev)
    assert gpu.status() == 0
    ora = h2o_oracle.OracleCache(1, heads, d, heavy, recent, scale=scale)
    g_out, g_ev = out.float().cpu().numpy(), ev.cpu().numpy()
    assert np.isfinite(g_out).all()
    for i in range(nt):
        res = ora.decode_step(q[i].float().cpu().numpy(), k[i].float().cpu().numpy(), v[i].float().cpu().numpy(),
                              hint=g_ev[i].reshape(-1), tie_rel=1e-6)
        assert (res["status"] != 2).all(), "token %d: evicted %s, oracle %s" % (i, g_ev[i].reshape(-1), res["evicted"])
        assert_close(g_out[i].reshape(heads, d), res["out"], "bf16", "token %d" % i)
    assert (g_ev[3].reshape(-1) == 1).all() or (g_ev[:16] == 1).any(), "the planted key was meant to be evicted early"
    pos, acc, count, t = gpu.export()
    for u in range(heads):
        opos, oacc = ora.export(u)
        order = np.argsort(pos[u, :count[u]])
        assert np.array_equal(pos[u, :count[u]][order], opos)
        assert_close(acc[u, :count[u]][order], oacc, "bf16", "acc unit %d" % u)
    gpu.close()
