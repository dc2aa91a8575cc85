"""CUDA path vs oracle, element by element, through the C ABI (needs a B200)."""
import dataclasses

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


def test_config1_tiny_fp32_full(H2OCache):
    from parity_harness import run_parity

    from parity_harness import record

    st = run_parity(CONFIGS["c1_tiny"], H2OCache, export_every=8)
    assert st.decisions == 4 + 4 * 64
    record(st, "c1 full")


@pytest.mark.parametrize("dtype,d", [("bf16", 128), ("bf16", 64), ("f32", 128), ("f32", 64)])
def test_small_ragged_all_dtypes(H2OCache, dtype, d):
    """Ragged batch spanning several tiles and ragged tails; one prompt shorter than its budget."""
    from parity_harness import run_parity

    wl = _wl("small", 4, 3, d, dtype, [300, 77, 513, 40], 48, [20, 9, 33, 30], [24, 5, 31, 30], seed=77 + d)
    st = run_parity(wl, H2OCache, export_every=8)
    print(st)


@pytest.mark.parametrize("heavy,recent", [([0, 0], [7, 16]), ([5, 12], [0, 0]), ([1, 0], [0, 1]), ([3, 2], [1, 2])])
def test_edge_budgets(H2OCache, heavy, recent):
    """k = 0 (sliding window), r = 0 (the new token may be the one dropped), single-slot caches."""
    from parity_harness import run_parity

    wl = _wl("edge", 2, 2, 64, "f32", [37, 21], 40, heavy, recent, seed=5)
    st = run_parity(wl, H2OCache, export_every=4)
    print(st)


@pytest.mark.parametrize("dtype,d", [("bf16", 128), ("f32", 64)])
def test_token_by_token_from_empty_cache(H2OCache, dtype, d):
    """No prefill: the fill phase of Algorithm 2, then steady-state eviction."""
    from parity_harness import run_parity

    wl = _wl("seq", 2, 2, d, dtype, [1, 1], 90, [10, 4], [6, 20], seed=9)
    st = run_parity(wl, H2OCache, prefill=False, export_every=5)
    print(st)


def test_peaky_softmax_stress(H2OCache):
    """Four times the default scale: many tiny probabilities, more near-equal scores."""
    from parity_harness import run_parity

    wl = _wl("peaky", 2, 4, 128, "bf16", [700, 450], 64, [40, 30], [40, 30], seed=21)
    st = run_parity(wl, H2OCache, scale=4.0 / np.sqrt(128.0), export_every=16)
    print(st)


@pytest.mark.parametrize("dtype,d,heavy,recent", [
    ("bf16", 128, [150, 30], [150, 40]),      # split over 4 thread blocks; the short sequence leaves blocks empty
    ("bf16", 128, [600, 500], [500, 600]),    # split over 8
    ("f32", 64, [100, 64], [100, 64]),
])
def test_units_split_over_a_cluster(H2OCache, dtype, d, heavy, recent):
    """Few units with long budgets: one unit is shared by several thread blocks of a cluster."""
    from parity_harness import run_parity

    wl = _wl("cluster", 2, 2, d, dtype, [1500, 1300], 40, heavy, recent, seed=31)
    st = run_parity(wl, H2OCache, export_every=8)
    print(st)


def test_cluster_split_fill_phase_from_empty(H2OCache):
    """Token-by-token fill of a cache that is split over a cluster: most blocks start empty."""
    from parity_harness import run_parity

    wl = _wl("clusterfill", 1, 2, 128, "bf16", [1], 330, [150], [150], seed=32)
    st = run_parity(wl, H2OCache, prefill=False, export_every=30)
    print(st)


def test_bf16_alu_prefill_path(H2OCache):
    """bf16 / head_dim 128 forced onto the fp32-FMA prefill kernels (the tensor-core path is the default)."""
    from parity_harness import run_parity

    wl = _wl("alu", 2, 2, 128, "bf16", [333, 129], 8, [20, 10], [20, 10], seed=41)
    st = run_parity(wl, H2OCache, export_every=4, prefill_path=1)
    print(st)


def test_tensor_core_prefill_tile_edges(H2OCache):
    """Prompt lengths around the 64/128 tile edges of the tensor-core kernels, ragged batch."""
    from parity_harness import run_parity

    lens = [1, 63, 64, 65, 127, 128, 129, 191, 192, 193, 255, 256, 257, 640]
    wl = _wl("edges", len(lens), 2, 128, "bf16", lens, 6, [5] * len(lens), [4] * len(lens), seed=43)
    st = run_parity(wl, H2OCache, export_every=3)
    print(st)


def test_tensor_core_prefill_long_and_short_kernels_mixed_lengths(H2OCache):
    """Both forward kernels of the tensor-core path: prompts up to 1024 tokens take the persistent
    one-query-block kernel (blocks walk over several (unit, query block) items, single-tile items included),
    longer ones the two-query-block kernel; the column-sum kernel runs persistent in the first case."""
    from parity_harness import run_parity

    short = [1024, 1, 130, 512, 64, 1000, 129, 700, 3, 256, 900, 65] * 3  # more items than resident blocks need
    wl = _wl("short", len(short), 8, 128, "bf16", short, 4, [6] * len(short), [5] * len(short), seed=45)
    st = run_parity(wl, H2OCache, units=[0, 9, 17, 100, 287], export_every=2)
    print(st)
    long_ = [1025, 300, 1500]
    wl = _wl("long", len(long_), 2, 128, "bf16", long_, 4, [6] * 3, [5] * 3, seed=46)
    st = run_parity(wl, H2OCache, export_every=2)
    print(st)
    # beyond 4096 tokens the two-query-block kernel runs the forward pass of the whole (ragged) batch
    longer = [4200, 130, 700]
    wl = _wl("longer", len(longer), 2, 128, "bf16", longer, 2, [6] * 3, [5] * 3, seed=48)
    st = run_parity(wl, H2OCache, units=[0, 3, 5], export_every=2)
    print(st)


def test_tensor_core_prefill_item_order_over_several_groups_of_units(H2OCache):
    """The persistent forward kernel orders its (unit, query block) items by groups of units whose K/V fit
    the L2 and gives a group as many levels as its longest sequence has query blocks: a very ragged batch
    whose groups end inside a sequence (5 heads, 24 units per group at this length)."""
    from parity_harness import run_parity

    lens = [4000, 1, 129, 64, 2500, 3, 700, 128, 33, 1024, 5, 3100]
    wl = _wl("groups", len(lens), 5, 128, "bf16", lens, 3, [6] * len(lens), [5] * len(lens), seed=47)
    st = run_parity(wl, H2OCache, units=[0, 4, 7, 21, 23, 24, 26, 39, 47, 48, 55, 59], export_every=2)
    print(st)


@pytest.mark.parametrize("lens,heads", [([512] * 12, 16), ([2048, 1100], 4), ([700, 33, 1024, 129, 5], 6), ([4300, 900], 4)])
def test_tensor_core_prefill_is_bit_reproducible(H2OCache, lens, heads):
    """Two issuing warps per query block add their products into the same accumulator; they are chained so
    that the order of those additions is fixed.  The same prompt twice: every bit of the outputs and of the
    column sums must agree (also with the output tensor at an address that is only 16-byte aligned, which
    takes the narrow stores)."""
    from workloads import make_prompt_inputs

    wl = _wl("repro", len(lens), heads, 128, "bf16", lens, 2, [4] * len(lens), [4] * len(lens), seed=47)
    q, k, v, cu = make_prompt_inputs(wl, layer=0, device="cuda")
    c = H2OCache(wl.batch, wl.n_heads, wl.head_dim, wl.dtype, wl.heavy, wl.recent)
    res = []
    backing = torch.empty(q.numel() + 8, dtype=q.dtype, device="cuda")
    for rep in range(6):
        out = torch.full_like(q, float("nan")) if rep < 5 else backing[8:].view_as(q)
        if rep == 5:
            assert out.data_ptr() % 32 == 16
        c.reset()
        c.prefill_select(q, k, v, cu, out)
        assert c.status() == 0
        res.append((out.clone().view(torch.int16), c.prefill_column_sums(wl.total_tokens).clone()))
    for o, a in res[1:]:
        assert torch.equal(o, res[0][0])
        assert torch.equal(a, res[0][1])
    c.close()


def test_rotating_caches_early_prefetch_equals_waiting_first(H2OCache):
    """Several caches stepped in rotation on one stream (the benchmark's pattern).  The kernels then
    prefetch their cache before the previous launch has finished; everything observable must be
    bit-identical to the run in which every launch waits first."""
    import paper_2306_14048_b200 as pkg
    from workloads import make_decode_inputs, make_prompt_inputs

    wl = _wl("rot", 6, 8, 128, "bf16", [700] * 6, 24, [60] * 6, [60] * 6, seed=51)
    n_caches = 3

    def run(early):
        prev = pkg.lib.h2o_debug_set_early_prefetch(1 if early else 0)
        try:
            caches = [H2OCache(wl.batch, wl.n_heads, wl.head_dim, wl.dtype, wl.heavy, wl.recent) for _ in range(n_caches)]
            for l, c in enumerate(caches):
                q, k, v, cu = make_prompt_inputs(wl, layer=l, device="cuda")
                c.prefill_select(q, k, v, cu, torch.empty_like(q))
            outs, evs = [], []
            ins = [[make_decode_inputs(wl, s, layer=l, device="cuda") for l in range(n_caches)] for s in range(wl.decode_steps)]
            torch.cuda.synchronize()
            for s in range(wl.decode_steps):
                for l, c in enumerate(caches):
                    q, k, v = ins[s][l]
                    o = torch.empty_like(q)
                    e = torch.empty(wl.batch, wl.n_heads, dtype=torch.int32, device="cuda")
                    c.decode_step(q, k, v, o, e)
                    outs.append(o)
                    evs.append(e)
            torch.cuda.synchronize()
            state = [c.export() for c in caches]
            assert all(c.status() == 0 for c in caches)
            for c in caches:
                c.close()
            return [o.float().cpu().numpy() for o in outs], [e.cpu().numpy() for e in evs], state
        finally:
            pkg.lib.h2o_debug_set_early_prefetch(prev)

    a, b = run(True), run(False)
    for x, y in zip(a[0], b[0]):
        assert np.array_equal(x, y)
    for x, y in zip(a[1], b[1]):
        assert np.array_equal(x, y)
    for sa, sb in zip(a[2], b[2]):
        for x, y in zip(sa, sb):
            assert np.array_equal(x, y)


def test_large_budget_per_unit(H2OCache):
    """A unit with thousands of slots: forced cluster split with large per-block chunks and deep score rows."""
    from parity_harness import run_parity

    wl = _wl("bigB", 1, 2, 128, "bf16", [9500], 12, [4600], [4400], seed=61)
    st = run_parity(wl, H2OCache, export_every=6)
    print(st)


@pytest.mark.parametrize("dtype,d", [("bf16", 128), ("f32", 64)])
def test_averaged_score_variant(H2OCache, dtype, d):
    """Ranking by accumulated score / number of attending queries ("Discussions and Limitations"): prefill
    selection, decode steps, a split unit, and h2o_decode_chunk (served by the step kernels in this mode)."""
    from parity_harness import run_parity

    wl = _wl("avg", 3, 3, d, dtype, [300, 77, 513], 48, [20, 9, 33], [24, 5, 31], seed=201)
    st = run_parity(wl, H2OCache, export_every=8, score_mode=1)
    assert st.decisions == 9 + 9 * 48
    print(st)
    st = run_parity(wl, H2OCache, export_every=16, score_mode=1, chunk=16)
    print(st)
    wl = _wl("avg0", 2, 2, d, dtype, [200, 150], 40, [12, 30], [0, 0], seed=202)  # no recent window
    st = run_parity(wl, H2OCache, export_every=8, score_mode=1)
    print(st)


def test_averaged_score_differs_from_accumulated_and_needs_an_empty_cache(H2OCache):
    """The two ranking rules keep different sets on the same inputs (old keys collect more), and the rule
    cannot change in the middle of a generation."""
    import paper_2306_14048_b200 as pkg
    from workloads import make_decode_inputs, make_prompt_inputs

    wl = _wl("avgdiff", 2, 4, 128, "bf16", [400, 380], 8, [16, 16], [8, 8], seed=203)
    q, k, v, cu = make_prompt_inputs(wl, layer=0, device="cuda")
    kept = []
    for mode in (0, 1):
        c = H2OCache(wl.batch, wl.n_heads, wl.head_dim, wl.dtype, wl.heavy, wl.recent)
        c.set_score_mode(mode)
        c.prefill_select(q, k, v, cu, torch.empty_like(q))
        with pytest.raises(pkg.H2OError):
            c.set_score_mode(1 - mode)
        pos, acc, count, t = c.export()
        kept.append([np.sort(pos[u, :count[u]]) for u in range(wl.units)])
        c.close()
    assert any(not np.array_equal(a, b) for a, b in zip(*kept))
    assert np.mean([a.mean() for a in kept[1]]) > np.mean([a.mean() for a in kept[0]])  # younger keys on average


def test_fscore_report(H2OCache):
    """Sum of h(accumulated score) per unit against the oracle's, for the three h of the paper's remark."""
    from oracle import h2o_oracle
    from workloads import make_decode_inputs, make_prompt_inputs

    wl = _wl("fs", 2, 3, 128, "bf16", [260, 90], 5, [10, 200], [6, 100], seed=204)  # the second sequence is not full
    q, k, v, cu = make_prompt_inputs(wl, layer=0, device="cuda")
    c = H2OCache(wl.batch, wl.n_heads, wl.head_dim, wl.dtype, wl.heavy, wl.recent)
    c.prefill_select(q, k, v, cu, torch.empty_like(q))
    for s_ in range(5):
        qs, ks, vs = make_decode_inputs(wl, s_, layer=0, device="cuda")
        c.decode_step(qs, ks, vs, torch.empty_like(qs), None)
    pos, acc, count, t = c.export()
    for hk in (0, 1, 2):
        f = c.fscore(hk).cpu().numpy().reshape(-1)
        for u in range(wl.units):
            assert f[u] == pytest.approx(h2o_oracle.fscore(acc[u, :count[u]], hk), rel=1e-12)
    c.close()


def test_kv4_slots_ragged(H2OCache):
    """4-bit group-quantised K/V slots (bf16 inputs): prefill selection quantises the kept rows, every decode
    step attends the new token at full precision and stores it quantised; against the oracle's quantiser."""
    from parity_harness import run_parity

    wl = _wl("kv4", 3, 3, 128, "bf16_kv4", [300, 77, 513], 80, [20, 9, 33], [24, 5, 31], seed=301)
    st = run_parity(wl, H2OCache, export_every=8)
    assert st.decisions == 9 + 9 * 80
    print(st)


@pytest.mark.parametrize("heavy,recent", [([0, 0], [7, 16]), ([5, 12], [0, 0]), ([1, 0], [0, 1])])
def test_kv4_edge_budgets_and_fill_phase(H2OCache, heavy, recent):
    from parity_harness import run_parity

    wl = _wl("kv4edge", 2, 2, 128, "bf16_kv4", [37, 21], 40, heavy, recent, seed=302)
    st = run_parity(wl, H2OCache, export_every=4)
    print(st)
    wl = _wl("kv4fill", 2, 2, 128, "bf16_kv4", [1, 1], 90, [10, 40], [6, 50], seed=303)
    st = run_parity(wl, H2OCache, prefill=False, export_every=8)  # Algorithm 1 from an empty cache, tiles fill up
    print(st)


def test_kv4_large_budget_chunk_call_and_averaged_score(H2OCache):
    """Several tiles per unit (budget 700), h2o_decode_chunk (step kernels in this format), averaged ranking."""
    from parity_harness import run_parity

    wl = _wl("kv4big", 2, 2, 128, "bf16_kv4", [1500, 900], 40, [350, 100], [350, 100], seed=304)
    st = run_parity(wl, H2OCache, export_every=8, chunk=8)
    print(st)
    wl = _wl("kv4avg", 2, 2, 128, "bf16_kv4", [300, 200], 40, [20, 12], [10, 0], seed=305)
    st = run_parity(wl, H2OCache, export_every=8, score_mode=1)
    print(st)


@pytest.mark.parametrize("plen,budget", [(60, 6), (330, 150)])
def test_kv4_many_units_four_warp_blocks(H2OCache, plen, budget):
    """More than 8 x 148 units: the decode step runs its four-warp instances (small and large block share)."""
    from parity_harness import run_parity

    batch, heads = 38, 32
    lens = [plen + (7 * i) % 23 for i in range(batch)]
    wl = _wl("kv4many", batch, heads, 128, "bf16_kv4", lens, 6, [budget] * batch, [budget] * batch, seed=305)
    st = run_parity(wl, H2OCache, units=[0, 31, 32, 500, 777, 1215], export_every=3)
    print(st)


def test_kv4_rejects_what_it_does_not_support(H2OCache):
    import paper_2306_14048_b200 as pkg

    with pytest.raises(pkg.H2OError):
        H2OCache(1, 1, 64, "bf16_kv4", [4], [4])  # head_dim 128 only
    with pytest.raises(pkg.H2OError):
        H2OCache(1, 1, 128, "bf16_kv4", [8000], [8000])  # more slots than one thread block stages


# ---------------------------------------------------------------------------------------------------------
# heavy hitters combined with a sparse pattern inside the recent window (h2o_cache_set_mask)
# ---------------------------------------------------------------------------------------------------------
MASKS = [(1, 8, 3), (1, 5, 1), (2, 16, 2), (2, 7, 3)]  # strided(stride, local window), fixed(block, summary columns)


@pytest.mark.parametrize("mask", MASKS)
@pytest.mark.parametrize("dtype,d", [("bf16", 128), ("f32", 64)])
def test_sparse_pattern_ragged(H2OCache, mask, dtype, d):
    """Prompt rows and decode steps under a pattern: ragged batch, several tiles, one prompt shorter than its budget."""
    from parity_harness import run_parity

    wl = _wl("mask", 4, 3, d, dtype, [300, 77, 513, 40], 48, [20, 9, 33, 30], [24, 5, 31, 30], seed=177 + d)
    st = run_parity(wl, H2OCache, export_every=8, mask=mask)
    print(st)


@pytest.mark.parametrize("heavy,recent", [([0, 0], [7, 16]), ([3, 2], [1, 2]), ([6, 1], [12, 9])])
def test_sparse_pattern_edge_budgets_token_by_token(H2OCache, heavy, recent):
    """No heavy hitters (the pattern alone), tiny windows, and the fill phase from an empty cache."""
    from parity_harness import run_parity

    wl = _wl("maskedge", 2, 2, 64, "f32", [1, 1], 60, heavy, recent, seed=15)
    for mask in ((1, 4, 2), (2, 5, 1)):
        st = run_parity(wl, H2OCache, prefill=False, export_every=5, mask=mask)
        print(st)


def test_sparse_pattern_units_split_over_a_cluster_and_chunk_call(H2OCache):
    """Long budgets (a unit shared by the blocks of a cluster) and the multi-token call, which takes one
    decode-step kernel per token when a pattern is set."""
    from parity_harness import run_parity

    wl = _wl("maskcluster", 2, 2, 128, "bf16", [1500, 1300], 40, [150, 30], [150, 40], seed=131)
    st = run_parity(wl, H2OCache, export_every=8, mask=(1, 16, 4))
    print(st)
    wl = _wl("maskchunk", 2, 3, 128, "bf16", [400, 300], 40, [20, 30], [24, 16], seed=132)
    st = run_parity(wl, H2OCache, export_every=8, mask=(2, 12, 2), chunk=16)
    print(st)


def test_sparse_pattern_argument_and_state_errors(H2OCache):
    import paper_2306_14048_b200 as pkg

    cache = H2OCache(1, 2, 64, "f32", [4], [4])
    for bad in ((3, 1, 0), (-1, 1, 0), (1, 0, 1), (1, 4, -1), (2, 4, 5)):
        assert pkg.lib.h2o_cache_set_mask(cache._h, *bad) == pkg.H2O_ERR_INVALID_ARG
    assert pkg.lib.h2o_cache_set_mask(None, 0, 1, 0) == pkg.H2O_ERR_INVALID_ARG
    cache.set_mask(1, 4, 2)
    x = torch.zeros(1, 2, 64, device="cuda")
    cache.decode_step(x, x, x, torch.empty_like(x))
    assert pkg.lib.h2o_cache_set_mask(cache._h, 0, 1, 0) == pkg.H2O_ERR_STATE  # one rule per generation
    cache.reset()
    cache.set_mask(0)
    cache.close()
    kv4 = H2OCache(1, 2, 128, "bf16_kv4", [4], [4])
    assert pkg.lib.h2o_cache_set_mask(kv4._h, 1, 4, 2) == pkg.H2O_ERR_UNSUPPORTED
    kv4.close()


# ---------------------------------------------------------------------------------------------------------
# heavy hitters combined with "Top-K" attention in decode steps (h2o_cache_set_topk)
# ---------------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("m", [1, 7, 40, 500])
@pytest.mark.parametrize("dtype,d", [("bf16", 128), ("f32", 64)])
def test_topk_attention_ragged(H2OCache, m, dtype, d):
    """m below, around and above the cache size (above: everything is attended, through the same code path)."""
    from parity_harness import run_parity

    wl = _wl("topk", 4, 3, d, dtype, [300, 77, 513, 40], 48, [20, 9, 33, 30], [24, 5, 31, 30], seed=277 + d)
    st = run_parity(wl, H2OCache, export_every=8, topk=m)  # bf16 / 128: the two-pass kernel's form (the library's choice)
    print(st)
    if dtype == "bf16":  # the same on the online-softmax kernel's "Top-K" instance
        print(run_parity(wl, H2OCache, export_every=8, topk=m, decode_path=1))


@pytest.mark.parametrize("heavy,recent", [([0, 0], [7, 16]), ([5, 12], [0, 0]), ([6, 1], [12, 9])])
def test_topk_attention_edge_budgets_token_by_token(H2OCache, heavy, recent):
    """Fill phase from an empty cache, no heavy hitters, no recent window (the new token may be the one dropped, and with
    Top-K attention it may not even attend itself)."""
    from parity_harness import run_parity

    wl = _wl("topkedge", 2, 2, 64, "f32", [1, 1], 60, heavy, recent, seed=25)
    for m in (1, 3):
        st = run_parity(wl, H2OCache, prefill=False, export_every=5, topk=m)
        print(st)
    wl = _wl("topkedge2", 2, 2, 128, "bf16", [1, 1], 60, heavy, recent, seed=26)  # the two-pass kernel's form
    for m in (1, 3):
        print(run_parity(wl, H2OCache, prefill=False, export_every=5, topk=m))


def test_topk_attention_long_budget_pattern_and_chunk_call(H2OCache):
    """A budget that would be split over a cluster stays in one block; Top-K on top of a sparse pattern; the
    multi-token call falls back to one decode-step kernel per token."""
    from parity_harness import run_parity

    wl = _wl("topklong", 2, 2, 128, "bf16", [1500, 1300], 24, [600, 500], [500, 600], seed=231)
    print(run_parity(wl, H2OCache, export_every=8, topk=64))
    wl = _wl("topkmask", 2, 3, 128, "bf16", [400, 300], 40, [20, 30], [24, 16], seed=232)
    print(run_parity(wl, H2OCache, export_every=8, topk=9, mask=(1, 8, 3)))
    print(run_parity(wl, H2OCache, export_every=8, topk=9, chunk=16))


def test_topk_argument_and_state_errors(H2OCache):
    import paper_2306_14048_b200 as pkg

    cache = H2OCache(1, 2, 64, "f32", [4], [4])
    assert pkg.lib.h2o_cache_set_topk(cache._h, -1) == pkg.H2O_ERR_INVALID_ARG
    cache.set_topk(3)
    assert pkg.lib.h2o_cache_set_decode_shape(cache._h, 2, 0) == pkg.H2O_ERR_UNSUPPORTED
    x = torch.zeros(1, 2, 64, device="cuda")
    cache.decode_step(x, x, x, torch.empty_like(x))
    assert pkg.lib.h2o_cache_set_topk(cache._h, 0) == pkg.H2O_ERR_STATE
    cache.close()
    kv4 = H2OCache(1, 2, 128, "bf16_kv4", [4], [4])
    assert pkg.lib.h2o_cache_set_topk(kv4._h, 2) == pkg.H2O_ERR_UNSUPPORTED
    kv4.close()
    big = H2OCache(1, 1, 64, "f32", [6000], [6000])
    assert pkg.lib.h2o_cache_set_topk(big._h, 2) == pkg.H2O_ERR_UNSUPPORTED
    big.close()


# ---------------------------------------------------------------------------------------------------------
# grouped-query attention: G query heads share a unit's keys and values, accumulated scores add up over the group
# ---------------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("group,dtype,d", [
    (2, "bf16", 128), (4, "bf16", 128), (8, "bf16", 128), (2, "f32", 64), (4, "f32", 64), (8, "f32", 64),
    (2, "bf16", 64), (4, "bf16", 64), (2, "f32", 128), (4, "f32", 128),
])
def test_grouped_query_attention_ragged(H2OCache, group, dtype, d):
    """Prompt, selection on the summed column sums, decode steps with one victim per unit."""
    from parity_harness import run_parity

    wl = _wl("gqa", 3, 2, d, dtype, [300, 77, 140], 40, [20, 9, 33], [24, 5, 31], seed=377 + d + group)
    st = run_parity(wl, H2OCache, export_every=8, group=group)
    print(st)


def test_grouped_query_attention_tensor_core_prompt_kernels(H2OCache):
    """bf16 / head_dim 128 prompts of a grouped cache run on the tensor-core kernels: the persistent forward kernel
    (prompts up to 4096 tokens), the two-query-block one (longer), and column sums that add up over the group's
    query heads; the fp32-FMA kernels on the same inputs give the same selection."""
    from parity_harness import run_parity

    wl = _wl("gqatc", 3, 2, 128, "bf16", [700, 129, 1025], 8, [40, 20, 60], [40, 12, 70], seed=911)
    for group in (2, 4, 8):
        print(run_parity(wl, H2OCache, export_every=4, group=group))
    print(run_parity(wl, H2OCache, export_every=4, group=4, prefill_path=1))
    wl = _wl("gqatclong", 1, 2, 128, "bf16", [4500], 4, [100], [120], seed=912)
    print(run_parity(wl, H2OCache, export_every=2, group=2))


@pytest.mark.parametrize("heavy,recent", [([0, 0], [7, 16]), ([5, 12], [0, 0]), ([6, 1], [12, 9])])
def test_grouped_query_attention_edge_budgets_token_by_token(H2OCache, heavy, recent):
    from parity_harness import run_parity

    wl = _wl("gqaedge", 2, 2, 64, "f32", [1, 1], 60, heavy, recent, seed=35)
    st = run_parity(wl, H2OCache, prefill=False, export_every=5, group=4)
    print(st)


def test_grouped_query_attention_long_budget_chunk_call_and_averaged_score(H2OCache):
    from parity_harness import run_parity

    wl = _wl("gqalong", 2, 2, 128, "bf16", [1500, 1300], 16, [600, 500], [500, 600], seed=331)
    print(run_parity(wl, H2OCache, export_every=8, group=2))
    wl = _wl("gqachunk", 2, 3, 128, "bf16", [400, 300], 40, [20, 30], [24, 16], seed=332)
    print(run_parity(wl, H2OCache, export_every=8, group=4, chunk=16))
    print(run_parity(wl, H2OCache, export_every=8, group=2, score_mode=1))


def test_grouped_query_attention_with_a_sparse_pattern(H2OCache):
    """Grouped bf16 / head_dim 128 caches combine with the strided / fixed patterns (fp32-FMA prompt kernels with the
    pattern over the group, streaming grouped step kernel); other grouped caches refuse a pattern."""
    import paper_2306_14048_b200 as pkg
    from parity_harness import run_parity

    wl = _wl("gqamask", 3, 2, 128, "bf16", [400, 300, 90], 30, [20, 30, 10], [40, 64, 30], seed=461)
    for group, mask in ((2, (1, 8, 3)), (4, (2, 16, 2)), (8, (1, 3, 1))):
        print(run_parity(wl, H2OCache, export_every=5, mask=mask, group=group))
    cache = H2OCache(1, 2, 64, "f32", [8], [8], query_group=2)
    assert pkg.lib.h2o_cache_set_mask(cache._h, 1, 4, 2) == pkg.H2O_ERR_UNSUPPORTED
    cache.close()


def test_grouped_query_attention_argument_errors(H2OCache):
    import ctypes

    import paper_2306_14048_b200 as pkg

    for bad in (3, 16, -1):
        cfg, keep = pkg.make_config(1, 2, 64, "f32", [4], [4], query_group=bad)
        assert pkg.h2o_cache_workspace_bytes(cfg) == 0
    cfg, keep = pkg.make_config(1, 2, 128, "bf16_kv4", [4], [4], query_group=2)
    assert pkg.h2o_cache_workspace_bytes(cfg) == 0
    cfg, keep = pkg.make_config(1, 1, 64, "f32", [4000], [4000], query_group=8)  # the group's scores would not fit
    assert pkg.h2o_cache_workspace_bytes(cfg) == 0
    cache = H2OCache(1, 2, 64, "f32", [4], [4], query_group=2)
    assert pkg.lib.h2o_cache_set_mask(cache._h, 1, 4, 2) == pkg.H2O_ERR_UNSUPPORTED
    assert pkg.lib.h2o_cache_set_topk(cache._h, 2) == pkg.H2O_ERR_UNSUPPORTED
    cache.close()

# ---------------------------------------------------------------------------------------------------------
# the two-pass streaming step kernel (h2o_cache_set_decode_path 2; automatic for many mid-sized units)
# ---------------------------------------------------------------------------------------------------------
def test_two_pass_step_kernel_ragged_fill_phase_and_edges(H2OCache):
    """Ragged batch over several tiles with a prompt shorter than its budget (fill phase), token-by-token from an
    empty cache, no recent window, no heavy budget, the averaged ranking, and the chunk call's per-token fallback."""
    from parity_harness import run_parity

    wl = _wl("tp", 4, 3, 128, "bf16", [300, 77, 513, 40], 48, [20, 9, 33, 30], [24, 5, 31, 30], seed=205)
    for path in (1, 2):
        print(run_parity(wl, H2OCache, export_every=8, decode_path=path))
    print(run_parity(wl, H2OCache, export_every=8, decode_path=2, score_mode=1))
    print(run_parity(wl, H2OCache, export_every=8, decode_path=2, chunk=16, chunk_path=1))
    for heavy, recent in (([0, 0], [7, 16]), ([5, 12], [0, 0]), ([6, 1], [12, 9])):
        wl = _wl("tpedge", 2, 2, 128, "bf16", [1, 1], 60, heavy, recent, seed=36)
        print(run_parity(wl, H2OCache, prefill=False, export_every=5, decode_path=2))
    wl = _wl("tplong", 1, 2, 128, "bf16", [3000], 12, [1200], [1100], seed=207)  # 72 tiles per matrix
    print(run_parity(wl, H2OCache, export_every=4, decode_path=2))


@pytest.mark.parametrize("budget,split", [(300, 2), (520, 2), (1040, 4), (2300, 8), (2048, 8)])
def test_two_pass_step_kernel_unit_split_over_a_cluster(H2OCache, budget, split):
    """The two-pass kernel with a unit split over a cluster: statistics exchanged between the passes, outputs and
    candidates after the value pass.  Shares of more than 256 slots wrap the block's ring while the consumers stand
    in the barrier between the passes (the producer warp must not wait there)."""
    from parity_harness import run_parity

    wl = _wl("tpsplit", 1, 2, 128, "bf16", [3000], 6, [budget // 2], [budget - budget // 2], seed=207)
    print(run_parity(wl, H2OCache, export_every=2, split=split, decode_path=2))
    wl = _wl("tpsplitfill", 1, 2, 128, "bf16", [1], 70, [20], [30], seed=208)
    print(run_parity(wl, H2OCache, prefill=False, export_every=8, split=min(split, 2), decode_path=2))


@pytest.mark.parametrize("budget,split", [(300, 2), (1040, 4), (2300, 8)])
def test_four_bit_slots_unit_split_over_a_cluster(H2OCache, budget, split):
    """4-bit slots with a unit split over a cluster (the library's choice for few long units): statistics and partial
    outputs exchanged after the stream, candidates after the final probabilities; also from an empty cache."""
    from parity_harness import run_parity

    wl = _wl("k4split", 1, 2, 128, "bf16_kv4", [3000], 6, [budget // 2], [budget - budget // 2], seed=217)
    print(run_parity(wl, H2OCache, export_every=2, split=split))
    wl = _wl("k4splitfill", 1, 2, 128, "bf16_kv4", [1], 70, [20], [30], seed=218)
    print(run_parity(wl, H2OCache, prefill=False, export_every=8, split=min(split, 4)))


def test_two_pass_step_kernel_where_it_does_not_apply(H2OCache):
    import paper_2306_14048_b200 as pkg

    for args in ((1, 2, 64, "bf16"), (1, 2, 128, "f32"), (1, 2, 128, "bf16_kv4")):
        cache = H2OCache(args[0], args[1], args[2], args[3], [8], [8])
        assert pkg.lib.h2o_cache_set_decode_path(cache._h, 2) == pkg.H2O_ERR_UNSUPPORTED
        assert pkg.lib.h2o_cache_set_decode_path(cache._h, 3) == pkg.H2O_ERR_INVALID_ARG
        assert pkg.lib.h2o_cache_set_decode_path(cache._h, 1) == pkg.H2O_OK
        cache.close()
    cache = H2OCache(1, 2, 128, "bf16", [8], [8])
    cache.set_topk(4)  # ("Top-K" attention has a form on either kernel)
    cache.set_decode_path(2)
    assert cache.decode_path() == 2
    cache.set_decode_path(1)
    assert cache.decode_path() == 1
    cache.close()


@pytest.mark.parametrize("mask", [(1, 8, 3), (2, 16, 2), (1, 3, 1)])
def test_two_pass_step_kernel_with_a_sparse_pattern(H2OCache, mask):
    """Heavy hitters combined with the strided / fixed patterns inside the recent window, on the two-pass kernel
    (also with a unit split over a cluster)."""
    from parity_harness import run_parity

    wl = _wl("tpmask", 3, 2, 128, "bf16", [400, 300, 90], 30, [20, 30, 10], [40, 64, 30], seed=451)
    print(run_parity(wl, H2OCache, export_every=5, mask=mask, decode_path=2))
    wl = _wl("tpmasksplit", 1, 2, 128, "bf16", [1500], 10, [300], [330], seed=452)
    print(run_parity(wl, H2OCache, export_every=5, mask=mask, decode_path=2, split=4))
