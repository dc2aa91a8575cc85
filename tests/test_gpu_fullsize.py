"""Parity at the full sizes of the benchmark configurations, on sampled units.

The CUDA path runs the whole configuration exactly as the benchmark launches it; the
oracle follows a sample of (sequence, head) units, which is exact because units never
interact.  Long prompts cost the oracle O(n^2 d) per unit, so the samples are small.
"""
import numpy as np
import pytest
import torch

from workloads import CONFIGS

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def H2OCache(oracle):
    import paper_2306_14048_b200 as pkg

    assert torch.cuda.is_available(), "these tests need a CUDA device; there is no CPU fallback"
    return pkg.H2OCache


def _sample(wl, count, seed):
    rng = np.random.default_rng(seed)
    return sorted(int(u) for u in rng.choice(wl.units, size=min(count, wl.units), replace=False))


def test_config2_opt6p7b_sampled_units(H2OCache):
    from parity_harness import run_parity

    wl = CONFIGS["c2_opt6p7b"]
    st = run_parity(wl, H2OCache, units=_sample(wl, 10, 2), export_every=64)
    print(st)


def test_config3_opt30b_sampled_units(H2OCache):
    from parity_harness import run_parity

    wl = CONFIGS["c3_opt30b"]
    st = run_parity(wl, H2OCache, units=_sample(wl, 48, 3), export_every=16)
    print(st)


def test_config4_long_context_one_unit(H2OCache):
    from parity_harness import run_parity

    wl = CONFIGS["c4_longctx"]
    st = run_parity(wl, H2OCache, units=_sample(wl, 1, 4), steps=64, export_every=32)
    print(st)


def test_config5_ragged_layer0_sampled_units(H2OCache):
    from parity_harness import run_parity

    wl = CONFIGS["c5_ragged_32layer"]
    lens = np.repeat(np.asarray(wl.prompt_lens), wl.n_heads)
    order = np.argsort(lens)
    picks = sorted({int(order[0]), int(order[len(order) // 3]), int(order[2 * len(order) // 3]), int(order[-1])})
    st = run_parity(wl, H2OCache, units=picks, steps=32, export_every=16)
    print(st)
