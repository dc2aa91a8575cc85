"""Parity at the full sizes of the benchmark configurations, on sampled units, for every decode step.

The CUDA path runs the whole configuration exactly as the benchmark launches it; the
oracle follows a sample of (sequence, head) units, which is exact because units never
interact.  Long prompts cost the oracle O(n^2 d) per unit, so the samples are small; the
decode steps cost it almost nothing, so every configuration runs its full step count
(accumulated-score drift, if there were any, would show on the long runs).  Every case
prints one JSON line of its statistics (units, decisions, near-ties, largest errors).

The stress cases multiply the softmax scale by 4 (peakier rows, many tiny probabilities,
more near-ties); the 4-bit case stores the slots group-quantised.
"""
import math

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


def _stress_scale(wl):
    return 4.0 / math.sqrt(wl.head_dim)


def _c5_units(wl, per_class=2):
    """Units of the shortest, the longest and middling prompts, and of the prompts closest to 4096 tokens."""
    lens = np.asarray(wl.prompt_lens)
    order = np.argsort(lens, kind="stable")
    seqs = list(order[:per_class]) + list(order[-per_class:]) + [order[len(order) // 3], order[2 * len(order) // 3]]
    seqs += list(np.argsort(np.abs(lens - 4096), kind="stable")[:per_class])
    picks = sorted({int(s) * wl.n_heads + (7 * i + 3) % wl.n_heads for i, s in enumerate(seqs)})
    return picks


def test_config2_opt6p7b_sampled_units(H2OCache):
    from parity_harness import record, run_parity

    wl = CONFIGS["c2_opt6p7b"]
    record(run_parity(wl, H2OCache, units=_sample(wl, 10, 2), export_every=64), "c2 full length")


def test_config2_opt6p7b_stress_scale(H2OCache):
    from parity_harness import record, run_parity

    wl = CONFIGS["c2_opt6p7b"]
    record(run_parity(wl, H2OCache, units=_sample(wl, 6, 12), export_every=64, scale=_stress_scale(wl)), "c2 scale x4")


def test_config2_opt6p7b_four_bit_slots(H2OCache):
    from parity_harness import record, run_parity

    wl = CONFIGS["c2_opt6p7b"].scaled(dtype="bf16_kv4")
    record(run_parity(wl, H2OCache, units=_sample(wl, 6, 22), export_every=64), "c2 4-bit slots")


def test_config3_opt30b_sampled_units(H2OCache):
    from parity_harness import record, run_parity

    wl = CONFIGS["c3_opt30b"]
    record(run_parity(wl, H2OCache, units=_sample(wl, 48, 3), export_every=16), "c3 full length")


def test_config3_opt30b_stress_scale(H2OCache):
    from parity_harness import record, run_parity

    wl = CONFIGS["c3_opt30b"]
    record(run_parity(wl, H2OCache, units=_sample(wl, 24, 13), export_every=16, scale=_stress_scale(wl)), "c3 scale x4")


def test_config4_long_context_all_steps(H2OCache):
    from parity_harness import record, run_parity

    wl = CONFIGS["c4_longctx"]
    record(run_parity(wl, H2OCache, units=_sample(wl, 2, 4), export_every=64), "c4 full length")


@pytest.mark.parametrize("layer", [0, 31])
def test_config5_ragged_all_steps(H2OCache, layer):
    from parity_harness import record, run_parity

    wl = CONFIGS["c5_ragged_32layer"]
    assert layer < wl.layers
    record(run_parity(wl, H2OCache, units=_c5_units(wl), export_every=32, layer=layer), "c5 layer %d full length" % layer)


def test_config5_ragged_stress_scale(H2OCache):
    from parity_harness import record, run_parity

    wl = CONFIGS["c5_ragged_32layer"]
    record(run_parity(wl, H2OCache, units=_c5_units(wl, per_class=1), export_every=32, layer=7, scale=_stress_scale(wl)),
           "c5 layer 7 scale x4")


def test_config5_ragged_online_softmax_kernel(H2OCache):
    """Config 5 takes the two-pass streaming step kernel by default (the cases above); the same steps on the
    online-softmax kernel."""
    from parity_harness import record, run_parity

    wl = CONFIGS["c5_ragged_32layer"]
    record(run_parity(wl, H2OCache, units=_c5_units(wl, per_class=1), export_every=32, layer=0, decode_path=1),
           "c5 layer 0, online-softmax kernel")


def test_config5_ragged_grouped_query(H2OCache):
    """Config 5's sequences with 8 K/V heads of 4 query heads each (1024 units): tensor-core prompt kernels over the
    group, the streaming grouped step kernel, every decode step."""
    from parity_harness import record, run_parity

    wl = CONFIGS["c5_ragged_32layer"].scaled(n_heads=8)
    lens = np.asarray(wl.prompt_lens)
    seqs = [int(np.argmin(lens)), int(np.argmax(lens)), int(np.argsort(lens)[len(lens) // 2])]
    units = [s * wl.n_heads + h for s, h in zip(seqs, (0, 5, 7))]
    record(run_parity(wl, H2OCache, units=units, export_every=32, layer=0, group=4), "c5 with 8 K/V heads x 4 query heads")

