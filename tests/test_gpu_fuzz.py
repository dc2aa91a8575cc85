"""Seeded random shapes through every step kernel: the parity protocol of the other GPU tests on small ragged
batches whose lengths, budgets (zero heavy budgets and zero recent windows included), head counts, cluster splits,
step-kernel choice and query groups are drawn from a fixed seed.  A case that fails prints its parameters."""
import numpy as np
import pytest
import torch

from workloads import Workload

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def H2OCache(oracle):
    import paper_2306_14048_b200 as pkg

    assert torch.cuda.is_available(), "these tests need a CUDA device; there is no CPU fallback"
    return pkg.H2OCache


def _draw(rng, i):
    batch = int(rng.integers(1, 5))
    heads = int(rng.integers(1, 4))
    lens = [int(rng.choice([1, 2, 17, 31, 64, 100, 129, 300, 515, 700])) for _ in range(batch)]
    heavy, recent = [], []
    for n in lens:
        b = int(rng.integers(2, max(3, min(n, 260))))
        k = int(rng.integers(0, b + 1))
        k = int(rng.choice([0, k, k, b]))  # some sequences without heavy hitters, some without a recent window
        heavy.append(k)
        recent.append(b - k)
    group = int(rng.choice([1, 1, 1, 2, 4, 8]))
    split = int(rng.choice([0, 0, 1, 2, 4])) if group == 1 else 0
    path = int(rng.choice([0, 1, 2])) if group == 1 else 0
    steps = int(rng.integers(3, 40))
    prefill = bool(rng.integers(0, 4) > 0) or min(lens) > 1
    if not prefill:
        lens = [1] * batch
    wl = Workload("fuzz%d" % i, batch, heads, 128, "bf16", tuple(lens), steps, tuple(heavy), tuple(recent), 1, 9000 + i)
    return wl, dict(group=group, split=split, decode_path=path, prefill=prefill, score_mode=int(rng.integers(0, 2)))


@pytest.mark.parametrize("block", range(4))
def test_random_shapes_bf16_head_dim_128(H2OCache, block):
    from parity_harness import run_parity

    rng = np.random.default_rng(20230614 + block)
    for i in range(8):
        wl, kw = _draw(rng, 8 * block + i)
        try:
            st = run_parity(wl, H2OCache, export_every=int(rng.integers(1, 9)), **kw)
        except Exception:
            print("failing case:", wl, kw)
            raise
        assert st.decisions > 0


@pytest.mark.parametrize("block", range(3))
def test_random_shapes_other_dtypes_and_slot_formats(H2OCache, block):
    """fp32, head_dim 64 and 4-bit slots: the online-softmax kernel, the plain grouped kernel, the 4-bit kernel."""
    from parity_harness import run_parity

    rng = np.random.default_rng(777 + block)
    for i in range(6):
        wl, kw = _draw(rng, 100 + 6 * block + i)
        dtype, d = [("f32", 64), ("f32", 128), ("bf16", 64), ("bf16_kv4", 128)][int(rng.integers(0, 4))]
        kw["decode_path"] = 0
        if dtype == "bf16_kv4":
            kw["group"], kw["split"] = 1, 0
        wl = wl.scaled(dtype=dtype, head_dim=d)
        try:
            st = run_parity(wl, H2OCache, export_every=int(rng.integers(1, 9)), **kw)
        except Exception:
            print("failing case:", wl, kw)
            raise
        assert st.decisions > 0
