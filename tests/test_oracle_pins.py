"""Pins for the fp64 CPU oracle: closed forms, brute force and textbook special cases.

None of these tests re-types the oracle's own loops.  Each compares it with
something fixed by the paper or by mathematics:

* uniform attention (q = 0) has a closed form in harmonic numbers, evaluated
  here in exact rational arithmetic;
* a pure-Python simulator materialises the whole (masked) probability matrix,
  takes accumulated scores as explicit column sums and picks the victim by the
  literal ``argmax_v F_score(G \\ {v})`` of the policy's definition, for three
  choices of ``h``;
* a budget at least as large as the sequence reduces to ordinary causal softmax
  attention, a zero heavy budget to sliding-window attention (library softmax);
* structural invariants of the eviction policy (budget, one eviction per step,
  no resurrection, recent window always present).
"""
import math
from fractions import Fraction

import numpy as np
import pytest
from scipy.special import softmax as scipy_softmax


def _rand_qkv(rng, n, d, heavy_tail=True):
    q = rng.standard_normal((n, d)).astype(np.float32)
    k = rng.standard_normal((n, d)).astype(np.float32)
    v = rng.standard_normal((n, d)).astype(np.float32)
    if heavy_tail:
        u = rng.standard_normal(d)
        u /= np.linalg.norm(u)
        q += (1.5 * u).astype(np.float32)
        hot = rng.random(n) < 0.1
        k[hot] += (4.0 * u).astype(np.float32)
    return q, k, v


def _as_thd(x):  # [n, d] -> [n, 1, d]
    return np.ascontiguousarray(x[:, None, :])


def _harmonic(m):
    return sum(Fraction(1, x) for x in range(1, m + 1))


# --------------------------------------------------------------------------
# closed form: uniform attention
# --------------------------------------------------------------------------
def test_uniform_attention_closed_form(oracle):
    n, d, k, r, steps = 23, 3, 4, 5, 9
    rng = np.random.default_rng(0)
    q = np.zeros((n + steps, d), dtype=np.float32)
    kk = rng.standard_normal((n + steps, d)).astype(np.float32)
    v = rng.standard_normal((n + steps, d)).astype(np.float32)

    O, acc0, P = oracle.causal_attention_colsum(q[:n], kk[:n], v[:n], 0.37, want_p=True)
    Hn = _harmonic(n)
    for j in range(n):
        assert acc0[j] == pytest.approx(float(Hn - _harmonic(j)), rel=1e-14)
    for i in range(n):
        np.testing.assert_allclose(P[i, : i + 1], 1.0 / (i + 1), rtol=1e-15)
        assert np.all(P[i, i + 1:] == 0.0)
        np.testing.assert_allclose(O[i], v[: i + 1].astype(np.float64).mean(axis=0), rtol=1e-13, atol=1e-15)

    # harmonic tails decrease with position, so the heavy hitters are the first k tokens
    kept, boundary = oracle.select(acc0, k, r)
    assert kept.tolist() == list(range(k)) + list(range(n - r, n))
    assert boundary[0] == pytest.approx(float(Hn - _harmonic(k - 1)), rel=1e-14)
    assert boundary[1] == pytest.approx(float(Hn - _harmonic(k)), rel=1e-14)

    cache = oracle.OracleCache(1, 1, d, [k], [r], scale=0.37)
    cache.prefill(_as_thd(q[:n]), _as_thd(kk[:n]), _as_thd(v[:n]), [0, n])
    B = k + r
    expect = {j: Hn - _harmonic(j) for j in kept.tolist()}
    for s in range(steps):
        t = n + s
        res = cache.decode_step(q[t][None, None], kk[t][None, None], v[t][None, None], want_p=True)
        # B cached entries plus the new token share the probability mass equally
        np.testing.assert_allclose(res["p"][0, : B + 1], 1.0 / (B + 1), rtol=1e-15)
        members = sorted(expect) + [t]
        np.testing.assert_allclose(res["out"][0], v[members].astype(np.float64).mean(axis=0), rtol=1e-12, atol=1e-14)
        expect[t] = Fraction(0)
        for j in expect:
            expect[j] += Fraction(1, B + 1)
        # the token that just left the recent window has the smallest accumulated score
        assert res["evicted"][0] == t - r
        del expect[t - r]
        pos, acc = cache.export(0)
        assert pos.tolist() == sorted(expect)
        np.testing.assert_allclose(acc, [float(expect[j]) for j in sorted(expect)], rtol=1e-13)


# --------------------------------------------------------------------------
# brute force of the literal definition
# --------------------------------------------------------------------------
class LiteralH2O:
    """Token-by-token policy, written for clarity only (pure Python, O(T^3)).

    Keeps the full T x T matrix of attention probabilities (zero where a token was
    not attended), so accumulated scores are explicit column sums, and evaluates
    F_score(G \\ {v}) = h(sum of accumulated scores of G without v) for every
    candidate v, taking the argmax.
    """

    def __init__(self, k, r, scale, h, attend=None):
        self.k, self.r, self.c, self.h = k, r, scale, h
        self.attend = attend  # optional predicate (key position, query position, r) -> attended?
        self.topk = 0  # > 0: a query attends only its topk largest logits (equal logits: the higher position)
        self.S = []  # kept positions
        self.rows = []  # rows[i][j] = probability token i gave token j
        self.K, self.V = {}, {}
        self.t = 0

    def preload_rows(self, rows):
        self.rows = [dict(r_) for r_ in rows]

    def column_sum(self, j):
        return math.fsum(row.get(j, 0.0) for row in self.rows)

    def step(self, q, k_new, v_new):
        t = self.t
        self.K[t], self.V[t] = k_new, v_new
        G = self.S + [t]
        seen = [j for j in G if self.attend is None or self.attend(j, t, self.r)]
        logits = [self.c * math.fsum(float(a) * float(b) for a, b in zip(q, self.K[j])) for j in seen]
        if self.topk and len(seen) > self.topk:
            order = sorted(range(len(seen)), key=lambda i: (logits[i], seen[i]), reverse=True)[:self.topk]
            seen = [seen[i] for i in sorted(order)]
            logits = [self.c * math.fsum(float(a) * float(b) for a, b in zip(q, self.K[j])) for j in seen]
        mx = max(logits)
        w = [math.exp(x - mx) for x in logits]
        tot = math.fsum(w)
        row = {j: x / tot for j, x in zip(seen, w)}
        probs = [row.get(j, 0.0) for j in G]
        self.rows.append(row)
        out = [math.fsum(p * float(self.V[j][x]) for j, p in zip(G, probs)) for x in range(len(q))]
        evicted = -1
        min_gap = math.inf
        if len(G) > self.k + self.r:
            cand = [j for j in G if j <= t - self.r]
            colsum = {j: self.column_sum(j) for j in G}
            best, best_val = None, None
            for v_ in sorted(cand):  # ascending position: first maximum wins = lowest position
                val = self.h(math.fsum(colsum[s] for s in G if s != v_))
                if best is None or val > best_val:
                    best, best_val = v_, val
            evicted = best
            cs = sorted(colsum[j] for j in cand)
            if len(cs) > 1:
                min_gap = (cs[1] - cs[0]) / max(abs(cs[1]), 1e-300)
            G.remove(evicted)
        self.S = G
        self.t += 1
        return out, evicted, probs, min_gap


@pytest.mark.parametrize("hname", ["identity", "sqrt", "log"])
@pytest.mark.parametrize("k,r", [(3, 0), (2, 2), (0, 3), (4, 1), (1, 4)])
def test_sequential_policy_matches_literal_argmax(oracle, hname, k, r):
    h = {"identity": lambda z: z, "sqrt": lambda z: math.sqrt(z + 1.0), "log": lambda z: math.log(z + 1.0)}[hname]
    T, d, scale = 16, 4, 0.6
    rng = np.random.default_rng(100 + 10 * k + r)
    q, kk, v = _rand_qkv(rng, T, d)
    lit = LiteralH2O(k, r, scale, h)
    cache = oracle.OracleCache(1, 1, d, [k], [r], scale=scale)
    ever_evicted = set()
    prev = set()
    checked = 0
    for t in range(T):
        out_l, ev_l, probs, gap = lit.step(q[t], kk[t], v[t])
        res = cache.decode_step(q[t][None, None], kk[t][None, None], v[t][None, None], want_p=True)
        m = len(probs)
        # every softmax row sums to one; same probabilities as the literal simulation
        assert math.fsum(res["p"][0, :m]) == pytest.approx(1.0, abs=1e-14)
        np.testing.assert_allclose(np.sort(res["p"][0, :m]), np.sort(probs), rtol=1e-12)
        np.testing.assert_allclose(res["out"][0], out_l, rtol=1e-11, atol=1e-13)
        if gap > 1e-9:  # the sum-minus-one form loses a few ulps; skip decisions it cannot resolve
            assert res["evicted"][0] == ev_l
            checked += 1
        else:
            pytest.skip("tiny accidental near-tie in random data")
        pos, acc = cache.export(0)
        # accumulated scores are explicit column sums of everything attended so far
        np.testing.assert_allclose(acc, [lit.column_sum(j) for j in pos], rtol=1e-12)
        now = set(pos.tolist())
        assert now == set(lit.S)
        assert len(now) <= k + r  # budget
        assert len(now - prev) <= 1  # at most one new entry per step
        if ev_l >= 0:
            ever_evicted.add(ev_l)
        assert not (now & ever_evicted)  # evicted entries never come back
        assert set(range(max(0, t - r + 1), t + 1)) <= now  # recent window always present
        prev = now
    assert checked >= T - (k + r)


def test_budget_three_example_structure(oracle):
    """Budget 3: the fourth step still sees four tokens, then drops one for good (Figure 2's story)."""
    rng = np.random.default_rng(5)
    q, kk, v = _rand_qkv(rng, 8, 4)
    cache = oracle.OracleCache(1, 1, 4, [3], [0], scale=0.5)
    gone = None
    for t in range(8):
        res = cache.decode_step(q[t][None, None], kk[t][None, None], v[t][None, None], want_p=True)
        if t < 3:
            assert res["evicted"][0] == -1 and cache.cnt[0] == t + 1
        if t == 3:
            assert np.count_nonzero(res["p"][0]) == 4
            gone = int(res["evicted"][0])
            assert 0 <= gone <= 3
        if t >= 3:
            assert cache.cnt[0] == 3
            assert gone not in cache.export(0)[0].tolist()


# --------------------------------------------------------------------------
# special cases that reduce to textbook attention
# --------------------------------------------------------------------------
def _textbook_causal(q, k, v, scale, window=None):
    n = q.shape[0]
    s = scale * (q.astype(np.float64) @ k.astype(np.float64).T)
    i, j = np.indices((n, n))
    mask = j <= i
    if window is not None:
        mask &= j >= i - window
    s = np.where(mask, s, -np.inf)
    p = scipy_softmax(s, axis=1)
    return p @ v.astype(np.float64), p


def test_budget_at_least_length_is_full_causal_attention(oracle):
    n, steps, d, scale = 40, 12, 8, 0.3
    rng = np.random.default_rng(7)
    q, kk, v = _rand_qkv(rng, n + steps, d)
    ref_out, ref_p = _textbook_causal(q, kk, v, scale)
    cache = oracle.OracleCache(1, 1, d, [30], [n + steps - 30], scale=scale)
    out, kept = cache.prefill(_as_thd(q[:n]), _as_thd(kk[:n]), _as_thd(v[:n]), [0, n])
    np.testing.assert_allclose(out[:, 0], ref_out[:n], rtol=1e-11, atol=1e-13)
    assert kept[0].tolist() == list(range(n))
    np.testing.assert_allclose(cache.export(0)[1], ref_p[:n].sum(axis=0)[:n], rtol=1e-12)
    for s in range(steps):
        t = n + s
        res = cache.decode_step(q[t][None, None], kk[t][None, None], v[t][None, None])
        assert res["evicted"][0] == -1
        np.testing.assert_allclose(res["out"][0], ref_out[t], rtol=1e-11, atol=1e-13)
    pos, acc = cache.export(0)
    assert pos.tolist() == list(range(n + steps))
    np.testing.assert_allclose(acc, ref_p.sum(axis=0), rtol=1e-12)


def test_prefill_outputs_are_full_causal_whatever_the_budget(oracle):
    n, d, scale = 64, 8, 0.4
    rng = np.random.default_rng(8)
    q, kk, v = _rand_qkv(rng, n, d)
    ref_out, ref_p = _textbook_causal(q, kk, v, scale)
    O, acc0, P = oracle.causal_attention_colsum(q, kk, v, scale, want_p=True)
    np.testing.assert_allclose(O, ref_out, rtol=1e-11, atol=1e-13)
    np.testing.assert_allclose(P, ref_p, rtol=1e-11, atol=1e-300)
    np.testing.assert_allclose(acc0, ref_p.sum(axis=0), rtol=1e-12)
    np.testing.assert_allclose(P.sum(axis=1), 1.0, rtol=1e-14)


def test_zero_heavy_budget_is_sliding_window(oracle):
    T, d, r, scale = 48, 8, 6, 0.5
    rng = np.random.default_rng(9)
    q, kk, v = _rand_qkv(rng, T, d)
    ref_out, _ = _textbook_causal(q, kk, v, scale, window=r)
    # token by token from an empty cache: every output is windowed attention
    cache = oracle.OracleCache(1, 1, d, [0], [r], scale=scale)
    for t in range(T):
        res = cache.decode_step(q[t][None, None], kk[t][None, None], v[t][None, None])
        np.testing.assert_allclose(res["out"][0], ref_out[t], rtol=1e-11, atol=1e-13)
        assert res["evicted"][0] == (t - r if t >= r else -1)
    # after a one-shot prefill the decode steps are windowed as well
    n = 30
    cache = oracle.OracleCache(1, 1, d, [0], [r], scale=scale)
    out, kept = cache.prefill(_as_thd(q[:n]), _as_thd(kk[:n]), _as_thd(v[:n]), [0, n])
    assert kept[0].tolist() == list(range(n - r, n))
    np.testing.assert_allclose(out[:, 0], _textbook_causal(q[:n], kk[:n], v[:n], scale)[0], rtol=1e-11, atol=1e-13)
    for t in range(n, T):
        res = cache.decode_step(q[t][None, None], kk[t][None, None], v[t][None, None])
        np.testing.assert_allclose(res["out"][0], ref_out[t], rtol=1e-11, atol=1e-13)


def test_sequential_fill_equals_prefill_when_nothing_is_evicted(oracle):
    n, steps, d, scale = 20, 6, 4, 0.7
    rng = np.random.default_rng(10)
    q, kk, v = _rand_qkv(rng, n + steps, d)
    a = oracle.OracleCache(1, 1, d, [n], [steps], scale=scale)
    b = oracle.OracleCache(1, 1, d, [n], [steps], scale=scale)
    out_a, _ = a.prefill(_as_thd(q[:n]), _as_thd(kk[:n]), _as_thd(v[:n]), [0, n])
    for t in range(n + steps):
        rb = b.decode_step(q[t][None, None], kk[t][None, None], v[t][None, None])
        if t < n:
            np.testing.assert_allclose(rb["out"][0], out_a[t, 0], rtol=1e-12, atol=1e-14)
        else:
            ra = a.decode_step(q[t][None, None], kk[t][None, None], v[t][None, None])
            np.testing.assert_allclose(rb["out"][0], ra["out"][0], rtol=1e-12, atol=1e-14)
    np.testing.assert_array_equal(a.export(0)[0], b.export(0)[0])
    np.testing.assert_allclose(a.export(0)[1], b.export(0)[1], rtol=1e-12)


# --------------------------------------------------------------------------
# selection and tie-breaking
# --------------------------------------------------------------------------
def _select_by_repeated_eviction(acc0, k, r):
    n = len(acc0)
    if n <= k + r:
        return list(range(n))
    cand = list(range(n - r))
    while len(cand) > k:
        worst = min(cand, key=lambda j: (acc0[j], j))
        cand.remove(worst)
    return sorted(cand) + list(range(n - r, n))


@pytest.mark.parametrize("seed", range(6))
def test_select_equals_repeated_min_eviction(oracle, seed):
    rng = np.random.default_rng(seed)
    n = int(rng.integers(5, 60))
    k = int(rng.integers(0, 12))
    r = int(rng.integers(0, 12))
    acc0 = rng.random(n)
    acc0[rng.integers(0, n, size=n // 2)] = 0.5  # plenty of exact ties
    kept, _ = oracle.select(acc0, k, r)
    assert kept.tolist() == _select_by_repeated_eviction(acc0.tolist(), k, r)


def test_select_ties_drop_lowest_position_first(oracle):
    acc0 = np.array([1.0, 1.0, 1.0, 1.0, 9.0, 0.1, 0.2], dtype=np.float64)
    kept, boundary = oracle.select(acc0, 2, 2)
    assert kept.tolist() == [3, 4, 5, 6]
    assert boundary.tolist() == [1.0, 1.0]
    kept, _ = oracle.select(acc0, 0, 3)
    assert kept.tolist() == [4, 5, 6]
    kept, _ = oracle.select(acc0, 3, 0)
    assert kept.tolist() == [2, 3, 4]


def test_decode_tie_evicts_lowest_position_and_hint_protocol(oracle):
    d = 2
    cache = oracle.OracleCache(1, 1, d, [2], [1], scale=1.0)
    kv = np.ones((3, d))
    # stored out of position order on purpose; positions 7 and 4 tie
    cache.load_unit(0, [7, 4, 9], [1.25, 1.25, 3.0], kv, kv, t=10)
    snap = {n_: getattr(cache, n_).copy() for n_ in ("t", "cnt", "pos", "acc", "K", "V")}
    z = np.zeros((1, 1, d), dtype=np.float32)
    res = cache.decode_step(z, z + 1, z + 1)
    assert res["evicted"][0] == 4 and res["status"][0] == 0 and res["gap"][0] == 0.0
    assert cache.export(0)[0].tolist() == [7, 9, 10]

    def restore():
        for n_, a in snap.items():
            getattr(cache, n_)[...] = a

    restore()
    res = cache.decode_step(z, z + 1, z + 1, hint=np.array([7], dtype=np.int32))
    assert res["evicted"][0] == 4 and res["status"][0] == 1  # excused, and the hint is applied
    assert cache.export(0)[0].tolist() == [4, 9, 10]
    restore()
    res = cache.decode_step(z, z + 1, z + 1, hint=np.array([9], dtype=np.int32))
    assert res["status"][0] == 2  # a real disagreement; oracle's own choice stands
    assert cache.export(0)[0].tolist() == [7, 9, 10]
    restore()
    res = cache.decode_step(z, z + 1, z + 1, hint=np.array([10], dtype=np.int32))
    assert res["status"][0] == 2  # the new token is inside the recent window, not a candidate


def test_entry_order_is_irrelevant(oracle):
    n, steps, d, scale = 50, 20, 8, 0.35
    rng = np.random.default_rng(11)
    q, kk, v = _rand_qkv(rng, n + steps, d)
    a = oracle.OracleCache(1, 1, d, [5], [4], scale=scale)
    b = oracle.OracleCache(1, 1, d, [5], [4], scale=scale)
    a.prefill(_as_thd(q[:n]), _as_thd(kk[:n]), _as_thd(v[:n]), [0, n])
    b.prefill(_as_thd(q[:n]), _as_thd(kk[:n]), _as_thd(v[:n]), [0, n])
    shuffler = np.random.default_rng(12)
    for t in range(n, n + steps):
        b.permute_entries(shuffler)
        ra = a.decode_step(q[t][None, None], kk[t][None, None], v[t][None, None])
        rb = b.decode_step(q[t][None, None], kk[t][None, None], v[t][None, None])
        assert ra["evicted"][0] == rb["evicted"][0]
        np.testing.assert_allclose(ra["out"], rb["out"], rtol=1e-12, atol=1e-14)
    np.testing.assert_array_equal(a.export(0)[0], b.export(0)[0])
    np.testing.assert_allclose(a.export(0)[1], b.export(0)[1], rtol=1e-12)


def test_heads_and_sequences_are_independent(oracle):
    """Batched, ragged call equals per-unit calls (different kept sets per head)."""
    rng = np.random.default_rng(13)
    lens, H, d = [9, 17, 5], 2, 4
    heavy, recent = [2, 3, 4], [2, 3, 4]
    tot = sum(lens)
    q = rng.standard_normal((tot, H, d)).astype(np.float32)
    k = rng.standard_normal((tot, H, d)).astype(np.float32)
    v = rng.standard_normal((tot, H, d)).astype(np.float32)
    cu = np.concatenate([[0], np.cumsum(lens)])
    cache = oracle.OracleCache(len(lens), H, d, heavy, recent)
    out, kept = cache.prefill(q, k, v, cu)
    for s, n in enumerate(lens):
        for h in range(H):
            sl = slice(cu[s], cu[s + 1])
            O, acc0 = oracle.causal_attention_colsum(q[sl, h], k[sl, h], v[sl, h], cache.scale)
            np.testing.assert_array_equal(out[sl, h], O)
            ks, _ = oracle.select(acc0, heavy[s], recent[s])
            np.testing.assert_array_equal(kept[s * H + h], ks)
    dq = rng.standard_normal((len(lens), H, d)).astype(np.float32)
    full = oracle.OracleCache(len(lens), H, d, heavy, recent)
    full.prefill(q, k, v, cu)
    r_all = cache.decode_step(dq, dq * 0.5, dq * 2)
    r_sub = full.decode_step(dq, dq * 0.5, dq * 2, units=[1, 4])
    np.testing.assert_array_equal(r_sub["out"], r_all["out"][[1, 4]])
    np.testing.assert_array_equal(r_sub["evicted"], r_all["evicted"][[1, 4]])
    assert full.t[1] == lens[0] + 1 and full.t[0] == lens[0]


# ---------------------------------------------------------------------------------------------------
# Score variants ("Discussions and Limitations": averaged attention score; remark on h: F_score reporting)
# ---------------------------------------------------------------------------------------------------
@pytest.fixture()
def averaged_mode(oracle):
    oracle.set_score_mode(1)
    yield oracle
    oracle.set_score_mode(0)


@pytest.mark.parametrize("k,r", [(3, 0), (2, 2), (4, 1), (1, 3)])
def test_averaged_score_variant_matches_a_literal_simulation(averaged_mode, k, r):
    """Rank by accumulated score / number of queries that attended the key (positions p .. t: t - p + 1),
    simulated literally in Python with explicit column sums; the accumulated scores themselves are
    unchanged.  The run must also differ somewhere from the accumulated-score policy, or it pins nothing."""
    oracle = averaged_mode
    T, d, scale = 20, 4, 0.7
    rng = np.random.default_rng(500 + 10 * k + r)
    q, kk, v = _rand_qkv(rng, T, d)
    cache = oracle.OracleCache(1, 1, d, [k], [r], scale=scale)
    S, rows, Kd = [], [], {}
    evictions = []
    for t in range(T):
        Kd[t] = kk[t]
        G = S + [t]
        logits = [scale * math.fsum(float(a) * float(b) for a, b in zip(q[t], Kd[j])) for j in G]
        mx = max(logits)
        w = [math.exp(x - mx) for x in logits]
        tot = math.fsum(w)
        rows.append({j: x / tot for j, x in zip(G, w)})
        ev = -1
        if len(G) > k + r:
            cand = [j for j in G if j <= t - r]
            avg = {j: math.fsum(row.get(j, 0.0) for row in rows) / (t - j + 1) for j in cand}
            ev = min(sorted(cand), key=lambda j: avg[j])  # first minimum in ascending position
            vals = sorted(avg.values())
            if len(vals) > 1 and (vals[1] - vals[0]) / max(vals[1], 1e-300) < 1e-9:
                pytest.skip("tiny accidental near-tie in random data")
            G.remove(ev)
        S = G
        res = cache.decode_step(q[t][None, None], kk[t][None, None], v[t][None, None])
        assert res["evicted"][0] == ev
        evictions.append(ev)
        pos, acc = cache.export(0)
        assert set(pos.tolist()) == set(S)
        np.testing.assert_allclose(acc, [math.fsum(row.get(j, 0.0) for row in rows) for j in pos], rtol=1e-12)
    oracle.set_score_mode(0)
    plain = oracle.OracleCache(1, 1, d, [k], [r], scale=scale)
    plain_ev = [int(plain.decode_step(q[t][None, None], kk[t][None, None], v[t][None, None])["evicted"][0]) for t in range(T)]
    if r < 3:  # with a long recent window and few candidates the two policies may coincide
        assert plain_ev != evictions


def test_averaged_score_prefill_selection_is_top_k_of_column_sum_over_age(averaged_mode):
    oracle = averaged_mode
    rng = np.random.default_rng(77)
    n, k, r = 40, 6, 5
    acc0 = rng.random(n) * np.linspace(3.0, 0.2, n)  # older keys have collected more, as in a real prompt
    kept, _ = oracle.select(acc0, k, r)
    avg = acc0[: n - r] / (n - np.arange(n - r))
    want = sorted(np.argsort(-avg, kind="stable")[:k].tolist() + list(range(n - r, n)))
    assert kept.tolist() == want
    oracle.set_score_mode(0)
    kept0, _ = oracle.select(acc0, k, r)
    assert kept0.tolist() != want  # the plain policy favours the old keys here


def test_fscore_reports_sum_of_h_of_accumulated_scores(oracle):
    acc = np.array([0.0, 3.0, 8.0, 0.25])
    assert oracle.fscore(acc, 0) == pytest.approx(11.25, rel=1e-15)
    assert oracle.fscore(acc, 1) == pytest.approx(1.0 + 2.0 + 3.0 + math.sqrt(1.25), rel=1e-15)
    assert oracle.fscore(acc, 2) == pytest.approx(0.0 + math.log(4.0) + math.log(9.0) + math.log(1.25), rel=1e-15)
    # removing the key with the smallest accumulated score keeps F_score largest, for every h (the reason
    # why h does not change the decisions)
    for hk in (0, 1, 2):
        drops = [oracle.fscore(np.delete(acc, j), hk) for j in range(len(acc))]
        assert int(np.argmax(drops)) == int(np.argmin(acc))


# ---------------------------------------------------------------------------------------------------
# 4-bit group quantisation of stored rows (the paper names the combination, not a quantiser: these pins
# are mathematical)
# ---------------------------------------------------------------------------------------------------
def test_kv4_quantiser_error_bound_end_points_and_idempotence():
    from oracle import kv_quant

    rng = np.random.default_rng(9)
    x = kv_quant.bf16_round(rng.standard_normal((64, 128)).astype(np.float32) * np.float32(3.0))
    x[5, 32:64] = np.float32(0.75)  # a constant group
    x[6, :32] = np.linspace(-4, 4, 32, dtype=np.float32)
    codes, scale, zero = kv_quant.quantize_rows(x)
    assert codes.dtype == np.uint8 and codes.max() <= 15
    xh = kv_quant.dequantize_rows(codes, scale, zero)
    g = x.reshape(64, 4, 32)
    # every value within half a step (+ one bf16 rounding of the step); the minimum is reproduced exactly
    step = scale[..., None]
    assert np.all(np.abs(xh.reshape(64, 4, 32) - g) <= 0.5 * step * (1 + 2.0 ** -7) + 1e-6)
    assert np.array_equal(xh.reshape(64, 4, 32).min(axis=-1), g.min(axis=-1))
    assert np.all(codes.reshape(64, 4, 32).min(axis=-1) == 0)
    nonconst = g.max(axis=-1) > g.min(axis=-1)
    assert np.all(codes.reshape(64, 4, 32).max(axis=-1)[nonconst] >= 14)  # the maximum lands on the last step or next to it
    assert np.array_equal(xh[5, 32:64], x[5, 32:64])  # constant group: exact
    # reading back and storing again changes nothing
    codes2, scale2, zero2 = kv_quant.quantize_rows(xh)
    assert np.array_equal(kv_quant.dequantize_rows(codes2, scale2, zero2), xh)
    # scale and zero are bf16 values
    assert np.array_equal(kv_quant.bf16_round(scale), scale) and np.array_equal(kv_quant.bf16_round(zero), zero)


def test_kv4_bf16_rounding_helper_matches_torch():
    import torch
    from oracle import kv_quant

    x = np.random.default_rng(3).standard_normal(10000).astype(np.float32) * np.float32(100.0)
    x[:4] = [1.00390625, 1.01171875, -1.00390625, 0.0]  # ties to even on both sides
    want = torch.from_numpy(x).to(torch.bfloat16).float().numpy()
    assert np.array_equal(kv_quant.bf16_round(x), want)


def test_kv4_cache_stores_quantised_rows_but_attends_the_new_token_exactly(oracle):
    from oracle import kv_quant

    rng = np.random.default_rng(12)
    d, k, r, T = 32, 2, 2, 9
    q, kk, v = _rand_qkv(rng, T, d)
    c4 = oracle.OracleCache(1, 1, d, [k], [r], scale=0.5, kv4=True)
    ref = oracle.OracleCache(1, 1, d, [k], [r], scale=0.5)
    for t in range(T):
        # a plain cache that is FED quantised rows for everything but the current token must behave the same
        res4 = c4.decode_step(q[t][None, None], kk[t][None, None], v[t][None, None])
        resr = ref.decode_step(q[t][None, None], kk[t][None, None], v[t][None, None])
        m = int(ref.cnt[0])
        hit = np.nonzero(ref.pos[0, :m] == t)[0]
        if hit.size:
            ref.K[0, hit[0]] = kv_quant.qdq(kk[t][None].astype(np.float32))[0]
            ref.V[0, hit[0]] = kv_quant.qdq(v[t][None].astype(np.float32))[0]
        assert res4["evicted"][0] == resr["evicted"][0]
        np.testing.assert_array_equal(res4["out"], resr["out"])
    m = int(c4.cnt[0])
    np.testing.assert_array_equal(c4.K[0, :m], kv_quant.qdq(c4.K[0, :m].astype(np.float32)))  # stored rows are on the grid


# --------------------------------------------------------------------------
# sparse patterns inside the recent window (heavy hitters combined with the strided / fixed masks)
# --------------------------------------------------------------------------
def _pattern(kind, a, b):
    """(key position p, query position t) -> allowed by the pattern, written on arrays."""
    if kind == "strided":
        return lambda p, t: ((t - p) < b) | ((t - p) % a == 0)
    return lambda p, t: ((p // a) == (t // a)) | ((p % a) >= a - b)


def _mask_matrix(T, r, pat):
    """M[t][j]: key j attended by query t under the reading: itself, everything older than the window,
    and of the window what the pattern allows."""
    t, j = np.indices((T, T))
    return (j <= t) & ((j == t) | (j <= t - r) | pat(j, t))


def _textbook_masked(q, k, v, scale, M):
    s = scale * (q.astype(np.float64) @ k.astype(np.float64).T)
    p = scipy_softmax(np.where(M, s, -np.inf), axis=1)
    return p @ v.astype(np.float64), p


MASKS = [("strided", 1, 4, 2), ("strided", 1, 3, 1), ("fixed", 2, 4, 1), ("fixed", 2, 5, 2)]  # (name, kind, a, b)


@pytest.fixture
def masked(oracle):
    def use(kind, a, b):
        oracle.set_mask(kind, a, b)

    yield use
    oracle.set_mask(0)


def test_a_pattern_that_allows_the_whole_window_changes_nothing(oracle, masked):
    n, steps, d, k, r, scale = 40, 30, 8, 5, 6, 0.5
    rng = np.random.default_rng(31)
    q, kk, v = _rand_qkv(rng, n + steps, d)

    def run():
        cache = oracle.OracleCache(1, 1, d, [k], [r], scale=scale)
        out, kept = cache.prefill(_as_thd(q[:n]), _as_thd(kk[:n]), _as_thd(v[:n]), [0, n])
        res = [cache.decode_step(q[t][None, None], kk[t][None, None], v[t][None, None]) for t in range(n, n + steps)]
        return out, kept[0], [x["out"] for x in res], [int(x["evicted"][0]) for x in res], cache.export(0)

    ref = run()
    for kind, a, b in ((1, 3, r), (1, 1, 0), (2, 4, 4), (2, 1000, 0)):  # local window >= r; stride 1; all columns summary; one block
        masked(kind, a, b)
        got = run()
        np.testing.assert_array_equal(got[0], ref[0])
        np.testing.assert_array_equal(got[1], ref[1])
        assert got[3] == ref[3]
        for x, y in zip(got[2], ref[2]):
            np.testing.assert_array_equal(x, y)
        np.testing.assert_array_equal(got[4][0], ref[4][0])
        np.testing.assert_array_equal(got[4][1], ref[4][1])


@pytest.mark.parametrize("name,kind,a,b", MASKS)
def test_masked_prompt_attention_is_textbook_masked_attention(oracle, masked, name, kind, a, b):
    n, d, r, scale = 48, 8, 9, 0.4
    rng = np.random.default_rng(32 + a)
    q, kk, v = _rand_qkv(rng, n, d)
    M = _mask_matrix(n, r, _pattern(name, a, b))
    assert not M[np.tril_indices(n)].all()  # the pattern really removes something
    ref_out, ref_p = _textbook_masked(q, kk, v, scale, M)
    masked(kind, a, b)
    O, acc0, P = oracle.causal_attention_colsum(q, kk, v, scale, want_p=True, window=r)
    np.testing.assert_allclose(O, ref_out, rtol=1e-11, atol=1e-13)
    np.testing.assert_allclose(P, ref_p, rtol=1e-11, atol=1e-300)
    np.testing.assert_allclose(acc0, ref_p.sum(axis=0), rtol=1e-12)
    np.testing.assert_allclose(P.sum(axis=1), 1.0, rtol=1e-14)


@pytest.mark.parametrize("name,kind,a,b", MASKS)
def test_masked_zero_heavy_budget_is_the_pattern_alone(oracle, masked, name, kind, a, b):
    """Without heavy hitters (k = 0) the token-by-token policy is plain masked attention: the window entries the
    pattern allows, the token that is just leaving the window, and the token itself."""
    T, d, r, scale = 40, 8, 7, 0.5
    rng = np.random.default_rng(33 + b)
    q, kk, v = _rand_qkv(rng, T, d)
    t, j = np.indices((T, T))
    M = (j <= t) & (j >= t - r) & _mask_matrix(T, r, _pattern(name, a, b))
    ref_out, _ = _textbook_masked(q, kk, v, scale, M)
    masked(kind, a, b)
    cache = oracle.OracleCache(1, 1, d, [0], [r], scale=scale)
    for step in range(T):
        res = cache.decode_step(q[step][None, None], kk[step][None, None], v[step][None, None])
        np.testing.assert_allclose(res["out"][0], ref_out[step], rtol=1e-11, atol=1e-13)
        assert res["evicted"][0] == (step - r if step >= r else -1)


@pytest.mark.parametrize("name,kind,a,b", MASKS)
def test_masked_cache_that_never_evicts_is_textbook_masked_attention(oracle, masked, name, kind, a, b):
    n, steps, d, r, scale = 30, 14, 8, 8, 0.35
    rng = np.random.default_rng(34 + a + b)
    q, kk, v = _rand_qkv(rng, n + steps, d)
    M = _mask_matrix(n + steps, r, _pattern(name, a, b))
    ref_out, ref_p = _textbook_masked(q, kk, v, scale, M)
    masked(kind, a, b)
    one_shot = oracle.OracleCache(1, 1, d, [n + steps], [r], scale=scale)
    token_by_token = oracle.OracleCache(1, 1, d, [n + steps], [r], scale=scale)
    out, kept = one_shot.prefill(_as_thd(q[:n]), _as_thd(kk[:n]), _as_thd(v[:n]), [0, n])
    np.testing.assert_allclose(out[:, 0], ref_out[:n], rtol=1e-11, atol=1e-13)
    for t in range(n + steps):
        rb = token_by_token.decode_step(q[t][None, None], kk[t][None, None], v[t][None, None])
        np.testing.assert_allclose(rb["out"][0], ref_out[t], rtol=1e-11, atol=1e-13)
        if t >= n:
            ra = one_shot.decode_step(q[t][None, None], kk[t][None, None], v[t][None, None])
            np.testing.assert_allclose(ra["out"][0], ref_out[t], rtol=1e-11, atol=1e-13)
    for cache in (one_shot, token_by_token):
        pos, acc = cache.export(0)
        assert pos.tolist() == list(range(n + steps))
        np.testing.assert_allclose(acc, ref_p.sum(axis=0), rtol=1e-12, atol=1e-300)


@pytest.mark.parametrize("name,kind,a,b", MASKS)
@pytest.mark.parametrize("k,r", [(3, 4), (2, 6), (5, 3)])
def test_masked_policy_matches_the_literal_simulation(oracle, masked, name, kind, a, b, k, r):
    """Evictions under a pattern: the literal argmax over explicit column sums of the masked probability matrix."""
    T, d, scale = 22, 4, 0.6
    rng = np.random.default_rng(500 + 7 * k + r + a)
    q, kk, v = _rand_qkv(rng, T, d)
    pat = _pattern(name, a, b)
    lit = LiteralH2O(k, r, scale, lambda z: z, attend=lambda p, t, r_: p == t or p <= t - r_ or bool(pat(p, t)))
    masked(kind, a, b)
    cache = oracle.OracleCache(1, 1, d, [k], [r], scale=scale)
    decided = 0
    for t in range(T):
        out_l, ev_l, probs, gap = lit.step(q[t], kk[t], v[t])
        res = cache.decode_step(q[t][None, None], kk[t][None, None], v[t][None, None], want_p=True)
        np.testing.assert_allclose(np.sort(res["p"][0, :len(probs)]), np.sort(probs), rtol=1e-12, atol=1e-300)
        np.testing.assert_allclose(res["out"][0], out_l, rtol=1e-11, atol=1e-13)
        if gap > 1e-9:
            assert res["evicted"][0] == ev_l
            decided += 1
        else:  # follow the simulation through an accidental near-tie so that later steps stay comparable
            cache = None
            break
        pos, acc = cache.export(0)
        assert set(pos.tolist()) == set(lit.S)
        np.testing.assert_allclose(acc, [lit.column_sum(j) for j in pos], rtol=1e-12, atol=1e-300)
    assert decided >= 8


# --------------------------------------------------------------------------
# "Top-K" attention in decode steps (each query keeps only its m largest logits)
# --------------------------------------------------------------------------
@pytest.fixture
def topk(oracle):
    def use(m):
        oracle.set_topk(m)

    yield use
    oracle.set_topk(0)


def _textbook_topk(q, k, v, scale, m):
    """Causal attention in which every row keeps its m largest logits (numpy argsort; ties cannot occur in random data)."""
    n = q.shape[0]
    s = scale * (q.astype(np.float64) @ k.astype(np.float64).T)
    s = np.where(np.tril(np.ones((n, n), dtype=bool)), s, -np.inf)
    keep = np.zeros((n, n), dtype=bool)
    for i in range(n):
        keep[i, np.argsort(-s[i, :i + 1], kind="stable")[:m]] = True
    p = scipy_softmax(np.where(keep, s, -np.inf), axis=1)
    return p @ v.astype(np.float64), p


@pytest.mark.parametrize("m", [1, 3, 8])
def test_topk_with_a_cache_that_never_evicts_is_textbook_top_m_attention(oracle, topk, m):
    T, d, scale = 36, 8, 0.45
    rng = np.random.default_rng(700 + m)
    q, kk, v = _rand_qkv(rng, T, d)
    ref_out, ref_p = _textbook_topk(q, kk, v, scale, m)
    topk(m)
    cache = oracle.OracleCache(1, 1, d, [T], [4], scale=scale)
    for t in range(T):
        res = cache.decode_step(q[t][None, None], kk[t][None, None], v[t][None, None], want_p=True)
        np.testing.assert_allclose(res["out"][0], ref_out[t], rtol=1e-11, atol=1e-13)
        assert int((res["p"][0, :t + 1] > 0).sum()) == min(m, t + 1)
        assert math.fsum(res["p"][0, :t + 1]) == pytest.approx(1.0, abs=1e-14)
    pos, acc = cache.export(0)
    np.testing.assert_allclose(acc, ref_p.sum(axis=0), rtol=1e-12, atol=1e-300)  # scores: column sums of what was attended


def test_topk_not_smaller_than_the_cache_changes_nothing(oracle, topk):
    n, steps, d, k, r, scale = 30, 25, 8, 4, 5, 0.5
    rng = np.random.default_rng(710)
    q, kk, v = _rand_qkv(rng, n + steps, d)

    def run():
        cache = oracle.OracleCache(1, 1, d, [k], [r], scale=scale)
        cache.prefill(_as_thd(q[:n]), _as_thd(kk[:n]), _as_thd(v[:n]), [0, n])
        res = [cache.decode_step(q[t][None, None], kk[t][None, None], v[t][None, None]) for t in range(n, n + steps)]
        return [x["out"] for x in res], [int(x["evicted"][0]) for x in res], cache.export(0)

    ref = run()
    topk(k + r + 1)  # the kept entries and the token itself
    got = run()
    assert got[1] == ref[1]
    for x, y in zip(got[0], ref[0]):
        np.testing.assert_array_equal(x, y)
    np.testing.assert_array_equal(got[2][1], ref[2][1])


@pytest.mark.parametrize("k,r,m", [(3, 3, 2), (4, 2, 4), (2, 5, 3), (5, 0, 2)])
def test_topk_policy_matches_the_literal_simulation(oracle, topk, k, r, m):
    """Evictions under Top-K attention: explicit column sums of the probability matrix that has zeros for the logits a
    query dropped, literal argmax of F_score."""
    T, d, scale = 22, 4, 0.6
    rng = np.random.default_rng(720 + 10 * k + r + m)
    q, kk, v = _rand_qkv(rng, T, d)
    lit = LiteralH2O(k, r, scale, lambda z: z)
    lit.topk = m
    topk(m)
    cache = oracle.OracleCache(1, 1, d, [k], [r], scale=scale)
    decided = 0
    for t in range(T):
        out_l, ev_l, probs, gap = lit.step(q[t], kk[t], v[t])
        res = cache.decode_step(q[t][None, None], kk[t][None, None], v[t][None, None], want_p=True)
        np.testing.assert_allclose(np.sort(res["p"][0, :len(probs)]), np.sort(probs), rtol=1e-12, atol=1e-300)
        np.testing.assert_allclose(res["out"][0], out_l, rtol=1e-11, atol=1e-13)
        if 0.0 < gap <= 1e-9:
            break  # an accidental near-tie: the two would drift apart from here
        # (an exact tie — two entries no query has attended yet both have score 0 — is decided by position on both sides)
        assert res["evicted"][0] == ev_l
        decided += 1
        pos, acc = cache.export(0)
        assert set(pos.tolist()) == set(lit.S)
        np.testing.assert_allclose(acc, [lit.column_sum(j) for j in pos], rtol=1e-12, atol=1e-300)
    assert decided >= 8


def test_topk_tie_keeps_the_higher_position_and_reports_the_gap(oracle, topk):
    d, scale = 4, 1.0
    key = np.array([[1.0, 0.0, 0.0, 0.0]], dtype=np.float32)
    cache = oracle.OracleCache(1, 1, d, [8], [2], scale=scale)
    zero = np.zeros((1, d), dtype=np.float32)
    for _ in range(3):  # three identical keys at positions 0, 1, 2
        cache.decode_step(zero[None], key[None], key[None])
    topk(2)
    res = cache.decode_step(key[None], (0.5 * key)[None], key[None], want_p=True)  # logits 1, 1, 1 and 0.5 for itself
    p = res["p"][0, :4]
    assert p[0] == 0.0 and p[3] == 0.0 and p[1] == pytest.approx(0.5) and p[2] == pytest.approx(0.5)
    assert res["topk_gap"][0] == 0.0  # weakest kept and strongest dropped logit are equal


# --------------------------------------------------------------------------
# grouped-query attention: several query heads share one unit's keys and values; scores add up over the group
# --------------------------------------------------------------------------
def test_group_of_identical_queries_is_one_head_with_scaled_scores(oracle):
    n, steps, d, k, r, scale, G = 30, 25, 8, 4, 5, 0.5, 3
    rng = np.random.default_rng(810)
    q, kk, v = _rand_qkv(rng, n + steps, d)
    one = oracle.OracleCache(1, 1, d, [k], [r], scale=scale)
    grp = oracle.OracleCache(1, 1, d, [k], [r], scale=scale, group=G)
    qg = np.repeat(q[:, None, :], G, axis=1)  # [tokens, G, d]: the same query in every head of the group
    o1, kept1 = one.prefill(_as_thd(q[:n]), _as_thd(kk[:n]), _as_thd(v[:n]), [0, n])
    og, keptg = grp.prefill(np.ascontiguousarray(qg[:n]), _as_thd(kk[:n]), _as_thd(v[:n]), [0, n])
    np.testing.assert_array_equal(kept1[0], keptg[0])
    for g in range(G):
        np.testing.assert_array_equal(og[:, g], o1[:, 0])
    for t in range(n, n + steps):
        r1 = one.decode_step(q[t][None, None], kk[t][None, None], v[t][None, None])
        rg = grp.decode_step(qg[t][None], kk[t][None, None], v[t][None, None])
        assert r1["evicted"][0] == rg["evicted"][0]
        for g in range(G):
            np.testing.assert_array_equal(rg["out"][0, g * d:(g + 1) * d], r1["out"][0])
    np.testing.assert_array_equal(one.export(0)[0], grp.export(0)[0])
    np.testing.assert_allclose(grp.export(0)[1], G * one.export(0)[1], rtol=1e-14)


def test_group_with_a_cache_that_never_evicts_is_textbook_attention_per_query_head(oracle):
    n, steps, d, scale, G = 24, 10, 8, 0.4, 4
    rng = np.random.default_rng(811)
    kk = rng.standard_normal((n + steps, d)).astype(np.float32)
    v = rng.standard_normal((n + steps, d)).astype(np.float32)
    qs = rng.standard_normal((n + steps, G, d)).astype(np.float32)
    refs = [_textbook_causal(qs[:, g], kk, v, scale) for g in range(G)]
    cache = oracle.OracleCache(1, 1, d, [n + steps], [3], scale=scale, group=G)
    out, kept = cache.prefill(np.ascontiguousarray(qs[:n]), _as_thd(kk[:n]), _as_thd(v[:n]), [0, n])
    for g in range(G):
        np.testing.assert_allclose(out[:, g], refs[g][0][:n], rtol=1e-11, atol=1e-13)
    for t in range(n, n + steps):
        res = cache.decode_step(qs[t][None], kk[t][None, None], v[t][None, None])
        for g in range(G):
            np.testing.assert_allclose(res["out"][0, g * d:(g + 1) * d], refs[g][0][t], rtol=1e-11, atol=1e-13)
    pos, acc = cache.export(0)
    assert pos.tolist() == list(range(n + steps))
    np.testing.assert_allclose(acc, sum(p.sum(axis=0) for _, p in refs), rtol=1e-12)  # column sums add up over the group


@pytest.mark.parametrize("k,r,G", [(3, 3, 2), (2, 4, 3), (4, 0, 2)])
def test_group_policy_matches_the_literal_simulation(oracle, k, r, G):
    """One simulation step per query head over the same kept set (the rows of all heads enter the explicit column
    sums), the eviction after the group's last head."""
    T, d, scale = 20, 4, 0.6
    rng = np.random.default_rng(820 + 10 * k + r + G)
    kk = rng.standard_normal((T, d)).astype(np.float32)
    v = rng.standard_normal((T, d)).astype(np.float32)
    qs = (rng.standard_normal((T, G, d)) + 0.7).astype(np.float32)
    lit = LiteralH2O(k, r, scale, lambda z: z)
    cache = oracle.OracleCache(1, 1, d, [k], [r], scale=scale, group=G)
    decided = 0
    for t in range(T):
        # literal: the first G - 1 heads attend without evicting (their rows are recorded), the last one evicts
        kept_before = list(lit.S)
        outs = []
        for g in range(G):
            lit.S, lit.t = list(kept_before), t
            budget = lit.k
            if g < G - 1:
                lit.k = 10 ** 6  # no eviction for this head
            out_l, ev_l, probs, gap = lit.step(qs[t, g], kk[t], v[t])
            lit.k = budget
            outs.append(out_l)
        res = cache.decode_step(qs[t][None], kk[t][None, None], v[t][None, None])
        for g in range(G):
            np.testing.assert_allclose(res["out"][0, g * d:(g + 1) * d], outs[g], rtol=1e-11, atol=1e-13)
        if 0.0 < gap <= 1e-9:
            break
        assert res["evicted"][0] == ev_l
        decided += 1
        pos, acc = cache.export(0)
        assert set(pos.tolist()) == set(lit.S)
        np.testing.assert_allclose(acc, [lit.column_sum(j) for j in pos], rtol=1e-12, atol=1e-300)
    assert decided >= 8
