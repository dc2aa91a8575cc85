"""ctypes front end of the fp64 CPU oracle (``h2o_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by the tests, the smoke check and the
benchmark's CPU-baseline leg.  The CUDA package never imports this module and
this module never imports the CUDA package.

The arithmetic lives in the C file; this wrapper only owns the per-unit state
arrays, slices ragged inputs into units and gathers the rows the C selection
named.  A *unit* is one (sequence, head); units never interact.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import List, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "h2o_oracle.c")
_LIB = os.path.join(_HERE, "libh2o_oracle.so")
_lib = None

NO_HINT = -2


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (OpenMP over independent rows/units)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-std=c99", "-fopenmp", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        c = ctypes
        dp, fp, ip = c.POINTER(c.c_double), c.POINTER(c.c_float), c.POINTER(c.c_int32)
        lib.h2o_oracle_num_threads.restype = c.c_int
        lib.h2o_oracle_causal_attention_colsum.restype = c.c_int
        lib.h2o_oracle_causal_attention_colsum.argtypes = [fp, fp, fp, c.c_long, c.c_long, c.c_long, c.c_long, c.c_double, c.c_long, dp, dp, dp, dp, dp]
        lib.h2o_oracle_select.restype = c.c_long
        lib.h2o_oracle_select.argtypes = [dp, c.c_long, c.c_long, c.c_long, ip, dp]
        lib.h2o_oracle_decode_step.restype = c.c_int
        lib.h2o_oracle_decode_step.argtypes = [c.c_long, c.c_long, c.c_long, c.c_long, ip, ip, ip, ip, ip, dp, dp, dp, fp, fp, fp,
                                               c.c_double, ip, c.c_double, dp, ip, ip, dp, dp, dp]
        lib.h2o_oracle_set_score_mode.restype = c.c_int
        lib.h2o_oracle_set_score_mode.argtypes = [c.c_int]
        lib.h2o_oracle_set_topk.restype = c.c_int
        lib.h2o_oracle_set_topk.argtypes = [c.c_long]
        lib.h2o_oracle_set_mask.restype = c.c_int
        lib.h2o_oracle_set_mask.argtypes = [c.c_int, c.c_long, c.c_long]
        lib.h2o_oracle_fscore.restype = c.c_double
        lib.h2o_oracle_fscore.argtypes = [dp, c.c_long, c.c_int]
        _lib = lib
    return _lib


def num_threads() -> int:
    return int(_load().h2o_oracle_num_threads())


def _p(a: Optional[np.ndarray], ty):
    return None if a is None else a.ctypes.data_as(ctypes.POINTER(ty))


def _f32(x) -> np.ndarray:
    """Widen any input (numpy or torch CPU tensor, f32 or bf16) to contiguous float32, exactly."""
    if hasattr(x, "detach"):
        x = x.detach().to("cpu").float().numpy()
    return np.ascontiguousarray(x, dtype=np.float32)


def causal_attention_colsum(q, k, v, scale: float, want_p: bool = False, window: int = 0):
    """One unit: q, k, v ``[n, d]`` views (row stride may exceed d).  Returns O, acc0, (P).
    ``window``: the unit's recent window r; only read when a sparse pattern is set (``set_mask``)."""
    n, d = q.shape
    assert q.dtype == np.float32 and k.dtype == np.float32 and v.dtype == np.float32
    stride_q, stride = q.strides[0] // 4, k.strides[0] // 4
    assert k.strides == v.strides and q.strides[1] == 4 and k.strides[1] == 4
    O = np.empty((n, d), dtype=np.float64)
    rowmax = np.empty(n, dtype=np.float64)
    rowsum = np.empty(n, dtype=np.float64)
    acc0 = np.empty(n, dtype=np.float64)
    P = np.empty((n, n), dtype=np.float64) if want_p else None
    rc = _load().h2o_oracle_causal_attention_colsum(
        _p(q, ctypes.c_float), _p(k, ctypes.c_float), _p(v, ctypes.c_float), n, d, stride_q, stride, float(scale), int(window),
        _p(O, ctypes.c_double), _p(rowmax, ctypes.c_double), _p(rowsum, ctypes.c_double), _p(acc0, ctypes.c_double),
        _p(P, ctypes.c_double))
    if rc != 0:
        raise RuntimeError("oracle attention failed: %d" % rc)
    return (O, acc0, P) if want_p else (O, acc0)


def set_score_mode(mode: int) -> None:
    """0: rank by the accumulated score (Algorithm 2); 1: by the averaged score (accumulated score over the
    number of queries that attended the key; the variant named in "Discussions and Limitations").
    Process-wide: the tests that use mode 1 set it back to 0 when they are done."""
    if _load().h2o_oracle_set_score_mode(int(mode)) != 0:
        raise ValueError("score mode must be 0 or 1")


MASK_NONE, MASK_STRIDED, MASK_FIXED = 0, 1, 2


def set_mask(kind: int, a: int = 1, b: int = 1) -> None:
    """Sparse pattern applied inside the recent window (combination of the heavy hitters with the strided / fixed
    Sparse Transformer patterns): 0 none; 1 strided(stride a, local window b); 2 fixed(block a, b summary columns).
    Process-wide, like the score mode: tests that set it put it back to 0."""
    if _load().h2o_oracle_set_mask(int(kind), int(a), int(b)) != 0:
        raise ValueError("bad mask parameters")


def set_topk(m: int) -> None:
    """"Top-K" attention in decode steps: each query attends only its m largest logits (0 = off).  Process-wide."""
    if _load().h2o_oracle_set_topk(int(m)) != 0:
        raise ValueError("m must be >= 0")


def fscore(acc: np.ndarray, hkind: int = 0) -> float:
    """F_score = sum of h(accumulated score) over the kept keys; h: 0 identity, 1 sqrt(z+1), 2 log(z+1)."""
    acc = np.ascontiguousarray(acc, dtype=np.float64)
    return float(_load().h2o_oracle_fscore(_p(acc, ctypes.c_double), acc.shape[0], int(hkind)))


def select(acc0: np.ndarray, k: int, r: int):
    """Kept positions (ascending) and the two boundary scores (weakest kept heavy, strongest dropped)."""
    n = acc0.shape[0]
    acc0 = np.ascontiguousarray(acc0, dtype=np.float64)
    kept = np.empty(max(1, min(n, k + r)), dtype=np.int32)
    boundary = np.empty(2, dtype=np.float64)
    m = _load().h2o_oracle_select(_p(acc0, ctypes.c_double), n, k, r, _p(kept, ctypes.c_int32), _p(boundary, ctypes.c_double))
    if m < 0:
        raise RuntimeError("oracle select failed")
    return kept[:m].copy(), boundary


class OracleCache:
    """State of ``batch * n_heads`` independent units; unit index = sequence * n_heads + head."""

    def __init__(self, batch: int, n_heads: int, head_dim: int, heavy: Sequence[int], recent: Sequence[int], scale: Optional[float] = None,
                 kv4: bool = False, group: int = 1):
        """kv4: stored K/V rows are 4-bit group-quantised (oracle/kv_quant.py): a row is quantised when it
        enters the cache — the kept prompt rows after selection, a new token's row after its own step, in
        which it still takes part at full precision."""
        assert len(heavy) == batch and len(recent) == batch
        self.kv4 = bool(kv4)
        # grouped-query attention: `group` query heads share the keys and values of one (sequence, head) unit; q and
        # out then have n_heads * group heads (query head = head * group + g), k and v n_heads
        self.group = int(group)
        self.batch, self.n_heads, self.d = batch, n_heads, head_dim
        self.units = batch * n_heads
        self.scale = float(scale) if scale and scale > 0 else 1.0 / float(np.sqrt(head_dim))
        self.kbud = np.repeat(np.asarray(heavy, dtype=np.int32), n_heads)
        self.rwin = np.repeat(np.asarray(recent, dtype=np.int32), n_heads)
        self.cap = int((self.kbud + self.rwin).max()) + 1
        self.t = np.zeros(self.units, dtype=np.int32)
        self.cnt = np.zeros(self.units, dtype=np.int32)
        self.pos = np.full((self.units, self.cap), -1, dtype=np.int32)
        self.acc = np.zeros((self.units, self.cap), dtype=np.float64)
        self.K = np.zeros((self.units, self.cap, head_dim), dtype=np.float64)
        self.V = np.zeros((self.units, self.cap, head_dim), dtype=np.float64)
        self.last_acc0: List[np.ndarray] = []
        self.last_boundary: List[np.ndarray] = []

    # -- prefill ---------------------------------------------------------
    def prefill(self, q, k, v, cu_seqlens, units: Optional[Sequence[int]] = None, forced_kept=None):
        """Causal attention, column sums and one-shot selection for every unit (or only ``units``).

        q, k, v: ``[total_tokens, n_heads, d]``.  Returns (out ``[total_tokens, n_heads, d]`` float64 with
        untouched units left NaN, kept: dict unit -> ascending positions).  ``forced_kept`` maps a unit to
        a kept set chosen elsewhere (used to re-synchronise after an excused near-tie).
        """
        q, k, v = _f32(q), _f32(k), _f32(v)
        cu = np.asarray(cu_seqlens, dtype=np.int64)
        out = np.full(q.shape, np.nan, dtype=np.float64)
        G = self.group
        todo = range(self.units) if units is None else units
        kept_all = {}
        self.last_acc0 = [None] * self.units
        self.last_boundary = [None] * self.units
        for u in todo:
            s, h = divmod(u, self.n_heads)
            lo, hi = int(cu[s]), int(cu[s + 1])
            acc0 = 0.0
            for g in range(G):  # every query head of the group over the shared keys; column sums add up
                O, a_g = causal_attention_colsum(q[lo:hi, h * G + g], k[lo:hi, h], v[lo:hi, h], self.scale,
                                                 window=int(self.rwin[u]))
                out[lo:hi, h * G + g] = O
                acc0 = acc0 + a_g
            kept, boundary = select(acc0, int(self.kbud[u]), int(self.rwin[u]))
            self.last_acc0[u], self.last_boundary[u] = acc0, boundary
            kept_all[u] = kept
            use = kept if forced_kept is None or u not in forced_kept else np.asarray(forced_kept[u], dtype=np.int32)
            self.load_unit(u, use, acc0[use], k[lo:hi, h][use], v[lo:hi, h][use], hi - lo)
        return out, kept_all

    def load_unit(self, u: int, positions, acc, k_rows, v_rows, t: int):
        m = len(positions)
        assert m <= self.cap - 1
        self.cnt[u] = m
        self.t[u] = t
        self.pos[u, :m] = positions
        self.acc[u, :m] = acc
        if self.kv4 and m > 0:
            from oracle import kv_quant
            k_rows, v_rows = kv_quant.qdq(_f32(k_rows)), kv_quant.qdq(_f32(v_rows))
        self.K[u, :m] = k_rows
        self.V[u, :m] = v_rows

    # -- decode ----------------------------------------------------------
    def decode_step(self, q, k_new, v_new, hint: Optional[np.ndarray] = None, tie_rel: float = 1e-6, want_p: bool = False,
                    units: Optional[Sequence[int]] = None):
        """One step for all units (or the listed ones).  q, k_new, v_new: ``[batch, n_heads, d]``.

        Returns dict(out [units, group * d], evicted [units], status [units], gap [units], p [units, cap] or None).
        """
        qf = _f32(q).reshape(self.units, self.group * self.d)
        kf = _f32(k_new).reshape(self.units, self.d)
        vf = _f32(v_new).reshape(self.units, self.d)
        t_before = self.t.copy()
        if units is not None:
            res = self._decode_subset(qf, kf, vf, hint, tie_rel, want_p, list(units))
        else:
            res = self._decode(self, qf, kf, vf, hint, tie_rel, want_p)
        if self.kv4:  # the new token's row, if it was kept, is stored quantised from now on
            from oracle import kv_quant
            kq, vq = kv_quant.qdq(kf), kv_quant.qdq(vf)
            for u in (range(self.units) if units is None else units):
                m = int(self.cnt[u])
                hit = np.nonzero(self.pos[u, :m] == t_before[u])[0]
                if hit.size:
                    self.K[u, hit[0]] = kq[u]
                    self.V[u, hit[0]] = vq[u]
        return res

    @staticmethod
    def _decode(st, qf, kf, vf, hint, tie_rel, want_p):
        n = st.cnt.shape[0]
        out = np.empty((n, st.group * st.d), dtype=np.float64)
        evicted = np.empty(n, dtype=np.int32)
        status = np.empty(n, dtype=np.int32)
        gap = np.empty(n, dtype=np.float64)
        p = np.zeros((n, st.cap), dtype=np.float64) if want_p else None
        tgap = np.empty(n, dtype=np.float64)
        h = None if hint is None else np.ascontiguousarray(hint, dtype=np.int32)
        rc = _load().h2o_oracle_decode_step(
            n, st.group, st.d, st.cap, _p(st.kbud, ctypes.c_int32), _p(st.rwin, ctypes.c_int32), _p(st.t, ctypes.c_int32),
            _p(st.cnt, ctypes.c_int32), _p(st.pos, ctypes.c_int32), _p(st.acc, ctypes.c_double), _p(st.K, ctypes.c_double),
            _p(st.V, ctypes.c_double), _p(qf, ctypes.c_float), _p(kf, ctypes.c_float), _p(vf, ctypes.c_float), st.scale,
            _p(h, ctypes.c_int32), float(tie_rel), _p(out, ctypes.c_double), _p(evicted, ctypes.c_int32),
            _p(status, ctypes.c_int32), _p(gap, ctypes.c_double), _p(p, ctypes.c_double), _p(tgap, ctypes.c_double))
        if rc != 0:
            raise RuntimeError("oracle decode step failed: inconsistent state (%d)" % rc)
        return dict(out=out, evicted=evicted, status=status, gap=gap, p=p, topk_gap=tgap)

    def _decode_subset(self, qf, kf, vf, hint, tie_rel, want_p, units):
        """Step only some units: copy their state out, step, copy back (units are independent)."""
        idx = np.asarray(units, dtype=np.int64)

        class _S:
            pass

        st = _S()
        st.d, st.cap, st.scale, st.group = self.d, self.cap, self.scale, self.group
        for name in ("kbud", "rwin", "t", "cnt", "pos", "acc", "K", "V"):
            setattr(st, name, np.ascontiguousarray(getattr(self, name)[idx]))
        res = self._decode(st, np.ascontiguousarray(qf[idx]), np.ascontiguousarray(kf[idx]), np.ascontiguousarray(vf[idx]),
                           None if hint is None else np.asarray(hint)[idx], tie_rel, want_p)
        for name in ("t", "cnt", "pos", "acc", "K", "V"):
            getattr(self, name)[idx] = getattr(st, name)
        return res

    # -- inspection ------------------------------------------------------
    def export(self, u: int):
        """Positions (ascending) and their accumulated scores for unit ``u``."""
        m = int(self.cnt[u])
        order = np.argsort(self.pos[u, :m], kind="stable")
        return self.pos[u, :m][order].copy(), self.acc[u, :m][order].copy()

    def permute_entries(self, rng: np.random.Generator):
        """Shuffle the storage order of every unit's entries (semantics must not change)."""
        for u in range(self.units):
            m = int(self.cnt[u])
            perm = rng.permutation(m)
            for a in (self.pos, self.acc, self.K, self.V):
                a[u, :m] = a[u, :m][perm]
