"""CPU oracle for the AMS compression step: Python face of ``ams_oracle.c``.

TEST INFRASTRUCTURE ONLY.  Nothing in the product path may import this package;
only the tests, the smoke check and the benchmark's CPU-baseline leg do.  It
shares no code with the CUDA library: it takes numpy arrays (bf16 as uint16 bit
patterns), calls the plain C functions, and returns numpy arrays.

Each function below names the passage of the paper that its C counterpart
follows; the arithmetic itself lives in ``ams_oracle.c``.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ams_oracle.c")
_LIB = os.path.join(_HERE, "libams_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no fast-math, no FMA contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fno-fast-math", "-fPIC", "-shared",
               "-Wall", "-Wextra", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


class _Params(ctypes.Structure):
    _fields_ = [("n_segments", ctypes.c_int32), ("l_min", ctypes.c_int32), ("l_max", ctypes.c_int32),
                ("q_min", ctypes.c_int32), ("n_sink", ctypes.c_int32), ("n_last", ctypes.c_int32),
                ("ema_lambda", ctypes.c_float), ("ema_beta", ctypes.c_float), ("eps", ctypes.c_float),
                ("fixed_segments", ctypes.c_int32), ("uniform_quotas", ctypes.c_int32)]


@dataclass
class Params:
    """Hyper-parameters of one event (defaults: the paper's hyper-parameter table;
    n_last and eps are readings, the table gives neither)."""
    n_segments: int = 10
    l_min: int = 16
    l_max: int = 256
    q_min: int = 1
    n_sink: int = 4
    n_last: int = 16
    ema_lambda: float = 0.9
    ema_beta: float = 0.9
    eps: float = 1e-8
    fixed_segments: bool = False    # ablation: equal-length instead of equal-mass segments
    uniform_quotas: bool = False    # ablation: budget shared by segment length instead of mass

    def c(self) -> _Params:
        return _Params(self.n_segments, self.l_min, self.l_max, self.q_min, self.n_sink, self.n_last,
                       self.ema_lambda, self.ema_beta, self.eps, int(self.fixed_segments), int(self.uniform_quotas))

    def max_segments(self, T: int) -> int:
        cap = self.n_segments
        if self.l_max > 0:
            cap += 2 * (T // self.l_max) + 2
        return cap + 2


def _p(a, ty):
    return a.ctypes.data_as(ctypes.POINTER(ty))


def lib():
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(_LIB)
        _lib.orc_select_unit.restype = ctypes.c_int32
        _lib.orc_cuts.restype = ctypes.c_int32
        _lib.orc_merge_split.restype = ctypes.c_int32
        _lib.orc_select.restype = ctypes.c_int32
        _lib.orc_score_tova.restype = ctypes.c_int
        _lib.orc_score_keydiff.restype = ctypes.c_int
        _lib.orc_score_expected.restype = ctypes.c_int
    return _lib


def _f32(a):
    return np.ascontiguousarray(a, dtype=np.float32)


def _i32(a):
    return np.ascontiguousarray(a, dtype=np.int32)


# --------------------------------------------------------------------------- scorers

def score_tova(k_pages, layer, h, table_row, T, q_rows, G, W, causal=True):
    """Observation-window usage u_t (Section 3.2, Algorithm 1 step 1).
    k_pages: uint16 [L][P][page][H][D]; q_rows: uint16 [G][W][D]."""
    L, P, page, H, D = k_pages.shape
    table_row = _i32(table_row)
    q_rows = np.ascontiguousarray(q_rows, dtype=np.uint16)
    assert q_rows.shape == (G, W, D)
    out = np.empty(T, dtype=np.float32)
    rc = lib().orc_score_tova(_p(k_pages, ctypes.c_uint16), ctypes.c_int64(P), ctypes.c_int32(page),
                              ctypes.c_int32(H), ctypes.c_int32(D), ctypes.c_int32(layer),
                              ctypes.c_int32(h), _p(table_row, ctypes.c_int32), ctypes.c_int32(T),
                              _p(q_rows, ctypes.c_uint16), ctypes.c_int32(G), ctypes.c_int32(W),
                              ctypes.c_int32(1 if causal else 0), _p(out, ctypes.c_float))
    if rc != 0:
        raise ValueError(f"orc_score_tova failed: {rc}")
    return out


def score_keydiff(k_pages, layer, h, table_row, T):
    """Key-only score: negative cosine similarity to the per-head mean key."""
    L, P, page, H, D = k_pages.shape
    table_row = _i32(table_row)
    out = np.empty(T, dtype=np.float32)
    rc = lib().orc_score_keydiff(_p(k_pages, ctypes.c_uint16), ctypes.c_int64(P), ctypes.c_int32(page),
                                 ctypes.c_int32(H), ctypes.c_int32(D), ctypes.c_int32(layer),
                                 ctypes.c_int32(h), _p(table_row, ctypes.c_int32), ctypes.c_int32(T),
                                 _p(out, ctypes.c_float))
    if rc != 0:
        raise ValueError(f"orc_score_keydiff failed: {rc}")
    return out


def score_expected(k_pages, v_pages, layer, h, table_row, T, mean, cov, eps):
    """Expected-attention score of one (layer, sequence, KV head): Gaussian closed form of the
    expected attention weight per query head of the group, softmax over the tokens, group
    mean, (+ eps) times the value norm (the scorer of the paper's "AMS-Expected" rows; the
    formula is a reading, see ams_oracle.c).  mean: float32 [G][D]; cov: uint16 (bf16) [G][D][D]."""
    L, P, page, H, D = k_pages.shape
    table_row = _i32(table_row)
    mean = _f32(mean)
    cov = np.ascontiguousarray(cov, dtype=np.uint16)
    G = mean.shape[0]
    assert mean.shape == (G, D) and cov.shape == (G, D, D)
    out = np.empty(T, dtype=np.float32)
    rc = lib().orc_score_expected(_p(k_pages, ctypes.c_uint16), _p(v_pages, ctypes.c_uint16), ctypes.c_int64(P),
                                  ctypes.c_int32(page), ctypes.c_int32(H), ctypes.c_int32(D), ctypes.c_int32(layer),
                                  ctypes.c_int32(h), _p(table_row, ctypes.c_int32), ctypes.c_int32(T),
                                  _p(mean, ctypes.c_float), _p(cov, ctypes.c_uint16), ctypes.c_int32(G),
                                  ctypes.c_float(eps), _p(out, ctypes.c_float))
    if rc != 0:
        raise ValueError(f"orc_score_expected failed: {rc}")
    return out


# --------------------------------------------------------------------------- stages

def smooth_usage(u, k):
    """Zero-padded 1-D average pooling of the usage scores, window k (odd), stride 1
    (Algorithm 1 step 1, optional smoothing)."""
    u = _f32(u)
    if k < 1 or k % 2 == 0:
        raise ValueError("pool kernel must be odd and >= 1")
    out = np.empty_like(u)
    lib().orc_smooth_usage(_p(u, ctypes.c_float), ctypes.c_int32(u.shape[0]), ctypes.c_int32(k),
                           _p(out, ctypes.c_float))
    return out


def mass(u, eps):
    """Eq. 1 on fixed-point weights.  Returns (A uint64[T], SA, m float32[T])."""
    u = _f32(u)
    T = u.shape[0]
    A = np.empty(T, dtype=np.uint64)
    SA = ctypes.c_uint64(0)
    m = np.empty(T, dtype=np.float32)
    lib().orc_mass(_p(u, ctypes.c_float), ctypes.c_int32(T), ctypes.c_float(eps),
                   _p(A, ctypes.c_uint64), ctypes.byref(SA), _p(m, ctypes.c_float))
    return A, int(SA.value), m


def history_mass(A, SA, m, credit, lam, beta):
    """EMA credit update and mixed mass (Algorithm 1 step 2).  Returns (Hm, credit_new)."""
    T = A.shape[0]
    credit = _f32(credit).copy()
    Hm = np.empty(T, dtype=np.uint64)
    lib().orc_history_mass(_p(A, ctypes.c_uint64), ctypes.c_uint64(SA), _p(_f32(m), ctypes.c_float),
                           _p(credit, ctypes.c_float), ctypes.c_int32(T), ctypes.c_float(lam),
                           ctypes.c_float(beta), _p(Hm, ctypes.c_uint64))
    return Hm, credit


def prefix(Hm):
    Hm = np.ascontiguousarray(Hm, dtype=np.uint64)
    C = np.empty_like(Hm)
    lib().orc_prefix(_p(Hm, ctypes.c_uint64), ctypes.c_int32(Hm.shape[0]), _p(C, ctypes.c_uint64))
    return C


def cuts(C, S):
    """Mass-quantile boundaries (Section 3.3 first paragraph; Algorithm 1 step 3)."""
    C = np.ascontiguousarray(C, dtype=np.uint64)
    b = np.empty(S + 1, dtype=np.int32)
    n = lib().orc_cuts(_p(C, ctypes.c_uint64), ctypes.c_int32(C.shape[0]), ctypes.c_int32(S),
                       _p(b, ctypes.c_int32))
    return b[:n].copy()


def merge_split(raw, l_min, l_max):
    raw = _i32(raw)
    T = int(raw[-1])
    cap = len(raw) + (2 * (T // l_max) + 2 if l_max > 0 else 0) + 2
    out = np.empty(cap, dtype=np.int32)
    n = lib().orc_merge_split(_p(raw, ctypes.c_int32), ctypes.c_int32(len(raw)), ctypes.c_int32(l_min),
                              ctypes.c_int32(l_max), _p(out, ctypes.c_int32), ctypes.c_int32(cap))
    if n < 0:
        raise ValueError("merge_split capacity")
    return out[:n].copy()


def must_keep(T, Tk, n_sink, n_last):
    ns, nl = ctypes.c_int32(0), ctypes.c_int32(0)
    lib().orc_must_keep(ctypes.c_int32(T), ctypes.c_int32(Tk), ctypes.c_int32(n_sink),
                        ctypes.c_int32(n_last), ctypes.byref(ns), ctypes.byref(nl))
    return int(ns.value), int(nl.value)


def quotas(C, bounds, q_min, Bq):
    """Segment quotas (Section 3.3 quota paragraph; Algorithm 1 step 4)."""
    C = np.ascontiguousarray(C, dtype=np.uint64)
    bounds = _i32(bounds)
    n_seg = len(bounds) - 1
    q = np.empty(n_seg, dtype=np.int32)
    lib().orc_quotas(_p(C, ctypes.c_uint64), _p(bounds, ctypes.c_int32), ctypes.c_int32(n_seg),
                     ctypes.c_int32(q_min), ctypes.c_int32(Bq), _p(q, ctypes.c_int32))
    return q


def select(g, bounds, q, ns, nl, Tk):
    """Per-segment top-q_i, must-keep union, backfill (Algorithm 1 step 5)."""
    g = _f32(g)
    bounds = _i32(bounds)
    q = _i32(q)
    keep = np.empty(Tk, dtype=np.int32)
    r = lib().orc_select(_p(g, ctypes.c_float), ctypes.c_int32(g.shape[0]), _p(bounds, ctypes.c_int32),
                         _p(q, ctypes.c_int32), ctypes.c_int32(len(q)), ctypes.c_int32(ns),
                         ctypes.c_int32(nl), ctypes.c_int32(Tk), _p(keep, ctypes.c_int32))
    if r < 0:
        raise ValueError("select: keep set larger than the budget")
    return keep, r


@dataclass
class UnitResult:
    n_seg: int
    mass: np.ndarray
    raw_bounds: np.ndarray
    bounds: np.ndarray
    quotas: np.ndarray
    keep_idx: np.ndarray
    credit: np.ndarray
    n_backfill: int


def select_unit(u, g, credit, Tk, prm: Params) -> UnitResult:
    """Algorithm 1 steps 1-5 for one (layer, sequence, KV head)."""
    u = _f32(u)
    g = u if g is None else _f32(g)
    T = u.shape[0]
    credit = np.zeros(T, np.float32) if credit is None else _f32(credit).copy()
    assert credit.shape[0] >= T
    cap = prm.max_segments(T)
    m = np.empty(T, np.float32)
    raw = np.empty(prm.n_segments + 1, np.int32)
    n_raw = ctypes.c_int32(0)
    bounds = np.empty(cap + 1, np.int32)
    q = np.empty(cap, np.int32)
    keep = np.empty(Tk, np.int32)
    nbf = ctypes.c_int32(0)
    cp = prm.c()
    n_seg = lib().orc_select_unit(_p(u, ctypes.c_float), _p(g, ctypes.c_float), _p(credit, ctypes.c_float),
                                  ctypes.c_int32(T), ctypes.c_int32(Tk), ctypes.byref(cp),
                                  ctypes.c_int32(cap), _p(m, ctypes.c_float), _p(raw, ctypes.c_int32),
                                  ctypes.byref(n_raw), _p(bounds, ctypes.c_int32), _p(q, ctypes.c_int32),
                                  _p(keep, ctypes.c_int32), ctypes.byref(nbf))
    if n_seg < 0:
        raise ValueError(f"orc_select_unit failed: {n_seg}")
    return UnitResult(n_seg, m, raw[:n_raw.value].copy(), bounds[:n_seg + 1].copy(), q[:n_seg].copy(),
                      keep, credit, int(nbf.value))


def gather_unit(k_pages, v_pages, layer, h, table_row, dst_row, keep_idx):
    """Paged head-wise compaction of one head (paged-compaction appendix). In place on the arrays."""
    L, P, page, H, D = k_pages.shape
    assert k_pages.flags.c_contiguous and v_pages.flags.c_contiguous
    table_row, dst_row, keep_idx = _i32(table_row), _i32(dst_row), _i32(keep_idx)
    lib().orc_gather_unit(_p(k_pages, ctypes.c_uint16), _p(v_pages, ctypes.c_uint16), ctypes.c_int64(P),
                          ctypes.c_int32(page), ctypes.c_int32(H), ctypes.c_int32(D),
                          ctypes.c_int32(layer), ctypes.c_int32(h), _p(table_row, ctypes.c_int32),
                          _p(dst_row, ctypes.c_int32), _p(keep_idx, ctypes.c_int32),
                          ctypes.c_int32(len(keep_idx)))


def retained_iou(keep_idx, prev_kept, budget):
    """Retained-set IoU between two consecutive compression events of one (layer, sequence, KV
    head) (mechanistic-diagnostics appendix): the previous event left its `prev_kept` retained
    tokens at positions [0, prev_kept) of the cache; `keep_idx` are the positions this event keeps.
    IoU = |R_prev & R_now| / |R_prev | R_now| on token identities; float32."""
    prev = set(range(int(prev_kept)))
    now = set(int(t) for t in keep_idx[:budget])
    union = len(prev | now)
    return np.float32(0.0) if union == 0 else np.float32(len(prev & now)) / np.float32(union)


# --------------------------------------------------------------------------- whole event

SCORER_TOVA, SCORER_KEYDIFF, SCORER_EXTERNAL, SCORER_EXPECTED = 0, 1, 2, 3


def compress(k_pages, v_pages, block_table, seq_lens, obs_queries, credit, budget, prm: Params,
             scorer_id, dst_pages, *, n_q_heads=None, causal=True, ext_scores=None, units=None,
             do_gather=True, threads=1, pool_kernel=1, decoupled=False, ext_usage=None, q_mean=None, q_cov=None,
             score_eps=1e-2):
    """One compression event over every layer, sequence and KV head.

    k_pages / v_pages: uint16 [L][P][page][H][D] (modified: kept rows are written into
    the pages named by dst_pages); block_table int32 [B][max_pages] and seq_lens int32 [B]
    (rewritten as the event leaves them); obs_queries uint16 [L][B][Hq][W][D] or None;
    credit float32 [L][B][H][T_cap] (updated in place); ext_scores float32 like credit for
    SCORER_EXTERNAL.  `units`: optional subset of (layer, b, h) to compute (for sampling);
    the table update is skipped then.

    Mass signal: by default the usage u that defines the mass is the scorer's score g.
    `decoupled` (SCORER_KEYDIFF with observation queries): u = window attention, g = key-only
    score.  `ext_usage` (SCORER_EXTERNAL): u given separately from g.  `pool_kernel` > 1
    smooths u (never g) before Eq. 1.  Returns {(layer,b,h): UnitResult} with `.scores` (g)
    and `.usage` (u after smoothing)."""
    L, P, page, H, D = k_pages.shape
    B = seq_lens.shape[0]
    T_cap = credit.shape[-1]
    todo = units if units is not None else [(l, b, h) for l in range(L) for b in range(B) for h in range(H)]
    todo = [(l, b, h) for (l, b, h) in todo if int(seq_lens[b]) > budget]
    G = (n_q_heads // H) if n_q_heads else None

    def one(unit):
        l, b, h = unit
        T = int(seq_lens[b])
        u = None
        if scorer_id == SCORER_TOVA:
            W = obs_queries.shape[3]
            s = score_tova(k_pages, l, h, block_table[b], T, obs_queries[l, b, h * G:(h + 1) * G], G, W, causal)
        elif scorer_id == SCORER_KEYDIFF:
            s = score_keydiff(k_pages, l, h, block_table[b], T)
            if decoupled:
                W = obs_queries.shape[3]
                u = score_tova(k_pages, l, h, block_table[b], T, obs_queries[l, b, h * G:(h + 1) * G], G, W, causal)
        elif scorer_id == SCORER_EXPECTED:
            s = score_expected(k_pages, v_pages, l, h, block_table[b], T, q_mean[l, b, h * G:(h + 1) * G],
                               q_cov[l, b, h * G:(h + 1) * G], score_eps)
            if decoupled and obs_queries is not None:
                W = obs_queries.shape[3]
                u = score_tova(k_pages, l, h, block_table[b], T, obs_queries[l, b, h * G:(h + 1) * G], G, W, causal)
        else:
            s = _f32(ext_scores[l, b, h, :T])
            if ext_usage is not None:
                u = _f32(ext_usage[l, b, h, :T])
        u = s if u is None else u
        if pool_kernel > 1:
            u = smooth_usage(u, pool_kernel)
        res = select_unit(u, s, credit[l, b, h, :T], budget, prm)
        res.scores = s
        res.usage = u
        return unit, res

    if threads > 1:
        with ThreadPoolExecutor(threads) as ex:
            results = dict(ex.map(one, todo))
    else:
        results = dict(map(one, todo))
    for (l, b, h), res in results.items():
        T = int(seq_lens[b])
        if prm.ema_beta != 1.0:
            credit[l, b, h, :T] = res.credit
        if do_gather:
            gather_unit(k_pages, v_pages, l, h, block_table[b], dst_pages[b], res.keep_idx)
    if units is None:
        n_dst = (budget + page - 1) // page
        for b in range(B):
            if int(seq_lens[b]) > budget:
                block_table[b, :] = -1
                block_table[b, :n_dst] = dst_pages[b, :n_dst]
                seq_lens[b] = budget
    return results
