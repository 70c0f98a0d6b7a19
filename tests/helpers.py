"""Shared plumbing of the GPU parity tests: run one event through libams and through the
oracle on the same bytes and compare."""
from __future__ import annotations

import numpy as np
import torch

import oracle
from paper_2605_23200_b200 import binding, inputs


def params_of(wl) -> oracle.Params:
    return oracle.Params(wl.n_segments, wl.l_min, wl.l_max, wl.q_min, wl.n_sink, wl.n_last, wl.ema_lambda,
                         wl.ema_beta, wl.eps, wl.fixed_segments, wl.uniform_quotas)


class HostSnapshot:
    """Host copies (numpy) of everything an event reads, taken before the GPU call."""

    def __init__(self, cache: inputs.Cache):
        self.k = inputs.as_u16(cache.k_pages)
        self.v = inputs.as_u16(cache.v_pages)
        self.table = cache.block_table.cpu().numpy().copy()
        self.lens = cache.seq_lens.cpu().numpy().copy()
        self.q = None if cache.obs_queries is None else inputs.as_u16(cache.obs_queries)


def gpu_event(comp: binding.AmsCompressor, cache: inputs.Cache, dst_pages: np.ndarray, scorer_id=None,
              ext_scores=None, want_dbg=True, ext_usage=None):
    wl = cache.wl
    dst = torch.from_numpy(dst_pages).to(cache.k_pages.device)
    dbg = comp.make_debug_views(wl.batch, wl.budget) if want_dbg else None
    sid = wl.scorer_id if scorer_id is None else scorer_id
    q = cache.obs_queries if (sid == inputs.SCORER_TOVA or wl.decoupled) else None
    comp.compress(cache.k_pages, cache.v_pages, cache.block_table, cache.seq_lens, q, wl.budget, wl.n_segments,
                  sid, dst, ext_scores=ext_scores, ext_usage=ext_usage, dbg=dbg)
    comp.status()
    return dbg


def compare_event(snap: HostSnapshot, cache: inputs.Cache, comp: binding.AmsCompressor, dbg, dst_pages, credit_before,
                  scores_for_oracle, units=None, check_bytes=True, usage_for_oracle=None, pool_kernel=1):
    """Oracle on `scores_for_oracle` (float32 [L][B][H][T_cap]; optionally a separate usage signal, smoothed by
    the oracle itself with `pool_kernel`) must reproduce the library's segments, quotas, keep indices, mass,
    credit, compacted bytes, block table and lengths exactly."""
    wl = cache.wl
    prm = params_of(wl)
    k, v = snap.k.copy(), snap.v.copy()
    table, lens = snap.table.copy(), snap.lens.copy()
    credit = credit_before.copy()
    res = oracle.compress(k, v, table, lens, None, credit, wl.budget, prm, oracle.SCORER_EXTERNAL, dst_pages,
                          ext_scores=scores_for_oracle, units=units, threads=8, ext_usage=usage_for_oracle,
                          pool_kernel=pool_kernel)
    n_seg = dbg.n_segments.cpu().numpy()
    bounds = dbg.seg_bounds.cpu().numpy()
    quotas = dbg.quotas.cpu().numpy()
    keep = dbg.keep_idx.cpu().numpy()
    mass = dbg.mass.cpu().numpy()
    for (l, b, h), r in res.items():
        T = int(snap.lens[b])
        assert n_seg[l, b, h] == r.n_seg, (l, b, h, n_seg[l, b, h], r.n_seg)
        assert bounds[l, b, h, : r.n_seg + 1].tolist() == r.bounds.tolist(), (l, b, h)
        assert quotas[l, b, h, : r.n_seg].tolist() == r.quotas.tolist(), (l, b, h)
        assert (keep[l, b, h] == r.keep_idx).all(), (l, b, h)
        assert (mass[l, b, h, :T] == r.mass).all(), (l, b, h)
    if wl.ema_beta != 1.0:
        got = comp.ema_state.cpu().numpy()
        for (l, b, h) in res:
            assert (got[l, b, h] == credit[l, b, h]).all(), (l, b, h)
    if check_bytes and units is None:
        assert (inputs.as_u16(cache.k_pages) == k).all()
        assert (inputs.as_u16(cache.v_pages) == v).all()
        assert (cache.block_table.cpu().numpy() == table).all()
        assert (cache.seq_lens.cpu().numpy() == lens).all()
    return res


def assert_scores_close(got, want, rtol=1e-3, atol=0.0):
    got = np.asarray(got, np.float64)
    want = np.asarray(want, np.float64)
    err = np.abs(got - want)
    tol = rtol * np.abs(want) + atol
    bad = err > tol
    assert not bad.any(), f"max rel err {np.max(err / np.maximum(np.abs(want), 1e-300)):.3e} at {np.argmax(err - tol)}"
