"""Parity on the other benchmark configurations, each at its true per-unit geometry (sequence
lengths, budget, observation window, query group, segment settings, scorer) with fewer layers
and sequences where the oracle would otherwise take minutes.  Configurations with decode steps
run two consecutive events with appended tokens in between, so that the EMA credit carried in
compacted order and the rewritten block table feed the second event.

Per event: sampled units' scores and mass against the oracle within 1e-3 relative, and on the
library's own scores the oracle must reproduce segments, quotas, kept indices, mass and credit
exactly."""
import numpy as np
import pytest

import oracle
from helpers import HostSnapshot, assert_scores_close, compare_event, gpu_event
from paper_2605_23200_b200 import binding, inputs

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _event(wl, cache, comp, sample, atol=0.0):
    snap = HostSnapshot(cache)
    credit0 = comp.ema_state.cpu().numpy()
    dst = inputs.alloc_dst_pages(cache)
    dbg = gpu_event(comp, cache, dst)
    got = dbg.scores.cpu().numpy()
    mass = dbg.mass.cpu().numpy()
    G = wl.group
    units = []
    for (l, b, h) in sample:
        T = int(snap.lens[b])
        if T <= wl.budget:
            continue
        units.append((l, b, h))
        if wl.scorer_id == inputs.SCORER_TOVA:
            want = oracle.score_tova(snap.k, l, h, snap.table[b], T, snap.q[l, b, h * G:(h + 1) * G], G, wl.window, True)
        else:
            want = oracle.score_keydiff(snap.k, l, h, snap.table[b], T)
        assert_scores_close(got[l, b, h, :T], want, 1e-3, atol)
        _, _, m_want = oracle.mass(want, wl.eps)
        # an absolute slack on a score is that slack over the sum of the weights on its mass (Eq. 1)
        sum_w = float(np.maximum(want.astype(np.float64), 0.0).sum() + wl.eps * T)
        assert_scores_close(mass[l, b, h, :T], m_want, 1e-3, 1e-3 * wl.eps + atol / sum_w)
    assert units
    compare_event(snap, cache, comp, dbg, dst, credit0, got, units=units)
    assert (cache.seq_lens.cpu().numpy()[snap.lens > wl.budget] == wl.budget).all()
    inputs.after_compress(cache, dst)


def test_config0_whole_workload():
    wl = inputs.CONFIGS[0]
    cache = inputs.make_cache(wl, DEV)
    comp = binding.AmsCompressor(binding.config_for(wl), DEV)
    _event(wl, cache, comp, [(0, 0, h) for h in range(wl.n_kv_heads)])


def test_config2_geometry_two_events():
    """Ragged batch (8192..32768 tokens), group of 7 query heads, window 1, EMA on."""
    wl = inputs.CONFIGS[2].scaled(n_layers=1, batch=4, resident_layers=0, steps=2)
    cache = inputs.make_cache(wl, DEV)
    comp = binding.AmsCompressor(binding.config_for(wl), DEV)
    _event(wl, cache, comp, [(0, 0, 0), (0, 1, 3), (0, 2, 1), (0, 3, 2)])
    inputs.append_tokens(cache, wl.append_per_step)
    _event(wl, cache, comp, [(0, 0, 1), (0, 2, 3), (0, 3, 0)])


def test_config3_geometry():
    """KeyDiff scorer, 32768 tokens, 16 segments with split length 4096, no EMA."""
    wl = inputs.CONFIGS[3].scaled(n_layers=1, batch=2, resident_layers=0)
    cache = inputs.make_cache(wl, DEV)
    comp = binding.AmsCompressor(binding.config_for(wl), DEV)
    _event(wl, cache, comp, [(0, 0, 0), (0, 1, 5), (0, 1, 7)], atol=1e-5)


def test_config4_geometry_two_events():
    """131072 tokens, window 64 x group 8 = 512 query rows, 32 segments, EMA on."""
    wl = inputs.CONFIGS[4].scaled(n_layers=1, resident_layers=0, steps=2)
    cache = inputs.make_cache(wl, DEV)
    comp = binding.AmsCompressor(binding.config_for(wl), DEV)
    _event(wl, cache, comp, [(0, 0, 2)])
    inputs.append_tokens(cache, wl.append_per_step)
    _event(wl, cache, comp, [(0, 0, 5)])
