"""GPU parity of the mass-signal options (Algorithm 1 step 1: optional smoothing of the usage
scores; the runtime section's decoupled mass and selection scores): the mass comes from the usage u,
the ranking inside a segment from the base score g.

Bit-exact whenever both sides start from the same fp32 arrays (the smoothing itself is a fixed
sequence of fp32 additions and one division on both sides); the scorers' outputs within 1e-3."""
import numpy as np
import pytest
import torch

import oracle
from helpers import HostSnapshot, assert_scores_close, compare_event, gpu_event
from paper_2605_23200_b200 import binding, inputs

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _small(cfg_id, **kw):
    base = dict(n_layers=2, batch=2, seq_len_min=1500, seq_len_max=1500, budget=384)
    base.update(kw)
    return inputs.CONFIGS[cfg_id].scaled(resident_layers=0, **base)


def _rand(wl, seed, kind):
    rng = np.random.default_rng(seed)
    shape = (wl.n_layers, wl.batch, wl.n_kv_heads, wl.max_seq_len)
    x = rng.standard_normal(shape)
    return (np.exp(2.0 * x) if kind == "lognormal" else x).astype(np.float32)


def _usage_rows_equal(dbg, snap, wl, want_fn):
    got = dbg.usage.cpu().numpy()
    for l in range(wl.n_layers):
        for b in range(wl.batch):
            T = int(snap.lens[b])
            if T <= wl.budget:
                continue
            for h in range(wl.n_kv_heads):
                assert (got[l, b, h, :T] == want_fn(l, b, h, T)).all(), (l, b, h)


@pytest.mark.parametrize("k,kw", [
    (3, dict()),
    (5, dict(seq_len_min=1000, seq_len_max=1777, batch=4, budget=1200)),                      # ragged; some skipped
    (9, dict(ema_beta=1.0, n_segments=7, q_min=3)),
    (63, dict(seq_len_min=20011, seq_len_max=20011, budget=3000, batch=1, n_layers=1)),       # two blocks per unit
    (7, dict(seq_len_min=3000, seq_len_max=3000, budget=700, l_min=1, l_max=5, n_segments=64, q_min=2)),
])
def test_smoothed_external_usage_bit_exact(k, kw):
    wl = _small(0, pool_kernel=k, **kw)
    cache = inputs.make_cache(wl, DEV)
    comp = binding.AmsCompressor(binding.config_for(wl), DEV)
    ext = _rand(wl, 99 + k, "lognormal")
    snap = HostSnapshot(cache)
    credit0 = comp.ema_state.cpu().numpy()
    dst = inputs.alloc_dst_pages(cache)
    dbg = gpu_event(comp, cache, dst, inputs.SCORER_EXTERNAL, torch.from_numpy(ext).to(DEV))
    assert comp.last_launch_count == 7           # validation, smoothing, three selection kernels, gather, table update
    _usage_rows_equal(dbg, snap, wl, lambda l, b, h, T: oracle.smooth_usage(ext[l, b, h, :T], k))
    compare_event(snap, cache, comp, dbg, dst, credit0, ext, pool_kernel=k)


@pytest.mark.parametrize("k", [1, 5])
def test_external_usage_separate_from_base_scores(k):
    wl = _small(0, pool_kernel=k, batch=3, seq_len_min=900, seq_len_max=2000)
    cache = inputs.make_cache(wl, DEV)
    comp = binding.AmsCompressor(binding.config_for(wl), DEV)
    g = _rand(wl, 5, "signed")
    u = _rand(wl, 6, "lognormal")
    snap = HostSnapshot(cache)
    credit0 = comp.ema_state.cpu().numpy()
    dst = inputs.alloc_dst_pages(cache)
    dbg = gpu_event(comp, cache, dst, inputs.SCORER_EXTERNAL, torch.from_numpy(g).to(DEV),
                    ext_usage=torch.from_numpy(u).to(DEV))
    assert (dbg.scores.cpu().numpy() == g).all()
    res = compare_event(snap, cache, comp, dbg, dst, credit0, g, usage_for_oracle=u, pool_kernel=k)
    # the two signals really play different roles: with u alone the kept sets differ
    alone = oracle.compress(snap.k.copy(), snap.v.copy(), snap.table.copy(), snap.lens.copy(), None, credit0.copy(),
                            wl.budget, oracle.Params(wl.n_segments, wl.l_min, wl.l_max, wl.q_min, wl.n_sink, wl.n_last,
                                                     wl.ema_lambda, wl.ema_beta, wl.eps),
                            oracle.SCORER_EXTERNAL, dst, ext_scores=u, units=[(0, 0, 0)], pool_kernel=k)
    assert (alone[(0, 0, 0)].bounds == res[(0, 0, 0)].bounds).all()
    assert (alone[(0, 0, 0)].keep_idx != res[(0, 0, 0)].keep_idx).any()


@pytest.mark.parametrize("k,window", [(1, 32), (5, 8), (3, 1)])
def test_tova_with_smoothed_mass(k, window):
    wl = _small(1, n_layers=1, pool_kernel=k, window=window, seq_len_min=2100, seq_len_max=2100, budget=256)
    cache = inputs.make_cache(wl, DEV)
    comp = binding.AmsCompressor(binding.config_for(wl), DEV)
    snap = HostSnapshot(cache)
    credit0 = comp.ema_state.cpu().numpy()
    dst = inputs.alloc_dst_pages(cache)
    dbg = gpu_event(comp, cache, dst)
    got = dbg.scores.cpu().numpy()
    G, T = wl.group, 2100
    for l in range(wl.n_layers):
        for b in range(wl.batch):
            for h in range(wl.n_kv_heads):
                want = oracle.score_tova(snap.k, l, h, snap.table[b], T, snap.q[l, b, h * G:(h + 1) * G], G, wl.window, True)
                assert_scores_close(got[l, b, h, :T], want, 1e-3, 0.0)
    # the usage is the smoothed copy of the library's own scores, bit for bit; g stays as scored
    _usage_rows_equal(dbg, snap, wl, lambda l, b, h, T: oracle.smooth_usage(got[l, b, h, :T], k))
    compare_event(snap, cache, comp, dbg, dst, credit0, got, pool_kernel=k)


@pytest.mark.parametrize("k", [1, 5])
def test_keydiff_ranking_with_window_attention_mass(k):
    wl = _small(3, n_layers=2, batch=3, seq_len_min=900, seq_len_max=2000, budget=256, n_segments=16, l_max=250,
                window=8, decoupled=True, pool_kernel=k)
    cache = inputs.make_cache(wl, DEV)
    assert cache.obs_queries is not None
    comp = binding.AmsCompressor(binding.config_for(wl), DEV)
    snap = HostSnapshot(cache)
    credit0 = comp.ema_state.cpu().numpy()
    dst = inputs.alloc_dst_pages(cache)
    dbg = gpu_event(comp, cache, dst)
    g_got = dbg.scores.cpu().numpy()
    u_got = dbg.usage.cpu().numpy()
    G = wl.group
    for l in range(wl.n_layers):
        for b in range(wl.batch):
            T = int(snap.lens[b])
            if T <= wl.budget:
                continue
            for h in range(wl.n_kv_heads):
                g_want = oracle.score_keydiff(snap.k, l, h, snap.table[b], T)
                assert_scores_close(g_got[l, b, h, :T], g_want, 1e-3, 1e-5)
                u_want = oracle.smooth_usage(
                    oracle.score_tova(snap.k, l, h, snap.table[b], T, snap.q[l, b, h * G:(h + 1) * G], G, wl.window, True), k)
                assert_scores_close(u_got[l, b, h, :T], u_want, 1e-3, 0.0)
    # on the library's own two signals the oracle takes the same decisions
    compare_event(snap, cache, comp, dbg, dst, credit0, g_got, usage_for_oracle=u_got, pool_kernel=1)
    # without the flag the queries are ignored and the key-only score is also the mass signal
    wl0 = wl.scaled(decoupled=False, pool_kernel=1)
    cache0 = inputs.make_cache(wl0, DEV)
    comp0 = binding.AmsCompressor(binding.config_for(wl0), DEV)
    dbg0 = gpu_event(comp0, cache0, inputs.alloc_dst_pages(cache0))
    assert torch.equal(dbg0.scores, dbg0.usage)
    for b in range(wl.batch):                       # positions beyond a sequence's length are never written
        T = int(snap.lens[b])
        if T > wl.budget:
            assert torch.equal(dbg0.scores[:, b, :, :T], dbg.scores[:, b, :, :T])


def test_mass_signal_argument_errors():
    wl = _small(0)
    for bad in (0, 2, 65, -3):
        with pytest.raises(binding.AmsError):
            binding.AmsCompressor(binding.config_for(wl.scaled(pool_kernel=bad)), DEV)
    cache = inputs.make_cache(wl, DEV)
    comp = binding.AmsCompressor(binding.config_for(wl), DEV)
    dst = torch.from_numpy(inputs.alloc_dst_pages(cache)).to(DEV)
    stray = torch.zeros((wl.n_layers, wl.batch, wl.n_kv_heads, wl.max_seq_len), device=DEV)
    with pytest.raises(binding.AmsError):     # a usage array only goes with external scores
        comp.compress(cache.k_pages, cache.v_pages, cache.block_table, cache.seq_lens, cache.obs_queries, wl.budget,
                      wl.n_segments, inputs.SCORER_TOVA, dst, ext_usage=stray)
