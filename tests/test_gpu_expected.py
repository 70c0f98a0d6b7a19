"""GPU parity of the expected-attention scorer (the scorer of the paper's "AMS-Expected" rows): the
library's scores against the oracle's within 1e-3, then every decision of the event (segments, quotas,
kept positions, credit, compacted bytes, table) bit-exact with the oracle selecting on the library's scores."""
import numpy as np
import pytest
import torch

import oracle
from helpers import HostSnapshot, assert_scores_close, compare_event, gpu_event
from paper_2605_23200_b200 import binding, inputs

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
EPS = 1e-2


def _wl(**kw):
    base = dict(n_layers=2, n_q_heads=8, n_kv_heads=2, batch=2, seq_len_min=1500, seq_len_max=1500, budget=384,
                window=0, scorer_id=inputs.SCORER_EXPECTED, resident_layers=0)
    base.update(kw)
    return inputs.CONFIGS[1].scaled(**base)


def _oracle_scores(snap, wl, mean, cov, units):
    G = wl.group
    out = {}
    for (l, b, h) in units:
        T = int(snap.lens[b])
        out[(l, b, h)] = oracle.score_expected(snap.k, snap.v, l, h, snap.table[b], T, mean[l, b, h * G:(h + 1) * G],
                                               cov[l, b, h * G:(h + 1) * G], EPS)
    return out


def _run(wl, units=None, seed_shift=0):
    cache = inputs.make_cache(wl, DEV)
    comp = binding.AmsCompressor(binding.config_for(wl), DEV)
    mean, cov = inputs.make_query_stats(cache)
    comp.set_query_stats(mean, cov, EPS)
    snap = HostSnapshot(cache)
    credit0 = comp.ema_state.cpu().numpy()
    dst = inputs.alloc_dst_pages(cache)
    dbg = gpu_event(comp, cache, dst)
    got = dbg.scores.cpu().numpy()
    if units is None:
        units = [(l, b, h) for l in range(wl.n_layers) for b in range(wl.batch) for h in range(wl.n_kv_heads)
                 if int(snap.lens[b]) > wl.budget]
    want = _oracle_scores(snap, wl, mean.cpu().numpy(), inputs.as_u16(cov), units)
    for (l, b, h), w in want.items():
        T = int(snap.lens[b])
        assert_scores_close(got[l, b, h, :T], w, rtol=1e-3)
    return cache, comp, snap, credit0, dst, dbg, got, units


@pytest.mark.parametrize("kw", [
    dict(),                                                                    # group of four: one launch, two K stages
    dict(n_q_heads=2),                                                         # one head per group, four K stages
    dict(n_q_heads=4),                                                         # two heads
    dict(n_q_heads=6, batch=1),                                                # three heads
    dict(n_q_heads=16, batch=1, n_layers=1),                                   # group of eight: two launches over K
    dict(seq_len_min=700, seq_len_max=2900, batch=4, budget=1000),             # ragged, some within the budget
    dict(n_kv_heads=8, n_q_heads=32, n_layers=1, batch=1, seq_len_min=4100, seq_len_max=4100, budget=512),
    dict(seq_len_min=129, seq_len_max=129, budget=64, batch=1, n_layers=1),    # a tile and one token
])
def test_expected_scores_and_event(kw):
    wl = _wl(**kw)
    cache, comp, snap, credit0, dst, dbg, got, units = _run(wl)
    assert comp.last_launch_count == 8 + (1 if wl.group > 4 else 0)   # validation, scorer (one launch per four heads of the group), scores, three selection kernels, gather, table update
    compare_event(snap, cache, comp, dbg, dst, credit0, got)


def test_expected_long_sequence_several_blocks_per_unit():
    """Twenty thousand tokens: a unit is shared by several blocks, whose running statistics are merged."""
    wl = _wl(n_layers=1, batch=1, n_kv_heads=2, n_q_heads=8, seq_len_min=20011, seq_len_max=20011, budget=2048)
    cache, comp, snap, credit0, dst, dbg, got, units = _run(wl, units=[(0, 0, 1)])
    compare_event(snap, cache, comp, dbg, dst, credit0, got, units=[(0, 0, 0), (0, 0, 1)])


def test_expected_with_window_attention_as_mass_signal():
    """Decoupled: the mass from the observation-window attention, the ranking from the expected-attention score."""
    wl = _wl(window=8, decoupled=True, n_layers=1)
    cache = inputs.make_cache(wl, DEV)
    comp = binding.AmsCompressor(binding.config_for(wl), DEV)
    mean, cov = inputs.make_query_stats(cache)
    comp.set_query_stats(mean, cov, EPS)
    snap = HostSnapshot(cache)
    credit0 = comp.ema_state.cpu().numpy()
    dst = inputs.alloc_dst_pages(cache)
    dbg = gpu_event(comp, cache, dst)
    g, u = dbg.scores.cpu().numpy(), dbg.usage.cpu().numpy()
    G = wl.group
    for l in range(wl.n_layers):
        for b in range(wl.batch):
            T = int(snap.lens[b])
            for h in range(wl.n_kv_heads):
                want_u = oracle.score_tova(snap.k, l, h, snap.table[b], T, snap.q[l, b, h * G:(h + 1) * G], G, wl.window, True)
                assert_scores_close(u[l, b, h, :T], want_u, rtol=1e-3)
    want = _oracle_scores(snap, wl, mean.cpu().numpy(), inputs.as_u16(cov),
                          [(l, b, h) for l in range(wl.n_layers) for b in range(wl.batch) for h in range(wl.n_kv_heads)])
    for (l, b, h), w in want.items():
        assert_scores_close(g[l, b, h, :int(snap.lens[b])], w, rtol=1e-3)
    compare_event(snap, cache, comp, dbg, dst, credit0, g, usage_for_oracle=u)


def test_expected_needs_room_and_statistics():
    wl = _wl(n_layers=1, batch=1)
    cache = inputs.make_cache(wl, DEV)
    dst = torch.from_numpy(inputs.alloc_dst_pages(cache)).to(DEV)
    comp = binding.AmsCompressor(binding.config_for(wl), DEV)
    with pytest.raises(binding.AmsError) as e:     # no statistics given yet
        comp.compress(cache.k_pages, cache.v_pages, cache.block_table, cache.seq_lens, None, wl.budget, wl.n_segments,
                      inputs.SCORER_EXPECTED, dst)
    assert e.value.code == binding.AMS_ERR_INVALID_ARG
    plain = binding.AmsCompressor(binding.config_for(wl, expected_scorer=0), DEV)
    mean, cov = inputs.make_query_stats(cache)
    plain.set_query_stats(mean, cov, EPS)
    with pytest.raises(binding.AmsError) as e:     # the configuration reserved no room for the logits
        plain.compress(cache.k_pages, cache.v_pages, cache.block_table, cache.seq_lens, None, wl.budget, wl.n_segments,
                       inputs.SCORER_EXPECTED, dst)
    assert e.value.code == binding.AMS_ERR_CAPACITY


def test_expected_two_events_with_credit_carried():
    """Two consecutive events with appended tokens in between (EMA on): the credit carried in compacted order, the
    rewritten block table and fresh query statistics feed the second event."""
    wl = _wl(n_layers=1, batch=2, seq_len_min=2000, seq_len_max=3000, budget=768, append_per_step=256, steps=2)
    cache = inputs.make_cache(wl, DEV)
    comp = binding.AmsCompressor(binding.config_for(wl), DEV)
    for ev in range(2):
        if ev:
            inputs.append_tokens(cache, wl.append_per_step)
        mean, cov = inputs.make_query_stats(cache)
        comp.set_query_stats(mean, cov, EPS)
        snap = HostSnapshot(cache)
        credit0 = comp.ema_state.cpu().numpy()
        assert (credit0 != 0).any() == bool(ev)
        dst = inputs.alloc_dst_pages(cache)
        dbg = gpu_event(comp, cache, dst)
        got = dbg.scores.cpu().numpy()
        units = [(0, b, h) for b in range(wl.batch) for h in range(wl.n_kv_heads)]
        want = _oracle_scores(snap, wl, mean.cpu().numpy(), inputs.as_u16(cov), units)
        for (l, b, h), w in want.items():
            assert_scores_close(got[l, b, h, :int(snap.lens[b])], w, rtol=1e-3)
        compare_event(snap, cache, comp, dbg, dst, credit0, got)
        assert (cache.seq_lens.cpu().numpy() == wl.budget).all()
        inputs.after_compress(cache, dst)


def test_expected_longest_sequence():
    """131072 tokens (the capacity limit): 1024 tiles per unit, shared by some thirty blocks whose statistics are merged."""
    wl = _wl(n_layers=1, batch=1, n_kv_heads=1, n_q_heads=2, seq_len_min=131072, seq_len_max=131072, budget=4096,
             n_segments=32, l_max=8192)
    cache, comp, snap, credit0, dst, dbg, got, units = _run(wl)
    compare_event(snap, cache, comp, dbg, dst, credit0, got)
