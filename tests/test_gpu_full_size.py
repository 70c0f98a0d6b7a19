"""Parity at the benchmark's full sizes and launch configurations: configuration 1 (32 layers, one sequence
of 16384 cached tokens, budget 2048, observation window 32, 256 units), the whole ragged batch of
configuration 2 (28 layers x 16 sequences of 8192..32768 tokens x 4 KV heads = 1792 units, budget 4096) and
one four-layer launch of configuration 3 (4 x 64 x 8 = 2048 units of 32768 tokens, key-only scorer).

The oracle cannot redo every unit in a test, so: sampled units are compared with it one by one (scores and
mass within 1e-3 relative; boundaries, quotas, kept indices and credit exactly, with the oracle selecting on
the library's scores), and every unit is checked through properties that hold at any size (kept indices
ascending, unique, inside the sequence, containing the must-keep prefix and suffix; quotas summing to the
segment budget and segments covering the sequence; compacted K/V rows byte-identical to the rows the kept
indices name; nothing outside the replacement pages written; block table and length rewritten)."""
import numpy as np
import pytest
import torch

import oracle
from helpers import assert_scores_close, gpu_event, params_of
from paper_2605_23200_b200 import binding, inputs

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


class _LightSnapshot:
    """Block table and lengths before the event; K and queries only for the layers asked for (a whole pool of
    these sizes does not belong in host memory twice)."""

    def __init__(self, cache):
        self.table = cache.block_table.cpu().numpy().copy()
        self.lens = cache.seq_lens.cpu().numpy().copy()


def _sampled_units_match_the_oracle(wl, cache, comp, snap, dbg, sample, k_before, credit_zero, atol=0.0, v_before=None, stats=None):
    """Scores and mass of the sampled units within 1e-3 of the oracle; on the library's own scores the oracle
    must select exactly what the library selected (segments, quotas, kept positions, mass, credit)."""
    G, Tk = wl.group, wl.budget
    prm = params_of(wl)
    for (l, b, h) in sample:
        T = int(snap.lens[b])
        k_l = inputs.as_u16(k_before[l:l + 1])
        if wl.scorer_id == inputs.SCORER_TOVA:
            q = inputs.as_u16(cache.obs_queries[l, b, h * G:(h + 1) * G])
            want = oracle.score_tova(k_l, 0, h, snap.table[b], T, q, G, wl.window, True)
        elif wl.scorer_id == inputs.SCORER_EXPECTED:
            mean, cov = stats
            want = oracle.score_expected(k_l, inputs.as_u16(v_before[l:l + 1]), 0, h, snap.table[b], T,
                                         mean[l, b, h * G:(h + 1) * G].cpu().numpy(), inputs.as_u16(cov[l, b, h * G:(h + 1) * G]), 1e-2)
        else:
            want = oracle.score_keydiff(k_l, 0, h, snap.table[b], T)
        got = dbg.scores[l, b, h, :T].cpu().numpy()
        assert_scores_close(got, want, 1e-3, atol)
        _, _, m_want = oracle.mass(want, wl.eps)
        sum_w = float(np.maximum(want.astype(np.float64), 0.0).sum() + wl.eps * T)
        mass = dbg.mass[l, b, h, :T].cpu().numpy()
        assert_scores_close(mass, m_want, 1e-3, 1e-3 * wl.eps + atol / sum_w)
        assert credit_zero                                           # first event: the credit starts from zero
        r = oracle.select_unit(got, got, None, Tk, prm)
        n = int(dbg.n_segments[l, b, h])
        assert n == r.n_seg, (l, b, h, n, r.n_seg)
        assert dbg.seg_bounds[l, b, h, : n + 1].cpu().numpy().tolist() == r.bounds.tolist(), (l, b, h)
        assert dbg.quotas[l, b, h, :n].cpu().numpy().tolist() == r.quotas.tolist(), (l, b, h)
        assert (dbg.keep_idx[l, b, h].cpu().numpy() == r.keep_idx).all(), (l, b, h)
        assert (mass == r.mass).all(), (l, b, h)
        if wl.ema_beta != 1.0:
            assert (comp.ema_state[l, b, h, :T].cpu().numpy() == r.credit[:T]).all(), (l, b, h)


def _properties_of_every_unit(wl, cache, comp, dbg, snap, dst, k_before, v_before):
    Tk = wl.budget
    keep = dbg.keep_idx                                             # [L][B][H][Tk] on the device
    lens = torch.from_numpy(snap.lens.astype(np.int64)).to(DEV)
    assert bool((snap.lens > Tk).all())
    assert int(keep.min()) >= 0 and bool((keep < lens[None, :, None, None]).all())
    assert bool((keep[..., 1:] > keep[..., :-1]).all())             # ascending, hence unique
    assert bool((keep[..., : wl.n_sink] == torch.arange(wl.n_sink, device=DEV)).all())
    tail = lens[None, :, None, None] - wl.n_last + torch.arange(wl.n_last, device=DEV)
    assert bool((keep[..., Tk - wl.n_last:] == tail).all())
    n_seg = dbg.n_segments
    assert int(n_seg.min()) >= 1 and int(n_seg.max()) <= comp.seg_cap
    nsg = n_seg.cpu().numpy()
    quotas = dbg.quotas.cpu().numpy()
    bounds = dbg.seg_bounds.cpu().numpy()
    L, B, H = nsg.shape
    col = np.arange(quotas.shape[-1])[None, None, None, :]
    assert ((quotas * (col < nsg[..., None])).sum(-1) == Tk - wl.n_sink - wl.n_last).all()
    for b in range(B):
        T = int(snap.lens[b])
        n = nsg[:, b, :]
        assert (bounds[:, b, :, 0] == 0).all()
        assert (np.take_along_axis(bounds[:, b], n[..., None], axis=-1)[..., 0] == T).all()   # segments cover the sequence
        d = np.diff(bounds[:, b], axis=-1)
        live = np.arange(d.shape[-1])[None, None, :] < n[..., None]
        assert (d[live] > 0).all()
        if wl.l_max:
            assert (d[live] <= wl.l_max).all()
    # kept per segment >= quota is implied by the oracle on samples; here: the compacted rows are the rows the kept
    # indices name, byte for byte, and nothing outside the replacement pages was written
    n_dst = dst.shape[1]
    j = torch.arange(Tk, device=DEV)
    dst_dev = torch.from_numpy(dst.astype(np.int64)).to(DEV)
    for pool_now, pool_before in ((cache.k_pages, k_before), (cache.v_pages, v_before)):
        now = pool_now.view(torch.int16).view(wl.layers_resident, -1, wl.n_kv_heads, 128)
        before = pool_before.view(torch.int16).view(wl.layers_resident, -1, wl.n_kv_heads, 128)
        for b in range(B):
            old_table = torch.from_numpy(snap.table[b].astype(np.int64)).to(DEV)
            new_slot = dst_dev[b][j // 16] * 16 + j % 16                        # [Tk]
            for l in range(L):
                pos = keep[l, b].long()                                         # [H][Tk]
                old_slot = old_table[pos // 16] * 16 + pos % 16                 # [H][Tk]
                for h in range(H):
                    assert torch.equal(now[l, new_slot, h], before[l, old_slot[h], h]), (l, b, h)
        live = torch.ones(now.shape[1], dtype=torch.bool, device=DEV)
        live[(dst_dev.reshape(-1)[:, None] * 16 + torch.arange(16, device=DEV)).reshape(-1)] = False
        for l in range(L):
            assert torch.equal(now[l, live], before[l, live])                   # (layer by layer: bounded temporaries)
    new_table = cache.block_table.long()
    assert bool((new_table[:, :n_dst] == dst_dev).all()) and bool((new_table[:, n_dst:] == -1).all())
    assert bool((cache.seq_lens == Tk).all())


def _run(wl, sample, atol=0.0, launches=None):
    cache = inputs.make_cache(wl, DEV)
    comp = binding.AmsCompressor(binding.config_for(wl), DEV)
    stats = None
    if wl.scorer_id == inputs.SCORER_EXPECTED:
        stats = inputs.make_query_stats(cache)
        comp.set_query_stats(stats[0], stats[1], 1e-2)
    snap = _LightSnapshot(cache)
    credit_zero = float(comp.ema_state.abs().sum()) == 0.0
    k_before = cache.k_pages.clone()
    v_before = cache.v_pages.clone()
    dst = inputs.alloc_dst_pages(cache)
    dbg = gpu_event(comp, cache, dst)
    if launches is not None:
        assert comp.last_launch_count == launches
    _sampled_units_match_the_oracle(wl, cache, comp, snap, dbg, sample, k_before, credit_zero, atol, v_before, stats)
    _properties_of_every_unit(wl, cache, comp, dbg, snap, dst, k_before, v_before)


def test_benchmark_workload_sampled_units_and_properties():
    # validation, two scorer passes, three selection kernels, gather, table update
    _run(inputs.CONFIGS[1], [(0, 0, 0), (5, 0, 3), (13, 0, 6), (22, 0, 1), (31, 0, 7)], launches=8)


def test_config2_whole_ragged_batch_properties():
    wl = inputs.CONFIGS[2]
    _run(wl, [(0, 0, 0), (11, 7, 2), (27, 15, 3)])


def test_config3_one_four_layer_launch_properties():
    wl = inputs.CONFIGS[3]
    _run(wl, [(0, 0, 0), (3, 63, 7)], atol=1e-5)


def test_expected_attention_workload_sampled_units_and_properties():
    """The extension workload of the benchmark (geometry of configuration 1, expected-attention scorer) at its timed size."""
    _run(inputs.CONFIGS[5], [(0, 0, 0), (17, 0, 5), (31, 0, 7)], launches=8)
