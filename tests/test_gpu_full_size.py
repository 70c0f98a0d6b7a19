"""Parity at the benchmark's full size and launch configuration (configuration 1: 32 layers,
one sequence of 16384 cached tokens, budget 2048, observation window 32, 256 units).

The oracle cannot redo all 256 units in a test, so: sampled units are compared with it one by
one (scores and mass within 1e-3 relative; boundaries, quotas, kept indices and credit exactly,
with the oracle selecting on the library's scores), and every unit is checked through
properties that hold at any size (kept indices ascending, unique, inside the sequence,
containing the must-keep prefix and suffix; compacted K/V rows byte-identical to the rows the
kept indices name; block table and length rewritten)."""
import numpy as np
import pytest
import torch

import oracle
from helpers import HostSnapshot, assert_scores_close, compare_event, gpu_event
from paper_2605_23200_b200 import binding, inputs

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
SAMPLE = [(0, 0, 0), (5, 0, 3), (13, 0, 6), (22, 0, 1), (31, 0, 7)]


def test_benchmark_workload_sampled_units_and_properties():
    wl = inputs.CONFIGS[1]
    cache = inputs.make_cache(wl, DEV)
    comp = binding.AmsCompressor(binding.config_for(wl), DEV)
    snap = HostSnapshot(cache)
    credit0 = comp.ema_state.cpu().numpy()
    k_before = cache.k_pages.clone()
    v_before = cache.v_pages.clone()
    dst = inputs.alloc_dst_pages(cache)
    dbg = gpu_event(comp, cache, dst)
    assert comp.last_launch_count == 8          # validation, two scorer passes, three selection kernels, gather, table
    got = dbg.scores.cpu().numpy()
    mass = dbg.mass.cpu().numpy()
    T, Tk, G = wl.seq_len_max, wl.budget, wl.group

    # ---- sampled units against the oracle
    for (l, b, h) in SAMPLE:
        want = oracle.score_tova(snap.k, l, h, snap.table[b], T, snap.q[l, b, h * G:(h + 1) * G], G, wl.window, True)
        assert_scores_close(got[l, b, h, :T], want, 1e-3, 0.0)
        _, _, m_want = oracle.mass(want, wl.eps)
        assert_scores_close(mass[l, b, h, :T], m_want, 1e-3, 1e-3 * wl.eps)
    compare_event(snap, cache, comp, dbg, dst, credit0, got, units=SAMPLE)

    # ---- properties of every unit
    keep = dbg.keep_idx                                             # [L][B][H][Tk] on the device
    assert int(keep.min()) >= 0 and int(keep.max()) < T
    assert bool((keep[..., 1:] > keep[..., :-1]).all())             # ascending, hence unique
    assert bool((keep[..., : wl.n_sink] == torch.arange(wl.n_sink, device=DEV)).all())
    assert bool((keep[..., Tk - wl.n_last:] == torch.arange(T - wl.n_last, T, device=DEV)).all())
    n_seg = dbg.n_segments
    assert int(n_seg.min()) >= T // wl.l_max and int(n_seg.max()) <= comp.seg_cap
    quotas = dbg.quotas.cpu().numpy()
    nsg = n_seg.cpu().numpy()
    for l in range(wl.n_layers):
        for h in range(wl.n_kv_heads):
            assert quotas[l, 0, h, : nsg[l, 0, h]].sum() == Tk - wl.n_sink - wl.n_last

    # ---- compacted rows are the rows the kept indices name, byte for byte; sources untouched
    old_table = torch.from_numpy(snap.table[0].astype(np.int64)).to(DEV)
    new_table = cache.block_table[0].long()
    assert bool((new_table[: Tk // 16] == torch.from_numpy(dst[0].astype(np.int64)).to(DEV)).all())
    assert bool((new_table[Tk // 16:] == -1).all()) and int(cache.seq_lens[0]) == Tk
    j = torch.arange(Tk, device=DEV)
    new_slot = new_table[j // 16] * 16 + j % 16                     # [Tk]
    for pool_now, pool_before in ((cache.k_pages, k_before), (cache.v_pages, v_before)):
        now = pool_now.view(torch.int16).view(wl.n_layers, -1, wl.n_kv_heads, 128)
        before = pool_before.view(torch.int16).view(wl.n_layers, -1, wl.n_kv_heads, 128)
        for l in range(wl.n_layers):
            pos = keep[l, 0].long()                                 # [H][Tk]
            old_slot = old_table[pos // 16] * 16 + pos % 16         # [H][Tk]
            for h in range(wl.n_kv_heads):
                assert torch.equal(now[l, new_slot, h], before[l, old_slot[h], h]), (l, h)
        live = torch.ones(now.shape[1], dtype=torch.bool, device=DEV)
        live[(torch.from_numpy(dst.reshape(-1).astype(np.int64)).to(DEV)[:, None] * 16 + torch.arange(16, device=DEV)).reshape(-1)] = False
        assert torch.equal(now[:, live], before[:, live])           # nothing outside the replacement pages was written
