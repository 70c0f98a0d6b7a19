"""GPU parity of the two component ablations of the paper's ablation table: segments of equal length
instead of equal mass (`fixed_segments`) and a budget shared by segment length instead of mass
(`uniform_quotas`).  External scores, so every decision and byte must match the oracle exactly."""
import numpy as np
import pytest
import torch

from helpers import HostSnapshot, compare_event, gpu_event
from paper_2605_23200_b200 import binding, inputs

pytestmark = pytest.mark.gpu
DEV = "cuda:0"

CASES = [
    dict(fixed_segments=True),
    dict(uniform_quotas=True),
    dict(fixed_segments=True, uniform_quotas=True, n_segments=7, l_min=1, l_max=0),
    dict(fixed_segments=True, seq_len_min=1000, seq_len_max=1777, batch=4, budget=1200),                 # ragged; some skipped
    dict(uniform_quotas=True, seq_len_min=20011, seq_len_max=20011, budget=3000, batch=1, n_layers=1),   # two blocks per unit
    dict(fixed_segments=True, uniform_quotas=True, seq_len_min=33000, seq_len_max=33000, budget=4000, batch=1, n_layers=1,
         n_segments=16, l_max=4096),                                                                     # joint search
    dict(fixed_segments=True, uniform_quotas=True, n_layers=4, batch=9, seq_len_min=500, seq_len_max=2600, budget=1203),  # work queue
    dict(fixed_segments=True, uniform_quotas=True, seq_len_min=16000, seq_len_max=16000, budget=2048, batch=1, n_layers=1,
         l_min=4, l_max=16),                                                                             # one-block fallback kernel
]


@pytest.mark.parametrize("kw", CASES)
def test_ablation_switches_bit_exact(kw):
    base = dict(n_layers=2, batch=2, seq_len_min=1500, seq_len_max=1500, budget=384)
    base.update(kw)
    wl = inputs.CONFIGS[0].scaled(resident_layers=0, **base)
    cache = inputs.make_cache(wl, DEV)
    comp = binding.AmsCompressor(binding.config_for(wl), DEV)
    rng = np.random.default_rng(4242)
    ext = np.exp(2.0 * rng.standard_normal((wl.n_layers, wl.batch, wl.n_kv_heads, wl.max_seq_len))).astype(np.float32)
    snap = HostSnapshot(cache)
    credit0 = comp.ema_state.cpu().numpy()
    dst = inputs.alloc_dst_pages(cache)
    dbg = gpu_event(comp, cache, dst, inputs.SCORER_EXTERNAL, torch.from_numpy(ext).to(DEV))
    res = compare_event(snap, cache, comp, dbg, dst, credit0, ext)
    assert res
    if wl.fixed_segments and wl.l_max == 0 and wl.l_min == 1:
        for (l, b, h), r in res.items():
            T = int(snap.lens[b])
            assert r.bounds.tolist() == sorted(set(k * T // wl.n_segments for k in range(wl.n_segments + 1)))


def test_retained_set_iou_between_consecutive_events():
    """Diagnostic of the mechanistic-diagnostics appendix: after an event the retained tokens sit at the
    front of the cache; the next event's IoU with them follows from its kept positions alone."""
    import oracle
    wl = inputs.CONFIGS[2].scaled(resident_layers=0, n_layers=2, batch=3, seq_len_min=700, seq_len_max=1300, budget=256,
                                  append_per_step=96, steps=3)
    cache = inputs.make_cache(wl, DEV)
    comp = binding.AmsCompressor(binding.config_for(wl), DEV)
    prev = torch.zeros(wl.batch, dtype=torch.int32, device=DEV)
    for step in range(wl.steps):
        dst_np = inputs.alloc_dst_pages(cache)
        lens = cache.seq_lens.cpu().numpy().copy()
        dbg = comp.make_debug_views(wl.batch, wl.budget)
        dbg.prev_kept = prev
        dbg.retained_iou = torch.full((wl.n_layers, wl.batch, wl.n_kv_heads), -1.0, device=DEV)
        comp.compress(cache.k_pages, cache.v_pages, cache.block_table, cache.seq_lens, cache.obs_queries, wl.budget,
                      wl.n_segments, wl.scorer_id, torch.from_numpy(dst_np).to(DEV), dbg=dbg)
        comp.status()
        keep = dbg.keep_idx.cpu().numpy()
        got = dbg.retained_iou.cpu().numpy()
        for l in range(wl.n_layers):
            for b in range(wl.batch):
                for h in range(wl.n_kv_heads):
                    if lens[b] <= wl.budget:
                        assert got[l, b, h] == -1.0                      # skipped sequences are left untouched
                    else:
                        assert got[l, b, h] == oracle.retained_iou(keep[l, b, h], int(prev[b]), wl.budget), (step, l, b, h)
        if step > 0:
            assert (got[got >= 0] > 0.3).all() and (got <= 1.0).all()    # most of a retained set survives 96 new tokens
        prev = torch.from_numpy(np.where(lens > wl.budget, wl.budget, 0).astype(np.int32)).to(DEV)
        inputs.after_compress(cache, dst_np)
        if step + 1 < wl.steps:
            inputs.append_tokens(cache, wl.append_per_step)
