"""Seeded workload generator and the oracle's whole-event driver on small workloads."""
import numpy as np
import torch

import oracle
from paper_2605_23200_b200 import inputs


def _params(wl):
    return oracle.Params(wl.n_segments, wl.l_min, wl.l_max, wl.q_min, wl.n_sink, wl.n_last, wl.ema_lambda,
                         wl.ema_beta, wl.eps)


def test_generator_is_seeded_and_structured():
    wl = inputs.CONFIGS[0].scaled(seq_len_min=1024, seq_len_max=1024, budget=256)
    a = inputs.make_cache(wl)
    b = inputs.make_cache(wl)
    assert torch.equal(a.k_pages.view(torch.int16), b.k_pages.view(torch.int16))
    assert torch.equal(a.block_table, b.block_table) and torch.equal(a.obs_queries.view(torch.int16),
                                                                     b.obs_queries.view(torch.int16))
    L, P, page, H, D = a.k_pages.shape
    assert (page, H, D) == (16, 8, 128) and a.obs_queries.shape == (1, 1, 32, 1, 128)
    table = a.host_table[0]
    assert len(set(table[:64].tolist())) == 64 and (table[64:] == -1).all()      # distinct live pages
    slots = table[np.arange(1024) // 16].astype(np.int64) * 16 + np.arange(1024) % 16
    K = a.k_pages[0].view(-1, H, D)[torch.from_numpy(slots)].float()
    norms = K.norm(dim=-1)[:, 0]
    heavy = (norms > 25).sum().item()
    assert 5 <= heavy <= 15                                                      # ~1 % of keys carry 3x norm
    proj = (K[:, 0] @ a.directions[0, 0])
    assert (proj > 1.0).float().mean() > 0.3                                     # spans shifted along u


def test_event_small_tova_multi_step_and_keydiff():
    wl = inputs.CONFIGS[2].scaled(n_layers=2, batch=3, seq_len_min=300, seq_len_max=700, budget=128,
                                  append_per_step=32, steps=3)
    cache = inputs.make_cache(wl)
    k, v = inputs.as_u16(cache.k_pages), inputs.as_u16(cache.v_pages)
    credit = np.zeros((wl.n_layers, wl.batch, wl.n_kv_heads, wl.max_seq_len), np.float32)
    prm = _params(wl)
    for step in range(wl.steps):
        dst = inputs.alloc_dst_pages(cache)
        table, lens = cache.host_table.copy(), cache.host_lens.copy()
        q = inputs.as_u16(cache.obs_queries)
        res = oracle.compress(k, v, table, lens, q, credit, wl.budget, prm, inputs.SCORER_TOVA, dst,
                              n_q_heads=wl.n_q_heads, threads=4)
        assert len(res) == wl.n_layers * wl.batch * wl.n_kv_heads
        assert (lens == wl.budget).all() and (table[:, : wl.budget // 16] == dst).all()
        for (l, b, h), r in res.items():
            assert abs(float(r.scores.astype(np.float64).sum()) - 1.0) < 1e-5     # W = 1: nothing padded
        inputs.after_compress(cache, dst)
        assert (cache.host_table == table).all() and (cache.host_lens == lens).all()
        # push the oracle's pages back so the next step's appended tokens land on top of them
        cache.k_pages.copy_(torch.from_numpy(k.view(np.int16)).view(torch.bfloat16))
        cache.v_pages.copy_(torch.from_numpy(v.view(np.int16)).view(torch.bfloat16))
        cache.block_table.copy_(torch.from_numpy(table)); cache.seq_lens.copy_(torch.from_numpy(lens))
        if step + 1 < wl.steps:
            inputs.append_tokens(cache, wl.append_per_step)
            k, v = inputs.as_u16(cache.k_pages), inputs.as_u16(cache.v_pages)
            assert (cache.host_lens == wl.budget + wl.append_per_step).all()
    assert (credit[..., : wl.budget] > 0).all() and (credit[..., wl.budget:] == 0).all()

    wl3 = inputs.CONFIGS[3].scaled(n_layers=1, resident_layers=0, batch=2, seq_len_min=500, seq_len_max=500,
                                   budget=64, n_segments=4, l_max=250)
    c3 = inputs.make_cache(wl3)
    assert c3.obs_queries is None
    k, v = inputs.as_u16(c3.k_pages), inputs.as_u16(c3.v_pages)
    credit = np.zeros((1, 2, wl3.n_kv_heads, wl3.max_seq_len), np.float32)
    dst = inputs.alloc_dst_pages(c3)
    res = oracle.compress(k, v, c3.host_table.copy(), c3.host_lens.copy(), None, credit, wl3.budget,
                          _params(wl3), inputs.SCORER_KEYDIFF, dst)
    for r in res.values():
        assert (np.abs(r.scores) <= 1.0 + 1e-6).all() and r.keep_idx.shape == (64,)
    assert (credit == 0).all()                                                    # beta = 1: credit unused
