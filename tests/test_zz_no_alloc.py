"""The allocation-free selection entry point (`ams_select_static`) against the regular one and the oracle.

Some users of the library cannot allocate device memory where they call it — a stream capture
is in progress, or the process's device memory pool belongs to the framework that hosts them —
so this entry point works out of a fixed scratch array inside the library.  The check: on the
same scores it must keep exactly the positions that `ams_compress` keeps (external-score mode,
credit off) and that the CPU oracle keeps, on calls in a row: the second one on different scores,
the third one with fewer and shorter rows, so that anything left in the shared scratch by an
earlier, larger call would show.  Collected last on purpose."""
import ctypes
import gc

import numpy as np
import pytest
import torch

import oracle
from paper_2605_23200_b200 import binding, inputs

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _regular_keep(wl, scores):
    """Kept indices from the handle-based entry point on the same scores (credit unused)."""
    cache = inputs.make_cache(wl, DEV)
    comp = binding.AmsCompressor(binding.config_for(wl), DEV)
    dbg = comp.make_debug_views(wl.batch, wl.budget)
    dst = torch.from_numpy(inputs.alloc_dst_pages(cache)).to(DEV)
    comp.compress(cache.k_pages, cache.v_pages, cache.block_table, cache.seq_lens, None, wl.budget, wl.n_segments,
                  inputs.SCORER_EXTERNAL, dst, ext_scores=scores, dbg=dbg)
    comp.status()
    return dbg.keep_idx.clone()


def test_static_scratch_selection_matches_regular_entry_point_twice():
    T, Tk = 5008, 640
    wl = inputs.CONFIGS[0].scaled(n_layers=1, n_q_heads=8, n_kv_heads=8, batch=1, seq_len_min=T, seq_len_max=T,
                                  budget=Tk, ema_beta=1.0, n_segments=12)
    cfg = binding.config_for(wl)
    rng = np.random.default_rng(99)
    for call in range(2):
        x = np.exp(2.0 * rng.standard_normal((1, 1, 8, wl.max_seq_len))).astype(np.float32)
        if call == 1:
            x = np.round(x * 2) / 2                                  # second call: many ties
        scores = torch.from_numpy(x).to(DEV)
        want = _regular_keep(wl, scores)[0, 0]                       # [8][Tk]
        free_before = torch.cuda.mem_get_info()[0]
        got = torch.full((8, Tk), -1, dtype=torch.int32, device=DEV)
        gc.collect()                                                 # tensors of earlier tests go now, not during the call
        torch.cuda.synchronize()
        allocated = torch.cuda.memory_allocated()
        n_allocs = torch.cuda.memory_stats()["allocation.all.allocated"]   # allocation events so far (never decreases)
        row = scores[0, 0]
        binding.select_static(cfg, row, T, Tk, wl.n_segments, got)
        torch.cuda.synchronize()
        assert torch.cuda.memory_stats()["allocation.all.allocated"] == n_allocs   # torch's allocator was not asked
        assert torch.cuda.memory_allocated() <= allocated
        assert torch.cuda.mem_get_info()[0] >= free_before - (64 << 20)
        assert torch.equal(got, want), f"call {call}"
        prm = oracle.Params(wl.n_segments, wl.l_min, wl.l_max, wl.q_min, wl.n_sink, wl.n_last, wl.ema_lambda, 1.0, wl.eps)
        for r in range(8):
            assert (got[r].cpu().numpy() == oracle.select_unit(x[0, 0, r, :T], None, None, Tk, prm).keep_idx).all(), (call, r)
        assert binding.select_static_status() == (binding.AMS_OK, [0, 0, 0, 0])
    # third call: fewer rows, a shorter sequence and another stride than the calls before it
    T3, Tk3, stride3 = 1203, 200, 1216
    x3 = np.exp(rng.standard_normal((3, stride3))).astype(np.float32)
    got3 = torch.full((3, Tk3), -1, dtype=torch.int32, device=DEV)
    binding.select_static(cfg, torch.from_numpy(x3).to(DEV), T3, Tk3, 7, got3)
    torch.cuda.synchronize()
    prm3 = oracle.Params(7, wl.l_min, wl.l_max, wl.q_min, wl.n_sink, wl.n_last, wl.ema_lambda, 1.0, wl.eps)
    for r in range(3):
        assert (got3[r].cpu().numpy() == oracle.select_unit(x3[r, :T3], None, None, Tk3, prm3).keep_idx).all(), r
    assert binding.select_static_status()[0] == binding.AMS_OK


def test_static_scratch_limits_are_rejected():
    cfg = binding.config_for(inputs.CONFIGS[0])
    lib = binding.lib()
    s = torch.zeros((9, 64), dtype=torch.float32, device=DEV)
    k = torch.zeros((9, 8), dtype=torch.int32, device=DEV)
    null = ctypes.c_void_p(0)
    args = lambda n_units, seq_len, stride, budget, nseg: lib.ams_select_static(
        ctypes.byref(cfg), ctypes.c_void_p(s.data_ptr()), stride, n_units, seq_len, budget, nseg,
        ctypes.c_void_p(k.data_ptr()), null)
    assert args(9, 64, 64, 8, 4) == binding.AMS_ERR_CAPACITY           # too many rows
    assert args(1, 32768 + 16, 32768 + 16, 8, 4) == binding.AMS_ERR_CAPACITY
    assert args(1, 64, 60, 8, 4) == binding.AMS_ERR_INVALID_ARG        # stride not a multiple of 16
    assert args(1, 64, 64, 64, 4) == binding.AMS_ERR_INVALID_ARG       # nothing to evict
    cfg.l_max = 16
    assert args(1, 32768, 32768, 8, 4) == binding.AMS_ERR_CAPACITY     # more segments than the array holds
