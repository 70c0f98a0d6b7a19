"""Failure handling and repeated events through the C ABI, without faulting, trapping or hanging the GPU:
bad page ids are caught by the event's first kernel before any address is formed from them, a bounded device
wait is made to run out by construction, and events that follow a skipped or reported one start from a clean
state."""
import numpy as np
import pytest
import torch

from helpers import HostSnapshot, compare_event, gpu_event
from paper_2605_23200_b200 import binding, inputs

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _wl(**kw):
    base = dict(n_layers=2, batch=3, seq_len_min=1500, seq_len_max=1500, budget=384, resident_layers=0)
    base.update(kw)
    return inputs.CONFIGS[0].scaled(**base)


def _ext(wl, seed):
    rng = np.random.default_rng(seed)
    return np.exp(2.0 * rng.standard_normal((wl.n_layers, wl.batch, wl.n_kv_heads, wl.max_seq_len))).astype(np.float32)


@pytest.mark.parametrize("where,bad_id", [("table", -7), ("table", 1 << 30), ("dst", -1), ("dst", 10 ** 9)])
def test_page_id_outside_the_pool_is_reported_and_the_sequence_left_alone(where, bad_id):
    wl = _wl()
    cache = inputs.make_cache(wl, DEV)
    comp = binding.AmsCompressor(binding.config_for(wl), DEV)
    ext = _ext(wl, 5)
    dst = inputs.alloc_dst_pages(cache)
    victim = 1
    if where == "table":
        cache.block_table[victim, 17] = bad_id          # injected on the host side of the call
    else:
        dst = dst.copy()
        dst[victim, 3] = bad_id
    snap = HostSnapshot(cache)
    k0, v0 = cache.k_pages.clone(), cache.v_pages.clone()
    credit0 = comp.ema_state.cpu().numpy()
    dbg = comp.make_debug_views(wl.batch, wl.budget)
    comp.compress(cache.k_pages, cache.v_pages, cache.block_table, cache.seq_lens, None, wl.budget, wl.n_segments,
                  inputs.SCORER_EXTERNAL, torch.from_numpy(dst).to(DEV), ext_scores=torch.from_numpy(ext).to(DEV), dbg=dbg)
    rc, detail = comp.status(check=False)
    assert rc == binding.AMS_ERR_INVALID_ARG and detail[1] == victim and detail[3] == np.int32(bad_id)
    assert detail[2] == (17 if where == "table" else -1 - 3)
    # the reported sequence: table row, length, credit and every page it names are as before
    assert (cache.block_table[victim].cpu().numpy() == snap.table[victim]).all()
    assert int(cache.seq_lens[victim]) == int(snap.lens[victim])
    assert (comp.ema_state[:, victim].cpu().numpy() == 0).all()
    good_dst = [int(x) for x in dst[victim] if 0 <= x < cache.num_pages]
    assert torch.equal(cache.k_pages[:, good_dst].view(torch.int16), k0[:, good_dst].view(torch.int16))
    assert torch.equal(cache.v_pages[:, good_dst].view(torch.int16), v0[:, good_dst].view(torch.int16))
    # the other sequences were compressed exactly as the oracle does it
    others = [(l, b, h) for l in range(wl.n_layers) for b in range(wl.batch) if b != victim for h in range(wl.n_kv_heads)]
    compare_event(snap, cache, comp, dbg, dst, credit0, ext, units=others)
    for b in range(wl.batch):
        if b != victim:
            assert int(cache.seq_lens[b]) == wl.budget
            assert (cache.block_table[b, : dst.shape[1]].cpu().numpy() == dst[b]).all()
    assert comp.status(check=False)[0] == binding.AMS_OK


def test_bounded_device_wait_runs_out_and_reports_timeout():
    wl = _wl(batch=1, n_layers=1)
    cache = inputs.make_cache(wl, DEV)
    comp = binding.AmsCompressor(binding.config_for(wl), DEV)
    comp.expire_wait(1000)                              # waits on a barrier nobody arrives at: 1000 polls, then gives up
    rc, detail = comp.status(check=False)
    assert rc == binding.AMS_ERR_TIMEOUT and detail[2] == 1000
    assert comp.status(check=False)[0] == binding.AMS_OK
    # the context is intact: a regular event right after it is still bit-exact
    ext = _ext(wl, 6)
    snap = HostSnapshot(cache)
    credit0 = comp.ema_state.cpu().numpy()
    dst = inputs.alloc_dst_pages(cache)
    dbg = gpu_event(comp, cache, dst, inputs.SCORER_EXTERNAL, torch.from_numpy(ext).to(DEV))
    compare_event(snap, cache, comp, dbg, dst, credit0, ext)
    with pytest.raises(binding.AmsError):
        comp.expire_wait(0)


@pytest.mark.parametrize("shape", ["many_units_first_sequence_idle", "one_sequence_idle_then_real"])
def test_event_after_an_event_with_nothing_to_evict(shape):
    """Two events on one handle.  In the first, sequence 0 is within the budget (nothing to evict) while the
    others are compressed; tokens are appended; in the second every sequence is over the budget.  Both must
    match the oracle bit for bit (more units than SMs in the first shape)."""
    if shape == "many_units_first_sequence_idle":
        wl = _wl(n_layers=6, batch=4, seq_len_min=2000, seq_len_max=2000, budget=1024, append_per_step=700)   # 192 units
        lens = [900, 2000, 1500, 1999]
    else:
        wl = _wl(n_layers=3, batch=1, seq_len_min=1200, seq_len_max=1200, budget=1024, append_per_step=700)
        lens = [1000]
    cache = inputs.make_cache(wl, DEV)
    lens_t = torch.tensor(lens, dtype=torch.int32)
    cache.seq_lens.copy_(lens_t)
    cache.host_lens[:] = lens_t.numpy()
    comp = binding.AmsCompressor(binding.config_for(wl), DEV)
    for event in range(2):
        ext = _ext(wl, 40 + event)
        snap = HostSnapshot(cache)
        credit0 = comp.ema_state.cpu().numpy()
        dst = inputs.alloc_dst_pages(cache)
        dbg = gpu_event(comp, cache, dst, inputs.SCORER_EXTERNAL, torch.from_numpy(ext).to(DEV))
        res = compare_event(snap, cache, comp, dbg, dst, credit0, ext)
        live = int((snap.lens > wl.budget).sum())
        assert len(res) == wl.n_layers * wl.n_kv_heads * live
        assert live == (len(lens) - 1 if event == 0 else len(lens))
        inputs.after_compress(cache, dst)
        if event == 0:
            inputs.append_tokens(cache, wl.append_per_step)


def test_second_device_state_is_kept_per_device():
    if torch.cuda.device_count() < 2:
        pytest.skip("one GPU visible")
    wl = _wl(batch=1, n_layers=1)
    for dev in ("cuda:0", "cuda:1"):
        with torch.cuda.device(dev):
            cache = inputs.make_cache(wl, dev)
            comp = binding.AmsCompressor(binding.config_for(wl), dev)
            dst = torch.from_numpy(inputs.alloc_dst_pages(cache)).to(dev)
            comp.compress(cache.k_pages, cache.v_pages, cache.block_table, cache.seq_lens, cache.obs_queries, wl.budget,
                          wl.n_segments, wl.scorer_id, dst)
            comp.status()
