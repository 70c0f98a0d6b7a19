"""GPU parity: libams (through its C ABI) against the CPU oracle on the same seeded bytes.

Bit-exact: segment boundaries, quotas, kept indices, mass, EMA credit, compacted K/V
bytes, block table and lengths, whenever both sides select on the same scores.
Within 1e-3 relative (fp32 accumulation from bf16): the scorers' scores and the mass
built from them."""
import numpy as np
import pytest
import torch

import oracle
from helpers import HostSnapshot, assert_scores_close, compare_event, gpu_event, params_of
from paper_2605_23200_b200 import binding, inputs

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _small(cfg_id, **kw):
    base = dict(n_layers=2, batch=2, seq_len_min=1500, seq_len_max=1500, budget=384)
    base.update(kw)
    return inputs.CONFIGS[cfg_id].scaled(resident_layers=0, **base)


def _ext_scores(wl, kind, seed):
    rng = np.random.default_rng(seed)
    shape = (wl.n_layers, wl.batch, wl.n_kv_heads, wl.max_seq_len)
    if kind == "lognormal":
        x = np.exp(2.0 * rng.standard_normal(shape))
    elif kind == "ties":
        x = rng.integers(0, 4, size=shape).astype(np.float64)
    elif kind == "constant":
        x = np.full(shape, 0.5)
    elif kind == "signed_nan":
        x = rng.standard_normal(shape)
        x[rng.random(shape) < 0.01] = np.nan
        x[rng.random(shape) < 0.01] = -0.0
        x[rng.random(shape) < 0.002] = np.inf
    elif kind == "spike":
        x = np.full(shape, 1e-4)
        x[..., 700] = 50.0
        x[..., 3] = 20.0
    else:
        raise ValueError(kind)
    return x.astype(np.float32)


EXT_CASES = [
    ("lognormal", dict()),
    ("lognormal", dict(n_segments=1, l_max=0, n_sink=0, n_last=0, q_min=0, ema_beta=1.0)),   # global top-k
    ("ties", dict(n_segments=7, q_min=3)),
    ("constant", dict(n_segments=10, budget=100)),
    ("signed_nan", dict(ema_beta=1.0, n_segments=16, l_min=1, l_max=64)),
    ("spike", dict(n_segments=10, l_min=16, l_max=256, budget=40, n_last=30)),
    ("lognormal", dict(seq_len_min=1000, seq_len_max=1777, batch=4, budget=1200, n_last=0)),  # ragged; some skipped
    ("lognormal", dict(budget=5, n_sink=4, n_last=16, q_min=2, n_segments=10)),               # budget below minima
    ("ties", dict(seq_len_min=9001, seq_len_max=9001, budget=2048, batch=1, n_layers=1, l_max=4096, n_segments=16)),
    # sequences that span a cluster of 2 / 4 / 8 blocks
    ("lognormal", dict(seq_len_min=20011, seq_len_max=20011, budget=3000, batch=1, n_layers=1)),
    ("ties", dict(seq_len_min=17000, seq_len_max=40000, budget=4096, batch=3, n_layers=1, l_max=4096, n_segments=16)),
    ("lognormal", dict(seq_len_min=70001, seq_len_max=70001, budget=8192, batch=1, n_layers=1, n_kv_heads=2, n_q_heads=8,
                       l_max=8192, n_segments=32)),
    ("ties", dict(seq_len_min=33000, seq_len_max=33000, budget=500, batch=1, n_layers=1, n_segments=1, l_max=0, n_sink=0,
                  n_last=0, q_min=0, ema_beta=1.0)),                                           # global top-k over 4 blocks
    ("spike", dict(seq_len_min=50000, seq_len_max=50000, budget=6000, batch=1, n_layers=1, n_kv_heads=2, n_q_heads=8)),
    ("ties", dict(seq_len_min=3000, seq_len_max=3000, budget=700, l_min=1, l_max=5, n_segments=64, q_min=2)),  # many tiny segments
    # more units than SMs (work-queue form of the segmentation kernel, row moves split with the gather kernel):
    # ragged with skipped sequences, and a budget that is not a multiple of the page size
    ("lognormal", dict(n_layers=4, batch=9, seq_len_min=500, seq_len_max=2600, budget=1203, n_last=5)),
    ("ties", dict(n_layers=5, batch=4, seq_len_min=4000, seq_len_max=9000, budget=2048, ema_beta=1.0, n_segments=12)),
    # backfill on a long sequence whose candidates all tie (the short candidate list overflows: every round re-reads the scores)
    ("constant", dict(seq_len_min=20000, seq_len_max=20000, budget=3000, batch=1, n_layers=1)),
    ("ties", dict(seq_len_min=21003, seq_len_max=21003, budget=2500, batch=1, n_layers=1, n_sink=40, n_last=300)),
    # NaN, infinities and signed zeros on a long sequence (keys of zero in the candidate search), long unsplit segments
    ("signed_nan", dict(seq_len_min=19001, seq_len_max=19001, budget=2048, batch=2, n_layers=1, ema_beta=1.0, l_max=0, n_segments=6)),
    # the smallest geometry (one page) and a few tokens more than the budget
    ("lognormal", dict(seq_len_min=16, seq_len_max=16, budget=5, batch=2, n_layers=1, n_segments=3, l_min=2, l_max=8, n_sink=1, n_last=2)),
    ("ties", dict(seq_len_min=41, seq_len_max=41, budget=40, batch=1, n_layers=2, n_segments=10)),
    # thousands of tiny segments on a long sequence (segment tables near their capacity)
    ("ties", dict(seq_len_min=30000, seq_len_max=30000, budget=9000, batch=1, n_layers=1, n_kv_heads=2, n_q_heads=8, l_min=1, l_max=17,
                  n_segments=64, q_min=2)),
    # many more must-keep positions than a block has threads (backfill count above the per-thread maxima's reach)
    ("lognormal", dict(seq_len_min=12000, seq_len_max=12000, budget=4000, batch=1, n_layers=1, n_sink=900, n_last=1200, l_max=1024)),
]


@pytest.mark.parametrize("kind,kw", EXT_CASES)
def test_external_scores_bit_exact(kind, kw):
    wl = _small(0, **kw)
    cache = inputs.make_cache(wl, DEV)
    comp = binding.AmsCompressor(binding.config_for(wl), DEV)
    ext = _ext_scores(wl, kind, 1234)
    snap = HostSnapshot(cache)
    credit0 = comp.ema_state.cpu().numpy()
    dst = inputs.alloc_dst_pages(cache)
    pool_before = inputs.as_u16(cache.k_pages)
    dbg = gpu_event(comp, cache, dst, inputs.SCORER_EXTERNAL, torch.from_numpy(ext).to(DEV))
    res = compare_event(snap, cache, comp, dbg, dst, credit0, ext)
    assert len(res) == wl.n_layers * wl.n_kv_heads * int((snap.lens > wl.budget).sum())
    # nothing outside the replacement pages was written
    mask = np.ones(cache.num_pages, bool)
    mask[dst.reshape(-1)] = False
    assert (inputs.as_u16(cache.k_pages)[:, mask] == pool_before[:, mask]).all()
    # skipped sequences keep their table row and length
    for b in range(wl.batch):
        if snap.lens[b] <= wl.budget:
            assert (cache.block_table[b].cpu().numpy() == snap.table[b]).all()
            assert int(cache.seq_lens[b]) == snap.lens[b]


def test_external_scores_multi_step_ema_and_checkpoint():
    wl = _small(2, n_layers=2, batch=3, seq_len_min=700, seq_len_max=1300, budget=256, append_per_step=64, steps=4)

    def run(restore_at=None):
        cache = inputs.make_cache(wl, DEV)
        comp = binding.AmsCompressor(binding.config_for(wl), DEV)
        keeps = []
        for step in range(wl.steps):
            if step == restore_at:           # checkpoint = copy of the credit tensor into a fresh handle
                saved = comp.ema_state.clone()
                comp = binding.AmsCompressor(binding.config_for(wl), DEV)
                comp.ema_state.copy_(saved)
            ext = _ext_scores(wl, "lognormal", 77 + step)
            snap = HostSnapshot(cache)
            credit0 = comp.ema_state.cpu().numpy()
            dst = inputs.alloc_dst_pages(cache)
            dbg = gpu_event(comp, cache, dst, inputs.SCORER_EXTERNAL, torch.from_numpy(ext).to(DEV))
            compare_event(snap, cache, comp, dbg, dst, credit0, ext)
            keeps.append(dbg.keep_idx.cpu().numpy().copy())
            inputs.after_compress(cache, dst)
            if step + 1 < wl.steps:
                inputs.append_tokens(cache, wl.append_per_step)
        return keeps, comp.ema_state.cpu().numpy()

    k1, c1 = run()
    k2, c2 = run(restore_at=2)
    assert all((a == b).all() for a, b in zip(k1, k2)) and (c1 == c2).all()
    assert (c1[..., : wl.budget] > 0).all() and (c1[..., wl.budget:] == 0).all()


def _check_scorer(wl, rtol=1e-3, atol=0.0, sample_units=None):
    cache = inputs.make_cache(wl, DEV)
    comp = binding.AmsCompressor(binding.config_for(wl), DEV)
    snap = HostSnapshot(cache)
    credit0 = comp.ema_state.cpu().numpy()
    dst = inputs.alloc_dst_pages(cache)
    dbg = gpu_event(comp, cache, dst)
    got = dbg.scores.cpu().numpy()
    mass = dbg.mass.cpu().numpy()
    units = sample_units or [(l, b, h) for l in range(wl.n_layers) for b in range(wl.batch)
                             for h in range(wl.n_kv_heads)]
    for (l, b, h) in units:
        T = int(snap.lens[b])
        if T <= wl.budget:
            continue
        if wl.scorer_id == inputs.SCORER_TOVA:
            G = wl.group
            want = oracle.score_tova(snap.k, l, h, snap.table[b], T, snap.q[l, b, h * G:(h + 1) * G], G, wl.window, True)
        else:
            want = oracle.score_keydiff(snap.k, l, h, snap.table[b], T)
        assert_scores_close(got[l, b, h, :T], want, rtol, atol)
        _, _, m_want = oracle.mass(want, wl.eps)
        # an absolute slack on a score is that slack over the sum of the weights on its mass (Eq. 1)
        sum_w = float(np.maximum(want.astype(np.float64), 0.0).sum() + wl.eps * T)
        assert_scores_close(mass[l, b, h, :T], m_want, rtol, 1e-3 * wl.eps + atol / sum_w)
    # selection on the library's own scores is exactly what the oracle selects on those scores
    compare_event(snap, cache, comp, dbg, dst, credit0, got, units=sample_units)
    return comp, cache


@pytest.mark.parametrize("window,group_heads,T,name", [
    (1, (32, 8), 1500, "rows4"),
    (1, (28, 4), 1237, "rows7_partial_page"),
    (5, (32, 8), 1500, "rows20_window"),
    (32, (32, 8), 2100, "rows128_window"),
    (24, (64, 8), 1333, "rows192_two_row_blocks"),
    (16, (32, 8), 1100, "rows64_padded_to_128"),
    (64, (64, 8), 2309, "rows512_four_row_blocks"),
    (32, (32, 8), 5000, "rows128_window_long"),
])
def test_tova_scores_and_selection(window, group_heads, T, name):
    wl = _small(0, n_layers=1, batch=2, seq_len_min=T, seq_len_max=T, window=window, n_q_heads=group_heads[0],
                n_kv_heads=group_heads[1], budget=256)
    _check_scorer(wl)


def test_tova_ragged_batch():
    wl = _small(2, n_layers=2, batch=4, seq_len_min=600, seq_len_max=2500, budget=512)
    _check_scorer(wl)


def test_tova_maximum_sequence_length():
    """131072 cached tokens (the largest supported): 1024 tiles per unit in the tensor-core scorer,
    a cluster of eight blocks in the segmentation kernel."""
    wl = _small(4, n_layers=1, batch=1, n_q_heads=4, n_kv_heads=1, window=16, seq_len_min=131072, seq_len_max=131072,
                budget=8192, n_segments=32, l_max=8192, append_per_step=0, steps=1)
    _check_scorer(wl)


def test_nothing_to_evict_leaves_everything_untouched():
    wl = _small(0, n_layers=2, batch=3, seq_len_min=600, seq_len_max=600, budget=384)
    cache = inputs.make_cache(wl, DEV)
    comp = binding.AmsCompressor(binding.config_for(wl), DEV)
    cache.seq_lens.copy_(torch.tensor([300, 384, 10], dtype=torch.int32))   # every sequence already within the budget
    k0, v0 = cache.k_pages.clone(), cache.v_pages.clone()
    table0, lens0 = cache.block_table.clone(), cache.seq_lens.clone()
    gpu_event(comp, cache, inputs.alloc_dst_pages(cache))
    assert torch.equal(cache.k_pages.view(torch.int16), k0.view(torch.int16))
    assert torch.equal(cache.v_pages.view(torch.int16), v0.view(torch.int16))
    assert torch.equal(cache.block_table, table0) and torch.equal(cache.seq_lens, lens0)
    assert float(comp.ema_state.abs().sum()) == 0.0


def test_keydiff_scores_and_selection():
    wl = _small(3, n_layers=2, batch=3, seq_len_min=900, seq_len_max=2000, budget=256, n_segments=16, l_max=250)
    _check_scorer(wl, rtol=1e-3, atol=1e-5)


def test_deterministic_and_attention_equivalence():
    wl = _small(1, n_layers=1, batch=1, seq_len_min=3000, seq_len_max=3000, budget=512, window=8)
    outs = []
    for _ in range(2):
        cache = inputs.make_cache(wl, DEV)
        comp = binding.AmsCompressor(binding.config_for(wl), DEV)
        snap = HostSnapshot(cache)
        dst = inputs.alloc_dst_pages(cache)
        dbg = gpu_event(comp, cache, dst)
        outs.append((dbg.scores[..., :3000].clone(), dbg.keep_idx.clone(), cache.k_pages.clone(), comp.ema_state.clone()))
    for a, b in zip(*outs):
        assert torch.equal(a.contiguous().view(torch.uint8), b.contiguous().view(torch.uint8))
    # attention over the compact pages equals attention over the dense gather of the kept rows
    keep = dbg.keep_idx[0, 0].long()                                    # [H][Tk]
    H, Tk = wl.n_kv_heads, wl.budget
    old_slots = torch.from_numpy(snap.table[0][np.arange(3000) // 16].astype(np.int64) * 16 + np.arange(3000) % 16).to(DEV)
    k_old = torch.from_numpy(snap.k.view(np.int16)).to(DEV).view(torch.bfloat16)[0].view(-1, H, 128)
    v_old = torch.from_numpy(snap.v.view(np.int16)).to(DEV).view(torch.bfloat16)[0].view(-1, H, 128)
    new_slots = cache.block_table[0, : Tk // 16].long().repeat_interleave(16) * 16 + torch.arange(Tk, device=DEV) % 16
    qv = torch.randn(H, 128, device=DEV, dtype=torch.float64)
    for h in range(H):
        kd = k_old[old_slots, h][keep[h]].double(); vd = v_old[old_slots, h][keep[h]].double()
        kc = cache.k_pages[0].view(-1, H, 128)[new_slots, h].double(); vc = cache.v_pages[0].view(-1, H, 128)[new_slots, h].double()
        o_dense = torch.softmax(kd @ qv[h] / 128 ** 0.5, 0) @ vd
        o_compact = torch.softmax(kc @ qv[h] / 128 ** 0.5, 0) @ vc
        assert torch.equal(o_dense, o_compact)


def test_argument_and_device_errors():
    wl = _small(0)
    cache = inputs.make_cache(wl, DEV)
    cfg = binding.config_for(wl)
    comp = binding.AmsCompressor(cfg, DEV)
    dst = torch.from_numpy(inputs.alloc_dst_pages(cache)).to(DEV)
    args = (cache.k_pages, cache.v_pages, cache.block_table, cache.seq_lens)
    with pytest.raises(binding.AmsError) as e:
        comp.compress(*args, cache.obs_queries, 0, wl.n_segments, inputs.SCORER_TOVA, dst)
    assert e.value.code == binding.AMS_ERR_INVALID_ARG
    with pytest.raises(binding.AmsError):
        comp.compress(*args, cache.obs_queries, wl.budget, 0, inputs.SCORER_TOVA, dst)
    with pytest.raises(binding.AmsError):
        comp.compress(*args, None, wl.budget, wl.n_segments, inputs.SCORER_TOVA, dst)
    with pytest.raises(binding.AmsError):
        comp.compress(*args, cache.obs_queries, wl.budget, wl.n_segments, 7, dst)
    bad = binding.config_for(wl)
    bad.head_dim = 64
    with pytest.raises(binding.AmsError):
        binding.AmsCompressor(bad, DEV)
    # a sequence longer than the configured capacity is reported by the device and skipped
    before = cache.k_pages.clone()
    lens = cache.seq_lens.clone()
    lens[0] = wl.max_seq_len + 16
    comp.compress(cache.k_pages, cache.v_pages, cache.block_table, lens, cache.obs_queries, wl.budget, wl.n_segments,
                  inputs.SCORER_TOVA, dst)
    rc, detail = comp.status(check=False)
    assert rc == binding.AMS_ERR_CAPACITY and detail[2] == wl.max_seq_len + 16
    assert int(lens[0]) == wl.max_seq_len + 16 and int(lens[1]) == wl.budget
    assert comp.status(check=False)[0] == binding.AMS_OK                 # status is cleared by reading it
    assert comp.last_launch_count >= 3


def test_event_captured_in_a_cuda_graph_replays_identically():
    """One event recorded into a CUDA graph (no allocation, no host synchronisation inside the call) and
    replayed on restored inputs gives the bytes of the directly enqueued event."""
    wl = _small(1, n_layers=2, batch=2, seq_len_min=1800, seq_len_max=2100, budget=256, window=32)
    cache = inputs.make_cache(wl, DEV)
    comp = binding.AmsCompressor(binding.config_for(wl), DEV)
    dst = torch.from_numpy(inputs.alloc_dst_pages(cache)).to(DEV)
    table0, lens0 = cache.block_table.clone(), cache.seq_lens.clone()
    dbg = comp.make_debug_views(wl.batch, wl.budget)

    def restore():
        cache.block_table.copy_(table0)
        cache.seq_lens.copy_(lens0)
        comp.ema_state.zero_()

    def event():
        comp.compress(cache.k_pages, cache.v_pages, cache.block_table, cache.seq_lens, cache.obs_queries, wl.budget,
                      wl.n_segments, wl.scorer_id, dst, dbg=dbg)

    event()                                              # direct call (also the warm-up the capture needs)
    comp.status()
    want = [t.clone() for t in (dbg.keep_idx, dbg.scores, cache.k_pages, cache.v_pages, cache.block_table,
                                cache.seq_lens, comp.ema_state)]
    restore()
    cache.k_pages[:, dst.reshape(-1).long()] = 0         # the replay must rewrite the replacement pages
    cache.v_pages[:, dst.reshape(-1).long()] = 0
    dbg.keep_idx.zero_()
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        event()
    restore()                                            # capture does not execute; state as before the event
    for _ in range(2):
        graph.replay()
        comp.status()
        got = (dbg.keep_idx, dbg.scores, cache.k_pages, cache.v_pages, cache.block_table, cache.seq_lens, comp.ema_state)
        for a, b in zip(got, want):
            assert torch.equal(a.view(torch.int16) if a.dtype == torch.bfloat16 else a,
                               b.view(torch.int16) if b.dtype == torch.bfloat16 else b)
        restore()


def test_stored_small_case_two_events():
    """The library against tests/golden/select_unit_small.json (written by the oracle alone): two consecutive events
    on caller-supplied scores with the credit carried through the compaction."""
    import importlib.util
    import json
    import os
    here = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")
    spec = importlib.util.spec_from_file_location("make_golden", os.path.join(here, "make_golden.py"))
    mg = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mg)
    gold = json.load(open(os.path.join(here, "select_unit_small.json")))
    prm = gold["params"]
    wl = inputs.CONFIGS[0].scaled(n_layers=1, batch=1, n_q_heads=1, n_kv_heads=1, seq_len_min=gold["T"], seq_len_max=gold["T"],
                                  budget=gold["Tk"], append_per_step=gold["append"], steps=2, resident_layers=0, **prm)
    cache = inputs.make_cache(wl, DEV)
    comp = binding.AmsCompressor(binding.config_for(wl), DEV)
    for event, want in enumerate(gold["events"]):
        n = want["n_tokens"]
        assert int(cache.seq_lens[0]) == n
        ext = np.zeros((1, 1, 1, wl.max_seq_len), np.float32)
        ext[0, 0, 0, :n] = mg.scores(event, n)
        dst = inputs.alloc_dst_pages(cache)
        dbg = gpu_event(comp, cache, dst, inputs.SCORER_EXTERNAL, torch.from_numpy(ext).to(DEV))
        ns = int(dbg.n_segments[0, 0, 0])
        assert ns == want["n_seg"]
        assert dbg.seg_bounds[0, 0, 0, : ns + 1].cpu().tolist() == want["bounds"]
        assert dbg.quotas[0, 0, 0, :ns].cpu().tolist() == want["quotas"]
        assert dbg.keep_idx[0, 0, 0].cpu().tolist() == want["keep_idx"]
        assert dbg.mass[0, 0, 0, :8].cpu().numpy().view(np.uint32).tolist() == want["mass_bits_first8"]
        assert comp.ema_state[0, 0, 0, :8].cpu().numpy().view(np.uint32).tolist() == want["credit_bits_first8"]
        assert abs(float(comp.ema_state[0, 0, 0].double().sum()) - want["credit_sum_f64"]) < 1e-12
        inputs.after_compress(cache, dst)
        if event == 0:
            inputs.append_tokens(cache, wl.append_per_step)
