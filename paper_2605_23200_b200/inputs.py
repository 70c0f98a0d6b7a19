"""Seeded synthetic workloads for the AMS compression step.

This module only *makes inputs*: paged bf16 K/V caches, block tables, sequence
lengths, observation-window queries and the free-page bookkeeping a serving
runtime would own.  It contains none of the method's arithmetic and is the one
module that both the CUDA path's callers and the CPU oracle's callers use, so
that both sides read the same bytes.

The inputs stand in for decode traces of real models (whose weights and prompts
are not available): they take over the model geometry, the budgets and the
workload structure the paper describes — a few contiguous spans that draw
moderate, distributed attention next to a few isolated heavy-hitter tokens.

Recipe (per layer, seed = 260523200 + 10^6*config + 10^3*step + layer):
  * one unit direction per (layer, KV head), shared by spans and queries;
  * keys ~ N(0,1); six spans per (layer, sequence), span i inside the i-th sixth
    of the cache, length uniform in [64, 256], shifted by +1.5 along the
    direction; then 1 % of positions (all heads) scaled by 3;
  * queries ~ N(0,1) + 2 * direction of their KV head; values ~ N(0,1);
  * appended tokens: same, without spans;
  * query statistics for the expected-attention scorer (the mean and covariance a runtime
    would estimate from recent queries): mean = 2 * direction + 0.1 * N(0,1); covariance =
    0.5 I + sum of eight rank-one terms lambda_i u_i u_i^T, u_0 the direction, the other u_i
    random unit vectors, lambda_i uniform in [0.5, 4]; rounded to bf16;
  * pages drawn from a seeded random permutation of the pool.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace

import numpy as np
import torch

SEED_BASE = 260523200
PAGE = 16
HEAD_DIM = 128

SCORER_TOVA, SCORER_KEYDIFF, SCORER_EXTERNAL, SCORER_EXPECTED = 0, 1, 2, 3


@dataclass(frozen=True)
class Workload:
    """Geometry and hyper-parameters of one benchmark configuration."""
    name: str
    cfg_id: int
    n_layers: int
    n_q_heads: int
    n_kv_heads: int
    batch: int
    seq_len_min: int
    seq_len_max: int
    budget: int
    window: int
    scorer_id: int
    n_segments: int = 10
    l_min: int = 16
    l_max: int = 256
    q_min: int = 1
    n_sink: int = 4
    n_last: int = 16
    ema_lambda: float = 0.9
    ema_beta: float = 0.9
    eps: float = 1e-8
    steps: int = 1
    append_per_step: int = 0
    resident_layers: int = 0  # 0 = all layers resident
    pool_kernel: int = 1      # width of the average pooling of the usage scores (1 = none)
    decoupled: bool = False   # key-only base scores with the window attention as mass signal
    fixed_segments: bool = False  # ablation: equal-length instead of equal-mass segments
    uniform_quotas: bool = False  # ablation: budget shared by segment length instead of mass

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    @property
    def layers_resident(self) -> int:
        return self.resident_layers or self.n_layers

    @property
    def max_seq_len(self) -> int:
        t = max(self.seq_len_max, self.budget + self.append_per_step)
        return (t + PAGE - 1) // PAGE * PAGE

    def scaled(self, **kw) -> "Workload":
        return replace(self, **kw)


# The five benchmark configurations.  Segment count 10 is the paper's segment mass 0.1;
# where the configuration fixes the count (3, 4) the split length follows it.
CONFIGS = {
    0: Workload("cfg0_L1_T4096_k1024_w1", 0, 1, 32, 8, 1, 4096, 4096, 1024, 1, SCORER_TOVA),
    1: Workload("cfg1_llama8b_L32_T16384_k2048_w32", 1, 32, 32, 8, 1, 16384, 16384, 2048, 32, SCORER_TOVA),
    2: Workload("cfg2_qwen7b_L28_B16_ragged_k4096_w1", 2, 28, 28, 4, 16, 8192, 32768, 4096, 1, SCORER_TOVA,
                steps=20, append_per_step=128),
    3: Workload("cfg3_qwen3_8b_L36_B64_T32768_k2048_keydiff", 3, 36, 32, 8, 64, 32768, 32768, 2048, 0,
                SCORER_KEYDIFF, n_segments=16, l_max=4096, ema_beta=1.0, resident_layers=4),
    4: Workload("cfg4_llama70b_L80_T131072_k8192_w64", 4, 80, 64, 8, 1, 131072, 131072, 8192, 64,
                SCORER_TOVA, n_segments=32, l_max=8192, steps=8, append_per_step=512),
    # not one of the five benchmark configurations: the geometry of configuration 1 with the expected-attention scorer
    5: Workload("cfg5_llama8b_L32_T16384_k2048_expected", 5, 32, 32, 8, 1, 16384, 16384, 2048, 0, SCORER_EXPECTED),
}


class PagePool:
    """Free-page bookkeeping of the caller (the serving runtime's allocator)."""

    def __init__(self, num_pages: int, rng: np.random.Generator, shuffle: bool = True):
        ids = np.arange(num_pages, dtype=np.int32)
        if shuffle:
            rng.shuffle(ids)
        self._free = list(ids[::-1])
        self.num_pages = num_pages

    def alloc(self, n: int) -> np.ndarray:
        if n > len(self._free):
            raise RuntimeError("page pool exhausted")
        out = [self._free.pop() for _ in range(n)]
        return np.asarray(out, dtype=np.int32)

    def free(self, ids) -> None:
        self._free.extend(int(i) for i in ids if i >= 0)


@dataclass
class Cache:
    """Device tensors of one workload instance plus the caller-side bookkeeping."""
    wl: Workload
    k_pages: torch.Tensor       # bf16 [L][P][16][H][128]
    v_pages: torch.Tensor
    block_table: torch.Tensor   # int32 [B][max_pages]
    seq_lens: torch.Tensor      # int32 [B]
    obs_queries: torch.Tensor | None  # bf16 [L][B][Hq][W][128]
    pool: PagePool
    directions: torch.Tensor    # fp32 [L][H][128]
    step: int = 0
    host_table: np.ndarray = field(default=None)
    host_lens: np.ndarray = field(default=None)

    @property
    def num_pages(self) -> int:
        return self.k_pages.shape[1]

    @property
    def max_pages(self) -> int:
        return self.block_table.shape[1]


def _seed(cfg_id: int, step: int, layer: int) -> int:
    return SEED_BASE + 1_000_000 * cfg_id + 1_000 * step + layer


def _gen(device, seed: int) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


def _slots(table_row: np.ndarray, t0: int, t1: int, device) -> torch.Tensor:
    t = np.arange(t0, t1, dtype=np.int64)
    return torch.from_numpy(table_row[t // PAGE].astype(np.int64) * PAGE + t % PAGE).to(device)


def _fill_tokens(cache_k, cache_v, layer, slots, n_tok, H, gen, device, direction, spans, heavy):
    k = torch.randn((n_tok, H, HEAD_DIM), generator=gen, device=device, dtype=torch.float32)
    for (a, b) in spans:
        k[a:b] += 1.5 * direction
    if len(heavy):
        k[torch.from_numpy(heavy).to(device)] *= 3.0
    v = torch.randn((n_tok, H, HEAD_DIM), generator=gen, device=device, dtype=torch.float32)
    kf = cache_k[layer].view(-1, H, HEAD_DIM)
    vf = cache_v[layer].view(-1, H, HEAD_DIM)
    kf[slots] = k.to(torch.bfloat16)
    vf[slots] = v.to(torch.bfloat16)


def _make_queries(wl: Workload, step: int, directions: torch.Tensor, device) -> torch.Tensor | None:
    if wl.window <= 0:
        return None
    L = wl.layers_resident
    q = torch.empty((L, wl.batch, wl.n_q_heads, wl.window, HEAD_DIM), device=device, dtype=torch.bfloat16)
    for l in range(L):
        gen = _gen(device, _seed(wl.cfg_id, step, l) + 500)
        x = torch.randn((wl.batch, wl.n_q_heads, wl.window, HEAD_DIM), generator=gen, device=device)
        d = directions[l].repeat_interleave(wl.group, dim=0)  # [Hq][128]
        q[l] = (x + 2.0 * d[None, :, None, :]).to(torch.bfloat16)
    return q


def make_query_stats(cache: "Cache"):
    """Mean (fp32 [L][B][Hq][128]) and covariance (bf16 [L][B][Hq][128][128]) of the future queries of every
    query head, as a serving runtime would estimate them; seeded by configuration, step and layer."""
    wl = cache.wl
    device = cache.k_pages.device
    L, B, Hq = wl.layers_resident, wl.batch, wl.n_q_heads
    mean = torch.empty((L, B, Hq, HEAD_DIM), device=device, dtype=torch.float32)
    cov = torch.empty((L, B, Hq, HEAD_DIM, HEAD_DIM), device=device, dtype=torch.bfloat16)
    eye = torch.eye(HEAD_DIM, device=device)
    for l in range(L):
        gen = _gen(device, _seed(wl.cfg_id, cache.step, l) + 700)
        d = cache.directions[l].repeat_interleave(wl.group, dim=0)  # [Hq][128]
        mean[l] = 2.0 * d[None] + 0.1 * torch.randn((B, Hq, HEAD_DIM), generator=gen, device=device)
        u = torch.randn((B, Hq, 8, HEAD_DIM), generator=gen, device=device)
        u = u / u.norm(dim=-1, keepdim=True)
        u[:, :, 0] = d[None]
        lam = 0.5 + 3.5 * torch.rand((B, Hq, 8), generator=gen, device=device)
        c = 0.5 * eye + torch.einsum("bhr,bhri,bhrj->bhij", lam, u, u)
        cov[l] = c.to(torch.bfloat16)
    return mean, cov


def make_cache(wl: Workload, device="cpu", shuffle_pages: bool = True) -> Cache:
    """Build the step-0 cache of a workload on `device`."""
    device = torch.device(device)
    L, B, H = wl.layers_resident, wl.batch, wl.n_kv_heads
    rng = np.random.default_rng(_seed(wl.cfg_id, 0, 0) + 999)
    if wl.seq_len_min == wl.seq_len_max:
        lens = np.full(B, wl.seq_len_max, dtype=np.int32)
    else:
        lens = rng.integers(wl.seq_len_min, wl.seq_len_max + 1, size=B).astype(np.int32)
    n_dst = (wl.budget + PAGE - 1) // PAGE
    live = int(sum((int(t) + PAGE - 1) // PAGE for t in lens))
    grow = B * ((wl.append_per_step + PAGE - 1) // PAGE + 1)
    num_pages = int((live + 2 * B * n_dst + grow) * 1.05) + 1
    max_pages = wl.max_seq_len // PAGE
    pool = PagePool(num_pages, rng, shuffle_pages)
    table = np.full((B, max_pages), -1, dtype=np.int32)
    for b in range(B):
        n = (int(lens[b]) + PAGE - 1) // PAGE
        table[b, :n] = pool.alloc(n)

    k_pages = torch.zeros((L, num_pages, PAGE, H, HEAD_DIM), device=device, dtype=torch.bfloat16)
    v_pages = torch.zeros_like(k_pages)
    directions = torch.empty((L, H, HEAD_DIM), device=device, dtype=torch.float32)
    for l in range(L):
        gen = _gen(device, _seed(wl.cfg_id, 0, l))
        d = torch.randn((H, HEAD_DIM), generator=gen, device=device)
        directions[l] = d / d.norm(dim=-1, keepdim=True)
        srng = np.random.default_rng(_seed(wl.cfg_id, 0, l) + 77)
        for b in range(B):
            T = int(lens[b])
            spans = []
            sixth = T // 6
            for i in range(6):
                ln = int(min(srng.integers(64, 257), max(sixth, 1)))
                lo = i * sixth
                st = lo + int(srng.integers(0, max(sixth - ln, 0) + 1))
                spans.append((st, min(st + ln, T)))
            heavy = np.sort(srng.choice(T, size=int(round(0.01 * T)), replace=False)).astype(np.int64)
            _fill_tokens(k_pages, v_pages, l, _slots(table[b], 0, T, device), T, H, gen, device,
                         directions[l], spans, heavy)
    cache = Cache(wl, k_pages, v_pages, torch.from_numpy(table).to(device), torch.from_numpy(lens).to(device),
                  None, pool, directions, 0, table.copy(), lens.copy())
    cache.obs_queries = _make_queries(wl, 0, directions, device)
    return cache


def alloc_dst_pages(cache: Cache) -> np.ndarray:
    """Replacement pages for one event: int32 [B][ceil(budget/16)] (the caller's allocator)."""
    n_dst = (cache.wl.budget + PAGE - 1) // PAGE
    return np.stack([cache.pool.alloc(n_dst) for _ in range(cache.wl.batch)]).astype(np.int32)


def after_compress(cache: Cache, dst_pages: np.ndarray) -> None:
    """Caller-side bookkeeping after an event: free the old pages of every compressed
    sequence and mirror the new table row and length on the host."""
    wl = cache.wl
    n_dst = dst_pages.shape[1]
    for b in range(wl.batch):
        if cache.host_lens[b] > wl.budget:
            cache.pool.free(cache.host_table[b])
            cache.host_table[b, :] = -1
            cache.host_table[b, :n_dst] = dst_pages[b]
            cache.host_lens[b] = wl.budget
        else:
            cache.pool.free(dst_pages[b])


def append_tokens(cache: Cache, n_new: int) -> None:
    """Decode `n_new` more synthetic tokens per sequence (no spans, 1 % heavy) and draw
    fresh observation queries; advances cache.step."""
    wl = cache.wl
    cache.step += 1
    device = cache.k_pages.device
    L, B, H = wl.layers_resident, wl.batch, wl.n_kv_heads
    for b in range(B):
        t0 = int(cache.host_lens[b])
        t1 = t0 + n_new
        have = (t0 + PAGE - 1) // PAGE
        need = (t1 + PAGE - 1) // PAGE
        if need > have:
            cache.host_table[b, have:need] = cache.pool.alloc(need - have)
        cache.host_lens[b] = t1
    for l in range(L):
        gen = _gen(device, _seed(wl.cfg_id, cache.step, l))
        srng = np.random.default_rng(_seed(wl.cfg_id, cache.step, l) + 77)
        for b in range(B):
            t1 = int(cache.host_lens[b])
            t0 = t1 - n_new
            heavy = np.sort(srng.choice(n_new, size=int(round(0.01 * n_new)), replace=False)).astype(np.int64)
            _fill_tokens(cache.k_pages, cache.v_pages, l, _slots(cache.host_table[b], t0, t1, device),
                         n_new, H, gen, device, cache.directions[l], [], heavy)
    cache.block_table.copy_(torch.from_numpy(cache.host_table))
    cache.seq_lens.copy_(torch.from_numpy(cache.host_lens))
    cache.obs_queries = _make_queries(wl, cache.step, cache.directions, device)


def as_u16(t: torch.Tensor) -> np.ndarray:
    """bf16 tensor -> numpy uint16 bit patterns on the host (what the oracle reads)."""
    return t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16)
