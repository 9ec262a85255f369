"""Seeded synthetic workloads shaped like the paper's agent traces.

This module only draws inputs (pool contents, page tables, queries, budgets, logits).  It
holds none of the method's arithmetic and is the one module that both the CUDA path's tests
and the CPU oracle's tests use.  Everything is plain torch on the device asked for, so the
same call fills a B200 pool or a small CPU tensor; bits are copied from that device to the
host for the oracle, never regenerated.

Recipe (one `Workload` per benchmark configuration):
  * values: K, V ~ N(0,1) in bf16; optionally keys = sqrt(1/2) N(0,1) + sqrt(D/2) u_t with
    `n_topics` random unit "topic" directions held constant over runs of 200-2000 tokens;
  * action window: q[w, g] = (mu + eps)/sqrt(2) with mu drawn once per (layer, request, KV
    head) — action queries share a direction, which is what makes some keys action-critical;
  * planted keys: a seeded `plant_frac` of the positions of each request gets
    k = 0.5 * mean(q over that head's window rows) + N(0, 0.1);
  * page tables: "permutation" (random prefix of a random permutation), "fragmented" (random
    subset of an oversized pool in random order) or "interleaved" (logical page i of request
    r -> physical i*R + r); every page not in a table is on the free list;
  * budgets: a fixed fraction of each request's length.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import List, Optional

import torch


@dataclass
class Workload:
    name: str
    n_layers: int
    n_kv_heads: int
    group: int                       # q-heads per KV head (G)
    seq_lens: List[int]
    windows: List[int]
    budgets: List[int]
    head_dim: int = 128
    page_size: int = 16
    causal: bool = False
    table_style: str = "permutation"  # permutation | fragmented | interleaved
    pool_slack: float = 1.25          # pool pages / pages in use (before adding fresh pages)
    n_topics: int = 0
    plant_frac: float = 0.02
    seed: int = 0
    poison_tail: bool = False         # NaN bit patterns in the unused slots of last pages

    @property
    def n_req(self) -> int:
        return len(self.seq_lens)

    @property
    def n_q_heads(self) -> int:
        return self.n_kv_heads * self.group

    @property
    def sm_scale(self) -> float:
        return 1.0 / math.sqrt(self.head_dim)


@dataclass
class Instance:
    wl: Workload
    pool: torch.Tensor               # bf16 [NL, 2, n_pages, P, Hkv, D]
    page_table: torch.Tensor         # int32 [R, max_pages]
    seq_len: torch.Tensor            # int32 [R]
    free_list: torch.Tensor          # int32 [n_pages]
    free_count: torch.Tensor         # int32 [1]
    q: torch.Tensor                  # bf16 [NL, sum_win, Hq, D]
    win_indptr: torch.Tensor         # int32 [R+1]
    tok_indptr: torch.Tensor         # int32 [R+1]
    budget: torch.Tensor             # int32 [R]
    planted: List[torch.Tensor] = field(default_factory=list)   # per request, int64 positions (cpu)


def _pages_needed(L: int, P: int) -> int:
    return -(-L // P)


def make_tables(wl: Workload, device, gen_cpu: torch.Generator, extra_free_pages: int = 0):
    """Page tables, free list and pool size for a workload (host-side integer work)."""
    P, R = wl.page_size, wl.n_req
    Y = [_pages_needed(L, P) for L in wl.seq_lens]
    X = [_pages_needed(min(b, L), P) for b, L in zip(wl.budgets, wl.seq_lens)]
    used = sum(Y)
    max_pages = max(Y + [1])
    if wl.table_style == "interleaved":
        n_used_span = max_pages * R
        n_pages = n_used_span + sum(X) + extra_free_pages + 8
        rows = [[i * R + r for i in range(Y[r])] for r in range(R)]
    else:
        n_pages = int(math.ceil(used * wl.pool_slack)) + sum(X) + extra_free_pages + 8
        perm = torch.randperm(n_pages, generator=gen_cpu).tolist()
        rows, o = [], 0
        if wl.table_style == "fragmented":
            # requests take pages round-robin from the permutation, so neighbours in a table
            # are neither adjacent nor ordered in memory
            take = perm[:used]
            rows = [[] for _ in range(R)]
            r = 0
            for p in take:
                while len(rows[r]) >= Y[r]:
                    r = (r + 1) % R
                rows[r].append(p)
                r = (r + 1) % R
        else:
            for r in range(R):
                rows.append(perm[o:o + Y[r]])
                o += Y[r]
    table = torch.full((R, max_pages), -1, dtype=torch.int32)
    in_use = torch.zeros(n_pages, dtype=torch.bool)
    for r in range(R):
        if Y[r]:
            table[r, :Y[r]] = torch.tensor(rows[r], dtype=torch.int32)
            in_use[torch.tensor(rows[r], dtype=torch.int64)] = True
    free = torch.nonzero(~in_use).flatten()
    free = free[torch.randperm(free.numel(), generator=gen_cpu)].to(torch.int32)
    free_list = torch.full((n_pages,), -1, dtype=torch.int32)
    free_list[:free.numel()] = free
    return (table.to(device), torch.tensor(wl.seq_lens, dtype=torch.int32, device=device),
            free_list.to(device), torch.tensor([free.numel()], dtype=torch.int32, device=device), n_pages)


def _logical_slots(table_row: torch.Tensor, L: int, P: int) -> torch.Tensor:
    j = torch.arange(L, device=table_row.device, dtype=torch.int64)
    return table_row.to(torch.int64)[j // P] * P + j % P


def generate(wl: Workload, device="cpu", extra_free_pages: int = 0) -> Instance:
    """Draw one instance of `wl` on `device`."""
    device = torch.device(device)
    g = torch.Generator(device=device)
    g.manual_seed(1000 + wl.seed)
    g_cpu = torch.Generator()
    g_cpu.manual_seed(2000 + wl.seed)
    NL, Hkv, G, D, P, R = wl.n_layers, wl.n_kv_heads, wl.group, wl.head_dim, wl.page_size, wl.n_req
    Hq = Hkv * G
    table, seq_len, free_list, free_count, n_pages = make_tables(wl, device, g_cpu, extra_free_pages)

    win_indptr = torch.zeros(R + 1, dtype=torch.int32)
    win_indptr[1:] = torch.cumsum(torch.tensor(wl.windows, dtype=torch.int32), 0)
    tok_indptr = torch.zeros(R + 1, dtype=torch.int32)
    tok_indptr[1:] = torch.cumsum(torch.tensor(wl.seq_lens, dtype=torch.int32), 0)
    sum_win = int(win_indptr[-1])

    # planted positions: per request, shared by layers and heads
    planted = []
    for r in range(R):
        L = wl.seq_lens[r]
        n_pl = int(round(wl.plant_frac * L))
        planted.append(torch.randperm(L, generator=g_cpu)[:n_pl].sort().values if n_pl else torch.zeros(0, dtype=torch.int64))

    # topic runs per request (shared by layers and heads): topic id per token
    topic_of = []
    if wl.n_topics > 0:
        for r in range(R):
            L = wl.seq_lens[r]
            ids = torch.empty(L, dtype=torch.int64)
            pos = 0
            while pos < L:
                run = int(torch.randint(200, 2001, (1,), generator=g_cpu))
                ids[pos:pos + run] = int(torch.randint(0, wl.n_topics, (1,), generator=g_cpu))
                pos += run
            topic_of.append(ids.to(device))

    pool = torch.empty((NL, 2, n_pages, P, Hkv, D), dtype=torch.bfloat16, device=device)
    q = torch.empty((NL, sum_win, Hq, D), dtype=torch.bfloat16, device=device)
    slots = [_logical_slots(table[r], wl.seq_lens[r], P) for r in range(R)]
    for l in range(NL):
        for kv in range(2):
            flat = pool[l, kv].view(n_pages * P, Hkv, D)
            # chunked fill keeps the float32 temporary small
            step = max(1, (1 << 26) // (Hkv * D))
            for a in range(0, n_pages * P, step):
                b = min(n_pages * P, a + step)
                flat[a:b] = torch.randn((b - a, Hkv, D), generator=g, device=device, dtype=torch.float32).to(torch.bfloat16)
        kflat = pool[l, 0].view(n_pages * P, Hkv, D)
        if wl.n_topics > 0:
            u = torch.randn((wl.n_topics, Hkv, D), generator=g, device=device)
            u = u / u.norm(dim=-1, keepdim=True)
        for r in range(R):
            L, W = wl.seq_lens[r], wl.windows[r]
            if L == 0 or W == 0:
                continue
            w0 = int(win_indptr[r])
            mu = torch.randn((1, Hkv, 1, D), generator=g, device=device)
            eps = torch.randn((W, Hkv, G, D), generator=g, device=device)
            q_r = ((mu + eps) / math.sqrt(2.0)).to(torch.bfloat16)          # [W, Hkv, G, D]
            q[l, w0:w0 + W] = q_r.view(W, Hq, D)
            if wl.n_topics > 0:
                base = torch.randn((L, Hkv, D), generator=g, device=device) * math.sqrt(0.5)
                k_r = base + math.sqrt(0.5 * D) * u[topic_of[r]]
                kflat[slots[r]] = k_r.to(torch.bfloat16)
            pl = planted[r].to(device)
            if pl.numel():
                q_mean = q_r.float().mean(dim=(0, 2))                          # [Hkv, D]
                noise = 0.1 * torch.randn((pl.numel(), Hkv, D), generator=g, device=device)
                kflat[slots[r][pl]] = (0.5 * q_mean[None] + noise).to(torch.bfloat16)
    if wl.poison_tail:
        nan_bits = torch.tensor([0x7FC0], dtype=torch.int16, device=device).view(torch.bfloat16)
        for r in range(R):
            L = wl.seq_lens[r]
            if L % P:
                last = int(table[r, (L - 1) // P])
                pool[:, :, last, L % P:, :, :] = nan_bits
    budget = torch.tensor(wl.budgets, dtype=torch.int32, device=device)
    return Instance(wl, pool, table, seq_len, free_list, free_count, q,
                    win_indptr.to(device), tok_indptr.to(device), budget, planted)


def confidence_logits(n_req: int, rows_per_req: int, vocab: int, seed: int, device="cpu",
                      sharp_lo: float = 0.5, sharp_hi: float = 4.0, drift: float = 0.3):
    """Action-token logits for the confidence monitor: z = sharp_r (1 + d_r i/T) N(0,1), fp32.

    sharp_r ~ U(sharp_lo, sharp_hi) per request, drift d_r ~ U(-drift, drift) so that the
    fitted confidence slope takes both signs.  Returns (logits [R*T, V], tok_indptr [R+1]).
    """
    device = torch.device(device)
    g = torch.Generator(device=device)
    g.manual_seed(3000 + seed)
    g_cpu = torch.Generator()
    g_cpu.manual_seed(4000 + seed)
    sharp = sharp_lo + (sharp_hi - sharp_lo) * torch.rand(n_req, generator=g_cpu)
    d = drift * (2.0 * torch.rand(n_req, generator=g_cpu) - 1.0)
    T = rows_per_req
    logits = torch.empty((n_req * T, vocab), dtype=torch.float32, device=device)
    i = torch.arange(T, dtype=torch.float32)
    for r in range(n_req):
        scale = (sharp[r] * (1.0 + d[r] * i / T)).to(device)
        logits[r * T:(r + 1) * T] = torch.randn((T, vocab), generator=g, device=device) * scale[:, None]
    tok_indptr = torch.arange(0, (n_req + 1) * T, T, dtype=torch.int32, device=device)
    return logits, tok_indptr


# --------------------------------------------------------------------------------------------
# The benchmark configurations (shapes of the paper's models and traces)


def config1(seed: int = 0) -> Workload:
    """Single layer, 8 KV heads x 4, 4096 tokens, window 32, B = 1024."""
    return Workload("c1_4k_x1", 1, 8, 4, [4096], [32], [1024], table_style="permutation", seed=seed)


def config2(n_layers: int = 36) -> Workload:
    """Qwen3-8B attention shape: 36 layers, 32 q / 8 KV heads, 32768 tokens, window 64, B = 25%."""
    return Workload("c2_qwen3_8b_32k_x1", n_layers, 8, 4, [32768], [64], [8192],
                    table_style="fragmented", pool_slack=1.5, seed=2)


def config3(n_layers: int = 48, n_req: int = 8) -> Workload:
    """Qwen3-30B-A3B attention shape: 48 layers, 32 q / 4 KV heads, 8 x 35000 tokens, B = 26%."""
    return Workload("c3_qwen3_30b_35k_x8", n_layers, 4, 8, [35000] * n_req, [64] * n_req, [9100] * n_req,
                    table_style="interleaved", n_topics=64, seed=3)


def table1_case(n_req: int, L: int, B: int) -> Workload:
    """Shapes of the paper's kernel table: page 16, 8 KV heads, head_dim 128 (G = 4, W = 32 assumed)."""
    return Workload(f"t1_r{n_req}_{L}_{B}", 1, 8, 4, [L] * n_req, [32] * n_req, [B] * n_req,
                    table_style="fragmented", seed=10 + n_req)


def config4(n_layers: int = 48, n_req: int = 64, seed: int = 4) -> Workload:
    """Serving mix on the Qwen3-30B-A3B shape: lengths log-uniform in 8K-64K, shared fragmented pool.
    Budgets are placeholders (20% of length): the workload's budgets come from actkv_budget."""
    g = torch.Generator()
    g.manual_seed(5000 + seed)
    u = torch.rand(n_req, generator=g)
    lens = [int(math.exp(math.log(8192) + float(x) * (math.log(65536) - math.log(8192)))) for x in u]
    return Workload("c4_serving_mix_x64", n_layers, 4, 8, lens, [64] * n_req, [L // 5 for L in lens],
                    table_style="fragmented", pool_slack=1.05, n_topics=64, seed=seed)


class AgentTrace:
    """Iterative agent trace (Qwen3-8B attention shape): every round appends an observation, a
    reasoning segment and an action to each request's paged cache; the action tokens are the window
    (causal: the last W cached tokens) and the budget is 25% of the uncompressed tokens so far.

    The owner of pool / tables between compression steps: `next_round()` pops pages from the free
    list for the new tokens and writes their K/V (host-side integer work + torch fills, no method
    arithmetic); the compression step itself is run by the caller on the tensors held here.
    """

    def __init__(self, n_layers=36, n_kv_heads=8, group=4, n_req=16, n_rounds=25, head_dim=128, page_size=16,
                 seed=5, device="cpu", prompt=(8192, 16384), obs=(1024, 2048), reason=(200, 800), action=(32, 96),
                 budget_frac=0.25, plant_frac=0.02, max_tokens_per_req=24576):
        self.NL, self.Hkv, self.G, self.R, self.D, self.P = n_layers, n_kv_heads, group, n_req, head_dim, page_size
        self.n_rounds, self.rng_ranges = n_rounds, dict(prompt=prompt, obs=obs, reason=reason, action=action)
        self.budget_frac, self.plant_frac = budget_frac, plant_frac
        self.dev = torch.device(device)
        self.g = torch.Generator(device=self.dev)
        self.g.manual_seed(6000 + seed)
        self.g_cpu = torch.Generator()
        self.g_cpu.manual_seed(7000 + seed)
        self.max_pages = -(-max_tokens_per_req // page_size)
        # every request may hold max_tokens_per_req tokens plus the fresh pages of one compaction
        self.n_pages = int(n_req * self.max_pages * 1.6) + 8
        self.pool = torch.zeros((n_layers, 2, self.n_pages, page_size, n_kv_heads, head_dim), dtype=torch.bfloat16,
                                device=self.dev)
        self.page_table = torch.full((n_req, self.max_pages), -1, dtype=torch.int32, device=self.dev)
        self.seq_len = torch.zeros(n_req, dtype=torch.int32, device=self.dev)
        perm = torch.randperm(self.n_pages, generator=self.g_cpu).to(torch.int32)
        self.free_list = perm.to(self.dev)
        self.free_count = torch.tensor([self.n_pages], dtype=torch.int32, device=self.dev)
        self.uncompressed = [0] * n_req
        self.round = 0
        # the shared direction of each (layer, request, KV head)'s action queries persists over rounds
        self.mu = torch.randn((n_layers, n_req, n_kv_heads, 1, head_dim), generator=self.g, device=self.dev)

    def _draw(self, key):
        lo, hi = self.rng_ranges[key]
        return int(torch.randint(lo, hi + 1, (1,), generator=self.g_cpu))

    def next_round(self):
        """Appends this round's tokens; returns (q, win_indptr, tok_indptr, budget, windows, seq_lens)."""
        NL, Hkv, G, R, D, P = self.NL, self.Hkv, self.G, self.R, self.D, self.P
        seq = self.seq_len.cpu().tolist()
        table = self.page_table.cpu()
        free = self.free_list.cpu()
        fc = int(self.free_count.cpu())
        windows, new_lens = [], []
        for r in range(R):
            n_new = self._draw("obs") + self._draw("reason")
            if self.round == 0:
                n_new += self._draw("prompt")
            W = self._draw("action")
            windows.append(W)
            new_lens.append(n_new + W)
        sum_win = sum(windows)
        q = torch.empty((NL, sum_win, Hkv * G, D), dtype=torch.bfloat16, device=self.dev)
        w0 = 0
        for r in range(R):
            L0, n_new, W = seq[r], new_lens[r], windows[r]
            L1 = L0 + n_new
            assert -(-L1 // P) <= self.max_pages, "request outgrew max_tokens_per_req"
            for lp in range(-(-L0 // P), -(-L1 // P)):              # pop pages for the new tokens
                fc -= 1
                table[r, lp] = free[fc]
            j = torch.arange(L0, L1, dtype=torch.int64)
            slots = (table[r].to(torch.int64)[j // P] * P + j % P).to(self.dev)
            n_pl = int(round(self.plant_frac * (n_new - W)))
            pl = torch.randperm(n_new - W, generator=self.g_cpu)[:n_pl].to(self.dev)
            for l in range(NL):
                eps = torch.randn((W, Hkv, G, D), generator=self.g, device=self.dev)
                q_r = ((self.mu[l, r][None] + eps) / math.sqrt(2.0)).to(torch.bfloat16)     # [W, Hkv, G, D]
                q[l, w0:w0 + W] = q_r.view(W, Hkv * G, D)
                for kv in range(2):
                    vals = torch.randn((n_new, Hkv, D), generator=self.g, device=self.dev)
                    if kv == 0 and n_pl:
                        q_mean = q_r.float().mean(dim=(0, 2))
                        vals[pl] = 0.5 * q_mean[None] + 0.1 * torch.randn((n_pl, Hkv, D), generator=self.g, device=self.dev)
                    self.pool[l, kv].view(self.n_pages * P, Hkv, D)[slots] = vals.to(torch.bfloat16)
            seq[r] = L1
            self.uncompressed[r] += n_new
            w0 += W
        self.page_table.copy_(table)
        self.free_count.fill_(fc)
        self.seq_len.copy_(torch.tensor(seq, dtype=torch.int32))
        budget = [int(math.ceil(self.budget_frac * u)) for u in self.uncompressed]
        win_indptr = torch.zeros(R + 1, dtype=torch.int32)
        win_indptr[1:] = torch.cumsum(torch.tensor(windows, dtype=torch.int32), 0)
        tok_indptr = torch.zeros(R + 1, dtype=torch.int32)
        tok_indptr[1:] = torch.cumsum(torch.tensor(seq, dtype=torch.int32), 0)
        self.round += 1
        return (q, win_indptr.to(self.dev), tok_indptr.to(self.dev),
                torch.tensor(budget, dtype=torch.int32, device=self.dev), windows, seq)
