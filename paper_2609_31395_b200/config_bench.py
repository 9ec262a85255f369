"""Per-configuration measurements behind `bench.py --all-configs`: every workload of the benchmark
definition (single layer 4K x 1; Qwen3-8B shape 32K x 1; Qwen3-30B-A3B shape 35K x 8; 64-request serving
mix with budgets from the confidence monitor; 25-round agent trace) and the twelve shapes of the paper's
kernel table (Section 8.4, Table 1: 1K -> 0.5K, 2K -> 1.5K, 6K -> 4K at 1 / 4 / 16 / 64 requests), each
as one JSON-able dict: per-stage CUDA-event times, KV tokens/s, the whole-step HBM roofline fraction
(algorithmic bytes 264 + 1032 rho per token, KV head and layer) against the measured copy bandwidth and
against 8 TB/s, and the fraction of the binding roof max(bytes / bandwidth, flops / tensor peak) / time,
with the LSE computed by the library and with the LSE supplied.

Buffer sizing and call order only; every step of the path runs in the library's kernels.
"""
from __future__ import annotations

import math
from typing import Dict, List, Optional

import torch

from . import binding as B
from . import harness as H
from . import synth

VOCAB = 151936
NOMINAL_HBM_GBS = 8000.0


def _event():
    return torch.cuda.Event(enable_timing=True)


def _roofs(tokens: int, keep: int, units_per_token: int, flops_pass: float, ms: float, passes: int, pk: dict) -> dict:
    """tokens: sum of L_r; keep: sum of n_r; units_per_token: KV heads x layers."""
    rho = keep / max(1, tokens)
    alg = (264.0 + 1032.0 * rho) * tokens * units_per_token
    t = ms * 1e-3
    t_hbm = alg / (pk["hbm_gbs"] * 1e9)
    t_tc = passes * flops_pass / (pk["tf_sustained"] * 1e12)
    return {"ms": ms, "tokens_per_s": tokens / t, "rho": rho, "algorithmic_bytes": alg,
            "hbm_roofline_frac_whole_step": t_hbm / t, "hbm_frac_of_8TBs": alg / (NOMINAL_HBM_GBS * 1e9) / t,
            "binding_roof": "tensor" if t_tc > t_hbm else "hbm", "binding_roof_frac": max(t_hbm, t_tc) / t}


class _Fixed:
    """A fixed workload (tables restored between repetitions; fresh-page compaction leaves the old pages'
    bytes intact, so the pool needs no restore)."""

    def __init__(self, wl: synth.Workload, dev, budget: Optional[torch.Tensor] = None):
        self.wl, self.dev = wl, dev
        self.inst = synth.generate(wl, dev)
        if budget is not None:
            self.inst.budget = budget
            wl.budgets = [int(b) for b in budget.cpu().tolist()]
        self.sz = H.sizes_of(self.inst)
        inst = self.inst
        self.comp = H.Compressor(inst.pool, inst.page_table, inst.seq_len, inst.free_list, inst.free_count, wl.n_q_heads,
                                 self.sz, want_lse=True)
        self.saved = [t.clone() for t in (inst.page_table, inst.seq_len, inst.free_list, inst.free_count)]

    def restore(self):
        inst = self.inst
        for dst, src in zip((inst.page_table, inst.seq_len, inst.free_list, inst.free_count), self.saved):
            dst.copy_(src)
        self.comp.status.zero_()

    def timed(self, lse_in, reps: int, warm: int = 2, inplace: bool = False, pool_backup=None) -> Dict[str, float]:
        """Mean per-stage and whole-step milliseconds of `reps` steps."""
        wl, inst, comp = self.wl, self.inst, self.comp
        acc: Dict[str, float] = {}
        for it in range(warm + reps):
            if pool_backup is not None:
                inst.pool.copy_(pool_backup)
            self.restore()
            ev = []

            def mark(name):
                e = _event()
                e.record()
                ev.append((name, e))
            mark("start")
            comp.step(inst.q, inst.win_indptr, inst.tok_indptr, inst.budget, wl.sm_scale, wl.causal, lse_in=lse_in,
                      marks=mark, inplace=inplace)
            mark("end")
            torch.cuda.synchronize()
            comp.check_status()
            if it >= warm:
                acc["total"] = acc.get("total", 0.0) + ev[0][1].elapsed_time(ev[-1][1])
                for (n0, e0), (n1, e1) in zip(ev, ev[1:]):
                    if n1 not in ("begin", "end"):
                        acc[n1] = acc.get(n1, 0.0) + e0.elapsed_time(e1)
        return {k: v / reps for k, v in acc.items()}

    def timed_graph(self, lse_in, reps: int) -> Optional[float]:
        """Whole-step milliseconds with the step captured once in a CUDA graph and replayed: for workloads of a few
        hundred microseconds, where the per-call cost of the Python harness would otherwise be what is measured.
        None when the capture fails."""
        wl, inst, comp = self.wl, self.inst, self.comp
        try:
            self.restore()
            torch.cuda.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                comp.step(inst.q, inst.win_indptr, inst.tok_indptr, inst.budget, wl.sm_scale, wl.causal, lse_in=lse_in)
            ms = []
            for it in range(3 + reps):
                self.restore()
                e0, e1 = _event(), _event()
                e0.record()
                g.replay()
                e1.record()
                torch.cuda.synchronize()
                comp.check_status()
                if it >= 3:
                    ms.append(e0.elapsed_time(e1))
            return sum(ms) / len(ms)
        except Exception:
            torch.cuda.synchronize()
            return None


    def timed_one_call(self, lse, reps: int) -> float:
        """Whole-step milliseconds through actkv_step_device: the step as ONE call of the library on inputs that are
        already on the device (`lse`: the supplied LSE, or None to have it computed)."""
        if getattr(self, "runner", None) is None:
            inst = self.inst
            self.runner = H.HostStepRunner(self.comp, inst.q, inst.win_indptr, inst.tok_indptr, inst.budget, self.wl.sm_scale,
                                           self.wl.causal)
            self.runner.stage_inputs()
        if lse is not None:
            self.comp.lse.copy_(lse)
        ms = []
        for it in range(3 + reps):
            self.restore()
            e0, e1 = _event(), _event()
            e0.record()
            self.runner.run_device(lse_supplied=lse is not None)
            e1.record()
            torch.cuda.synchronize()
            self.comp.check_status()
            if it >= 3:
                ms.append(e0.elapsed_time(e1))
        return sum(ms) / len(ms)


def _fixed_line(name: str, wl: synth.Workload, dev, pk: dict, reps: int, budget=None, scale_layers_to: Optional[int] = None,
                inplace_too: bool = False, graph: bool = False) -> dict:
    fx = _Fixed(wl, dev, budget)
    tokens = sum(wl.seq_lens)
    keep = sum(min(b, L) for b, L in zip(wl.budgets, wl.seq_lens))
    upt = wl.n_kv_heads * wl.n_layers
    flops_pass = 2.0 * sum(W * wl.group * L for W, L in zip(wl.windows, wl.seq_lens)) * wl.head_dim * upt
    path = B.actkv_score_path(fx.comp.pd, wl.n_q_heads, max(wl.windows), wl.sm_scale, fx.inst.q)
    st_int = fx.timed(None, reps)
    lse = fx.comp.lse.clone()
    st_sup = fx.timed(lse, reps)
    g_int = g_sup = None
    if graph:
        g_int, g_sup = fx.timed_graph(None, reps), fx.timed_graph(lse, reps)
    out = {"config": name, "requests": wl.n_req, "tokens": tokens, "layers_resident": wl.n_layers, "kv_heads": wl.n_kv_heads,
           "group": wl.group, "window_rows": max(wl.windows) * wl.group, "score_path": "tensor cores" if path == 1 else "fma",
           "stage_ms_lse_internal": st_int, "stage_ms_lse_supplied": st_sup,
           "lse_internal": _roofs(tokens, keep, upt, flops_pass, st_int["total"], 2, pk),
           "lse_supplied": _roofs(tokens, keep, upt, flops_pass, st_sup["total"], 1, pk)}
    if graph:
        out["graph_replay_ms_lse_internal"], out["graph_replay_ms_lse_supplied"] = g_int, g_sup
        out["one_call_ms_lse_internal"], out["one_call_ms_lse_supplied"] = fx.timed_one_call(None, reps), fx.timed_one_call(lse, reps)
    if inplace_too:
        backup = fx.inst.pool.clone()
        st_ip = fx.timed(lse, reps, inplace=True, pool_backup=backup)
        out["stage_ms_lse_supplied_inplace"] = st_ip
        out["lse_supplied_inplace_ms"] = st_ip["total"]
        del backup
    if scale_layers_to is not None and scale_layers_to != wl.n_layers:
        # layers are independent repetitions of the same work: the step over all layers takes proportionally longer
        f = scale_layers_to / wl.n_layers
        out["scaled_to_layers"] = scale_layers_to
        for k in ("lse_internal", "lse_supplied"):
            out[k + "_scaled"] = {"ms": out[k]["ms"] * f, "tokens_per_s": out[k]["tokens_per_s"] / f}
    del fx
    torch.cuda.empty_cache()
    return out


def _config4(dev, pk: dict, reps: int) -> dict:
    """64 requests, lengths log-uniform in 8K-64K, budgets from actkv_budget (256 logit rows per request,
    clamped to 15-40 % of the length); as many of the 48 layers as fit beside the logits."""
    probe = synth.config4(n_layers=1)
    free, _ = torch.cuda.mem_get_info()
    P, R = probe.page_size, probe.n_req
    used = sum(-(-L // P) for L in probe.seq_lens)
    fresh = sum(-(-(L * 2 // 5) // P) for L in probe.seq_lens)                 # budgets up to 40 %
    pages = int(math.ceil(used * probe.pool_slack)) + fresh + 8
    per_layer = pages * P * probe.n_kv_heads * probe.head_dim * 2 * 2 + sum(probe.windows) * probe.n_q_heads * probe.head_dim * 2 \
        + 2 * probe.n_kv_heads * sum(probe.seq_lens) * 4
    batch, rows = 16, 256
    logits_bytes = batch * rows * VOCAB * 4
    layers = int(max(1, min(48, (free * 0.88 - logits_bytes - 4e9) // per_layer)))
    # budgets on the device, logits in request batches through one reused buffer
    hist_cap = 512
    conf_hist = torch.zeros((R, hist_cap), dtype=torch.float32, device=dev)
    hist_len = torch.zeros(R, dtype=torch.int32, device=dev)
    seq_len = torch.tensor(probe.seq_lens, dtype=torch.int32, device=dev)
    budget_in = torch.tensor([L // 5 for L in probe.seq_lens], dtype=torch.int32, device=dev)
    budget_out = torch.zeros(R, dtype=torch.int32, device=dev)
    status = torch.zeros(4, dtype=torch.int32, device=dev)
    params = B.BudgetParams.paper_defaults(clamp_lo_ppm=150000, clamp_hi_ppm=400000)
    ws = torch.empty(B.actkv_budget_workspace_bytes(batch * rows, batch, hist_cap) + 256, dtype=torch.uint8, device=dev)
    budget_ms = 0.0
    for b0 in range(0, R, batch):
        logits, ltok = synth.confidence_logits(batch, rows, VOCAB, seed=40 + b0, device=dev)
        e0, e1 = _event(), _event()
        e0.record()
        B.actkv_budget(logits, ltok, batch * rows, VOCAB, conf_hist[b0:b0 + batch], hist_len[b0:b0 + batch], hist_cap, params,
                       seq_len[b0:b0 + batch], budget_in[b0:b0 + batch], budget_out[b0:b0 + batch], None, batch, ws, status)
        e1.record()
        torch.cuda.synchronize()
        budget_ms += e0.elapsed_time(e1)
        del logits
    assert status.cpu().tolist()[0] == 0
    del ws
    torch.cuda.empty_cache()
    wl = synth.config4(n_layers=layers)
    line = _fixed_line("c4_serving_mix_x64", wl, dev, pk, reps, budget=budget_out, scale_layers_to=48)
    line["budget_ms_all_requests"] = budget_ms
    line["budget_gbs"] = R * rows * VOCAB * 4.0 / (budget_ms * 1e-3) / 1e9
    line["note"] = (f"{layers} of 48 layers resident (all 48 need 159 GiB of KV plus fresh pages); budgets produced by "
                    f"actkv_budget, clamp 15-40 %; the *_scaled figures multiply the time by 48 / {layers}")
    return line


def _config5(dev, pk: dict, n_layers: int = 36) -> dict:
    """16 requests x 25 rounds on the Qwen3-8B shape: every round appends observation + reasoning + action
    tokens (untimed) and compresses the already-compressed cache (timed), budget 25 % of the uncompressed length.
    Fresh-page form: both LSE modes on the same state (tables restored in between).  In-place form
    (Algorithm 4): a second trace from the same seed."""
    sm_scale = 1.0 / math.sqrt(128)
    out = {"config": "c5_agent_trace_x16_25_rounds", "requests": 16, "rounds": 25, "layers_resident": n_layers}

    def one_trace(inplace: bool):
        tr = synth.AgentTrace(n_layers=n_layers, device=dev)
        tot = {"internal": 0.0, "supplied": 0.0, "lse": 0.0}
        tokens = keep_sum = moved_rows = 0
        flops_pass = 0.0
        for rnd in range(tr.n_rounds):
            q, win_indptr, tok_indptr, budget, windows, seq = tr.next_round()
            budgets = budget.cpu().tolist()
            keep = [min(b, L) for b, L in zip(budgets, seq)]
            sz = H.StepSizes(tr.R, sum(windows), max(windows), sum(seq), max(seq), max(1, sum(keep)), max(keep))
            comp = H.Compressor(tr.pool, tr.page_table, tr.seq_len, tr.free_list, tr.free_count, tr.Hkv * tr.G, sz, want_lse=True)
            saved = [t.clone() for t in (tr.page_table, tr.seq_len, tr.free_list, tr.free_count)]
            tokens += sum(seq)
            keep_sum += sum(keep)
            flops_pass += 2.0 * sum(W * tr.G * L for W, L in zip(windows, seq)) * tr.D * tr.Hkv * n_layers
            e = [_event() for _ in range(4)]
            if not inplace:
                e[0].record()
                comp.step(q, win_indptr, tok_indptr, budget, sm_scale, True)                      # LSE internal
                e[1].record()
                torch.cuda.synchronize()
                comp.check_status()
                lse = comp.lse.clone()
                for dst, src in zip((tr.page_table, tr.seq_len, tr.free_list, tr.free_count), saved):
                    dst.copy_(src)
                e[2].record()
                comp.step(q, win_indptr, tok_indptr, budget, sm_scale, True, lse_in=lse)          # LSE supplied
                e[3].record()
                torch.cuda.synchronize()
                comp.check_status()
                tot["internal"] += e[0].elapsed_time(e[1])
                tot["supplied"] += e[2].elapsed_time(e[3])
            else:
                e[0].record()
                comp.run_lse(q, win_indptr, tok_indptr, sm_scale, True, 0, n_layers, comp.lse)
                e[1].record()
                comp.step(q, win_indptr, tok_indptr, budget, sm_scale, True, lse_in=comp.lse, inplace=True)
                e[2].record()
                torch.cuda.synchronize()
                comp.check_status()
                tot["lse"] += e[0].elapsed_time(e[1])
                tot["supplied"] += e[1].elapsed_time(e[2])
                tot["internal"] += e[0].elapsed_time(e[2])
                # rows that had to move: kept indices outside the tail region of their request
                ki = comp.keep_indptr.cpu().tolist()
                for r, (L, b) in enumerate(zip(seq, budgets)):
                    if b < L:
                        start = (-(-L // tr.P) - -(-b // tr.P)) * tr.P
                        seg = comp.sel_idx[:, ki[r]:ki[r + 1]]
                        moved_rows += int(((seg < start) | (seg >= start + b)).sum())
            del comp
        upt = tr.Hkv * n_layers
        res = {"tokens": tokens, "final_uncompressed_tokens_per_request": [min(tr.uncompressed), max(tr.uncompressed)],
               "lse_internal": _roofs(tokens, keep_sum, upt, flops_pass, tot["internal"], 2, pk),
               "lse_supplied": _roofs(tokens, keep_sum, upt, flops_pass, tot["supplied"], 1, pk)}
        if inplace:
            res["rows_moved_fraction_of_kept"] = moved_rows / max(1, keep_sum * upt)
            res["bytes_moved"] = moved_rows * 4.0 * tr.D * 2
            res["note"] = ("the roofline fractions divide the algorithmic bytes of the fresh-page form (every survivor's K and V "
                           "row read and written) by the time; in place only the survivors outside the tail region move, so a "
                           "fraction above 1 means fewer bytes than that, not more bandwidth")
        else:
            res["bytes_moved"] = keep_sum * upt * 4.0 * tr.D * 2
        del tr
        torch.cuda.empty_cache()
        return res

    out["fresh_pages"] = one_trace(False)
    out["in_place"] = one_trace(True)
    return out


def _table1(dev, pk: dict, reps: int) -> List[dict]:
    cells = []
    for (L, Bk) in ((1024, 512), (2048, 1536), (6144, 4096)):
        for R in (1, 4, 16, 64):
            wl = synth.table1_case(R, L, Bk)
            line = _fixed_line(wl.name, wl, dev, pk, reps, graph=True)
            gi, gs = line["graph_replay_ms_lse_internal"], line["graph_replay_ms_lse_supplied"]
            cells.append({"config": f"table1 {L} -> {Bk}, r = {R}", "requests": R, "tokens": line["tokens"],
                          "us_graph_replay_lse_internal": None if gi is None else gi * 1e3,
                          "us_graph_replay_lse_supplied": None if gs is None else gs * 1e3,
                          "us_lse_internal": line["lse_internal"]["ms"] * 1e3, "us_lse_supplied": line["lse_supplied"]["ms"] * 1e3,
                          "us_one_call_lse_internal": line["one_call_ms_lse_internal"] * 1e3,
                          "us_one_call_lse_supplied": line["one_call_ms_lse_supplied"] * 1e3,
                          "stage_us_lse_internal": {k: v * 1e3 for k, v in line["stage_ms_lse_internal"].items()},
                          "tokens_per_s_lse_supplied": line["lse_supplied"]["tokens_per_s"],
                          "score_path": line["score_path"]})
    return cells


def run_all(dev, pk: dict, only: Optional[List[str]] = None) -> List[dict]:
    """Every configuration; `only`: subset of {"c1", "c2", "c3", "c4", "c5", "table1"}."""
    want = set(only) if only else {"c1", "c2", "c3", "c4", "c5", "table1"}
    out: List[dict] = []
    if "c1" in want:
        l1 = _fixed_line("c1_4k_x1", synth.config1(), dev, pk, reps=20, graph=True)
        for k in ("graph_replay_ms_lse_internal", "graph_replay_ms_lse_supplied", "one_call_ms_lse_internal",
                  "one_call_ms_lse_supplied"):
            v = l1.pop(k)
            l1[k.replace("_ms_", "_us_")] = None if v is None else v * 1e3
        # a step of a few kernels on 17 MB that fit in L2: bound by launch latency, reported in microseconds
        for k in ("lse_internal", "lse_supplied"):
            l1[k] = {"us": l1[k]["ms"] * 1e3, "tokens_per_s": l1[k]["tokens_per_s"]}
        l1["stage_us_lse_internal"] = {k: v * 1e3 for k, v in l1.pop("stage_ms_lse_internal").items()}
        l1["stage_us_lse_supplied"] = {k: v * 1e3 for k, v in l1.pop("stage_ms_lse_supplied").items()}
        out.append(l1)
    if "c2" in want:
        out.append(_fixed_line("c2_qwen3_8b_32k_x1", synth.config2(), dev, pk, reps=10, inplace_too=True))
    if "c3" in want:
        out.append(_fixed_line("c3_qwen3_30b_35k_x8", synth.config3(), dev, pk, reps=10, inplace_too=True))
    if "c4" in want:
        out.append(_config4(dev, pk, reps=3))
    if "c5" in want:
        out.append(_config5(dev, pk))
    if "table1" in want:
        out.extend(_table1(dev, pk, reps=20))
    return out
