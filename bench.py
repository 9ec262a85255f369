#!/usr/bin/env python
"""Benchmark of the ActKV compression hot path on B200.

One step = one pass of the whole path over one batch of synthetic input:
  actkv_budget (64 action-token logit rows per request) -> actkv_keep_indptr ->
  actkv_score_lse + actkv_score -> actkv_select -> actkv_compact   over all layers.
Metric: KV tokens compressed per second (tokens = cached tokens examined, counted once per
request whatever the number of layers and heads).  Default workload: the 8 x 35000-token
Qwen3-30B-A3B attention shape (48 layers, 32 q / 4 KV heads, head_dim 128, page 16, window 64,
budget 26%).

  python bench.py --gpus 1 --steps 5 --warmup 3
  python -m torch.distributed.run --nproc-per-node N ... bench.py --gpus N   (N independent replicas)
  python bench.py --impl reference     (the CPU oracle on a bounded sample of the same workload)
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

from paper_2609_31395_b200 import synth

METRIC = "KV tokens compressed/s (score+select+compact)"
UNIT = "tokens/s"
VOCAB = 151936
LOGIT_ROWS = 64          # action-token logit rows per request fed to actkv_budget each step
BUDGET_PPM = 260000      # config: budget 26% of the length (clamp of the monitor's output)


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": d["hbm_gbs"], "tf_burst": d["bf16_tflops"], "tf_sustained": d["bf16_tflops_sustained"],
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "tf_burst": 1590.0, "tf_sustained": 1400.0, "source": "fallback"}


def make_workload(name: str, layers):
    if name == "c3":
        wl = synth.config3(48 if layers is None else layers)
    elif name == "c2":
        wl = synth.config2(36 if layers is None else layers)
    elif name == "c1":
        wl = synth.config1()
    else:
        raise SystemExit(f"unknown workload {name}")
    return wl


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []          # (host time the line was read, line)
        self.t_begin = self.t_end = None

    def start(self):
        """Starts nvidia-smi (it needs a moment to produce its first sample, so this is called before
        the warm-up); only samples read between begin() and end() count."""
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "20", "-i", str(self.index)], stdout=subprocess.PIPE, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.perf_counter(), line.strip()))

    def begin(self):
        self.t_begin = time.perf_counter()

    def end(self):
        self.t_end = time.perf_counter()

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        t_lo = self.t_begin if self.t_begin is not None else -1.0
        t_hi = (self.t_end if self.t_end is not None else float("inf")) + 0.02       # a sample covers the 20 ms before it
        for t, ln in self.lines:
            if not (t_lo <= t <= t_hi):
                continue
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1]))
            except ValueError:
                continue
            for n, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def aggregate_replicas(ms_local: float, tokens_per_replica: int, world: int, dist, device):
    """Replicas only (no data-path collective): every rank compresses its own batch; the job's time
    is the slowest rank's (max over ranks), the job's throughput all replicas' tokens over that time."""
    t = torch.tensor([ms_local], dtype=torch.float64, device=device)
    if dist is not None and world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    ms_max = float(t.item())
    return ms_max, world * tokens_per_replica / (ms_max * 1e-3)


def count_inplace_moves(comp, wl) -> int:
    """Rows the in-place compaction of the last call had to move: kept indices outside the tail region
    [Start, End) of their request (counted from the index lists; reporting only)."""
    P = wl.page_size
    ki = comp.keep_indptr.cpu().tolist()
    moved = 0
    for r, (L, b) in enumerate(zip(wl.seq_lens, wl.budgets)):
        if b >= L:
            continue
        start = (-(-L // P) - -(-b // P)) * P
        seg = comp.sel_idx[:, ki[r]:ki[r + 1]]
        moved += int(((seg < start) | (seg >= start + b)).sum())
    return moved


def visible_gpu_index(local_rank: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_rank])
        except Exception:
            return local_rank
    return local_rank


# ---------------------------------------------------------------------------------------------
# the CPU oracle on a bounded sample (cpu_baseline and --impl reference)


_UNIT_CACHE = {}


def _oracle_unit(task):
    """Worker (one process per host core): the oracle's budget + score + select + compact on ONE unit of the
    workload's shape, i.e. one request x one KV head x one layer, drawn on the CPU from the unit's own seed.
    Returns the CPU seconds the call took.  The instance is built on the first call and kept."""
    (name, group, L, W, Bud, head_dim, page, causal, n_topics, seed), timed = task
    os.environ.setdefault("OMP_NUM_THREADS", "1")
    from oracle import actkv_oracle as O
    key = (name, seed)
    if key not in _UNIT_CACHE:
        torch.set_num_threads(1)
        small = synth.Workload(name + "_sample", 1, 1, group, [L], [W], [Bud], head_dim=head_dim, page_size=page,
                               causal=causal, table_style="permutation", n_topics=n_topics, seed=seed)
        inst = synth.generate(small, "cpu")
        bits = lambda t: t.contiguous().view(torch.int16).numpy().view(np.uint16)
        logits, tind = synth.confidence_logits(1, LOGIT_ROWS, VOCAB, seed=seed, device="cpu")
        _UNIT_CACHE[key] = (small, inst, bits(inst.pool), bits(inst.q), logits.numpy(), tind.numpy())
    small, inst, pool_b, q_b, logits_np, tind = _UNIT_CACHE[key]
    if not timed:
        return 0.0
    c0 = time.process_time()
    pt, sl = inst.page_table.numpy(), inst.seq_len.numpy()
    bp = O.BudgetParams(clamp_lo_ppm=BUDGET_PPM, clamp_hi_ppm=BUDGET_PPM)
    hist = np.zeros((1, 4096), dtype=np.float32)
    _, _, bud, _, _ = O.budget(logits_np, tind, hist, [0], small.budgets, bp, sl)
    sc, _, tok = O.score(pool_b, pt, sl, q_b, inst.win_indptr.numpy(), small.n_q_heads, small.sm_scale, small.causal)
    sel = [[[O.select_unit(sc[0, 0], int(bud[0]))]]]
    tables = O.Tables(pt.copy(), sl.copy(), inst.free_list.numpy().copy(), int(inst.free_count))
    O.compact(pool_b, tables, sel, bud)
    return time.process_time() - c0


class OracleSample:
    """The oracle, as it stands, on a bounded sample of the workload spread over ALL host cores: one unit
    (request x KV head x layer) per core and step, each in its own process.  Used by the cpu_baseline leg and by
    --impl reference alike (the same sample)."""

    def __init__(self, wl):
        import multiprocessing as mp
        self.wl = wl
        self.cores = os.cpu_count() or 1
        n_units_all = wl.n_req * wl.n_kv_heads * wl.n_layers
        # (at most one layer's worth of units, and at most 32 worker processes: each holds its own interpreter)
        self.n_units = max(1, min(self.cores, n_units_all, wl.n_req * wl.n_kv_heads, 32))
        # unit u: request u % R (its length, window and budget), a seed of its own
        R = wl.n_req
        self.tasks = [(wl.name, wl.group, wl.seq_lens[u % R], wl.windows[u % R], wl.budgets[u % R], wl.head_dim,
                       wl.page_size, wl.causal, wl.n_topics, wl.seed * 1000 + u) for u in range(self.n_units)]
        self.pool = mp.get_context("spawn").Pool(self.n_units)
        self.pool.map(_oracle_unit, [(t, False) for t in self.tasks], chunksize=1)      # build the instances (untimed)
        tok_units = sum(wl.seq_lens[u % R] for u in range(self.n_units))
        # a unit covers 1 / (KV heads x layers) of its request's tokens
        self.tokens_equiv = tok_units / (wl.n_kv_heads * wl.n_layers)
        self.desc = (f"{self.n_units} units (request x KV head x layer) of {n_units_all}, one per host core, each "
                     f"{wl.seq_lens[0]} tokens, window {wl.windows[0]}, budget {wl.budgets[0]}, + {LOGIT_ROWS} logit rows "
                     f"per unit's request; tokens/s scaled by the unit count")

    def step(self):
        """One step: every worker runs its unit once.  Returns (wall seconds, CPU seconds summed over workers)."""
        w0 = time.perf_counter()
        cpu = self.pool.map(_oracle_unit, [(t, True) for t in self.tasks], chunksize=1)
        return time.perf_counter() - w0, float(sum(cpu))

    def timed(self, steps):
        wall = cpu = 0.0
        for _ in range(steps):
            w, c = self.step()
            wall += w
            cpu += c
        return wall / steps, max(1, int(round(cpu / max(wall, 1e-9))))

    def close(self):
        self.pool.close()
        self.pool.join()


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    wl = make_workload(args.workload, args.layers)
    smp = OracleSample(wl)
    for _ in range(min(args.warmup, 1)):
        smp.step()
    dt, cores = smp.timed(args.steps)
    smp.close()
    v = smp.tokens_equiv / dt
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": wl.name, "note": "CPU oracle on a bounded sample per step: " + smp.desc},
        "cpu_baseline": {"value": v, "unit": UNIT, "cores": cores, "host_cores": smp.cores, "kind": "oracle",
                         "sample": smp.desc},
        "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}))


# ---------------------------------------------------------------------------------------------
# the CUDA path


def run_ours(args):
    from paper_2609_31395_b200 import binding as B
    from paper_2609_31395_b200 import harness as H

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; the CUDA path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    B.load()
    pk = peaks()

    wl = make_workload(args.workload, args.layers)
    wl.seed += 100 * rank                      # every replica draws its own batch
    R, NL, Hkv, G, D = wl.n_req, wl.n_layers, wl.n_kv_heads, wl.group, wl.head_dim
    sampler = ClockSampler(visible_gpu_index(local_rank))
    sampler.start()                            # early: nvidia-smi takes a moment to deliver its first sample
    inst = synth.generate(wl, dev)
    sz = H.sizes_of(inst)
    pipe_groups = None
    if args.pipeline and args.pipeline != "none":
        sizes = [NL // 3, NL // 3, NL - 2 * (NL // 3)] if args.pipeline == "auto" else [int(x) for x in args.pipeline.split(",")]
        sizes = [x for x in sizes if x > 0]
        if sum(sizes) != NL:
            raise SystemExit(f"--pipeline: group sizes must add up to {NL} layers")
        pipe_groups = [(sum(sizes[:i]), sum(sizes[:i + 1])) for i in range(len(sizes))]
    comp = H.Compressor(inst.pool, inst.page_table, inst.seq_len, inst.free_list, inst.free_count, wl.n_q_heads, sz,
                        layers_per_call=args.layers_per_call if args.layers_per_call else (8 if args.overlap else None),
                        want_lse=True, want_ties=True)
    # budget inputs: LOGIT_ROWS action-token logit rows per request
    logits, ltok = synth.confidence_logits(R, LOGIT_ROWS, VOCAB, seed=wl.seed, device=dev)
    n_rows = logits.shape[0]
    hist_cap = 4096
    conf_hist = torch.zeros((R, hist_cap), dtype=torch.float32, device=dev)
    hist_len = torch.zeros(R, dtype=torch.int32, device=dev)
    budget_in = torch.full((R,), 512, dtype=torch.int32, device=dev)
    budget_dev = torch.zeros(R, dtype=torch.int32, device=dev)
    ws_budget = torch.empty(B.actkv_budget_workspace_bytes(n_rows, R, hist_cap) + 256, dtype=torch.uint8, device=dev)
    bparams = B.BudgetParams.paper_defaults(clamp_lo_ppm=BUDGET_PPM, clamp_hi_ppm=BUDGET_PPM)
    assert all(b == L * BUDGET_PPM // 1000000 for b, L in zip(wl.budgets, wl.seq_lens)) or args.workload != "c3"
    if args.workload != "c3":                  # other shapes: fixed budgets, the monitor still runs
        bparams = B.BudgetParams.paper_defaults()

    saved = [t.clone() for t in (inst.page_table, inst.seq_len, inst.free_list, inst.free_count)]

    def restore():
        for dst, src in zip((inst.page_table, inst.seq_len, inst.free_list, inst.free_count), saved):
            dst.copy_(src)
        hist_len.zero_()
        comp.status.zero_()

    lse_supplied = None
    # The timed step hides the compaction of a layer group under the pooled-score kernel of the next group
    # (actkv_compact_begin / actkv_score_overlap / actkv_compact_end) unless --pipeline none; the other form
    # (one score, one select and one compact call over all layers) is timed as a secondary line.
    pipelined = pipe_groups is not None and not args.overlap
    pipe_stats = torch.zeros((len(pipe_groups) if pipe_groups else 1, 2), dtype=torch.int32, device=dev)
    pipe_comp = None
    if pipelined:
        pipe_comp = H.Compressor(inst.pool, inst.page_table, inst.seq_len, inst.free_list, inst.free_count, wl.n_q_heads,
                                 sz, layers_per_call=max(l1 - l0 for l0, l1 in pipe_groups), want_lse=False, want_ties=True,
                                 lse_layers_per_call=NL)
        pipe_comp.lse, pipe_comp.status = comp.lse, comp.status
    lrfu_state = None                          # set for the secondary LRFU-policy line only
    inplace_mode = False                       # set for the secondary in-place-compaction line only
    inplace_pipe = False                       # ... its pipelined form
    stage_names = ["budget", "lse", "score", "select", "compact"]

    def one_step(events=None):
        # events: list of (name, event); stage time = time since the previous event on the SAME stream
        # ("begin" / "begin_aux" only open an interval).  Main stream: budget, lse, score; second
        # stream (overlapped mode): select, compact.
        def mark(name, stream=None):
            if events is not None:
                e = torch.cuda.Event(enable_timing=True)
                e.record(stream if stream is not None else torch.cuda.current_stream())
                events.append((name, e))
        mark("start")
        B.actkv_budget(logits, ltok, n_rows, VOCAB, conf_hist, hist_len, hist_cap, bparams, inst.seq_len, budget_in,
                       budget_dev, None, R, ws_budget, comp.status)
        bud = budget_dev if args.workload == "c3" else inst.budget
        mark("budget")
        if args.overlap:
            n = comp.step_overlapped(inst.q, inst.win_indptr, inst.tok_indptr, bud, wl.sm_scale, wl.causal,
                                     lse_in=lse_supplied, marks=mark)
        elif pipelined and (not inplace_mode or inplace_pipe) and not (inplace_mode and lrfu_state is not None):
            n = pipe_comp.step_pipelined(inst.q, inst.win_indptr, inst.tok_indptr, bud, wl.sm_scale, wl.causal,
                                         lse_in=lse_supplied, marks=(lambda nm: mark(nm)), groups=pipe_groups,
                                         stats=pipe_stats, inplace=inplace_mode, lrfu=lrfu_state)
        else:
            n = comp.step(inst.q, inst.win_indptr, inst.tok_indptr, bud, wl.sm_scale, wl.causal,
                          lse_in=lse_supplied, marks=(lambda nm: mark(nm)), lrfu=lrfu_state, inplace=inplace_mode)
        mark("end")
        return n + 3          # the monitor: sweep, exact redo of overflowed rows, trend

    for _ in range(args.warmup):
        restore()
        one_step()
    torch.cuda.synchronize()
    comp.check_status()
    if args.lse == "supplied":
        lse_supplied = comp.lse.clone()

    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    all_events, launches = [], 0
    sampler.begin()
    t_wall0 = time.perf_counter()
    for _ in range(args.steps):
        restore()
        ev = []
        launches = one_step(ev)
        all_events.append(ev)
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    t_wall = time.perf_counter() - t_wall0
    sampler.end()
    clocks = sampler.stop()
    comp.check_status()

    # ties at the k-th threshold, as actkv_select reported them for the units of the last call of the timed step
    tie_t = (pipe_comp if pipelined else comp).ties.cpu()
    n_eq_total, n_eq_kept = tie_t[:, 2], tie_t[:, 1]
    ties_line = {"units_reported": int(tie_t.shape[0]), "units_with_a_tie_at_the_threshold": int((n_eq_total > n_eq_kept).sum()),
                 "entries_equal_to_the_threshold": int(n_eq_total.sum()), "of_them_kept": int(n_eq_kept.sum())}
    stage_ms = {k: 0.0 for k in stage_names}
    total_ms = 0.0
    aux_names = ("begin_aux", "select", "compact") if args.overlap else ()
    for ev in all_events:
        total_ms += ev[0][1].elapsed_time(ev[-1][1])
        prev_main, prev_aux = ev[0][1], None
        for name, e in ev[1:]:
            if name in aux_names:
                if name != "begin_aux":
                    stage_ms[name] += prev_aux.elapsed_time(e)
                prev_aux = e
            else:
                if name not in ("begin", "end"):
                    stage_ms[name] += prev_main.elapsed_time(e)
                prev_main = e
    ms_per_step = total_ms / args.steps
    stage_ms = {k: v / args.steps for k, v in stage_ms.items()}
    tokens = sum(wl.seq_lens)
    ms_max, value = aggregate_replicas(ms_per_step, tokens, world, dist, dev)

    # ---- roofline of the dominant kernel --------------------------------------------------------
    rho = sum(min(b, L) for b, L in zip(wl.budgets, wl.seq_lens)) / max(1, tokens)
    flops_pass = 2.0 * sum(W * G * L for W, L in zip(wl.windows, wl.seq_lens)) * D * Hkv * NL
    bytes_k = 2.0 * D * tokens * Hkv * NL
    alg_bytes = (264.0 + 1032.0 * rho) * tokens * Hkv * NL
    n_calls = len(pipe_groups) if pipelined else -(-NL // comp.lpc)
    stages = {
        "lse": {"bound": "tensor", "achieved": flops_pass / (stage_ms["lse"] * 1e-3) / 1e12 if stage_ms["lse"] else None,
                "peak": pk["tf_sustained"], "unit": "TFLOP/s"},
        "score": {"bound": "tensor", "achieved": flops_pass / (stage_ms["score"] * 1e-3) / 1e12, "peak": pk["tf_sustained"],
                  "unit": "TFLOP/s"},
        "compact": {"bound": "hbm", "achieved": 1024.0 * rho * tokens * Hkv * NL / (stage_ms["compact"] * 1e-3) / 1e9,
                    "peak": pk["hbm_gbs"], "unit": "GB/s"},
        "budget": {"bound": "hbm", "achieved": 4.0 * n_rows * VOCAB / (stage_ms["budget"] * 1e-3) / 1e9,
                   "peak": pk["hbm_gbs"], "unit": "GB/s"},
    }
    if pipelined:
        # the copies run inside the pooled-score kernels; "compact" times only what was left for the drain kernel
        stages["compact"].update({"achieved": None, "note": "hidden under the pooled-score kernels of the next layer group; "
                                                             "stage_ms.compact is the part that was not"})
        stages["score"]["note"] = "with the copies of the previous layer group inside"
    for s in stages.values():
        s["frac"] = None if s["achieved"] is None else s["achieved"] / s["peak"]
    dom = max(("lse", "score", "compact"), key=lambda k: stage_ms[k])
    if pipelined and dom == "lse":
        n_calls = -(-NL // pipe_comp.lse_lpc)      # the LSE pass of the pipelined step: all layers per launch
    roofline = dict(stages[dom])
    # DRAM bytes per (token, KV head, layer) of each kernel, measured with ncu on a small cut of the workload and kept
    # in a data file beside the capture's summary; scaled to one launch of this run by its unit count (traffic grows
    # in proportion to the units processed).  null when the file has no entry for the kernel this run launched.
    traffic, traffic_src = None, None
    kernel_of = {"lse": "score_tc_lse_kernel", "score": "score_tc_pool_kernel", "compact": "compact_copy_kernel"}
    tpath = os.path.join(ROOT, "profiles", f"traffic_{args.workload}.json")
    if os.path.exists(tpath):
        tj = json.load(open(tpath))
        ent = tj.get("kernels", {}).get(kernel_of[dom])
        if ent is not None and tj.get("library_version") == B.actkv_version():
            per_unit = ent["dram_bytes_per_unit"]
            ent2 = tj["kernels"].get(kernel_of[dom] + "_with_copies")
            if pipelined and dom == "score" and ent2 is not None:
                # every launch but the first carries the copies of the group before it
                g0 = (pipe_groups[0][1] - pipe_groups[0][0]) / NL
                per_unit = g0 * per_unit + (1.0 - g0) * ent2["dram_bytes_per_unit"]
            traffic = per_unit * tokens * Hkv * NL / n_calls
            traffic_src = tj.get("capture")
    roofline.update({"kernel": dom, "kernel_name": kernel_of[dom], "launches_per_step": n_calls,
                     "ms_per_launch": stage_ms[dom] / n_calls,
                     "traffic": traffic, "traffic_unit": "bytes per launch (ncu dram__bytes_read.sum + dram__bytes_write.sum of a "
                                                         "small capture, scaled by the units processed)",
                     "traffic_capture": traffic_src, "peak_source": pk["source"] + (" sustained bf16" if stages[dom]["bound"] == "tensor" else " copy")})
    hbm_frac_whole = alg_bytes / (ms_max * 1e-3) / 1e9 / pk["hbm_gbs"]
    # The LSE pass evaluates one exp2 per (window row, key): besides the contraction it is bound by the
    # special function units, 16 results per clock per SM on 148 SMs at the maximum SM clock.
    n_exp = sum(W * G * L for W, L in zip(wl.windows, wl.seq_lens)) * Hkv * NL
    exp_peak = 148 * 16 * (clocks.get("sm_max_mhz") or 1965.0) * 1e6 / 1e9
    lse_exp = None
    if stage_ms["lse"]:
        ach = n_exp / (stage_ms["lse"] * 1e-3) / 1e9
        lse_exp = {"bound": "alu", "achieved": ach, "peak": exp_peak, "unit": "Gexp2/s", "frac": ach / exp_peak,
                   "kernel": "lse", "peak_source": "148 SMs x 16 MUFU results per clock x the maximum SM clock"}
        if clocks.get("sm_mhz"):
            # the same against the clock the SMs actually ran at under the power cap (median of the samples taken
            # during the timed region, all phases of the step): how close the kernel is to the unit's limit there
            lse_exp["frac_at_sampled_clock"] = ach / (148 * 16 * clocks["sm_mhz"] * 1e6 / 1e9)
            lse_exp["sampled_sm_mhz"] = clocks["sm_mhz"]

    # ---- end to end: host buffers in, host results out, every step -------------------------------
    e2e = None
    if not args.no_e2e:
        # restore the device tables first: the runner snapshots them as the host-side state of the engine
        restore()
        torch.cuda.synchronize()
        runner = H.HostStepRunner(pipe_comp if pipelined else comp, inst.q, inst.win_indptr, inst.tok_indptr, budget_in, wl.sm_scale, wl.causal,
                                  logits=logits, logit_indptr=ltok, hist_cap=hist_cap, params=bparams)
        h2d, d2h = runner.h2d_bytes, runner.d2h_bytes
        e2e_ms = []
        for it in range(1 + min(args.steps, 5)):
            torch.cuda.synchronize()
            if dist is not None:
                dist.barrier()
            t0 = time.perf_counter()
            out = runner.run()                 # one C-ABI call: H2D copies, the whole path, D2H copies, stream sync
            if it > 0:
                e2e_ms.append((time.perf_counter() - t0) * 1e3)
            if out["st"].tolist()[0] != 0:
                raise SystemExit(f"actkv_step_host: device status {out['st'].tolist()}")
        te = torch.tensor([sum(e2e_ms) / len(e2e_ms)], dtype=torch.float64, device=dev)
        if dist is not None:
            dist.all_reduce(te, op=dist.ReduceOp.MAX)
        e2e = {"value": world * tokens / (float(te.item()) * 1e-3), "unit": UNIT, "ms_per_step": float(te.item()),
               "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h),
               "note": "one actkv_step_host call per step: queries, logits, index arrays, tables and budgets come from "
                       "pinned host memory, new tables / free list / budgets / status go back; the KV pool stays "
                       "resident in HBM (it is the cache being compressed)"}

    # ---- the same step when the attention backend hands the LSE over (the paper's own mode, Section 7.1):
    # reported beside the headline, which computes the LSE itself
    lse_supplied_line = None
    if args.lse == "internal" and not args.no_secondary:
        lse_supplied = comp.lse.clone()
        ms = []
        for it in range(2 + min(args.steps, 5)):
            restore()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            one_step()
            e1.record()
            torch.cuda.synchronize()
            if it >= 2:
                ms.append(e0.elapsed_time(e1))
        lse_supplied = None
        tl = torch.tensor([sum(ms) / len(ms)], dtype=torch.float64, device=dev)
        if dist is not None:
            dist.all_reduce(tl, op=dist.ReduceOp.MAX)
        lse_supplied_line = {"ms_per_step": float(tl.item()), "value": world * tokens / (float(tl.item()) * 1e-3),
                             "unit": UNIT, "hbm_roofline_frac_whole_step":
                                 alg_bytes / (float(tl.item()) * 1e-3) / 1e9 / pk["hbm_gbs"]}
        comp.check_status()

    # ---- the other form of the step (one score / select / compact call over all layers when the timed step is the
    # pipelined one, and the other way round), both LSE modes
    other_line = None
    if pipe_groups is not None and not args.overlap and not args.no_secondary:
        was = pipelined
        pipelined = not was
        other_line = {"form": "one call per stage over all layers" if was else "pipelined",
                      "groups": None if was else [l1 - l0 for l0, l1 in pipe_groups]}
        for mode in ("internal", "supplied"):
            lse_supplied = comp.lse.clone() if mode == "supplied" else None
            ms = []
            for it in range(2 + min(args.steps, 5)):
                restore()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                one_step()
                e1.record()
                torch.cuda.synchronize()
                if it >= 2:
                    ms.append(e0.elapsed_time(e1))
            comp.check_status()
            tl = torch.tensor([sum(ms) / len(ms)], dtype=torch.float64, device=dev)
            if dist is not None:
                dist.all_reduce(tl, op=dist.ReduceOp.MAX)
            other_line[mode] = {"ms_per_step": float(tl.item()), "value": world * tokens / (float(tl.item()) * 1e-3), "unit": UNIT,
                                "hbm_roofline_frac_whole_step": alg_bytes / (float(tl.item()) * 1e-3) / 1e9 / pk["hbm_gbs"]}
        lse_supplied = None
        pipelined = was

    # ---- the same step ranking by the attention-aware LRFU keep-score (Section 5.1): score -> keepscore
    # -> select -> gather keep-scores -> compact, p = 0.9, lambda = 0.5, 512 protected tokens per request
    lrfu_line = None
    if not args.overlap and not args.no_lrfu:
        lrfu_state = H.LrfuState(NL * Hkv, sz, dev, 0.9, 0.5,
                                 torch.full((R,), 512, dtype=torch.int32, device=dev))
        lrfu_state.keep_score.uniform_(0.0, 1e-3, generator=torch.Generator(device=dev).manual_seed(wl.seed))
        ms, ks_ms = [], []
        for it in range(2 + min(args.steps, 5)):
            restore()
            ev = []
            one_step(ev)
            torch.cuda.synchronize()
            if it >= 2:
                ms.append(ev[0][1].elapsed_time(ev[-1][1]))
                ks_ms.append(sum(ev[i - 1][1].elapsed_time(ev[i][1]) for i in range(1, len(ev))
                                 if ev[i][0] == "keepscore"))
        lrfu_state = None
        tl = torch.tensor([sum(ms) / len(ms)], dtype=torch.float64, device=dev)
        if dist is not None:
            dist.all_reduce(tl, op=dist.ReduceOp.MAX)
        ks = sum(ks_ms) / len(ks_ms)
        # algorithmic bytes of the keep-score stage: score read + KS read + KS write + key write
        ks_bytes = 16.0 * tokens * Hkv * NL
        lrfu_line = {"ms_per_step": float(tl.item()), "value": world * tokens / (float(tl.item()) * 1e-3), "unit": UNIT,
                     "keepscore_ms": ks, "keepscore_gbs": ks_bytes / (ks * 1e-3) / 1e9,
                     "keepscore_frac_of_hbm_peak": ks_bytes / (ks * 1e-3) / 1e9 / pk["hbm_gbs"],
                     "keepscore_stage": "keep-score update and TopK in one launch (actkv_keepscore_select); the separate "
                                        "select stage is empty",
                     "top_p": 0.9, "lambda": 0.5, "n_protect": 512,
                     "form": "pipelined like the timed step" if pipelined else "one call per stage"}
        comp.check_status()
        if pipe_comp is not None:
            pipe_comp.check_status()

    # ---- streaming form (Algorithm 3 as triggered per decode step): one action query per request per call,
    # LSE supplied, running mean updated in place; all layers in one call.  Bound by the K reads.
    stream_line = None
    if not args.no_stream and comp.lse is not None:
        restore()
        first = inst.win_indptr[:-1].to(torch.int64)
        q1 = inst.q[:, first].contiguous()
        lse1 = comp.lse[:, first].contiguous()
        win1 = torch.arange(R + 1, dtype=torch.int32, device=dev)
        steps1 = torch.ones(R, dtype=torch.int32, device=dev)
        run_io = torch.zeros((NL, Hkv, sz.sum_tok), dtype=torch.float32, device=dev)
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
        n_it = 3 + min(args.steps, 10)
        for it in range(n_it):
            if it == 3:
                ev[0].record()
            B.actkv_score_accumulate(comp.pd, comp.td, 0, NL, q1, win1, wl.n_q_heads, lse1, wl.sm_scale, wl.causal,
                                     inst.tok_indptr, steps1, run_io, R, 1, sz.sum_tok, sz.max_tok, comp.ws_score,
                                     comp.status)
        ev[1].record()
        torch.cuda.synchronize()
        comp.check_status()
        ms1 = ev[0].elapsed_time(ev[1]) / (n_it - 3)
        st_bytes = (2.0 * D + 8.0) * tokens * Hkv * NL          # K row read + running mean read and write
        stream_line = {"ms_per_call": ms1, "value": world * tokens / (ms1 * 1e-3), "unit": "KV tokens examined/s",
                       "gbs": st_bytes / (ms1 * 1e-3) / 1e9, "frac_of_hbm_peak": st_bytes / (ms1 * 1e-3) / 1e9 / pk["hbm_gbs"],
                       "queries_per_request": 1, "layers_per_call": NL}
        del run_io

    # ---- the confidence monitor on a serving-mix sized batch of logit rows (64 requests x 64 action tokens,
    # 2.5 GB): the 512 rows of the step above are too few launches to show the kernel's rate.
    budget_line = None
    if not args.no_stream:
        Rb, Tb = 64, 64
        lg, lt = synth.confidence_logits(Rb, Tb, VOCAB, seed=wl.seed + 7, device=dev)
        ch = torch.zeros((Rb, hist_cap), dtype=torch.float32, device=dev)
        hl = torch.zeros(Rb, dtype=torch.int32, device=dev)
        sl = torch.full((Rb,), 35000, dtype=torch.int32, device=dev)
        bi = torch.full((Rb,), 512, dtype=torch.int32, device=dev)
        bo = torch.zeros(Rb, dtype=torch.int32, device=dev)
        wsb = torch.empty(B.actkv_budget_workspace_bytes(Rb * Tb, Rb, hist_cap) + 256, dtype=torch.uint8, device=dev)
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
        n_it = 3 + min(args.steps, 10)
        for it in range(n_it):
            if it == 3:
                ev[0].record()
            hl.zero_()
            B.actkv_budget(lg, lt, Rb * Tb, VOCAB, ch, hl, hist_cap, B.BudgetParams.paper_defaults(), sl, bi, bo, None,
                           Rb, wsb, comp.status)
        ev[1].record()
        torch.cuda.synchronize()
        comp.check_status()
        msb = ev[0].elapsed_time(ev[1]) / (n_it - 3)
        gb = 4.0 * Rb * Tb * VOCAB / (msb * 1e-3) / 1e9
        budget_line = {"ms_per_call": msb, "rows": Rb * Tb, "vocab": VOCAB, "gbs": gb, "frac_of_hbm_peak": gb / pk["hbm_gbs"]}
        del lg, ch, wsb

    # ---- the same step compacting in place into the tail blocks (Algorithm 4) instead of fresh pages.
    # Run last: it overwrites evicted slots of the original layout, which the fresh-page form never does.
    inplace_line = None
    if not args.overlap and not args.no_inplace:
        inplace_mode = True
        ms, cp_ms = [], []
        pool_backup = inst.pool.clone()        # the pool is restored (untimed) before every in-place step
        for it in range(2 + min(args.steps, 5)):
            inst.pool.copy_(pool_backup)
            restore()
            ev = []
            one_step(ev)
            torch.cuda.synchronize()
            if it >= 2:
                ms.append(ev[0][1].elapsed_time(ev[-1][1]))
                cp_ms.append(sum(ev[i - 1][1].elapsed_time(ev[i][1]) for i in range(1, len(ev))
                                 if ev[i][0] == "compact"))
        comp.check_status()
        # rows that had to move: survivors outside the tail region, counted from the last step's lists
        moved = count_inplace_moves(comp, wl)
        tl = torch.tensor([sum(ms) / len(ms)], dtype=torch.float64, device=dev)
        if dist is not None:
            dist.all_reduce(tl, op=dist.ReduceOp.MAX)
        cp = sum(cp_ms) / len(cp_ms)
        moved_bytes = 4.0 * D * 2 * moved * (-(-NL // comp.lpc))      # K and V rows, read + write, bf16; lists of the last call
        # ... and with the LSE supplied as well: the paper's own mode (Section 7.1) with the paper's own compaction
        # (Algorithm 4), the cheapest step the library has
        lse_supplied = comp.lse.clone()
        ms2 = []
        for it in range(2 + min(args.steps, 5)):
            inst.pool.copy_(pool_backup)
            restore()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            one_step()
            e1.record()
            torch.cuda.synchronize()
            if it >= 2:
                ms2.append(e0.elapsed_time(e1))
        # ... and both with the moves of a layer group inside the pooled-score kernel of the next one
        pipe_ip = None
        if pipelined:
            inplace_pipe = True
            tp = []
            for mode in ("internal", "supplied"):
                lse_supplied = comp.lse.clone() if mode == "supplied" else None
                ms3 = []
                for it in range(2 + min(args.steps, 5)):
                    inst.pool.copy_(pool_backup)
                    restore()
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    e0.record()
                    one_step()
                    e1.record()
                    torch.cuda.synchronize()
                    if it >= 2:
                        ms3.append(e0.elapsed_time(e1))
                t3 = torch.tensor([sum(ms3) / len(ms3)], dtype=torch.float64, device=dev)
                if dist is not None:
                    dist.all_reduce(t3, op=dist.ReduceOp.MAX)
                tp.append(float(t3.item()))
            inplace_pipe = False
            pipe_comp.check_status()
            pipe_ip = {"groups": [l1 - l0 for l0, l1 in pipe_groups],
                       "ms_per_step": tp[0], "value": world * tokens / (tp[0] * 1e-3), "unit": UNIT,
                       "with_lse_supplied": {"ms_per_step": tp[1], "value": world * tokens / (tp[1] * 1e-3), "unit": UNIT,
                                             "hbm_roofline_frac_whole_step_fresh_page_bytes": alg_bytes / (tp[1] * 1e-3) / 1e9 / pk["hbm_gbs"]}}
        lse_supplied = None
        inplace_mode = False
        del pool_backup
        comp.check_status()
        t2 = torch.tensor([sum(ms2) / len(ms2)], dtype=torch.float64, device=dev)
        if dist is not None:
            dist.all_reduce(t2, op=dist.ReduceOp.MAX)
        inplace_line = {"ms_per_step": float(tl.item()), "value": world * tokens / (float(tl.item()) * 1e-3), "unit": UNIT,
                        "with_lse_supplied": {"ms_per_step": float(t2.item()),
                                              "value": world * tokens / (float(t2.item()) * 1e-3), "unit": UNIT},
                        "compact_ms": cp, "rows_moved_fraction_of_kept": moved / max(1.0, rho * tokens * Hkv * comp.lpc),
                        "compact_gbs": moved_bytes / (cp * 1e-3) / 1e9,
                        "compact_frac_of_hbm_peak": moved_bytes / (cp * 1e-3) / 1e9 / pk["hbm_gbs"],
                        "pipelined": pipe_ip}

    # ---- the oracle on the host cores (rank 0, single GPU only) ----------------------------------
    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        smp = OracleSample(make_workload(args.workload, args.layers))
        n_rep = 3
        dt, cores = smp.timed(n_rep)
        smp.close()
        cpu_baseline = {"value": smp.tokens_equiv / dt, "unit": UNIT, "cores": cores, "host_cores": smp.cores,
                        "kind": "oracle", "sample": smp.desc, "seconds": n_rep * dt}

    if rank == 0:
        out = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_max, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": wl.name, "requests": R, "tokens_per_request": wl.seq_lens[0], "layers": NL,
                       "kv_heads": Hkv, "q_heads": wl.n_q_heads, "head_dim": D, "page": wl.page_size,
                       "window": wl.windows[0], "budget": wl.budgets[0], "lse": args.lse,
                       "layers_per_call": pipe_comp.lpc if pipelined else comp.lpc, "replicas": world,
                       "overlap": "select+compact of a layer group on a second stream under the score kernels "
                                  "of the next group" if args.overlap else
                                  ("copies of a layer group inside the pooled-score kernel of the next one, groups of "
                                   + "+".join(str(l1 - l0) for l0, l1 in pipe_groups) + " layers (one stream)"
                                   if pipelined else "none (one stream)"),
                       "l2": "inputs (KV pool %.1f GB) far larger than the 126 MB L2" % (inst.pool.numel() * 2 / 1e9)},
            "stage_ms": stage_ms, "hbm_roofline_frac_whole_step": hbm_frac_whole,
            "hbm_roofline_frac_whole_step_of_nominal_8TBs": alg_bytes / (ms_max * 1e-3) / 8e12,
            "hbm_roofline_target": {"north_star": 0.70, "met": bool(hbm_frac_whole >= 0.70)},
            "with_lse_supplied": lse_supplied_line, "other_step_form": other_line,
            "copy_items_taken_by_score_kernels": ([round(b / a, 3) if a else None for a, b in pipe_stats.cpu().tolist()]
                                                  if pipelined else None),
            "with_lrfu_policy": lrfu_line,
            "with_inplace_compaction": inplace_line, "streaming_update": stream_line,
            "algorithmic_bytes_per_step": alg_bytes, "k_bytes_per_pass": bytes_k,
            "roofline": roofline, "roofline_stages": stages, "roofline_lse_exp_rate": lse_exp,
            "budget_4096_rows": budget_line,
            "cpu_baseline": cpu_baseline, "e2e": e2e,
            "ties_at_threshold": ties_line,
            "clocks": clocks, "gpu_launches": launches, "wall_s_timed_region": t_wall,
        }
    if dist is not None:
        dist.destroy_process_group()
    return out if rank == 0 else None


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c3", choices=["c1", "c2", "c3"])
    ap.add_argument("--layers", type=int, default=None, help="override the layer count (debugging only)")
    ap.add_argument("--layers-per-call", type=int, default=None,
                    help="layers per score/select/compact call (default: 8 when overlapped, else all)")
    ap.add_argument("--overlap", action="store_true",
                    help="run select + compact of a layer group on a second stream under the score kernels of the "
                         "next group (measured: no gain, the score CTAs fill the register file of every SM)")
    ap.add_argument("--pipeline", default="auto",
                    help="layer groups of the timed step, whose copies run inside the pooled-score kernel of the next group: "
                         "'auto' (three equal groups), comma-separated group sizes, or 'none' (one call per stage)")
    ap.add_argument("--lse", default="internal", choices=["internal", "supplied"])
    ap.add_argument("--all-configs", action="store_true",
                    help="after the timed workload, measure every configuration of the benchmark definition and the "
                         "paper's kernel-table shapes (adds a per_config list; takes several minutes)")
    ap.add_argument("--configs", default=None, help="like --all-configs for a subset: c1,c2,c3,c4,c5,table1")
    ap.add_argument("--no-secondary", action="store_true",
                    help="only the timed step: none of the secondary lines (LSE supplied, other step form, LRFU, in place, "
                         "streaming, monitor batch, end to end, CPU baseline); for launch lists")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-lrfu", action="store_true", help="skip the secondary LRFU-policy line")
    ap.add_argument("--no-inplace", action="store_true", help="skip the secondary in-place-compaction line")
    ap.add_argument("--no-stream", action="store_true", help="skip the secondary streaming-update line")
    args = ap.parse_args()
    if args.no_secondary:
        args.no_e2e = args.no_cpu_baseline = args.no_lrfu = args.no_inplace = args.no_stream = True
    if args.warmup < 3 and args.impl == "ours":
        print("note: fewer than 3 warm-up steps", file=sys.stderr)
    if args.impl == "reference":
        run_reference(args)
        return
    out = run_ours(args)
    if out is not None and (args.all_configs or args.configs) and out["n_gpus"] == 1:
        # every other configuration of the benchmark definition, one after the other on the freed device
        import gc
        from paper_2609_31395_b200 import config_bench
        gc.collect()
        torch.cuda.empty_cache()
        out["per_config"] = config_bench.run_all(torch.device("cuda", 0), peaks(),
                                                 args.configs.split(",") if args.configs else None)
    if out is not None:
        print(json.dumps(out))


if __name__ == "__main__":
    main()
