"""Developer tool: per-job timestamps of one CTA of the two tensor-core score kernels, and the SM clock
inside them.

    python -m paper_2609_31395_b200.dev_trace [--layers 32] [--loop 25]

Builds the sources a second time with -DACTKV_LSE_TRACE -DACTKV_POOL_TRACE (into libactkv_trace.so beside
the library; the product library is untouched), runs the LSE pass and the pooled-score pass of the bench
shape `--loop` times and prints, for CTA 200 of the last launch of each:
  * the SM clock inside the kernel (clock64 over the nanosecond timer around the CTA), every few iterations:
    under the power cap it is far below what nvidia-smi reports for the whole step;
  * LSE pass (Section 7.1, LSE equation): cycles per pair of jobs of one epilogue group, its fold time and
    the time to fetch the next accumulator, and the phase between the two groups;
  * pooled-score pass (Algorithm 3 steps 4-5): cycles per job, how long the MMA issuer waits for an
    accumulator, and where an epilogue warp spends a job (waiting, holding the accumulator, folding, end-of-tile
    work).
A job is one (key tile, row block) product; the stamps themselves cost the traced CTA some 40 cycles each.
"""
from __future__ import annotations

import argparse
import ctypes
import os

import numpy as np


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--layers", type=int, default=32)
    ap.add_argument("--loop", type=int, default=25)
    args = ap.parse_args()
    from . import build
    lib_path = os.path.join(build.HERE, "libactkv_trace.so")
    build.build(out=lib_path, extra_flags=["-DACTKV_LSE_TRACE", "-DACTKV_POOL_TRACE"])
    os.environ["ACTKV_LIB"] = lib_path
    import torch
    from . import binding as B, harness as H, synth
    lib = B.load()
    dev = torch.device("cuda", 0)
    wl = synth.config3(args.layers)
    inst = synth.generate(wl, dev)
    comp = H.Compressor(inst.pool, inst.page_table, inst.seq_len, inst.free_list, inst.free_count, wl.n_q_heads,
                        H.sizes_of(inst), want_lse=True)

    def read(fn, rows):
        out = np.zeros((rows, 1024), dtype=np.int64)
        fn.argtypes = [ctypes.c_void_p]
        if fn(out.ctypes.data_as(ctypes.c_void_p)) != 0:
            raise RuntimeError("trace read failed")
        return out

    for it in range(args.loop):
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
        ev[0].record()
        comp.run_lse(inst.q, inst.win_indptr, inst.tok_indptr, wl.sm_scale, wl.causal, 0, wl.n_layers, comp.lse)
        ev[1].record()
        comp.run_score(inst.q, inst.win_indptr, inst.tok_indptr, wl.sm_scale, wl.causal, lse_in=comp.lse)
        ev[2].record()
        torch.cuda.synchronize()
        if it < 2 or it % 5 == 0 or it == args.loop - 1:
            mhz = []
            for fn, rows in ((lib.actkv_debug_lse_trace, 6), (lib.actkv_debug_pool_trace, 8)):
                t = read(fn, rows)
                mhz.append(1000.0 * (t[0, 1002] - t[0, 1000]) / max(1, t[0, 1003] - t[0, 1001]))
            print(f"iteration {it}: LSE pass {ev[0].elapsed_time(ev[1]):.2f} ms at {mhz[0]:.0f} MHz inside the kernel, "
                  f"pooled-score pass {ev[1].elapsed_time(ev[2]):.2f} ms at {mhz[1]:.0f} MHz")
    comp.check_status()

    t = read(lib.actkv_debug_lse_trace, 6)       # rows: MMA issue, commit, loaded, released, folded, wait begins
    nj = int((t[2, :1000] != 0).sum())
    a = np.arange(nj // 4 & ~1, nj - 4, 2)       # even jobs (epilogue group 0) of the steady part
    print(f"LSE pass, CTA 200: {nj} jobs in {t[0, 1002] - t[0, 1000]} cycles; per pair of jobs "
          f"{np.diff(t[2, a]).mean():.0f} (group 0) / {np.diff(t[2, a + 1]).mean():.0f} (group 1), "
          f"fold {(t[4, a] - t[3, a]).mean():.0f}, fetch {(t[2, a] - t[5, a]).mean():.0f}, "
          f"group 1 behind group 0 by {(t[2, a + 1] - t[2, a]).mean():.0f}")
    t = read(lib.actkv_debug_pool_trace, 8)      # rows: K tile there, accumulator free, issued | wait begins,
    nj = int((t[2, :1000] != 0).sum())           # accumulator full, folded, released, end-of-tile work done
    j = np.arange(nj // 4, nj - 4)
    print(f"pooled-score pass, CTA 200: {nj} jobs in {t[0, 1002] - t[0, 1000]} cycles; per job {np.diff(t[2, j]).mean():.0f}; "
          f"issuer waits {(t[1, j] - t[0, j]).mean():.0f} for its accumulator and issues in {(t[2, j] - t[1, j]).mean():.0f}")
    for wg in (0, 1):                            # warpgroup wg takes the jobs of parity wg
        k = j[(j & 1) == wg]
        print(f"  epilogue warpgroup {wg}, per job of its own: waits {(t[4, k] - t[3, k]).mean():.0f} for the accumulator, "
              f"holds it {(t[6, k] - t[4, k]).mean():.0f}, folds the rest in {(t[5, k] - t[6, k]).mean():.0f}, "
              f"end of tile {(t[7, k] - t[5, k]).mean():.0f}, to its next wait {(t[3, k + 2] - t[7, k]).mean():.0f}")


if __name__ == "__main__":
    main()
