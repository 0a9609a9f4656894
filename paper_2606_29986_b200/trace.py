"""Per-warp timing of the attention kernel, from the instrumented build of the library (-DHMA_TRACE).

    python -m paper_2606_29986_b200.trace [--workload NAME] [--layers N] [--reps R] [--self-planned]

Builds libhma_trace.so if needed, runs hma_decode_attention_planned (with --self-planned: hma_decode_attention, which
repeats the set-up in every call) on a benchmark workload with that image, reads the
time stamps every worker (warp) left behind its partial tiles, and prints a summary: when warps start, when their
first record lands, when they leave the record loop, how that spreads inside an SM and between SMs, what the CTA-level
reduction costs, and how three consecutive calls hand over to one another.  The default
library carries none of the instrumentation; the numbers printed here are about where time goes, not bench values.
"""
import argparse
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
TRACE_WORDS = 16


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="qwen3-32b-b32-ctx8k")
    ap.add_argument("--layers", type=int, default=4)
    ap.add_argument("--reps", type=int, default=5)
    ap.add_argument("--self-planned", action="store_true")
    args = ap.parse_args()

    from paper_2606_29986_b200 import build
    os.environ["HMA_LIBRARY"] = os.environ.get("HMA_LIBRARY") or build.build(trace=True)
    sys.path.insert(0, ROOT)
    import torch
    import bench
    from paper_2606_29986_b200 import hma
    dev = torch.device("cuda", 0)
    wl = bench.Workload(args.workload, dev, with_bf16=False, with_ingest=False, layers=args.layers)
    ws_bytes = hma.hma_decode_attention_workspace_bytes(wl.caches["bfp8"].desc, wl.B)
    n_workers = 192 * 16
    trace_off = ws_bytes - n_workers * TRACE_WORDS * 8
    assert wl.workspace.numel() >= ws_bytes
    cache = wl.caches["bfp8"]
    plan = hma.hma_decode_attention_plan(cache, wl.table, wl.ctx)

    def attention(l, ws):
        if args.self_planned:
            hma.hma_decode_attention(cache, l, wl.q[l], wl.out[l], wl.table, wl.ctx, wl.sm_scale, ws)
        else:
            hma.hma_decode_attention_planned(cache, l, wl.q[l], wl.out[l], wl.table, wl.ctx, wl.sm_scale, plan, ws)

    def run(l):
        wl.workspace[trace_off:ws_bytes].zero_()
        # two calls back to back: the second one starts the way a call inside a decode pass does
        attention((l + 1) % wl.L, wl.workspace)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        attention(l, wl.workspace)
        e1.record()
        torch.cuda.synchronize()
        tr = wl.workspace[trace_off:ws_bytes].view(torch.int64).cpu().numpy().reshape(-1, TRACE_WORDS).copy()
        return tr[tr[:, 1] > 0], e0.elapsed_time(e1) * 1e3

    for i in range(3):
        run(i % wl.L)
    rows = []
    for rep in range(args.reps):
        tr, call_us = run(rep % wl.L)
        t0 = tr[:, 1].min()
        us = lambda col: (tr[:, col] - t0) / 1e3
        smid, wait, pro, first, loop_end, done, recs = tr[:, 0], us(1), us(2), us(3), us(4), us(5), tr[:, 6]
        epi = tr[:, 8] > 0
        cyc = lambda a, b: ((tr[:, a] - tr[:, b])[epi & (tr[:, a] > 0) & (tr[:, b] > 0)] / 1.9e3)      # us at about 1.9 GHz
        sms = np.unique(smid)
        sm_end = np.array([loop_end[smid == s].max() for s in sms])
        sm_mean = np.array([loop_end[smid == s].mean() for s in sms])
        within = np.array([loop_end[smid == s].max() - loop_end[smid == s].min() for s in sms])
        rows.append(dict(call_us=call_us, workers=len(tr), sms=len(sms), enter_spread=wait.max(), prologue_end=pro.mean(),
                         range_known_mean=us(13).mean(), range_known_max=us(13).max(), first_request_mean=us(14).mean(),
                         first_request_max=us(14).max(), planned_mean=us(15).mean(), planned_max=us(15).max(),
                         first_mean=first.mean(), first_max=first.max(), end_min=loop_end.min(), end_mean=loop_end.mean(),
                         end_p90=np.percentile(loop_end, 90), end_max=loop_end.max(), done_max=done.max(),
                         sm_mean_min=sm_mean.min(), sm_mean_max=sm_mean.max(), sm_mean_std=sm_mean.std(),
                         epi_reduce_us=cyc(9, 8).mean(), epi_arrive_us=cyc(10, 9).mean(),
                         epi_merge_us=cyc(11, 10).mean(), epi_total_us_mean=cyc(11, 8).mean(), epi_total_us_max=cyc(11, 8).max(),
                         within_mean=within.mean(), within_max=within.max(), recs_min=int(recs.min()), recs_max=int(recs.max()),
                         slow=[int(x) for x in sms[np.argsort(sm_end)[-8:]]]))
    # three consecutive calls, each with a workspace of its own so that all three traces survive: where one kernel ends
    # and the next begins on the same clock (the hand-off under programmatic stream serialisation)
    wss = [hma.new_workspace(wl.caches["bfp8"].desc, wl.B, dev) for _ in range(3)]
    for i in range(24):
        l = i % wl.L
        attention(l, wss[i % 3])
    torch.cuda.synchronize()
    chain = []
    for ws in wss:
        tr = ws[trace_off:ws_bytes].view(torch.int64).cpu().numpy().reshape(-1, TRACE_WORDS)
        chain.append(tr[tr[:, 1] > 0])
    c0 = chain[0][:, 1].min()
    print("three consecutive calls in one stream (calls 22, 23, 24 of 24), us after the first warp of the first passed its wait:")
    print("| call | CTAs enter (min .. max) | wait passed (min .. max) | first record lands (mean) | record loop ends (mean, max) | CTA leaves (min, mean, max) |")
    print("|---|---|---|---|---|---|")
    for i, T in enumerate(chain):
        f = lambda x: (x - c0) / 1e3
        ex = T[:, 12][T[:, 12] > 0]
        print("| %d | %.1f .. %.1f | %.1f .. %.1f | %.1f | %.1f, %.1f | %.1f, %.1f, %.1f |" % (
            i, f(T[:, 7].min()), f(T[:, 7].max()), f(T[:, 1].min()), f(T[:, 1].max()), f(T[:, 3].mean()), f(T[:, 4].mean()), f(T[:, 4].max()),
            f(ex.min()), f(ex.mean()), f(ex.max())))
    keys = [k for k in rows[0] if k != "slow"]
    print("workload %s, %d layers built, %d traced %s calls (all times in us after the first warp passed the grid-dependency wait)" %
          (args.workload, wl.L, len(rows), "self-planning" if args.self_planned else "planned"))
    print("| quantity | " + " | ".join("call %d" % i for i in range(len(rows))) + " |")
    print("|---|" + "---|" * len(rows))
    for k in keys:
        print("| %s | " % k + " | ".join(("%.2f" % r[k]) if isinstance(r[k], float) else str(r[k]) for r in rows) + " |")
    print("SMs whose last warp leaves the loop last, per call:", [r["slow"] for r in rows])


if __name__ == "__main__":
    main()
