"""Run one of the synthetic workloads a few times through the C ABI and print its
device time.  Handy for profiling a single kernel:

    python -m paper_2605_05802_b200.run_case --case c3 --reps 3
    ncu --set full --clock-control none -k regex:gate_single -c 1 \\
        python -m paper_2605_05802_b200.run_case --case c3 --reps 3

Cases: c1, c2, c2x128 (65536 groups x N=8, K=15), c3 (4096 groups x N=16), c3x16
(65536 groups), c4 (token level), c4s (256 groups), c4d (token level through sr_gate_decide at --threshold), c5 (streaming, --groups to
shrink), adv (advantages, 4M groups), orr (OR rule, 4M groups), bstats (batch
statistics, 4M groups), keep (kept-group index list, 4M groups), sig (Appendix-B
signals, 65536 groups x N=16), packed (token level from packed host input, 256 groups).
"""
from __future__ import annotations

import argparse
import statistics

import torch

import paper_2605_05802_b200 as sr
from paper_2605_05802_b200 import workloads as W


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--case", default="c3")
    ap.add_argument("--reps", type=int, default=5)
    ap.add_argument("--groups", type=int, default=0)
    ap.add_argument("--threshold", type=float, default=0.3)
    args = ap.parse_args()
    dev = torch.device("cuda:0")
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    sweep = torch.zeros(64 << 20, dtype=torch.float32, device=dev)
    times = []

    def timed(fn):
        # flush L2: write 256 MiB, then read another 256 MiB so that the dirty lines of
        # the write are already back in DRAM when the timed launch starts
        flush.fill_(1)
        sweep.sum()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        fn()
        b.record()
        torch.cuda.synchronize()
        times.append(a.elapsed_time(b) * 1e3)

    if args.case in ("c1", "c2", "c2x128", "c3", "c3x16", "c4", "c4s", "c4d"):
        w = {"c1": lambda: W.tiny_gate(), "c2": lambda: W.agent_gate(K=15),
             "c2x128": lambda: W.agent_gate(K=15, n_groups=args.groups or 65536),
             "c3": lambda: W.large_group_gate(n_groups=args.groups or 4096),
             "c3x16": lambda: W.large_group_gate(n_groups=65536),
             "c4": lambda: W.token_gate(n_groups=args.groups or 1024),
             "c4s": lambda: W.token_gate(n_groups=256),
             "c4d": lambda: W.token_gate(n_groups=args.groups or 1024)}[args.case]()
        G, N, stride = w.seqs.shape
        seqs = torch.from_numpy(w.seqs).to(dev)
        lens = torch.from_numpy(w.lens).to(dev)
        ps = torch.empty(G, dtype=torch.int32, device=dev)
        mean = torch.empty(G, dtype=torch.float64, device=dev)
        stop = torch.empty(G, dtype=torch.uint8, device=dev)
        wsb = sr.sr_gate_workspace_bytes(G, N, stride, w.K)
        ws = torch.empty(wsb, dtype=torch.uint8, device=dev) if wsb else None
        if args.case == "c4d":
            ex = torch.empty(G, dtype=torch.uint8, device=dev)
            call = lambda: sr.sr_gate_decide(seqs, lens, w.K, args.threshold, w.norm_mode, pair_sum=ps, mean=mean,
                                             stop=stop, exact=ex, workspace=ws)
        else:
            call = lambda: sr.sr_gate(seqs, lens, w.K, w.threshold, w.norm_mode, pair_sum=ps, mean=mean,
                                      stop=stop, workspace=ws)
        for _ in range(args.reps):
            timed(call)
        print(f"{w.name}: {G} groups x N={N}, K={w.K}: median {statistics.median(times):.1f} us, "
              f"{W.dp_cells(w.lens, w.K) / statistics.median(times) / 1e3:.0f} GCUPS, stopped {int(stop.sum())}")
    elif args.case == "c5":
        s = W.streaming_gate(n_groups=args.groups or 65536)
        acts = torch.from_numpy(s.actions).to(dev)
        state = torch.empty(sr.sr_incr_state_bytes(s.n_groups, s.N, s.steps), dtype=torch.uint8, device=dev)
        mean = torch.empty(s.n_groups, dtype=torch.float64, device=dev)
        stop = torch.empty(s.n_groups, dtype=torch.uint8, device=dev)
        for _ in range(args.reps):
            sr.sr_incr_init(state, s.n_groups, s.N, s.steps)
            for t in range(s.steps):
                timed(lambda: sr.sr_gate_step_incremental(state, acts[t], s.threshold, s.norm_mode,
                                                          mean=mean, stop=stop))
        per_step = [statistics.median(times[t::s.steps]) for t in range(s.steps)]
        print(f"{s.name}: {s.n_groups} groups, {s.steps} steps: median step {statistics.median(times):.1f} us, "
              f"stopped at the end {int(stop.sum())}")
        print("  per step (us): " + " ".join(f"{v:.0f}" for v in per_step))
    elif args.case == "adv":
        G = args.groups or (64 * 65536)
        r = torch.rand((G, 8), device=dev)
        adv = torch.empty_like(r)
        zv = torch.empty(G, dtype=torch.uint8, device=dev)
        for _ in range(args.reps):
            timed(lambda: sr.sr_grpo_advantage(r, None, 1e-6, adv=adv, zero_var=zv))
        print(f"advantages: {G} groups x N=8: median {statistics.median(times):.1f} us")
    elif args.case in ("orr", "bstats", "keep"):
        G = args.groups or (64 * 65536)
        adv = torch.rand((G, 8), device=dev)
        adv[::3] = 0.0
        flags = (torch.rand(G, device=dev) < 0.2).to(torch.uint8)
        if args.case == "orr":
            lens = torch.randint(0, 31, (G, 8), dtype=torch.int32, device=dev)
            mean = torch.rand(G, dtype=torch.float64, device=dev)
            tau = torch.empty(G, dtype=torch.float64, device=dev)
            fn = lambda: sr.sr_gate_or_rule(mean, lens, None, 8, 15, 0.12, 0.9, tau=tau, stop=flags)
        elif args.case == "bstats":
            cnt = torch.empty(3, dtype=torch.int64, device=dev)
            ssq = torch.empty(2, dtype=torch.float64, device=dev)
            fn = lambda: sr.sr_batch_stats(adv, flags, counts=cnt, sumsq=ssq)
        else:
            idx = torch.empty(G, dtype=torch.int32, device=dev)
            cnt = torch.empty(1, dtype=torch.int32, device=dev)
            ws = torch.empty(sr.sr_kept_groups_workspace_bytes(G), dtype=torch.uint8, device=dev)
            fn = lambda: sr.sr_kept_groups(flags, None, index=idx, count=cnt, workspace=ws)
        for _ in range(args.reps):
            timed(fn)
        print(f"{args.case}: {G} groups x N=8: median {statistics.median(times):.1f} us")
    elif args.case == "sig":
        w = W.large_group_gate(n_groups=args.groups or 65536)
        seqs = torch.from_numpy(w.seqs).to(dev)
        outs = [torch.empty(w.n_groups, dtype=torch.float64, device=dev) for _ in range(4)]
        for _ in range(args.reps):
            timed(lambda: sr.sr_group_signals(seqs, None, w.K, unique_prefix_ratio=outs[0],
                                              unique_action_ratio=outs[1], action_entropy=outs[2],
                                              bigram_jaccard_mean=outs[3]))
        print(f"signals: {w.n_groups} groups x N={w.N}, K={w.K}: median {statistics.median(times):.1f} us")
    elif args.case == "packed":
        w = W.token_gate(n_groups=args.groups or 256)
        G, N, stride = w.seqs.shape
        symbols, row_start = W.pack_rows(w.seqs, w.lens)
        h_sym = torch.from_numpy(symbols).pin_memory()
        h_rs = torch.from_numpy(row_start).pin_memory()
        h_stop = torch.empty(G, dtype=torch.uint8).pin_memory()
        arena = torch.empty(sr.sr_gate_host_packed_arena_bytes(G, N, stride, w.K), dtype=torch.uint8, device=dev)
        for _ in range(args.reps):
            timed(lambda: sr.sr_gate_host_packed(h_sym, h_rs, N, stride, w.K, w.threshold, w.norm_mode,
                                                 stop=h_stop, arena=arena))
        print(f"packed host input: {G} groups x N={N}: median {statistics.median(times):.1f} us")
    else:
        raise SystemExit(f"unknown case {args.case}")


if __name__ == "__main__":
    main()
