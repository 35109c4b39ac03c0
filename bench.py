#!/usr/bin/env python
"""Benchmark of the Selective Rollout gate on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

One step = one pass of the hot path over one batch: the gate (stage, match
streams, pair distances, d_K, threshold) on the token-level workload (1024 groups
x N=8 rollouts, prefix lengths 256..1024) followed by the group-relative
advantages of the same groups with the stop mask as drop mask.  Prints ONE JSON
line.  Under torchrun every rank runs its own shard of groups (weak scaling, no
data-path collective); time is the max over ranks.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

FLUSH_BYTES = 256 << 20
SM_INT32_LANES = 64          # 32-bit integer add / logic results per clock per SM (compute capability 10.0)
METRIC = "prefix_edit_distance_gcups"
UNIT = "GCUPS"


def read_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "sm_max_mhz": float(p.get("sm_max_mhz", 1965.0)),
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "sm_max_mhz": 1965.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while a region runs."""
    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.path = None

    def start(self):
        fd, self.path = tempfile.mkstemp(suffix=".csv")
        os.close(fd)
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.gpu), f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "50"],
                stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        with open(self.path) as f:
            for ln in f:
                parts = [x.strip() for x in ln.split(",")]
                if len(parts) < 9:
                    continue
                try:
                    sm.append(float(parts[1]))
                    mx.append(float(parts[2]))
                except ValueError:
                    continue
                for name, val in zip(names, parts[5:9]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
        os.unlink(self.path)
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), reasons=sorted(reasons),
                       samples=len(sm))
        return out


def traffic_from_profiles(kernel: str, source_file: str):
    """DRAM bytes per launch recorded from an ncu capture, valid only while the
    kernel's source file is unchanged (a `traffic:` line in profiles/*.md)."""
    sha = hashlib.sha256(open(source_file, "rb").read()).hexdigest()[:16]
    pdir = os.path.join(ROOT, "profiles")
    if not os.path.isdir(pdir):
        return None
    for name in sorted(os.listdir(pdir)):
        if not name.endswith(".md"):
            continue
        for ln in open(os.path.join(pdir, name)):
            if ln.startswith("traffic:") and f"kernel={kernel}" in ln and f"source_sha={sha}" in ln:
                for tok in ln.split():
                    if tok.startswith("dram_bytes_per_full_launch="):
                        return float(tok.split("=")[1])
    return None


def run_reference(args):
    """Reference arm: the CPU oracle, as it stands, timed on the host cores."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    from paper_2605_05802_b200 import workloads as W
    cores = min(os.cpu_count() or 1, oracle.max_threads())
    w = W.token_gate()
    sample = max(8, min(w.n_groups, 16 * cores))          # about a second of work per step
    seqs, lens, rewards = w.seqs[:sample], w.lens[:sample], w.rewards[:sample]
    cells = W.dp_cells(lens, w.K)

    def step():
        _, _, _, stop = oracle.gate(seqs, lens, w.K, w.threshold, w.norm_mode, threads=cores)
        oracle.advantage(rewards, stop, 1e-6)

    for _ in range(args.warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
    dt = time.perf_counter() - t0
    value = cells * args.steps / dt / 1e9
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int32",
        "data": "synthetic",
        "config": {"workload": "C4-token: N=8 rollouts/group, token prefixes U{256..1024}, vocab 151936, K=1024",
                   "groups_per_step": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                         "sample": f"first {sample} of 1024 groups per step"},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "groups_per_s": sample * args.steps / dt,
    }
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=300)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--groups", type=int, default=1024,
                    help="groups per GPU of the token-level workload (1024 = the benchmark configuration)")
    ap.add_argument("--no-extras", action="store_true", help="skip the per-config side measurements")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
        return

    import torch
    import torch.distributed as dist
    import paper_2605_05802_b200 as sr
    from paper_2605_05802_b200 import workloads as W

    sr.load()                                   # fail loudly if the CUDA library is missing
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    peaks = read_peaks()
    props = torch.cuda.get_device_properties(dev)
    sms = props.multi_processor_count

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    flush = torch.empty(FLUSH_BYTES, dtype=torch.uint8, device=dev)
    sweep = torch.zeros(FLUSH_BYTES // 4, dtype=torch.float32, device=dev)

    def flush_l2(tag: int):
        """Write 256 MiB, then read another 256 MiB: the L2 ends up holding clean lines
        of unrelated data, so the timed launch neither hits in L2 nor has to wait for
        the write-back of the flush itself."""
        flush.fill_(tag & 0xFF)
        sweep.sum()

    def timed(fn, reps, warm=3, do_flush=True):
        """Per-launch device times (ms) of fn, L2 flushed before every launch."""
        for _ in range(warm):
            fn()
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(reps)]
        torch.cuda.synchronize()
        for i, (a, b) in enumerate(evs):
            if do_flush:
                flush_l2(i)
            a.record()
            fn()
            b.record()
        torch.cuda.synchronize()
        return [a.elapsed_time(b) for a, b in evs]

    # ------------------------------------------------------------ headline workload
    w = W.token_gate(seed=3 + 1000 * rank, n_groups=args.groups)      # every rank gates its own 1024 groups
    G, N, stride, K = w.n_groups, w.N, w.stride, w.K
    P = N * (N - 1) // 2
    cells = W.dp_cells(w.lens, K)
    wcols_full = W.word_columns(w.lens, K)
    wcols = W.word_columns(w.lens, K, w.seqs)          # what is left after the pairs' common prefixes
    seqs = torch.from_numpy(w.seqs).to(dev)
    lens = torch.from_numpy(w.lens).to(dev)
    rewards = torch.from_numpy(w.rewards).to(dev)
    ps = torch.empty(G, dtype=torch.int32, device=dev)
    mean = torch.empty(G, dtype=torch.float64, device=dev)
    stop = torch.empty(G, dtype=torch.uint8, device=dev)
    adv = torch.empty_like(rewards)
    zv = torch.empty(G, dtype=torch.uint8, device=dev)
    ws = torch.empty(sr.sr_gate_workspace_bytes(G, N, stride, K), dtype=torch.uint8, device=dev)

    def step():
        sr.sr_gate(seqs, lens, K, w.threshold, w.norm_mode, pair_sum=ps, mean=mean, stop=stop, workspace=ws)
        sr.sr_grpo_advantage(rewards, stop, 1e-6, adv=adv, zero_var=zv)

    # ---- before any timing: the outputs of this very configuration against the oracle on a
    # sample of groups, at the paper's threshold and at one where the mask is mixed
    verify = None
    if rank == 0:
        import oracle
        cores = min(os.cpu_count() or 1, oracle.max_threads())
        n_check = min(G, 96)
        pd = torch.empty((G, P), dtype=torch.int32, device=dev)
        verify = {"groups_checked": n_check, "thresholds": [], "cut_in_sample": []}
    for thr in ((w.threshold, 0.5) if rank == 0 else ()):
        sr.sr_gate(seqs, lens, K, thr, w.norm_mode, pair_dist=pd, pair_sum=ps, mean=mean, stop=stop, workspace=ws)
        torch.cuda.synchronize()
        o_pd, o_ps, o_mean, o_stop = oracle.gate(w.seqs[:n_check], w.lens[:n_check], K, thr, w.norm_mode, threads=cores)
        assert np.array_equal(pd[:n_check].cpu().numpy(), o_pd), "pair distances differ from the oracle"
        assert np.array_equal(ps[:n_check].cpu().numpy(), o_ps), "pair sums differ from the oracle"
        assert np.array_equal(mean[:n_check].cpu().numpy().view(np.uint64), o_mean.view(np.uint64)), "d_K differs from the oracle"
        assert np.array_equal(stop[:n_check].cpu().numpy(), o_stop), "stop mask differs from the oracle"
        verify["thresholds"].append(thr)
        verify["cut_in_sample"].append(int(o_stop.sum()))

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    for _ in range(max(args.warmup, 3)):
        step()
    barrier()
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    barrier()
    for i, (a, b) in enumerate(evs):
        flush_l2(i)
        a.record()
        step()
        b.record()
    barrier()
    total_ms = sum(a.elapsed_time(b) for a, b in evs)
    if world > 1:
        t = torch.tensor([total_ms], dtype=torch.float64, device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        total_ms = float(t.item())

    # stage pass: same steps with events at the pipeline's stage boundaries
    stage_evs = []
    for _ in range(args.steps):
        e5 = [torch.cuda.Event(enable_timing=True) for _ in range(5)]
        for e in e5:
            e.record()
        stage_evs.append(e5)
    torch.cuda.synchronize()
    for i, e5 in enumerate(stage_evs):
        flush_l2(i)
        sr.sr_gate_stages(seqs, lens, K, w.threshold, w.norm_mode, pair_sum=ps, mean=mean, stop=stop,
                          workspace=ws, events=e5)
    torch.cuda.synchronize()
    clocks = sampler.stop() if rank == 0 else None
    stage_ms = [statistics.median(e5[k].elapsed_time(e5[k + 1]) for e5 in stage_evs) for k in range(4)]
    dp_ms = stage_ms[2]

    # ------------------------------------------------------------------ end to end
    # host side: the batch as a rollout buffer holds it, prefixes back to back plus row offsets
    symbols, row_start = W.pack_rows(w.seqs, w.lens)
    h_sym = torch.from_numpy(symbols).pin_memory()
    h_rs = torch.from_numpy(row_start).pin_memory()
    h_rew = torch.from_numpy(w.rewards).pin_memory()
    h_ps = torch.empty(G, dtype=torch.int32).pin_memory()
    h_mean = torch.empty(G, dtype=torch.float64).pin_memory()
    h_stop = torch.empty(G, dtype=torch.uint8).pin_memory()
    h_adv = torch.empty((G, N), dtype=torch.float32).pin_memory()
    h_zv = torch.empty(G, dtype=torch.uint8).pin_memory()
    arena = torch.empty(sr.sr_gate_host_packed_arena_bytes(G, N, stride, K), dtype=torch.uint8, device=dev)
    d_rew = torch.empty_like(rewards)
    d_stop = torch.empty_like(stop)

    copy_stream = torch.cuda.Stream(device=dev)

    def e2e_tail():
        d_rew.copy_(h_rew, non_blocking=True)
        d_stop.copy_(h_stop, non_blocking=True)      # stream-ordered after the D2H that filled h_stop
        sr.sr_grpo_advantage(d_rew, d_stop, 1e-6, adv=adv, zero_var=zv)
        h_adv.copy_(adv, non_blocking=True)
        h_zv.copy_(zv, non_blocking=True)

    def e2e_step():
        sr.sr_gate_host_packed(h_sym, h_rs, N, stride, K, w.threshold, w.norm_mode, pair_sum=h_ps, mean=h_mean,
                               stop=h_stop, arena=arena, copy_stream=copy_stream)
        e2e_tail()

    h2d = h_sym.numel() * 4 + h_rs.numel() * 8 + h_rew.numel() * 4 + h_stop.numel()
    d2h = h_ps.numel() * 4 + h_mean.numel() * 8 + h_stop.numel() + h_adv.numel() * 4 + h_zv.numel()
    e2e_ms = sum(timed(e2e_step, args.steps))
    if world > 1:
        t = torch.tensor([e2e_ms], dtype=torch.float64, device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        e2e_ms = float(t.item())
    assert np.array_equal(h_stop.numpy(), stop.cpu().numpy())

    value = cells * world * args.steps / (total_ms * 1e-3) / 1e9
    e2e_value = cells * world * args.steps / (e2e_ms * 1e-3) / 1e9
    alu_peak = sms * SM_INT32_LANES * peaks["sm_max_mhz"] * 1e6 / 1e9          # Gop/s
    achieved = 10.0 * wcols / (dp_ms * 1e-3) / 1e9
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": total_ms / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "int32", "data": "synthetic",
        "config": {"workload": f"C4-token: {args.groups} groups x N=8 rollouts per GPU, token prefixes U[256..1024], "
                               "vocab 151936, K=1024, d_L=0.12; gate + advantages",
                   "groups_per_gpu": G, "pairs_per_group": P, "dp_cells_per_gpu": cells,
                   "l2": "flushed before every step (256 MiB write + 256 MiB read)", "parallelism": f"groups sharded x{world}, no collective"},
        "groups_per_s": G * world * args.steps / (total_ms * 1e-3),
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "ms_per_step": e2e_ms / args.steps,
                "input": "packed prefixes + int64 row offsets in pinned host memory (sr_gate_host_packed), "
                         "sent in four pieces on a copy stream under the per-group pass; one recurrence launch"},
        "gpu_launches": 5 * args.steps,
        "clocks": clocks,
        "stage_ms": {"prep": stage_ms[0], "order": stage_ms[1], "dp": stage_ms[2], "finish": stage_ms[3]},
        "roofline": {"kernel": "multi_dp_kernel", "bound": "alu", "achieved": achieved, "peak": alu_peak,
                     "unit": "Gop/s (int32 lane-ops, 10 per 32-row block per column, common prefixes of a pair not counted)",
                     "frac": achieved / alu_peak,
                     "peak_basis": f"{sms} SMs x {SM_INT32_LANES} int32 lanes/clk x {peaks['sm_max_mhz']:.0f} MHz (derived)",
                     "traffic": traffic_from_profiles("multi_dp_kernel", os.path.join(ROOT, "paper_2605_05802_b200", "csrc", "gate_multi.cu")),
                     "word_columns": wcols, "word_columns_before_prefix_removal": wcols_full,
                     "ms_per_launch": dp_ms},
        "verified_against_oracle": verify,
    }

    # ------------------------------------------------ side measurements (1 GPU only)
    if world == 1 and not args.no_extras:
        extras = {}
        sink = torch.empty(sms * 8 * 256, dtype=torch.int32, device=dev)
        probe = {}
        for name, var in (("logic", sr.SR_PROBE_LOGIC), ("add", sr.SR_PROBE_ADD), ("mix8l2a", sr.SR_PROBE_MIX)):
            ms = min(timed(lambda: sr.sr_probe_int32(var, 2000, sms * 8, 256, sink), 5, do_flush=False))
            probe[name] = sr.sr_probe_int32_ops(2000, sms * 8, 256) / (ms * 1e-3) / 1e9
        extras["int32_probe_gops"] = probe
        # the recurrence is 8 logic : 2 add; logic issues on the int32 ALU only, adds can also
        # issue on the FMA pipe, so the logic-only rate is the pipe's own ceiling
        line["roofline"]["peak_probe_logic"] = probe["logic"]
        line["roofline"]["frac_of_probe_logic"] = achieved / probe["logic"]
        # the recurrence's own mix (8 logic : 2 add) measured register-only on this GPU: the
        # adds also issue on the FMA pipe, so this ceiling is a little above the logic rate
        line["roofline"]["peak_probe_mix"] = probe["mix8l2a"]
        line["roofline"]["frac_of_probe_mix"] = achieved / probe["mix8l2a"]

        def gate_case(wl, reps=20):
            g, n, st = wl.seqs.shape
            p = n * (n - 1) // 2
            s_ = torch.from_numpy(wl.seqs).to(dev)
            l_ = torch.from_numpy(wl.lens).to(dev)
            o_ps = torch.empty(g, dtype=torch.int32, device=dev)
            o_mean = torch.empty(g, dtype=torch.float64, device=dev)
            o_stop = torch.empty(g, dtype=torch.uint8, device=dev)
            wsb = sr.sr_gate_workspace_bytes(g, n, st, wl.K)
            ws_ = torch.empty(wsb, dtype=torch.uint8, device=dev) if wsb else None
            ms = timed(lambda: sr.sr_gate(s_, l_, wl.K, wl.threshold, wl.norm_mode, pair_sum=o_ps,
                                          mean=o_mean, stop=o_stop, workspace=ws_), reps)
            med = statistics.median(ms)
            c = W.dp_cells(wl.lens, wl.K)
            m = np.minimum(wl.lens, wl.K).astype(np.int64)
            cols = 0
            for i in range(n):
                for j in range(i + 1, n):
                    cols += int(np.minimum(m[:, i], m[:, j]).sum())
            ach = 10.0 * cols / (med * 1e-3) / 1e9
            return {"groups": g, "N": n, "us_median": med * 1e3, "us_best": min(ms) * 1e3,
                    "gcups": c / (med * 1e-3) / 1e9, "groups_per_s": g / (med * 1e-3),
                    "alu_gops": ach, "alu_frac": ach / alu_peak}

        extras["C1_tiny"] = gate_case(W.tiny_gate())
        extras["C2_agent_K15"] = gate_case(W.agent_gate(K=15))
        extras["C3_large_group"] = gate_case(W.large_group_gate())
        extras["C3_x16_groups"] = gate_case(W.large_group_gate(n_groups=65536), reps=10)

        s5 = W.streaming_gate()
        acts = torch.from_numpy(s5.actions).to(dev)
        state = torch.empty(sr.sr_incr_state_bytes(s5.n_groups, s5.N, s5.steps), dtype=torch.uint8, device=dev)
        o_mean = torch.empty(s5.n_groups, dtype=torch.float64, device=dev)
        o_stop = torch.empty(s5.n_groups, dtype=torch.uint8, device=dev)
        per_step = [[] for _ in range(s5.steps)]
        for rep in range(4):
            sr.sr_incr_init(state, s5.n_groups, s5.N, s5.steps)
            evs5 = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(s5.steps)]
            for t_, (a, b) in enumerate(evs5):
                flush_l2(t_)
                a.record()
                sr.sr_gate_step_incremental(state, acts[t_], s5.threshold, s5.norm_mode, mean=o_mean, stop=o_stop)
                b.record()
            torch.cuda.synchronize()
            if rep > 0:
                for t_, (a, b) in enumerate(evs5):
                    per_step[t_].append(a.elapsed_time(b))
        step_ms = [statistics.median(x) for x in per_step]
        Pn = s5.N * (s5.N - 1) // 2
        # algorithmic bytes per group and step: pair state read + written (16 B each way),
        # history so far read (4 B per stored action) + one appended action per rollout,
        # lengths read + written, new actions, d_K and stop mask written
        bytes_steps = []
        for t_ in range(s5.steps):
            per_group = Pn * 32 + s5.N * (4 * t_ + 4) + s5.N * 8 + s5.N * 4 + 9
            bytes_steps.append(per_group * s5.n_groups)
        gbs = [b / (ms * 1e-3) / 1e9 for b, ms in zip(bytes_steps, step_ms)]
        # DP cells that are new at step t: every pair's matrix grows from (t-1)^2 to t^2 cells
        new_cells = s5.n_groups * Pn * s5.steps * s5.steps
        extras["C5_stream"] = {"groups": s5.n_groups, "steps": s5.steps, "us_per_step_median": statistics.median(step_ms) * 1e3,
                               "us_total": sum(step_ms) * 1e3,
                               "us_per_step": [round(x * 1e3, 1) for x in step_ms],
                               "group_gates_per_s": s5.n_groups * s5.steps / (sum(step_ms) * 1e-3),
                               "new_cells_per_s": new_cells / (sum(step_ms) * 1e-3),
                               "bytes_per_group_step": "28*32 pair state both ways + 8*(4t+4) stored actions read + append "
                                                       "+ 8*8 lengths both ways + 8*4 new actions + 9 outputs",
                               "hbm_gbs_mean": statistics.mean(gbs), "hbm_gbs_last_step": gbs[-1],
                               "hbm_frac_mean": statistics.mean(gbs) / peaks["hbm_gbs"],
                               "hbm_peak_source": peaks["source"]}
        big = 64 * s5.n_groups
        r_ = torch.rand((big, 8), device=dev)
        a_ = torch.empty_like(r_)
        z_ = torch.empty(big, dtype=torch.uint8, device=dev)
        ms = timed(lambda: sr.sr_grpo_advantage(r_, None, 1e-6, adv=a_, zero_var=z_), 10)
        med = statistics.median(ms)
        adv_bytes = big * (8 * 8 + 1)
        extras["advantage_x64"] = {"groups": big, "us_median": med * 1e3, "hbm_gbs": adv_bytes / (med * 1e-3) / 1e9,
                                   "hbm_frac": adv_bytes / (med * 1e-3) / 1e9 / peaks["hbm_gbs"]}
        ms = timed(lambda: sr.sr_grpo_advantage(rewards, stop, 1e-6, adv=adv, zero_var=zv), 20)
        extras["advantage_C4"] = {"groups": G, "us_median": statistics.median(ms) * 1e3}
        # decide mode on the headline workload: same mask, groups dismissed from lower bounds
        ex = torch.empty(G, dtype=torch.uint8, device=dev)
        stop_d = torch.empty(G, dtype=torch.uint8, device=dev)
        ms = timed(lambda: sr.sr_gate_decide(seqs, lens, K, w.threshold, w.norm_mode, pair_sum=ps, mean=mean,
                                             stop=stop_d, exact=ex, workspace=ws), 20)
        assert torch.equal(stop_d, stop)
        extras["decide_C4"] = {"groups": G, "us_median": statistics.median(ms) * 1e3,
                               "groups_per_s": G / (statistics.median(ms) * 1e-3),
                               "groups_computed_exactly": int(ex.sum().item()),
                               "note": "mask-equivalent mode; not the headline (work is skipped by design)"}
        # the same mode at a threshold the bounds alone cannot settle: open groups run in bands
        # cut to what the threshold still allows (compared with sr_gate's mask at that threshold)
        thr_mid = 0.3
        stop_ref = torch.empty(G, dtype=torch.uint8, device=dev)
        ms_gate = timed(lambda: sr.sr_gate(seqs, lens, K, thr_mid, w.norm_mode, pair_sum=ps, mean=mean,
                                           stop=stop_ref, workspace=ws), 10)
        ms = timed(lambda: sr.sr_gate_decide(seqs, lens, K, thr_mid, w.norm_mode, pair_sum=ps, mean=mean,
                                             stop=stop_d, exact=ex, workspace=ws), 10)
        assert torch.equal(stop_d, stop_ref)
        extras["decide_C4_thr0.3"] = {"groups": G, "us_median": statistics.median(ms) * 1e3,
                                      "us_sr_gate_same_threshold": statistics.median(ms_gate) * 1e3,
                                      "groups_computed_exactly": int(ex.sum().item()),
                                      "groups_cut": int(stop_ref.sum().item()),
                                      "note": "above about 0.35 most groups have to be computed anyway and sr_gate is the faster call"}
        # restore the headline outputs for the checks below
        sr.sr_gate(seqs, lens, K, w.threshold, w.norm_mode, pair_sum=ps, mean=mean, stop=stop, workspace=ws)
        torch.cuda.synchronize()
        # end to end with the padded [groups][N][stride] host array instead of packed prefixes
        h_seqs = torch.from_numpy(w.seqs).pin_memory()
        h_lens = torch.from_numpy(w.lens).pin_memory()

        def e2e_padded():
            sr.sr_gate_host(h_seqs, h_lens, K, w.threshold, w.norm_mode, pair_sum=h_ps, mean=h_mean,
                            stop=h_stop, arena=arena, copy_stream=copy_stream)
            e2e_tail()

        ms = timed(e2e_padded, 20)
        extras["e2e_padded_input"] = {"ms_per_step": statistics.median(ms),
                                      "gcups": cells / (statistics.median(ms) * 1e-3) / 1e9,
                                      "h2d_bytes_per_step": h_seqs.numel() * 4 + h_lens.numel() * 4 + h_rew.numel() * 4 + h_stop.numel()}
        # the same pipeline on inputs without common prefixes (odd groups diverge from the
        # first token): nothing is removed, so this line shows the dp kernel on whole matrices
        w0 = W.token_gate(seed=3, n_groups=args.groups, shared_head=False)
        s0 = torch.from_numpy(w0.seqs).to(dev)
        l0 = torch.from_numpy(w0.lens).to(dev)
        ev0 = []
        for i in range(20):
            e5 = [torch.cuda.Event(enable_timing=True) for _ in range(5)]
            for e in e5:
                e.record()
            flush_l2(i)
            sr.sr_gate_stages(s0, l0, K, w0.threshold, w0.norm_mode, pair_sum=ps, mean=mean, stop=stop_d,
                              workspace=ws, events=e5)
            ev0.append(e5)
        torch.cuda.synchronize()
        dp0 = statistics.median(e5[2].elapsed_time(e5[3]) for e5 in ev0)
        all0 = statistics.median(e5[0].elapsed_time(e5[4]) for e5 in ev0)
        wc0 = W.word_columns(w0.lens, K, w0.seqs)
        extras["C4_no_shared_head"] = {"groups": w0.n_groups, "us_gate": all0 * 1e3, "us_dp": dp0 * 1e3,
                                       "gcups": W.dp_cells(w0.lens, K) / (all0 * 1e-3) / 1e9,
                                       "word_columns": wc0, "dp_alu_gops": 10.0 * wc0 / (dp0 * 1e-3) / 1e9,
                                       "dp_alu_frac": 10.0 * wc0 / (dp0 * 1e-3) / 1e9 / alu_peak}
        # small token-level batches (teams of up to a whole warp per pair)
        for small in (16, 64):
            ws_ = W.token_gate(seed=3, n_groups=small)
            r_ = gate_case(ws_)
            r_.pop("alu_gops"), r_.pop("alu_frac")        # those two count single-word columns
            extras[f"C4_{small}_groups"] = r_
        # a large batch of action-level groups at the paper's G = 8, K = 15
        extras["C2_x128_groups"] = gate_case(W.agent_gate(K=15, n_groups=65536), reps=10)
        # the rows beyond the gate proper: OR rule, Appendix-B signals, batch statistics
        w3 = W.large_group_gate(n_groups=65536)
        s3 = torch.from_numpy(w3.seqs).to(dev)
        outs = [torch.empty(w3.n_groups, dtype=torch.float64, device=dev) for _ in range(4)]
        ms = timed(lambda: sr.sr_group_signals(s3, None, w3.K, unique_prefix_ratio=outs[0],
                                               unique_action_ratio=outs[1], action_entropy=outs[2],
                                               bigram_jaccard_mean=outs[3]), 5)
        sig_bytes = w3.n_groups * (w3.N * 32 * 4 + 32)
        extras["group_signals_C3x16"] = {"groups": w3.n_groups, "N": w3.N, "us_median": statistics.median(ms) * 1e3,
                                         "groups_per_s": w3.n_groups / (statistics.median(ms) * 1e-3),
                                         "hbm_gbs": sig_bytes / (statistics.median(ms) * 1e-3) / 1e9,
                                         "bound": "instruction issue (hashing 480 bigrams per group); far from the HBM roofline"}
        l5 = torch.randint(0, 31, (big, 8), dtype=torch.int32, device=dev)
        m5 = torch.rand(big, dtype=torch.float64, device=dev)
        t5 = torch.empty(big, dtype=torch.float64, device=dev)
        ms = timed(lambda: sr.sr_gate_or_rule(m5, l5, None, 8, 15, 0.12, 0.9, tau=t5, stop=z_), 10)
        med = statistics.median(ms)
        or_bytes = big * (8 * 4 + 8 + 8 + 1)
        extras["or_rule_x64"] = {"groups": big, "us_median": med * 1e3, "hbm_gbs": or_bytes / (med * 1e-3) / 1e9,
                                 "hbm_frac": or_bytes / (med * 1e-3) / 1e9 / peaks["hbm_gbs"]}
        cnt = torch.empty(3, dtype=torch.int64, device=dev)
        ssq = torch.empty(2, dtype=torch.float64, device=dev)
        ms = timed(lambda: sr.sr_batch_stats(a_, z_, counts=cnt, sumsq=ssq), 10)
        med = statistics.median(ms)
        bs_bytes = big * (8 * 4 + 1)
        extras["batch_stats_x64"] = {"groups": big, "us_median": med * 1e3, "hbm_gbs": bs_bytes / (med * 1e-3) / 1e9,
                                     "hbm_frac": bs_bytes / (med * 1e-3) / 1e9 / peaks["hbm_gbs"]}
        flags = (torch.rand(big, device=dev) < 0.2).to(torch.uint8)
        kidx = torch.empty(big, dtype=torch.int32, device=dev)
        kcnt = torch.empty(1, dtype=torch.int32, device=dev)
        kws = torch.empty(sr.sr_kept_groups_workspace_bytes(big), dtype=torch.uint8, device=dev)
        ms = timed(lambda: sr.sr_kept_groups(flags, z_, index=kidx, count=kcnt, workspace=kws), 10)
        med = statistics.median(ms)
        kept_bytes = big * 2 + int(kcnt.item()) * 4 + 4
        extras["kept_groups_x64"] = {"groups": big, "kept": int(kcnt.item()), "us_median": med * 1e3,
                                     "hbm_gbs": kept_bytes / (med * 1e-3) / 1e9,
                                     "hbm_frac": kept_bytes / (med * 1e-3) / 1e9 / peaks["hbm_gbs"]}
        # host link: the end-to-end step cannot beat the copy of its own input
        ms = timed(lambda: arena[:h_sym.numel() * 4].view(torch.int32).copy_(h_sym, non_blocking=True), 10)
        med = statistics.median(ms)
        extras["h2d_link"] = {"bytes": h_sym.numel() * 4, "ms": med, "gbs": h_sym.numel() * 4 / (med * 1e-3) / 1e9,
                              "note": "pinned host -> device copy of the packed symbols alone: the floor of the e2e step"}
        line["extras"] = extras

        # CPU baseline: the oracle as it stands on this machine's host cores
        import oracle
        cores = min(os.cpu_count() or 1, oracle.max_threads())
        est_gcups = 0.4 * cores
        sample = int(max(16, min(G, G * 15.0 * est_gcups * 1e9 / cells)))
        c_s = W.dp_cells(w.lens[:sample], K)
        t0 = time.perf_counter()
        _, _, _, o_stop_cpu = oracle.gate(w.seqs[:sample], w.lens[:sample], K, w.threshold, w.norm_mode, threads=cores)
        oracle.advantage(w.rewards[:sample], o_stop_cpu, 1e-6)
        dt = time.perf_counter() - t0
        assert np.array_equal(o_stop_cpu, stop.cpu().numpy()[:sample])
        one = max(8, sample // (2 * cores))
        c_1 = W.dp_cells(w.lens[:one], K)
        t0 = time.perf_counter()
        oracle.gate(w.seqs[:one], w.lens[:one], K, w.threshold, w.norm_mode, threads=1)
        dt1 = time.perf_counter() - t0
        line["cpu_baseline"] = {"value": c_s / dt / 1e9, "unit": UNIT, "cores": cores, "kind": "oracle",
                                "sample": f"first {sample} of {G} groups, one pass, {dt:.1f} s",
                                "single_thread": {"value": c_1 / dt1 / 1e9, "unit": UNIT, "cores": 1,
                                                  "sample": f"first {one} groups, one pass, {dt1:.1f} s"}}
        # groups whose ordered fp64 d_K and exact rational d_K fall on different sides of the
        # threshold (none expected: the two differ by about 1e-16)
        razor = {}
        for name, wl in (("C1", W.tiny_gate()), ("C1_normalised", W.tiny_gate(raw_threshold=False)),
                         ("C2_K15", W.agent_gate(K=15)), ("C2_K30", W.agent_gate(K=30)),
                         ("C3", W.large_group_gate()), ("C4", w)):
            o_pd, _, _, o_st = oracle.gate(wl.seqs, wl.lens, wl.K, wl.threshold, wl.norm_mode, threads=cores)
            razor[name] = int((oracle.exact_mask(o_pd, wl.lens, wl.K, wl.threshold, wl.norm_mode) != o_st).sum())
        sq, ln = W.stream_prefix(s5.actions[:, :8192], s5.steps)
        o_pd, _, _, o_st = oracle.gate(sq, ln, 32, s5.threshold, s5.norm_mode, threads=cores)
        razor["C5_final_step_8192_groups"] = int((oracle.exact_mask(o_pd, ln, 32, s5.threshold, s5.norm_mode) != o_st).sum())
        line["extras"]["razor_edge_groups"] = razor
    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
