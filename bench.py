"""Benchmark of the batched what-if evaluation hot path on the largest workload configuration.

One step = the whole hot path over one batch: forward + backward pass for all policies with the
per-node slack matrix materialised (emo_slack_batch), the all-max-frequency baseline (emo_baseline)
and the constrained arg-min (emo_select), on the cfg4-llm graph (200 000 kernels + 50 000 CPU
nodes, ~470 k edges, 32 levels, 16 384 policies) with seeded synthetic inputs.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

Prints ONE JSON line (rank 0).  With N > 1 (torchrun) every rank runs a replica of the same
workload on its own GPU; the path has no exchange between GPUs.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "policy_edge_relaxations_per_s"
UNIT = "relaxations/s"


def measured_traffic(kernel: str):
    """DRAM bytes per node x policy of a pass kernel, from the committed ncu summary
    (profiles/dram_traffic.json, taken on a scaled-down case; traffic is proportional to n x B)."""
    p = os.path.join(ROOT, "profiles", "dram_traffic.json")
    if not os.path.exists(p):
        return None
    with open(p) as f:
        d = json.load(f)
    return d.get(kernel, {}).get("dram_bytes_per_node_policy")


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        return float(d["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "100", "-i", str(self.gpu)], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, smax, reasons = [], [], set()
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                smax.append(float(f[2]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def oracle_sample(g, lv_cols, threads, want_slack=True, keep=None):
    """Times the CPU oracle as it stands on the given policy columns; returns seconds."""
    import oracle
    t0 = time.perf_counter()
    r = oracle.batch(g, lv_cols, want_slack=want_slack, threads=threads)
    dt = time.perf_counter() - t0
    if keep is not None:
        keep.update(r)
    return dt


def workload_config(name, scale, g, B, ppm):
    """What both arms print as `config` (the same keys and values in both)."""
    return {"workload": name if scale == 1.0 else f"{name} x{scale}", "n": int(g.n), "m": int(g.m), "L": int(g.L),
            "policies": int(B), "passes": "forward+backward", "slack_materialised": True, "delta_ppm": int(ppm),
            "l2": "inputs larger than L2 (levels %.1f GB, slack %.1f GB per step)" % (g.n * B / 1e9, g.n * B * 8 / 1e9)}


def run_reference(args, rank, world):
    """The reference arm: the CPU oracle on the host cores, a bounded sample per step."""
    if rank != 0:
        return
    import numpy as np
    from paper_2607_12324_b200 import workloads as W
    g = W.make_graph(args.workload, args.scale)
    B = args.policies or g.meta["B"]
    ppm = (g.meta["delta_ppm"] or [50_000])[-1]
    threads = os.cpu_count() or 1
    per_step = max(threads, 2 * threads)
    total = per_step * (args.steps + args.warmup)
    cols = np.linspace(0, B - 1, total).astype(np.int64)
    lv = np.empty((g.n, total), dtype=np.uint8)
    for j0 in range(0, total, 64):
        js = cols[j0:j0 + 64]
        for k, c in enumerate(js):
            lv[:, j0 + k] = W.policy_levels(g.meta["policy_seed"], g.n, g.L, B, g.meta["policy_mode"], g.meta["q_max"],
                                            cols=(int(c), int(c) + 1)).numpy()[:, 0]
    for w in range(args.warmup):
        oracle_sample(g, np.ascontiguousarray(lv[:, w * per_step:(w + 1) * per_step]), threads)
    t = 0.0
    for s in range(args.steps):
        a = (args.warmup + s) * per_step
        t += oracle_sample(g, np.ascontiguousarray(lv[:, a:a + per_step]), threads)
    value = per_step * args.steps * g.m * 2 / t
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * t / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int64", "data": "synthetic",
            "config": workload_config(args.workload, args.scale, g, B, ppm),
            "policies_per_s": per_step * args.steps / t,
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle",
                             "sample": f"{per_step} of {B} policies per step, forward+backward with slack sums"},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


def other_workloads_leg(sm_mhz, hbm_gbs):
    """The smaller configurations (parity-test cases, not the headline): forward + backward pass with the slack matrix,
    default kernels, CUDA events, median of five calls after three; each beside its depth floor and its HBM time."""
    import numpy as np
    import torch
    from paper_2607_12324_b200 import emo, workloads as W
    names = {5: "32-bit spine forward + lane-stream backward", 4: "32-bit spine", 3: "generic", 2: "32-bit lane-stream", 1: "staged 64-bit", 0: "plain 64-bit"}
    out = []
    for name in ("cfg0-tiny", "cfg1-train", "cfg2-packed", "cfg3-8dev"):
        g = W.make_graph(name)
        B = g.meta["B"]
        lv = W.policies_for(g, B=B, device="cuda")
        h = emo.load_workload(g)
        info = h.info
        slack = torch.empty((g.n, B), dtype=torch.int64, device="cuda")
        T = torch.zeros(B, dtype=torch.int64, device="cuda")
        E = torch.zeros(B, dtype=torch.float64, device="cuda")
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        ws = torch.empty(emo.emo_workspace_bytes(h, B, 1), dtype=torch.uint8, device="cuda")
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
        for e in ev:
            e.record()
        fw, bw = [], []
        for it in range(8):
            emo.emo_set_pass_events(*ev)
            emo.emo_slack_batch(h, B, lv, lv.stride(0), None, None, slack, B, T, E, None, None, ws, status)
            emo.emo_set_pass_events(None, None, None, None)
            torch.cuda.synchronize()
            if it >= 3:
                fw.append(ev[0].elapsed_time(ev[1]))
                bw.append(ev[2].elapsed_time(ev[3]))
        assert int(status.item()) == 0
        out.append({"workload": name, "n": int(g.n), "policies": int(B),
                    "kernels": names[emo.emo_call_path(h, B, lv, lv.stride(0), B, True, 0)],
                    "fwd_ms": float(np.median(fw)), "bwd_ms": float(np.median(bw)),
                    "depth_floor_ms": 2 * info.depth * 30.0 / (sm_mhz * 1e6) * 1e3,
                    "t_hbm_ms": 9.0 * g.n * B / (hbm_gbs * 1e9) * 1e3})
        h.free()
        del slack, lv, ws
    return out


def intervals_leg(args, g, B, m, T0_ns, check):
    """Times emo_eval_intervals (device-resident inputs, CUDA events) and checks a few policies against the oracle."""
    import numpy as np
    import torch
    from paper_2607_12324_b200 import emo, workloads as W
    dev_of = W.device_of(g)
    D = int(dev_of.max()) + 1
    I = max(2, min(4096, int(T0_ns * 1.05 / 20e6) + 1))
    breaks = W.interval_breaks(T0_ns, I)
    F = W.interval_policies(g.meta["policy_seed"], D, I, g.L, B, device="cuda")
    ldb = F.shape[2]
    h = emo.load_workload(g, flags=args.flags | emo.EMO_F_INTERVALS, group_of=dev_of)
    T = torch.zeros(B, dtype=torch.int64, device="cuda")
    E = torch.zeros(B, dtype=torch.float64, device="cuda")
    Ei = torch.zeros(B, dtype=torch.float64, device="cuda")
    pi = torch.from_numpy(W.idle_power(g.L)).cuda()
    ws = torch.empty(emo.emo_workspace_bytes_intervals(h, B, I, True), dtype=torch.uint8, device="cuda")
    k = max(1, min(args.steps, 5))
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
    for it in range(min(args.warmup, 3) + k):
        if it == min(args.warmup, 3):
            ev[0].record()
        emo.emo_eval_intervals(h, B, F, ldb, I, breaks, pi, T, E, Ei, ws)
    ev[1].record()
    torch.cuda.synchronize()
    ms = ev[0].elapsed_time(ev[1]) / k
    out = {"ms_per_call": ms, "value": B * m / (ms * 1e-3), "unit": UNIT, "passes": "forward", "policies_per_s": B / (ms * 1e-3),
           "intervals": I, "devices": D, "grid_ns": int(breaks[1]), "idle_energy": True,
           "bound": "latency of a schedule step (the level look-up depends on the recurrence); no HBM or tensor roofline applies"}
    if check:
        nb = 8
        cols = np.linspace(0, B - 1, nb).astype(np.int64)
        Fh = F[:, :, torch.as_tensor(cols, device="cuda")].contiguous().cpu().numpy()
        import oracle      # the CPU oracle: checks only, never on the product path
        r = oracle.intervals(g, dev_of, breaks, Fh, W.idle_power(g.L))
        bad = int((T.cpu().numpy()[cols] != r["makespan"]).sum()) + int((~np.isclose(E.cpu().numpy()[cols], r["energy"], rtol=1e-9, atol=0)).sum())
        out["checked"] = {"policies": nb, "mismatches": bad}
        assert bad == 0, "interval evaluation disagrees with the oracle"
    if not args.no_search:
        # Alg. 2 on top of it: dynamic programming over the intervals, every stage's candidates as one batch
        T_max = T0_ns + T0_ns * int(args.search_ppm) // 1000000
        ws2 = torch.empty(emo.emo_workspace_bytes_search(h, I, 0, True), dtype=torch.uint8, device="cuda")
        t_start = time.perf_counter()
        r = emo.emo_search_dp(h, breaks, pi, T_max, 1000000, ws2)
        dt = time.perf_counter() - t_start
        Fb = torch.from_numpy(np.repeat(r["F"][None, :, None], D, axis=0).repeat(16, axis=2).copy()).cuda()
        emo.emo_eval_intervals(h, 1, torch.full((D, I, 16), g.L - 1, dtype=torch.uint8, device="cuda"), 16, I, breaks, pi, T, E, Ei, ws)
        torch.cuda.synchronize()
        E_default = float(E[0].item())
        out["search"] = {"found": r["found"], "budget_ppm": int(args.search_ppm), "bin_ns": 1000000, "predictions": r["n_pred"], "seconds": dt,
                         "predictions_per_s": r["n_pred"] / dt, "T_over_T0": r["T"] / T0_ns, "energy": r["E"],
                         "energy_default": E_default, "saving": 1.0 - r["E"] / E_default}
        if check and r["found"]:
            import oracle      # the CPU oracle: checks only, never on the product path
            ro = oracle.intervals(g, dev_of, breaks, Fb[:, :, :1].cpu().numpy(), W.idle_power(g.L))
            ok = int(ro["makespan"][0]) == r["T"] and bool(np.isclose(ro["energy"][0], r["E"], rtol=1e-9, atol=0))
            out["search"]["policy_checked_against_oracle"] = ok
            assert ok, "the searched policy's time and energy disagree with the oracle"
    h.free()
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg4-llm")
    ap.add_argument("--policies", type=int, default=0, help="override the number of policies (profiling a small case)")
    ap.add_argument("--scale", type=float, default=1.0, help="shrink the graph (profiling a small case)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--sums", action="store_true", help="also produce per-policy slack sums and critical counts")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--flags", type=int, default=0, help="extra EMO_F_* load flags (lanes / look-ahead)")
    ap.add_argument("--call-flags", type=int, default=0, help="EMO_F_* flags of the pass calls (kernel choice)")
    ap.add_argument("--no-intervals", action="store_true", help="skip the time-interval policy leg (Alg. 1 in its own form)")
    ap.add_argument("--no-others", action="store_true", help="skip the report-only timings of the smaller configurations")
    ap.add_argument("--no-search", action="store_true", help="skip the policy search (Alg. 2) inside the time-interval leg")
    ap.add_argument("--search-ppm", type=int, default=50000, help="latency budget of the policy search, parts per million of T_0")
    args = ap.parse_args()
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        run_reference(args, rank, world)
        return

    import numpy as np
    import torch
    from paper_2607_12324_b200 import build, emo, workloads as W

    if rank == 0:
        build.build()
    assert torch.cuda.is_available(), "bench.py needs a CUDA device (there is no CPU path)"
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
        dist.barrier()

    g = W.make_graph(args.workload, args.scale)
    B = args.policies or g.meta["B"]
    ppm = (g.meta["delta_ppm"] or [50_000])[-1]
    lv = W.policies_for(g, B=B, device="cuda")
    ldb = lv.stride(0)
    t_load = time.perf_counter()
    h = emo.load_workload(g, flags=args.flags)
    t_load = time.perf_counter() - t_load
    info = h.info
    fl = emo.emo_graph_flow(h, arrays=False)
    n, m = g.n, g.m
    slack = torch.empty((n, B), dtype=torch.int64, device="cuda")
    T = torch.zeros(B, dtype=torch.int64, device="cuda")
    E = torch.zeros(B, dtype=torch.float64, device="cuda")
    ss = torch.zeros(B, dtype=torch.int64, device="cuda")
    nc = torch.zeros(B, dtype=torch.int32, device="cuda")
    T0 = torch.zeros(1, dtype=torch.int64, device="cuda")
    E0 = torch.zeros(1, dtype=torch.float64, device="cuda")
    sel = torch.zeros(2, dtype=torch.int64, device="cuda")
    selE = torch.zeros(1, dtype=torch.float64, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    ws = torch.empty(emo.emo_workspace_bytes(h, B, 2, args.call_flags), dtype=torch.uint8, device="cuda")

    def step(events=None):
        if events is not None:
            emo.emo_set_pass_events(*events)
        emo.emo_slack_batch(h, B, lv, ldb, None, None, slack, B, T, E, sums[0], sums[1], ws, status, T0=T0, E0=E0,
                            flags=args.call_flags)
        if events is not None:
            emo.emo_set_pass_events(None, None, None, None)
        emo.emo_select(B, T, E, 0, sel[0:1], sel[1:2], selE, ws, target_dev=T0, delta_ppm=ppm)

    sums = (ss, nc) if args.sums else (None, None)
    launches_per_step = 4          # forward pass (with the baseline column), backward pass, 2 selection kernels
    for _ in range(max(args.warmup, 0)):
        step()
    torch.cuda.synchronize()

    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(args.steps)]
    for e4 in evs:
        for e in e4:
            e.record()                      # creates the handles before the timed region
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    start.record()
    for s in range(args.steps):
        step(evs[s])
    stop.record()
    torch.cuda.synchronize()
    total_ms = start.elapsed_time(stop)
    fwd_ms = [e4[0].elapsed_time(e4[1]) for e4 in evs]
    bwd_ms = [e4[2].elapsed_time(e4[3]) for e4 in evs]
    clocks = sampler.stop() if rank == 0 else None
    if dist is not None:
        tt = torch.tensor([total_ms], dtype=torch.float64, device="cuda")
        dist.all_reduce(tt, op=dist.ReduceOp.MAX)
        total_ms = float(tt.item())
        dist.barrier()
    assert int(status.item()) == 0, f"device status {int(status.item())}"
    ms_per_step = total_ms / args.steps
    passes = 2
    value = world * B * m * passes / (ms_per_step * 1e-3)

    # roofline of the dominant kernel (the backward pass: reads the levels, writes the slack matrix)
    peak, peak_kind = measured_peaks()
    bwd = sum(bwd_ms) / len(bwd_ms)        # average launch duration over the timed region
    fwd = sum(fwd_ms) / len(fwd_ms)
    dom_is_bwd = bwd >= fwd
    alg_bwd = n * B * 9 + B * 12            # 1 B level in + 8 B slack out per node x policy, per-policy sums out
    alg_fwd = n * B * 1 + B * 16            # 1 B level in per node x policy, makespan + energy out
    dom_ms, dom_bytes = (bwd, alg_bwd) if dom_is_bwd else (fwd, alg_fwd)
    achieved = dom_bytes / (dom_ms * 1e-3) / 1e9
    per_unit = measured_traffic("backward" if dom_is_bwd else "forward")
    traffic = None if per_unit is None else per_unit * n * B          # bytes per launch, scaled from the capture
    roofline = {"bound": "hbm", "kernel": "backward pass" if dom_is_bwd else "forward pass", "achieved": achieved,
                "peak": peak, "peak_source": peak_kind, "unit": "GB/s", "frac": achieved / peak, "traffic": traffic,
                "kernel_ms": dom_ms, "fwd_ms": fwd, "bwd_ms": bwd}
    step_bytes = n * B * 9 + B * 28
    roofline_step = {"bound": "hbm", "algorithmic_bytes": step_bytes, "achieved": step_bytes / (ms_per_step * 1e-3) / 1e9,
                     "peak": peak, "unit": "GB/s", "frac": step_bytes / (ms_per_step * 1e-3) / 1e9 / peak}

    # the three bounds of the step: HBM (algorithmic bytes at the measured copy rate), integer issue (one add per
    # node and one max per edge, per pass and policy, at the measured issue rate of 32-bit adds and maxima) and
    # the depth floor (the graph's hop levels times a dependent step of about 30 cycles; not a roofline, it
    # explains low fractions on shallow batches)
    scratch = torch.zeros(16, dtype=torch.int64, device="cuda")
    ipk = emo.emo_measure_int_issue(scratch)
    t_hbm = step_bytes / (peak * 1e9) * 1e3
    t_issue = passes * B / 32.0 * (n / ipk["add32"] + m / ipk["max32"]) * 1e3
    sm_mhz = (clocks or {}).get("sm_mhz") or 1965.0
    t_depth = passes * info.depth * 30.0 / (sm_mhz * 1e6) * 1e3
    # what one warp alone pays for the kernels' steps, and the measured time per schedule step: the passes walk a
    # dependency chain as long as the schedule, so the per-step latency times the steps is the time
    costs = emo.emo_measure_warp_costs(scratch)
    bounds = {"t_hbm_ms": t_hbm, "t_issue_ms": t_issue, "depth_floor_ms": t_depth,
              "binding": "hbm" if t_hbm >= t_issue else "int_issue",
              "int_issue_peak_warp_ops_per_s": ipk,
              "frac_of_binding": max(t_hbm, t_issue) / ms_per_step,
              "warp_costs_cycles": {k: round(v, 2) for k, v in costs.items()}}
    path = emo.emo_call_path(h, B, lv, ldb, B, True, args.call_flags)
    if path in (2, 5) and fl["steps"]:
        bounds["cycles_per_schedule_step"] = {"forward": fwd * 1e-3 * sm_mhz * 1e6 / fl["steps"], "backward": bwd * 1e-3 * sm_mhz * 1e6 / fl["steps"]}
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "int64", "data": "synthetic",
            "config": workload_config(args.workload, args.scale, g, B, ppm),
            "details": {"kernels": {5: "32-bit spine forward + lane-stream backward", 4: "32-bit spine", 3: "generic", 2: "32-bit lane-stream", 1: "staged 64-bit", 0: "plain 64-bit"}[path],
                        "slack_sums": bool(args.sums), "lanes": fl["lanes"] if path in (2, 5) else info.lanes,
                        "steps": fl["steps"] if path in (2, 5) else info.steps_fwd, "stage_steps": fl["K"], "barrier_steps": fl["sync"],
                        "restore_rows": fl["pushes"], "depth": info.depth, "graph_load_s": t_load,
                        "workspace_gb": ws.numel() / 1e9,
                        "parallelism": "replicas" if world > 1 else "single"},
            "policies_per_s": world * B / (ms_per_step * 1e-3),
            "gpu_launches": launches_per_step * args.steps,
            "roofline": roofline, "roofline_step": roofline_step, "bounds": bounds, "clocks": clocks,
            "selected": {"index": int(sel[0].item()), "T": int(sel[1].item()), "E": float(selE.item()),
                         "T0": int(T0.item()), "E0": float(E0.item())}}

    if path in (4, 5):
        line["details"]["spine"] = emo.emo_graph_spine(h)
    # end to end through the host-buffer entry point: the levels come from pinned host memory every step, packed
    # at ceil(log2 L) bits each (the call spreads them to bytes on the device), per-policy results and the
    # selection go back to the host; the slack matrix stays on the device
    if not args.no_e2e:
        bits = max(1, int(np.ceil(np.log2(max(g.L, 2)))))
        ldp = ((B + 7) // 8 * bits + 15) // 16 * 16
        dev_packed = torch.empty((g.n, ldp), dtype=torch.uint8, device="cuda")
        emo.emo_pack_levels(bits, g.n, B, lv, ldb, dev_packed, ldp)
        lv_host = torch.empty((g.n, ldp), dtype=torch.uint8).pin_memory()
        lv_host.copy_(dev_packed)
        hT = torch.zeros(B, dtype=torch.int64).pin_memory()
        hE = torch.zeros(B, dtype=torch.float64).pin_memory()
        hss = torch.zeros(B, dtype=torch.int64).pin_memory()
        hnc = torch.zeros(B, dtype=torch.int32).pin_memory()
        hsel = torch.zeros(4, dtype=torch.int64)
        dev_lvl = torch.empty_like(lv)
        hsums = (hss, hnc) if args.sums else (None, None)

        def e2e_step():
            emo.emo_slack_batch_host_packed(h, B, bits, lv_host, ldp, dev_packed, dev_lvl, ldb, slack, B, ppm, hT, hE,
                                            hsums[0], hsums[1], hsel, ws, flags=args.call_flags)
        e2e_step()
        torch.cuda.synchronize()
        k = max(1, min(args.steps, 5))
        if dist is not None:
            dist.barrier()
        t0 = time.perf_counter()
        for _ in range(k):
            e2e_step()
        torch.cuda.synchronize()
        serial_s = (time.perf_counter() - t0) / k
        assert int(hsel[0]) == int(sel[0].item())
        assert torch.equal(hT, T.cpu()), "the host-buffer call and the device call disagree"

        # the same steps with two device buffers: the copy of step s + 1 runs under the kernels of step s (every step's
        # levels still come from pinned host memory inside the timed region, every step's results still go back)
        dev_packed2 = torch.empty_like(dev_packed)
        bufs = (dev_packed, dev_packed2)
        copy_stream = torch.cuda.Stream()
        ready = (torch.cuda.Event(), torch.cuda.Event())

        def e2e_pipelined(steps):
            emo.emo_levels_prefetch(h, lv_host, ldp, bufs[0], copy_stream, ready[0])
            for s_ in range(steps):
                if s_ + 1 < steps:
                    emo.emo_levels_prefetch(h, lv_host, ldp, bufs[(s_ + 1) & 1], copy_stream, ready[(s_ + 1) & 1])
                emo.emo_slack_batch_prefetched(h, B, bits, bufs[s_ & 1], ldp, ready[s_ & 1], dev_lvl, ldb, slack, B, ppm, hT, hE,
                                               hsums[0], hsums[1], hsel, ws, flags=args.call_flags)
        hT.zero_()
        e2e_pipelined(2)
        torch.cuda.synchronize()
        k2 = max(1, min(args.steps, 10))
        if dist is not None:
            dist.barrier()
        t0 = time.perf_counter()
        e2e_pipelined(k2)
        torch.cuda.synchronize()
        e2e_s = (time.perf_counter() - t0) / k2
        if dist is not None:
            tt = torch.tensor([e2e_s, serial_s], dtype=torch.float64, device="cuda")
            dist.all_reduce(tt, op=dist.ReduceOp.MAX)
            e2e_s, serial_s = float(tt[0].item()), float(tt[1].item())
        assert int(hsel[0]) == int(sel[0].item())
        assert torch.equal(hT, T.cpu()), "the prefetched host-buffer call and the device call disagree"
        line["e2e"] = {"value": world * B * m * passes / e2e_s, "unit": UNIT, "ms_per_step": e2e_s * 1e3,
                       "h2d_bytes_per_step": int(g.n * ldp), "d2h_bytes_per_step": int(B * (28 if args.sums else 16) + 80),
                       "steps": k2, "ms_per_step_one_call": serial_s * 1e3,
                       "note": f"levels cross the bus packed at {bits} bits each, the copy of the next step under the kernels of "
                               "the current one (emo_levels_prefetch + emo_slack_batch_prefetched; ms_per_step_one_call: copy, "
                               "then kernels, in one call); the slack matrix stays on the device"}
        del dev_packed2
        del lv_host, dev_packed, dev_lvl

    # the next row of the path: Alg. 1 with time-interval policies (20 ms grid as in the paper's experiments) and
    # idle energy, on the same graph and batch size; a separate figure, not part of `value`
    if rank == 0 and not args.no_intervals:
        line["intervals"] = intervals_leg(args, g, B, m, T0_ns=int(T0.item()), check=not args.no_cpu)

    # the other configurations: report-only figures that explain themselves (depth floor, HBM time)
    if rank == 0 and not args.no_others and args.workload == "cfg4-llm" and args.scale == 1.0:
        line["other_workloads"] = other_workloads_leg(sm_mhz, peak)

    if rank == 0 and not args.no_cpu:
        threads = os.cpu_count() or 1
        # a probe of a few policies per thread sizes the sample for about 15 s of CPU work
        cnt = min(B, 8 * threads)
        cols = np.linspace(0, B - 1, cnt).astype(np.int64)
        sub = lv[:, torch.as_tensor(cols, device="cuda")].contiguous().cpu().numpy()
        oracle_sample(g, sub[:, :threads].copy(), threads)           # start the threads, touch the tables
        t1 = oracle_sample(g, sub, threads)
        cnt2 = int(min(B, max(threads, (15.0 / max(t1, 1e-3)) * cnt)))
        cols = np.linspace(0, B - 1, cnt2).astype(np.int64)
        cols_dev = torch.as_tensor(cols, device="cuda")
        sub = lv[:, cols_dev].contiguous().cpu().numpy()
        ref = {}
        t2 = oracle_sample(g, sub, threads, keep=ref)
        line["cpu_baseline"] = {"value": cnt2 * m * passes / t2, "unit": UNIT, "cores": threads, "kind": "oracle",
                                "sample": f"{cnt2} of {B} policies, forward+backward with slack sums, {t2:.1f} s",
                                "policies_per_s": cnt2 / t2}
        # the outputs of the last timed step against what the oracle just computed for the same policies:
        # makespan and slack sums (column sums of the materialised slack matrix) exact, energy to 1e-9
        Tg = T[cols_dev].cpu().numpy()
        Eg = E[cols_dev].cpu().numpy()
        bad = int((Tg != ref["makespan"]).sum()) + int((np.abs(Eg - ref["energy"]) > 1e-9 * np.abs(ref["energy"])).sum())
        nsum = min(cnt2, 512)
        ssg = slack[:, cols_dev[:nsum]].sum(dim=0).cpu().numpy()
        ncg = (slack[:, cols_dev[:nsum]] == 0).sum(dim=0).cpu().numpy()
        bad += int((ssg != ref["slack_sum"][:nsum]).sum()) + int((ncg != ref["n_critical"][:nsum]).sum())
        import oracle
        base = oracle.batch(g, np.full((g.n, 1), g.L - 1, dtype=np.uint8))
        bad += int(int(T0.item()) != int(base["makespan"][0]))
        line["checked"] = {"policies_makespan_energy": cnt2, "policies_slack_sum_and_critical_count": nsum,
                           "baseline_makespan": True, "mismatches": bad}
        assert bad == 0, f"{bad} outputs of the timed step differ from the oracle"
    if rank == 0:
        print(json.dumps(line), flush=True)
    h.free()
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
