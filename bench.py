#!/usr/bin/env python
"""Benchmark of the ESPO hot path on B200: fused decode step (rows/s, GB/s vs HBM peak) + advantage pass.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

A timed "step" is one espo_step call over the rollout batch (B=512 trajectories x V=152064
bf16 logits, temperature 1: the paper's 64 prompts x 8 rollouts at a Qwen-sized vocabulary).
The timed region is a rollout of K such steps followed by ONE espo_advantages pass over the
K*B tokens that rollout generated -- the whole path, at the cadence the method runs it.
The advantage kernel is additionally timed on its own workload (1024 ragged trajectories of
256..16384 tokens) and reported under "advantage_pass".

Prints one JSON line: the metric, the roofline of the step kernel, the advantage pass, an end-to-end figure with
host buffers, sampled clocks and the CPU oracle timed on the same box.
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
sys.path.insert(0, ROOT)

B_ROWS = 512
VOCAB = 152064
N_BUFFERS = 4                 # 4 x 155.7 MB of logits rotate, so no step finds its rows in the 126 MB L2
ADV_B = 1024
# dram bytes read + written per launch of the step kernel at (B_ROWS, VOCAB, bf16, hierarchical sampler): a constant
# copied from the ncu capture summarised under profiles/, not measured by this run
TRAFFIC_STEP_BYTES = 160.0e6
TARGET_REGION_MS = 250.0      # short timed regions are repeated until about this much device time has been timed

PARAMS = dict(temperature=1.0, mu_g=6.0, sigma2_g=9.0, delta=1e-8, clip_c=10.0, alpha_s=0.9, beta=7.0, eps=0.2,
              warmup_complete=1, t_max=1 << 30, eos_token=-1)
FILTER = {}   # top_p / top_k of the timed step when --top-p / --top-k ask for the filtered step


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.rows = []
        self.proc = None
        self.gpu = gpu_index
        self.thread = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "50", "-i", str(self.gpu)],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None
            return

        def pump():
            for line in self.proc.stdout:
                self.rows.append((time.time(), line.strip()))
        self.thread = threading.Thread(target=pump, daemon=True)
        self.thread.start()

    def stop(self):
        if self.proc is not None:
            self.proc.terminate()       # the exact process started above
            try:
                self.proc.wait(timeout=5)
            except Exception:
                pass

    def summary(self, t0: float, t1: float) -> dict:
        def parse(rows):
            sm, mx, reasons = [], [], set()
            for _, line in rows:
                f = [x.strip() for x in line.split(",")]
                if len(f) < 7:
                    continue
                try:
                    sm.append(float(f[0])); mx.append(float(f[1]))
                except ValueError:
                    continue
                for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[3:7]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
            return sm, mx, reasons
        inside = [r for r in self.rows if t0 <= r[0] <= t1]
        window = "timed region"
        if not inside:
            inside, window = self.rows, "whole run (timed region shorter than the sampling period)"
        sm, mx, reasons = parse(inside)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0, "window": "nvidia-smi unavailable"}
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "reasons": sorted(reasons),
                "samples": len(sm), "window": window}


def cpu_threads() -> int:
    try:
        return len(os.sched_getaffinity(0))
    except Exception:
        return os.cpu_count() or 1


def oracle_step_rate(rows_f32, values, seconds_target: float, sampler: int, cores: int | None = None):
    """Time the CPU oracle (as it stands) on a bounded sample of the benchmark's rows; returns rows/s.

    The sample rows are advanced decode step after decode step (new draws each step) on `cores` threads (default:
    all host cores) until about `seconds_target` seconds have passed.
    """
    import oracle
    cores = cores or cpu_threads()
    p = oracle.make_params(sampler=sampler, **PARAMS, **FILTER)
    n = rows_f32.shape[0]
    ro = oracle.Rollout(n, seed=1)
    done, t0 = 0, time.perf_counter()
    while True:
        ro.step_f32(rows_f32, values, p, n_threads=cores)
        done += n
        dt = time.perf_counter() - t0
        if dt >= seconds_target:
            break
    return done / dt, cores, done, dt


def oracle_advantage_rate(r, v, L, s, n_traj: int, cores: int):
    """Tokens/s of the oracle's advantage pass (backward recursion, float64) on the first `n_traj` trajectories."""
    import numpy as np
    import oracle
    Ls = L[:n_traj]
    n = int(Ls.astype(np.int64).sum())
    t0 = time.perf_counter()
    oracle.advantages_f32(r[:n], v[:n], Ls, s[:n_traj], 1.0, 0.95, -1.0, n_threads=cores)
    return n / (time.perf_counter() - t0), n


def run_reference(args):
    """--impl reference: the CPU oracle on the host cores, same metric and config, bounded sample per step."""
    import numpy as np
    import torch
    import oracle
    from paper_2605_29860_b200 import synth
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cores = cpu_threads()
    sample_rows = 32
    x = synth.logits_batch(sample_rows, VOCAB, dtype=torch.bfloat16, sd=3.0, seed=100, device="cpu").float().numpy()
    vals = np.full(sample_rows, 0.5)
    p = oracle.make_params(sampler=oracle.SAMPLER_HIER, **PARAMS)
    ro = oracle.Rollout(sample_rows, seed=1)
    for _ in range(args.warmup):
        ro.step_f32(x, vals, p, n_threads=cores)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        ro.step_f32(x, vals, p, n_threads=cores)
    dt = time.perf_counter() - t0
    value = sample_rows * args.steps / dt
    sample = f"{sample_rows} rows of the {B_ROWS}x{VOCAB} bf16 batch per step, hierarchical sampler"
    print(json.dumps({
        "impl": "reference", "metric": "fused ESPO step logit rows/s at V=152064 bf16", "value": value, "unit": "rows/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": f"rollout-batch scale: B={B_ROWS}, V={VOCAB}, bf16 logits, temperature 1.0 "
                               f"(CPU oracle on a {sample_rows}-row sample per step)"},
        "cpu_baseline": {"value": value, "unit": "rows/s", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "rows/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--rows", type=int, default=B_ROWS, help="rollout batch size B (default: the headline 512)")
    ap.add_argument("--sampler", default="hier", choices=["hier", "flat"])
    ap.add_argument("--top-p", type=float, default=1.0, help="time the filtered step instead (needs --sampler flat)")
    ap.add_argument("--top-k", type=int, default=0, help="time the filtered step instead (needs --sampler flat)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-sweep", action="store_true", help="skip the single-step timings at other shapes")
    ap.add_argument("--eager", action="store_true", help="launch every step separately instead of replaying a CUDA graph")
    ap.add_argument("--no-dependent-launch", action="store_true",
                    help="launch the step kernel plainly (default: as a programmatic dependent of the kernel before it)")
    ap.add_argument("--repeats", type=int, default=None,
                    help="times the K-step region is timed (default: enough repeats for ~150 ms; the median is reported)")
    args = ap.parse_args()
    if args.impl == "reference":
        args.steps = args.steps or 4
        args.warmup = args.warmup if args.warmup is not None else 1
        return run_reference(args)
    args.steps = args.steps or 20000
    args.warmup = max(3, args.warmup if args.warmup is not None else 200)

    import numpy as np
    import torch
    import paper_2605_29860_b200 as espo
    from paper_2605_29860_b200 import shard, synth

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU implementation")
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    dev = torch.device("cuda", local_rank)

    B, V, K, W = args.rows, VOCAB, args.steps, args.warmup
    sampler = espo.ESPO_SAMPLER_HIER if args.sampler == "hier" else espo.ESPO_SAMPLER_FLAT
    filtered = args.top_p < 1.0 or args.top_k > 0
    if filtered:
        if args.sampler != "flat":
            raise SystemExit("--top-p / --top-k need --sampler flat (the filtered step draws with the flat sampler)")
        FILTER.update(top_p=args.top_p, top_k=args.top_k)
    params = espo.make_params(sampler=sampler, **PARAMS, **FILTER)
    # ---- synthetic inputs, resident in HBM: every rank owns its own B rows (rows are independent) ----
    plan = shard.rank_plan(rank, world, B)
    bufs = [synth.logits_batch(B, V, dtype=torch.bfloat16, sd=3.0, seed=100 + plan["data_seed_offset"] + i, device=dev)
            for i in range(N_BUFFERS)]
    values = torch.full((B,), 0.5, dtype=torch.bfloat16, device=dev)
    tokens = torch.empty(B, dtype=torch.int32, device=dev)
    stop = torch.empty(B, dtype=torch.uint8, device=dev)
    state = espo.espo_init_state(B, V, seed=plan["state_seed"])
    # The step kernel is launched as a programmatic dependent of whatever precedes it in the stream (in a decode loop:
    # the LM head; here: the previous step): the GPU places its thread blocks and runs its set-up while that kernel
    # winds down, and the kernel waits for that kernel's completion before it touches global memory.
    use_pdl = not args.no_dependent_launch
    espo.espo_set_dependent_launch(state, use_pdl)
    view = espo.espo_state_view(state)
    # rollout record for the closing advantage pass: K tokens per trajectory, reward 0 except the end
    adv_tokens = B * K
    adv_r = torch.zeros(adv_tokens, device=dev)
    adv_v = torch.full((adv_tokens,), 0.5, device=dev)
    adv_out = torch.empty(adv_tokens, device=dev)
    adv_len = torch.full((B,), K, dtype=torch.int32, device=dev)
    adv_stopped = torch.zeros(B, dtype=torch.uint8, device=dev)
    espo.espo_advantages_reserve(max(B, ADV_B), max(adv_tokens, ADV_B * 16384))

    def rollout(n_steps):
        for i in range(n_steps):
            espo.espo_step(bufs[i % N_BUFFERS], values, state, params, tokens, stop)

    # The decode loop is launch-latency sensitive (one ~30 us kernel per step), so the timed rollout replays a CUDA
    # graph of GRAPH_STEPS consecutive steps (the remainder, and everything with --eager, is launched one by one).
    graph, graph_steps = None, 0
    if not args.eager and K >= 2 * N_BUFFERS:
        graph_steps = min(400, K) // N_BUFFERS * N_BUFFERS
        graph = torch.cuda.CUDAGraph()
        cap_stream = torch.cuda.Stream()
        cap_stream.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(cap_stream):
            rollout(N_BUFFERS)                      # warm the capture stream
            with torch.cuda.graph(graph, stream=cap_stream):
                rollout(graph_steps)
        torch.cuda.current_stream().wait_stream(cap_stream)

    def timed_rollout(n_steps):
        done = 0
        if graph is not None:
            while done + graph_steps <= n_steps:
                graph.replay()
                done += graph_steps
        rollout(n_steps - done)

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    def region(ev):
        """One timed region: K decode steps, then the advantage pass over the tokens they generated."""
        ev[0].record()
        timed_rollout(K)
        ev[1].record()
        espo.espo_advantages(adv_r, adv_v, adv_len, adv_stopped, 1.0, 0.95, -1.0, adv_out)
        ev[2].record()

    # Warm-up: W eager steps, then one untimed pass of exactly what is timed (so the graph that is timed has been
    # replayed before), which also gives the region's duration.
    rollout(W)
    ev_w = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
    region(ev_w)
    torch.cuda.synchronize()
    region(ev_w)                     # (the first pass pays for the graph's first replay: the second one is the estimate)
    torch.cuda.synchronize()
    est_ms = max(ev_w[0].elapsed_time(ev_w[2]), 1e-3)
    # A region of K steps that lasts less than TARGET_REGION_MS is repeated back to back (R times, every repeat
    # timed by its own events) and the median repeat is reported: one 0.6 ms region is shorter than a clock sample
    # and at the mercy of whatever the GPU did just before.
    R = int(min(1000, max(1, round(TARGET_REGION_MS / est_ms)))) if args.repeats is None else max(1, args.repeats)
    if dist is not None:
        R = int(shard.max_over_ranks([R], dist, device=dev)[0])
    espo.espo_reset_state(state, 0)
    sampler_proc = ClockSampler(local_rank) if rank == 0 else None
    if sampler_proc:
        sampler_proc.start()
        time.sleep(0.3)
    barrier()
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(R)]
    t_wall0 = time.time()
    for ev in evs:
        region(ev)
    barrier()
    t_wall1 = time.time()
    tot = sorted(ev[0].elapsed_time(ev[2]) for ev in evs)
    stp = sorted(ev[0].elapsed_time(ev[1]) for ev in evs)
    ms_total, ms_steps = statistics.median(tot), statistics.median(stp)
    ms_total, ms_steps = shard.max_over_ranks([ms_total, ms_steps], dist, device=dev)
    if sampler_proc:
        time.sleep(0.1)
        sampler_proc.stop()
    dev_status = espo.espo_state_status(state) | espo.espo_advantages_status()
    n_stopped = int((view["status"] != espo.ESPO_ROW_ACTIVE).sum().item())
    assert int(view["t"].min().item()) == K * R or n_stopped > 0, "the timed rollout did not advance every trajectory"

    rows_per_s = world * B * K / (ms_total * 1e-3)
    bytes_per_launch = B * V * 2
    kernel_ms = ms_steps / K
    peak, peak_kind = measured_peaks()
    achieved = bytes_per_launch / (kernel_ms * 1e-3) / 1e9

    traffic_known = (B == B_ROWS and args.sampler == "hier")
    out = {
        "metric": "fused ESPO step logit rows/s at V=152064 bf16", "value": rows_per_s, "unit": "rows/s",
        "n_gpus": world, "steps": K, "warmup": W, "ms_per_step": ms_total / K, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {
            "workload": f"rollout-batch scale: B={B} trajectories per GPU, V={V}, bf16 logits ~N(0,3) + 5 Zipf peaks, "
                        f"temperature 1.0, {args.sampler} Philox Gumbel-max sampler"
                        + (f" over the top-p {args.top_p} / top-k {args.top_k} support" if filtered else "")
                        + f", full active set; timed region = "
                        f"{K} decode steps + 1 advantage pass over the {adv_tokens} tokens generated",
            "logits_dtype": "bf16", "arithmetic": "f32 (f64 for the advantage scan's composition)",
            "launch": ("eager launches" if graph is None else f"CUDA graph of {graph_steps} steps, replayed once before timing")
                      + ("; step kernel launched as a programmatic dependent (set-up overlaps the previous kernel's end, no "
                         "global memory touched before that kernel has completed)" if use_pdl else "; plain launches"),
            "l2": f"{N_BUFFERS} logit buffers of {bytes_per_launch / 1e6:.1f} MB rotate (each larger than the 126 MB L2)",
            "parallelism": f"rows sharded over {world} GPU(s), no collective",
            "stopped_rows": n_stopped, "device_status": dev_status,
        },
        "timing": {"repeats": R, "region_ms_median": ms_total, "region_ms_min": tot[0], "region_ms_max": tot[-1],
                   "steps_ms_median": ms_steps, "steps_ms_min": stp[0], "steps_ms_max": stp[-1],
                   "note": "the K-step region (+ advantage pass) is timed `repeats` times back to back, each by its own "
                           "CUDA events; value, ms_per_step and roofline use the median repeat (max over ranks)"},
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "traffic": TRAFFIC_STEP_BYTES if traffic_known else None,
                     "traffic_source": ("constant from the ncu capture summarised under profiles/ (same kernel, same workload), "
                                        "not measured by this run") if traffic_known else "no capture at this shape",
                     "kernel": ("espo_filtered_kernel<bf16>" if filtered else "espo_step_hier_kernel<bf16,bulk>" if args.sampler == "hier"
                                else "espo_step_kernel<bf16,flat,bulk>"),
                     "peak_kind": f"of {peak_kind} copy bandwidth", "frac_of_nominal_8TBs": achieved / 8000.0,
                     "launch_us": kernel_ms * 1e3, "launch_us_min": stp[0] / K * 1e3, "launch_us_max": stp[-1] / K * 1e3,
                     "bytes_per_launch": bytes_per_launch},
        "gpu_launches": K + 2,
    }

    if rank == 0:
        # ---- the advantage kernel on its own workload (ragged batch of 1024 trajectories) ----
        r, v, L, s = synth.ragged_trajectories(ADV_B, seed=0, device=dev)
        a_out = torch.empty_like(r)
        n_tok = r.numel()
        for lam in (0.95,):
            for _ in range(5):
                espo.espo_advantages(r, v, L, s, 1.0, lam, -1.0, a_out)
            torch.cuda.synchronize()
            reps = 50
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(reps):
                espo.espo_advantages(r, v, L, s, 1.0, lam, -1.0, a_out)
            e1.record()
            torch.cuda.synchronize()
            adv_ms = e0.elapsed_time(e1) / reps
        adv_gbs = 12.0 * n_tok / (adv_ms * 1e-3) / 1e9
        out["advantage_pass"] = {
            "workload": f"B={ADV_B} ragged trajectories, lengths U[256,16384] ({n_tok} tokens, "
                        f"{12.0 * n_tok / 1e6:.1f} MB of traffic > L2), 35% stopped, gamma=1, lambda=0.95",
            "tokens_per_s": n_tok / (adv_ms * 1e-3), "ms": adv_ms,
            "roofline": {"bound": "hbm", "achieved": adv_gbs, "peak": peak, "unit": "GB/s", "frac": adv_gbs / peak,
                         "traffic": None, "bytes_per_token": 12},
        }
        ADV_TOKENS_NOMINAL = n_tok
        if not args.no_sweep:
            # ---- the other entry points of the advantage pass on the same batch ----
            def adv_us(fn, reps=30):
                for _ in range(3):
                    fn()
                torch.cuda.synchronize()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                for _ in range(reps):
                    fn()
                e1.record()
                torch.cuda.synchronize()
                return e0.elapsed_time(e1) * 1e3 / reps
            ret = torch.empty_like(r)
            sums = torch.zeros(2, dtype=torch.float64, device=dev)
            t_pad = int(L.max().item())
            pad_r = torch.zeros(ADV_B, t_pad, device=dev)
            pad_v = torch.zeros(ADV_B, t_pad, device=dev)
            keep = torch.arange(t_pad, device=dev)[None, :] < L[:, None]
            pad_r[keep] = r
            pad_v[keep] = v
            pad_out = torch.empty_like(pad_r)
            out["advantage_variants"] = {
                "lambda_1_us": adv_us(lambda: espo.espo_advantages(r, v, L, s, 1.0, 1.0, -1.0, a_out)),
                "with_returns_us": adv_us(lambda: espo.espo_advantages_returns(r, v, L, s, 1.0, 0.95, -1.0, a_out, ret)),
                "with_batch_sums_us": adv_us(lambda: espo.espo_advantages_stats(r, v, L, s, 1.0, 0.95, -1.0, a_out, sums)),
                "padded_layout_us": adv_us(lambda: espo.espo_advantages_padded(pad_r, pad_v, L, s, 1.0, 0.95, -1.0, pad_out)),
                "note": f"same batch as advantage_pass; padded: [{ADV_B}, {t_pad}] ({ADV_B * t_pad} entries, {n_tok} of them tokens)",
            }
            del ret, pad_r, pad_v, pad_out, keep
        del r, v, L, s, a_out

        # ---- library operations that move the same number of bytes, timed the same way: at these sizes (one launch
        #      of 100-160 MB) launch, ramp and tail keep even a plain copy well below the large-buffer copy bandwidth
        #      that `peak` is ----
        if not args.no_sweep:
            def time_us(fn, reps=100):
                for i in range(5):
                    fn(i)
                torch.cuda.synchronize()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                for i in range(reps):
                    fn(i)
                e1.record()
                torch.cuda.synchronize()
                return e0.elapsed_time(e1) * 1e3 / reps
            half = [torch.empty(B // 2, V, dtype=torch.bfloat16, device=dev) for _ in range(2)]
            row_max = torch.empty(B, dtype=torch.bfloat16, device=dev)
            adv_src = torch.empty(int(12.0 * ADV_TOKENS_NOMINAL / 8), dtype=torch.float32, device=dev).normal_()
            adv_dst = torch.empty_like(adv_src)
            lib = {
                "copy_moving_step_bytes_us": time_us(lambda i: half[i % 2].copy_(bufs[i % N_BUFFERS][:B // 2])),
                "torch_amax_over_step_logits_us": time_us(lambda i: torch.amax(bufs[i % N_BUFFERS], dim=1, out=row_max)),
                "copy_moving_advantage_bytes_us": time_us(lambda i: adv_dst.copy_(adv_src)),
                "note": f"step launch: {bytes_per_launch / 1e6:.1f} MB read; copy: {bytes_per_launch / 2e6:.1f} MB read + as much "
                        f"written; advantage pass: {12.0 * ADV_TOKENS_NOMINAL / 1e6:.1f} MB moved",
            }
            out["library_ops_same_bytes"] = lib
            del half, adv_src, adv_dst

        # Times launch(i) (i picks the input variant, so that consecutive launches read different buffers) as a CUDA
        # graph of >= 40 launches: replayed once untimed, then for about 30 ms; returns microseconds per launch.
        def graph_time_us(launch, n_variants, total_ms=30.0):
            n = n_variants * max(1, -(-40 // n_variants))
            g = torch.cuda.CUDAGraph()
            side = torch.cuda.Stream()
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(side):
                for i in range(max(3, n_variants)):
                    launch(i)
                with torch.cuda.graph(g, stream=side):
                    for i in range(n):
                        launch(i)
            torch.cuda.current_stream().wait_stream(side)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(); g.replay(); e1.record()
            torch.cuda.synchronize()
            reps = int(min(200, max(1, round(total_ms / max(e0.elapsed_time(e1), 1e-3)))))
            e0.record()
            for _ in range(reps):
                g.replay()
            e1.record()
            torch.cuda.synchronize()
            us = e0.elapsed_time(e1) * 1e3 / (reps * n)
            del g
            return us

        # ---- the bench's step under both launch modes, timed the same way (graph of 40 steps over the rotating buffers)
        if not args.no_sweep:
            modes = {}
            for name, flag in (("plain_launch_us", False), ("dependent_launch_us", True)):
                mst = espo.espo_init_state(B, V, seed=3)
                espo.espo_set_dependent_launch(mst, flag)
                modes[name] = graph_time_us(lambda i: espo.espo_step(bufs[i % N_BUFFERS], values, mst, params, tokens, stop), N_BUFFERS)
                espo.espo_free_state(mst)
            out["launch_modes"] = modes

        # ---- single-step bandwidth at other shapes: the large-batch sweep, every (B, V, dtype) with the hierarchical
        #      sampler and the V=152064 column with the flat one too; rotating buffers of > 2 x L2 in total ----
        if not args.no_sweep:
            sweep = []
            flat_params = espo.make_params(sampler=espo.ESPO_SAMPLER_FLAT, **PARAMS)
            hier_params = espo.make_params(sampler=espo.ESPO_SAMPLER_HIER, **PARAMS)
            for sV in (32000, 128256, VOCAB):
                for sdt in (torch.bfloat16, torch.float32):
                    for sB in (128, 256, 512, 1024, 2048):
                        es = 2 if sdt == torch.bfloat16 else 4
                        per = sB * sV * es
                        nb = max(2, int(280e6 // per) + 1)
                        sbufs = [synth.logits_batch(sB, sV, dtype=sdt, sd=3.0, seed=500 + i, device=dev) for i in range(nb)]
                        sst = espo.espo_init_state(sB, sV, seed=99)
                        espo.espo_set_dependent_launch(sst, use_pdl)      # the main region's launch mode
                        sval = torch.full((sB,), 0.5, dtype=torch.bfloat16, device=dev)
                        stok = torch.empty(sB, dtype=torch.int32, device=dev)
                        sstop = torch.empty(sB, dtype=torch.uint8, device=dev)
                        row = {"B": sB, "V": sV, "logits": "bf16" if es == 2 else "f32", "MB": per / 1e6}
                        for name, pp in (("hier", hier_params),) + ((("flat", flat_params),) if sV == VOCAB else ()):
                            us = graph_time_us(lambda i: espo.espo_step(sbufs[i % nb], sval, sst, pp, stok, sstop), nb)
                            gbs = per / us / 1e3
                            row[name] = {"us": us, "GB/s": gbs, "frac_of_measured_peak": gbs / peak,
                                         "frac_of_nominal_8TBs": gbs / 8000.0, "rows/s": sB / (us * 1e-6)}
                        sweep.append(row)
                        espo.espo_free_state(sst)
                        del sbufs
            out["bandwidth_sweep"] = {"shapes": sweep,
                                      "note": "one espo_step per launch, CUDA graph of >= 40 launches over rotating buffers "
                                              "(> 280 MB in total), full active set; GB/s = B*V*sizeof(logit) / time; "
                                              + ("hierarchical step launched as a programmatic dependent, like the main region"
                                                 if use_pdl else "plain launches")}

            # ---- shrinking active set: as rows stop, the caller passes the n_active surviving rows (compacted
            #      logits plus the slot list from espo_compact_active); per-step time vs n_active ----
            act = []
            sst = espo.espo_init_state(B, V, seed=7)
            espo.espo_set_dependent_launch(sst, use_pdl)
            all_ids = torch.arange(B, dtype=torch.int32, device=dev)
            n_act_dev = torch.zeros(1, dtype=torch.int32, device=dev)
            for n_act in (B, (3 * B) // 4, B // 2, B // 4, B // 8):
                ids = all_ids[:n_act].contiguous()
                us = graph_time_us(lambda i: espo.espo_step(bufs[i % N_BUFFERS][:n_act], values[:n_act], sst, params, tokens, stop,
                                                            row_ids=ids, n_rows=n_act), N_BUFFERS)
                act.append({"n_active": n_act, "us": us, "GB/s": n_act * V * 2 / us / 1e3, "rows/s": n_act / (us * 1e-6)})
            ids_out = torch.empty(B, dtype=torch.int32, device=dev)

            def step_then_compact(i):
                espo.espo_step(bufs[i % N_BUFFERS], values, sst, params, tokens, stop)
                espo.espo_compact_active(sst, ids_out, n_act_dev)
            espo.espo_set_dependent_launch(sst, True)
            pair_us = graph_time_us(step_then_compact, N_BUFFERS)
            step_alone_us = graph_time_us(lambda i: espo.espo_step(bufs[i % N_BUFFERS], values, sst, params, tokens, stop), N_BUFFERS)
            espo.espo_set_dependent_launch(sst, False)
            out["active_set"] = {"steps": act,
                                 "compact_extra_us_dependent_launch": pair_us - step_alone_us,
                                 "compact_us": graph_time_us(lambda i: espo.espo_compact_active(sst, ids_out, n_act_dev), 1),
                                 "note": f"capacity {B} slots, bf16, V={V}; CUDA graphs, "
                                         + ("step launched as a programmatic dependent" if use_pdl else "plain launches")
                                         + "; compaction is a separate one-CTA kernel"}
            espo.espo_free_state(sst)

        # ---- the other routes through the step: flat sampler, top-p filter, vocabulary shards ----
        if not args.no_sweep:
            def step_us(p, fn=None, n_var=N_BUFFERS):
                sst = espo.espo_init_state(B, V, seed=5)
                espo.espo_set_dependent_launch(sst, use_pdl)          # (only the hierarchical kernels are launched that way)
                call = (lambda i: espo.espo_step(bufs[i % N_BUFFERS], values, sst, p, tokens, stop)) if fn is None else (lambda i: fn(i, sst))
                us = graph_time_us(call, n_var)
                espo.espo_free_state(sst)
                return us
            flat = espo.make_params(sampler=espo.ESPO_SAMPLER_FLAT, **PARAMS)
            top_p = espo.make_params(sampler=espo.ESPO_SAMPLER_FLAT, top_p=0.7, **PARAMS)
            top_p_wide = espo.make_params(sampler=espo.ESPO_SAMPLER_FLAT, top_p=0.9999, **PARAMS)
            cuts = shard.vocab_shards(V, 8, multiple=1024)
            lo, n_ids = cuts[3]
            shard_bufs = [synth.logits_batch(B, n_ids, dtype=torch.bfloat16, sd=3.0, seed=700 + i, device=dev) for i in range(16)]
            parts = torch.zeros(8, B, 8, dtype=torch.float32, device=dev)
            out["other_routes"] = {
                "flat_sampler_us": step_us(flat),
                "top_p_0.7_us": step_us(top_p),
                "top_p_0.9999_us": step_us(top_p_wide),
                "vocab_shard_partial_us": step_us(flat, lambda i, sst: espo.espo_step_partial(shard_bufs[i % 16], lo, sst, flat, parts[3]), 16),
                "vocab_shard_partial_hier_us": step_us(hier_params, lambda i, sst: espo.espo_step_partial(shard_bufs[i % 16], lo, sst, hier_params, parts[3]), 16),
                "vocab_shard_merge_us": step_us(flat, lambda i, sst: espo.espo_step_merge(parts, values, sst, flat, tokens, stop), 1),
                "note": f"same batch (B={B}, V={V}, bf16), CUDA graphs; partial: one of 8 shards ({n_ids} ids) as its own buffer; "
                        f"merge: 8 x {B} partials",
            }
            del shard_bufs

        # ---- end to end through the public API with HOST buffers (pinned), copies inside the timed region ----
        host_logits = [torch.empty(B, V, dtype=torch.bfloat16).pin_memory() for _ in range(2)]
        for i in range(2):
            host_logits[i].copy_(bufs[i])
        host_values = torch.full((B,), 0.5, dtype=torch.bfloat16).pin_memory()
        host_tokens = torch.empty(B, dtype=torch.int32).pin_memory()
        host_stop = torch.empty(B, dtype=torch.uint8).pin_memory()
        dev_logits = torch.empty(B, V, dtype=torch.bfloat16, device=dev)
        dev_values = torch.empty(B, dtype=torch.bfloat16, device=dev)
        espo.espo_reset_state(state, 1)

        def e2e_step(i):
            dev_logits.copy_(host_logits[i % 2], non_blocking=True)
            dev_values.copy_(host_values, non_blocking=True)
            espo.espo_step(dev_logits, dev_values, state, params, tokens, stop)
            host_tokens.copy_(tokens, non_blocking=True)
            host_stop.copy_(stop, non_blocking=True)
            torch.cuda.synchronize()       # the caller needs the tokens before the next decode step

        for i in range(3):
            e2e_step(i)
        n_e2e = 20
        t0 = time.perf_counter()
        for i in range(n_e2e):
            e2e_step(i)
        dt = time.perf_counter() - t0
        out["e2e"] = {"value": B * n_e2e / dt, "unit": "rows/s", "h2d_bytes_per_step": B * V * 2 + B * 2,
                      "d2h_bytes_per_step": B * 4 + B, "steps": n_e2e, "n_gpus": 1,
                      "note": "pinned host logits copied in, tokens and stop mask copied out, every step"}
        del host_logits, dev_logits

        # ---- clocks ----
        out["clocks"] = sampler_proc.summary(t_wall0, t_wall1) if sampler_proc else None

        # ---- the CPU oracle on this machine's host cores, on a bounded sample of the same rows ----
        if not args.no_cpu_baseline:
            sample_src = bufs[0][:256].float().cpu().numpy()
            rate, cores, n_rows, secs = oracle_step_rate(sample_src, np.full(256, 0.5), 10.0, sampler)
            out["cpu_baseline"] = {"value": rate, "unit": "rows/s", "cores": cores, "kind": "oracle",
                                   "sample": f"{n_rows} row-steps: rows 0..255 of buffer 0 advanced step after step "
                                             f"for {secs:.1f} s on {cores} threads"}
            rate1, _, n1, secs1 = oracle_step_rate(sample_src[:16], np.full(16, 0.5), 3.0, sampler, cores=1)
            out["cpu_baseline"]["one_core"] = {"value": rate1, "unit": "rows/s", "cores": 1,
                                               "sample": f"{n1} row-steps: rows 0..15 of buffer 0 for {secs1:.1f} s on 1 thread"}
            # the oracle's advantage pass on a bounded slice of the advantage workload (tokens/s)
            ar, av, aL, a_s = (t.cpu().numpy() for t in synth.ragged_trajectories(ADV_B, seed=0, device=dev))
            a_all, n_all = oracle_advantage_rate(ar, av, aL, a_s, 256, cores)
            a_one, n_one = oracle_advantage_rate(ar, av, aL, a_s, 64, 1)
            out["cpu_baseline"]["advantages"] = {
                "value": a_all, "unit": "tokens/s", "cores": cores, "kind": "oracle",
                "sample": f"first 256 of the {ADV_B} trajectories of the advantage workload ({n_all} tokens), backward recursion "
                          f"in float64, gamma=1, lambda=0.95",
                "one_core": {"value": a_one, "unit": "tokens/s", "cores": 1, "sample": f"first 64 trajectories ({n_one} tokens)"}}
        print(json.dumps(out))
    espo.espo_free_state(state)
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
