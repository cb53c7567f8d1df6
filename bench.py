#!/usr/bin/env python
"""Benchmark of the HilbertA hot path on B200.

One step = one pass of the whole path over one batch of synthetic Flux-shaped
activations that are already resident in HBM (original token order):
    permute(Q), permute(K), permute(V) -> sparse attention forward, whose epilogue
    writes O back in the original token order (hilberta_forward_unpermute)
The plan (Hilbert LUT, permutation, key ranges) is built once, outside the
steps, and its build time is reported separately.  Inputs (Q+K+V+O = 415 MB at
2048^2) are larger than the 126 MB L2, so nothing is L2-resident between steps.

Prints ONE JSON line (rank 0).  `--impl reference` times the CPU fp64 oracle
instead (rank 0 only), on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

NOMINAL_BF16_TFLOPS = 2250.0
L2_BYTES = 126 * 2**20   # B200 L2
# Idle time before a side row is timed: the GPU's clock follows a moving average of its power draw
# (1 kW cap), so a row measured right after seconds of full load runs at 1.3-1.5 GHz instead of the
# 1.6-1.9 GHz a short run sees.  Every row also reports the SM clock its last launch ran at.
COOL_DOWN_S = 1.0
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
# dram__bytes_read.sum + dram__bytes_write.sum of one forward launch: one ncu capture of the
# single-CTA bf16 kernel at this workload, taken on the kernel revision with a four-slot K/V ring and
# the output staging area (559.7 MB read + 99.7 MB written; the revisions before it measured 651.6 and
# 647.5 MB).
FORWARD_DRAM_TRAFFIC_BYTES = {"flux2048": 659.4e6}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            d = json.load(f)
        return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d["bf16_tflops"]),
                "bf16_tflops_sustained": float(d.get("bf16_tflops_sustained", d["bf16_tflops"])),
                "source": "measured"}
    except Exception:
        return dict(FALLBACK_PEAKS, source="fallback")


class ClockSampler(threading.Thread):
    """Polls SM clock and throttle reasons through NVML (read-only) while the
    timed region runs."""

    def __init__(self, index: int, period_s: float = 0.001):
        super().__init__(daemon=True)
        self.index, self.period = index, period_s
        self.samples, self.stamps, self.reasons = [], [], set()
        self.max_mhz = None
        self._stop_evt = threading.Event()
        self.ok = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            self.ok = True
        except Exception:
            self.ok = False

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        names = {
            "hw_slowdown": getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8),
            "hw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40),
            "sw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20),
            "sw_power_cap": getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4),
            "hw_power_brake": getattr(nv, "nvmlClocksEventReasonHwPowerBrakeSlowdown", 0x80),
        }
        while not self._stop_evt.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                self.stamps.append(time.perf_counter())
                try:
                    mask = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for k, bit in names.items():
                    if mask & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            time.sleep(self.period)

    def stop(self, window=None):
        """window = (t0, t1) in time.perf_counter() seconds: also report the samples taken inside it."""
        self._stop_evt.set()
        self.join(timeout=2)
        out = {"sm_mhz": statistics.median(self.samples) if self.samples else None,
               "sm_min_mhz": min(self.samples) if self.samples else None,
               "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples),
               "period_ms": 1e3 * self.period}
        if window:
            inside = [m for m, t in zip(self.samples, self.stamps) if window[0] <= t <= window[1]]
            out["samples_in_timed_region"] = len(inside)
            out["sm_mhz_in_timed_region"] = statistics.median(inside) if inside else None
        return out


def oracle_sample(wl, seconds_target: float, heads: int = 2):
    """Time the oracle (as it stands) on a seeded sample of query rows of the
    workload; returns (useful TFLOP/s, threads, description, seconds)."""
    import numpy as np

    from oracle import attn_c
    from oracle import hilberta_oracle as orc
    from paper_2509_26538_b200.inputs import make_qkv, sample_rows

    ig, grp = orc.token_classes(wl.H, wl.W, wl.tile, wl.layer_offset, wl.shared_region, wl.n_text)
    n_glob = int(ig.sum())
    per_group = np.bincount(grp[(grp >= 0) & (ig == 0)], minlength=wl.HW // wl.tile)

    def pairs_of(rows, n_heads):
        tot = 0
        for r in rows:
            tot += wl.S if ig[r] else n_glob + int(per_group[grp[r]])
        return tot * n_heads * wl.batch

    # calibrate on a small sample, then size the timed sample for the target:
    # first widen to all query rows, then add heads
    q, k, v = make_qkv(wl, heads=heads)
    qf, kf, vf = (t.float().numpy() for t in (q, k, v))
    rows = sample_rows(wl, 256, seed=1)
    attn_c.attention_rows(qf, kf, vf, ig, grp, rows=rows[:8])  # thread start-up
    t0 = time.perf_counter()
    attn_c.attention_rows(qf, kf, vf, ig, grp, rows=rows)
    dt = time.perf_counter() - t0
    rate = pairs_of(rows, heads) / max(dt, 1e-6)
    budget = seconds_target * rate
    all_rows = list(range(wl.S))
    full_per_head = pairs_of(all_rows, 1)
    if budget >= full_per_head:
        n_heads = int(max(1, min(wl.heads, budget // full_per_head)))
        rows = all_rows
    else:
        n_heads = 1
        n_rows = int(max(64, wl.S * budget / full_per_head))
        rows = sorted(np.random.default_rng(wl.seed).choice(wl.S, size=n_rows, replace=False).tolist())
    if n_heads != heads:
        q, k, v = make_qkv(wl, heads=n_heads)
        qf, kf, vf = (t.float().numpy() for t in (q, k, v))
    t0 = time.perf_counter()
    _, threads = attn_c.attention_rows(qf, kf, vf, ig, grp, rows=rows, return_threads=True)
    dt = time.perf_counter() - t0
    flops = 4.0 * wl.head_dim * pairs_of(rows, n_heads)
    desc = (f"{len(rows)} query rows (of {wl.S}) x {n_heads} heads (of {wl.heads}) of {wl.name}, "
            f"all kept keys, fp64")
    return flops / dt / 1e12, int(threads), desc, dt


def run_reference(args, wl):
    """CPU oracle arm: rank 0 only; other ranks exit without work."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    if "TORCHELASTIC_RUN_ID" in os.environ and os.environ.get("OMP_NUM_THREADS") == "1":
        # torch.distributed.run pins every rank to one OpenMP thread; this arm runs on rank 0 alone
        del os.environ["OMP_NUM_THREADS"]
    total_budget = 150.0
    per_step = max(0.05, min(20.0, total_budget / (args.steps + args.warmup + 1)))
    vals, times = [], []
    threads, desc = 0, ""
    for i in range(args.warmup + args.steps):
        tf, threads, desc, dt = oracle_sample(wl, per_step)
        if i >= args.warmup:
            vals.append(tf)
            times.append(dt)
    value = statistics.mean(vals)
    line = {
        "impl": "reference", "metric": "sparse-attn useful TFLOP/s at 2048^2 (Flux shape)", "value": value,
        "unit": "TFLOP/s", "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": 1e3 * statistics.mean(times), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(wl, args.gpus),
        "cpu_baseline": {"value": value, "unit": "TFLOP/s", "cores": threads, "kind": "oracle",
                         "sample": desc + " per step"},
        "e2e": {"value": value, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def workload_config(wl, n_gpus, shard="replicas"):
    return {"workload": f"{wl.name}: {wl.H}x{wl.W} image tokens + {wl.n_text} text, batch {wl.batch} per GPU, "
                        f"{wl.heads} heads x {wl.head_dim}, tile {wl.tile}, shared {wl.shared_region}x"
                        f"{wl.shared_region}, offset {wl.layer_offset}",
            "S": wl.S, "tile": wl.tile, "shared_region": wl.shared_region, "layer_offset": wl.layer_offset,
            "step": "permute(Q,K,V) + sparse forward with the exit unpermute fused into its epilogue",
            "l2": ("inputs larger than L2 (Q+K+V+O = %d MB)" if 4 * wl.batch * wl.heads * wl.S * wl.head_dim * 2 > L2_BYTES
                   else "Q+K+V+O = %d MB fits in L2: the steps rotate through several copies of their buffers") %
                  (4 * wl.batch * wl.heads * wl.S * wl.head_dim * 2 // 2**20),
            "parallelism": (f"replicas x{n_gpus} (independent batches, no collective)" if shard == "replicas" else
                            f"one batch, its (batch, head) units split over {n_gpus} GPUs ({wl.heads} heads on this rank), no collective")}


def device_qkv(torch, wl, seed_offset=0):
    """Q, K, V ~ N(0,1) drawn on the device from the workload's seed (the timing-only rows of the other
    workload sizes; the parity tests and the main workload use the CPU draw of inputs.make_qkv)."""
    g = torch.Generator(device="cuda")
    g.manual_seed(wl.seed + seed_offset)
    shape = (wl.batch, wl.heads, wl.S, wl.head_dim)
    return tuple(torch.randn(shape, generator=g, device="cuda", dtype=torch.float32).to(torch.bfloat16) for _ in range(3))


def n_buffer_sets(wl, tensors_per_set=4):
    """Workloads whose tensors fit in L2 rotate through several copies so that no call finds its inputs cached."""
    set_bytes = tensors_per_set * wl.batch * wl.heads * wl.S * wl.head_dim * 2
    return 1 if set_bytes >= 2 * L2_BYTES else min(8, -(-3 * L2_BYTES // set_bytes))


def time_forward_config(hb, torch, wl, peaks, stream, n_calls=30):
    """ms per forward call (CUDA events around each launch) of one workload configuration."""
    n_sets = n_buffer_sets(wl)
    sets = [device_qkv(torch, wl, 17 * i) for i in range(n_sets)]   # used as if already in physical order
    out = torch.empty_like(sets[0][0])
    t0 = time.perf_counter()
    plan = hb.Plan(wl.H, wl.W, wl.tile, wl.layer_offset, wl.shared_region, wl.n_text)
    plan.bind_like(out)
    torch.cuda.synchronize()
    plan_ms = 1e3 * (time.perf_counter() - t0)
    nnz = int(plan.export(hb.EXPORT_NNZ)[0])
    flops = 4.0 * wl.head_dim * wl.heads * wl.batch * nnz
    for i in range(4):
        plan.forward(*sets[i % n_sets], out)
    torch.cuda.synchronize()
    time.sleep(COOL_DOWN_S)   # the rows before this one ran the GPU into its power cap
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n_calls)]
    for i, (a, b_) in enumerate(ev):
        a.record(stream)
        plan.forward(*sets[i % n_sets], out)
        b_.record(stream)
    torch.cuda.synchronize()
    assert plan.status() == 0, "device-side wait timed out"
    assert torch.isfinite(out.float()).all()
    lc = plan.export(hb.EXPORT_LAUNCH_CLOCK)
    ms = sorted(a.elapsed_time(b_) for a, b_ in ev)
    med = ms[len(ms) // 2]
    tf = flops / (med * 1e-3) / 1e12
    plan.destroy()
    del sets, out
    torch.cuda.empty_cache()
    return {"workload": "%s: %dx%d + %d text, %d heads x %d, tile %d, shared %d, offset %d" % (
                wl.name, wl.H, wl.W, wl.n_text, wl.heads, wl.head_dim, wl.tile, wl.shared_region, wl.layer_offset),
            "ms_per_call_median": med, "ms_per_call_min": ms[0], "useful_tflops": tf, "nnz": nnz,
            "useful_gflop_per_call": flops / 1e9,
            "frac_of_measured_burst_peak": tf / peaks["bf16_tflops"],
            "frac_of_measured_sustained_peak": tf / peaks["bf16_tflops_sustained"],
            "frac_of_nominal_peak": tf / NOMINAL_BF16_TFLOPS,
            "effective_sm_mhz_last_launch": (1e3 * float(lc[0]) / float(lc[1])) if lc[1] > 0 else None,
            "buffer_sets": n_sets, "calls": n_calls, "plan_build_ms": plan_ms,
            "data": "synthetic, N(0,1) drawn on the device"}


def run_schedule57(hb, torch, wl, stream, steps):
    """The full per-step layer schedule (Sec. 3.4 with the per-layer offsets of Sec. 3.2): one entry
    permute of Q, K, V, 57 attention layers whose offsets are (layer * tile / 4) mod HW, the last of
    which writes its output in the original order."""
    from paper_2509_26538_b200.inputs import SCHEDULE_LAYERS, schedule_offset
    n_sets = max(4, n_buffer_sets(wl, 3))
    qd, kd, vd = device_qkv(torch, wl)                       # original order
    qp, kp, vp, op, od = (torch.empty_like(qd) for _ in range(5))
    layer_sets = [device_qkv(torch, wl, 31 * (i + 1)) for i in range(n_sets)]   # the layers' own activations
    offs = [schedule_offset(layer, wl.tile, wl.HW) for layer in range(SCHEDULE_LAYERS)]
    # only offset mod tile changes the mask: the 57 layers share a few plans
    offs = [o % wl.tile for o in offs]
    plans = {}
    for o in sorted(set(offs)):
        plans[o] = hb.Plan(wl.H, wl.W, wl.tile, o, wl.shared_region, wl.n_text)
        plans[o].bind_like(qp)
    any_plan = plans[offs[0]]
    sched_flops = sum(4.0 * wl.head_dim * wl.heads * wl.batch * int(plans[o].export(hb.EXPORT_NNZ)[0]) for o in offs)

    def sched_step():
        # the physical layout does not depend on the offset: one permute serves all layers
        any_plan.permute(qd, qp)
        any_plan.permute(kd, kp)
        any_plan.permute(vd, vp)
        plans[offs[0]].forward(qp, kp, vp, op)
        for li, o in enumerate(offs[1:-1]):
            lq, lk, lv = layer_sets[li % n_sets]
            plans[o].forward(lq, lk, lv, op)
        plans[offs[-1]].forward_unpermute(qp, kp, vp, od)

    l0 = hb.launch_count()
    sched_step()
    per_step_launches = hb.launch_count() - l0
    for _ in range(2):
        sched_step()
    torch.cuda.synchronize()
    time.sleep(COOL_DOWN_S)
    reps = max(3, min(steps, 10))
    s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    s0.record(stream)
    for _ in range(reps):
        sched_step()
    s1.record(stream)
    torch.cuda.synchronize()
    sched_ms = s0.elapsed_time(s1) / reps
    for p_ in plans.values():
        assert p_.status() == 0, "device-side wait timed out"
        p_.destroy()
    assert torch.isfinite(od.float()).all()
    return {"workload": "%s: %dx%d + %d text, %d heads x %d, tile %d, shared %d" % (
                wl.name, wl.H, wl.W, wl.n_text, wl.heads, wl.head_dim, wl.tile, wl.shared_region),
            "layers": SCHEDULE_LAYERS, "distinct_plans": len(plans), "ms_per_step": sched_ms,
            "ms_per_layer": sched_ms / SCHEDULE_LAYERS, "useful_tflops": sched_flops / (sched_ms * 1e-3) / 1e12,
            "useful_gflop_per_step": sched_flops / 1e9, "launches_per_step": int(per_step_launches),
            "offsets": "(layer * tile / 4) mod HW", "reps": reps,
            "note": "timed: permute(Q), permute(K), permute(V) + 57 forward launches (the last with the exit unpermute "
                    "fused into its epilogue); the middle layers rotate through %d sets of Q/K/V buffers so that no "
                    "layer finds its inputs in L2" % n_sets}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="flux2048")
    ap.add_argument("--tile", type=int, default=0)
    ap.add_argument("--groups", type=int, default=0,
                    help="use the Appendix-A tiling with this many equal groups over the non-shared tokens "
                         "(the paper's Table 1 settings: --groups 4|16 --shared 16 at 1024^2, 32 at 2048^2)")
    ap.add_argument("--shared", type=int, default=-1, help="override the side of the central shared region")
    ap.add_argument("--head-dim", type=int, default=0, help="override the head dim (bf16: 128 or 64)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-context", action="store_true", help="skip the dense / SDPA context rows")
    ap.add_argument("--no-backward", action="store_true", help="skip the backward-pass row")
    ap.add_argument("--no-fp8", action="store_true", help="skip the e4m3-operand forward row")
    ap.add_argument("--schedule", action="store_true",
                    help="time the 57-layer per-step schedule (one permute, 57 forwards with the per-layer "
                         "offsets, one unpermute) on the chosen workload's shape instead of the 1024^2 one")
    ap.add_argument("--no-configs", action="store_true",
                    help="skip the rows for the other workload sizes (1024^2 tile sweep, 4096^2) and the 57-layer schedule")
    ap.add_argument("--no-sustained", action="store_true", help="skip the 2-second back-to-back row")
    ap.add_argument("--shard", default="replicas", choices=["replicas", "heads"],
                    help="N > 1: 'replicas' = one independent batch per GPU (weak scaling); 'heads' = one batch whose "
                         "(batch, head) units are split across the GPUs (strong scaling); no collective either way")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # started as a plain process: become N ranks (one per GPU) of a single-node job
        import socket
        with socket.socket() as sk:
            sk.bind(("127.0.0.1", 0))
            port = sk.getsockname()[1]
        os.execvp(sys.executable, [sys.executable, "-m", "torch.distributed.run", "--nnodes=1",
                                   f"--nproc-per-node={args.gpus}", "--master-addr", "127.0.0.1",
                                   "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:])

    from paper_2509_26538_b200.inputs import WORKLOADS, make_qkv
    wl = WORKLOADS[args.workload]
    if args.tile:
        wl = wl.with_(tile=args.tile, layer_offset=args.tile // 2)
    if args.shared >= 0:
        wl = wl.with_(shared_region=args.shared)
    if args.head_dim:
        wl = wl.with_(head_dim=args.head_dim)
    if args.groups:
        if args.impl == "reference" or args.schedule:
            raise SystemExit("--groups is a timing-only option of the CUDA arm")
        size = (wl.HW - wl.shared_region ** 2) // args.groups
        wl = wl.with_(tile=size, layer_offset=size // 2, name=wl.name + f"-groups{args.groups}")

    if args.impl == "reference":
        run_reference(args, wl)
        return

    import torch
    import torch.distributed as dist

    from paper_2509_26538_b200 import binding as hb
    from paper_2509_26538_b200 import build as _build

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    distributed = world > 1
    if distributed:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    if rank == 0:
        _build.build_library()
    if distributed:
        dist.barrier()

    peaks = load_peaks()
    # ---- inputs: seeded, resident in HBM.  replicas: one independent batch per rank; heads: every rank
    # takes its contiguous slice of the (batch, head) units of ONE batch (no data is exchanged)
    shard_heads = distributed and args.shard == "heads"
    if shard_heads:
        from paper_2509_26538_b200.sharding import unit_slice
        if wl.batch != 1:
            raise SystemExit("--shard heads expects batch 1")
        h0, h1 = unit_slice(wl.heads, world, rank)
        q, k, v = (t[:, h0:h1].contiguous() for t in make_qkv(wl))
        full_heads = wl.heads
        wl = wl.with_(heads=h1 - h0)
    else:
        q, k, v = make_qkv(wl.with_(seed=wl.seed + 100 * rank))
        full_heads = wl.heads * (world if distributed else 1)
    qd, kd, vd = (t.cuda() for t in (q, k, v))
    qp, kp, vp, op, od = (torch.empty_like(qd) for _ in range(5))
    # Workloads whose tensors fit in L2 (126 MB) rotate through several copies of the step's
    # buffers, so that no step finds its inputs cached by the previous one.
    step_bytes = 7 * qd.numel() * qd.element_size()      # q, k, v, their permuted copies, out
    n_sets = 1 if step_bytes >= 2 * L2_BYTES else min(8, -(-3 * L2_BYTES // step_bytes))
    sets = [(qd, kd, vd, qp, kp, vp, od)]
    for _ in range(n_sets - 1):
        sets.append(tuple(t.clone() for t in sets[0]))

    t0 = time.perf_counter()
    plan = hb.Plan(wl.H, wl.W, wl.tile, wl.layer_offset, wl.shared_region, wl.n_text, groups=args.groups)
    plan.bind_like(qp)
    torch.cuda.synchronize()
    plan_ms = 1e3 * (time.perf_counter() - t0)
    nnz = int(plan.export(hb.EXPORT_NNZ)[0])
    flops = 4.0 * wl.head_dim * wl.heads * wl.batch * nnz
    tensor_bytes = qd.numel() * qd.element_size()

    stream = torch.cuda.current_stream()

    def step(ev=None, i=0):
        a_q, a_k, a_v, a_qp, a_kp, a_vp, a_o = sets[i % n_sets]
        if ev:
            ev[0].record(stream)
        plan.permute(a_q, a_qp)
        plan.permute(a_k, a_kp)
        plan.permute(a_v, a_vp)
        if ev:
            ev[1].record(stream)
        plan.forward_unpermute(a_qp, a_kp, a_vp, a_o)   # exit gather fused into the epilogue
        if ev:
            ev[2].record(stream)

    for i in range(args.warmup):
        step(None, i)
    torch.cuda.synchronize()
    assert plan.status() == 0, "device-side wait timed out"

    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler = ClockSampler(local)
    if distributed:
        dist.barrier()
    torch.cuda.synchronize()
    launches0 = hb.launch_count()
    sampler.start()
    t_region0 = time.perf_counter()
    start.record(stream)
    for i in range(args.steps):
        step(evs[i], args.warmup + i)
    stop.record(stream)
    torch.cuda.synchronize()
    t_region1 = time.perf_counter()
    launches = hb.launch_count() - launches0
    # SM cycles / nanoseconds the first CTA of the last timed forward launch was resident: the
    # clock the kernel really ran at (NVML samples are too coarse for a region of a few milliseconds)
    lc = plan.export(hb.EXPORT_LAUNCH_CLOCK)
    kernel_clock = {"sm_cycles": int(lc[0]), "ns": int(lc[1]),
                    "effective_sm_mhz": (1e3 * float(lc[0]) / float(lc[1])) if lc[1] > 0 else None}
    # The timed region is short; the same steps go on, untimed, until the sampler has seen at
    # least 0.3 s of this load, so that the clock record has enough samples to mean something.
    i_extra = 0
    while time.perf_counter() - t_region0 < 0.3:
        step(None, args.warmup + args.steps + i_extra)
        i_extra += 1
        if i_extra % 8 == 0:
            torch.cuda.synchronize()
    torch.cuda.synchronize()
    if distributed:
        dist.barrier()
    clocks = sampler.stop(window=(t_region0, t_region1))
    clocks["kernel"] = kernel_clock
    clocks["note"] = ("NVML polled every ms while the timed steps and %d further untimed repeats of the same step ran "
                      "(>= 0.3 s of load); kernel = SM cycles / ns of one forward launch, read from the kernel" % i_extra)
    total_ms = start.elapsed_time(stop)
    if distributed:
        t = torch.tensor([total_ms], device="cuda")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        total_ms = float(t.item())
    ms_per_step = total_ms / args.steps
    fwd_ms = [e[1].elapsed_time(e[2]) for e in evs]
    perm_ms = [e[0].elapsed_time(e[1]) for e in evs]
    # the standalone exit gather is not part of the step any more; time it on its own
    plan.forward(qp, kp, vp, op)
    ue = [torch.cuda.Event(enable_timing=True) for _ in range(11)]
    plan.unpermute(op, od)
    for i in range(10):
        ue[i].record(stream)
        plan.unpermute(op, od)
    ue[10].record(stream)
    torch.cuda.synchronize()
    unperm_ms = [ue[i].elapsed_time(ue[i + 1]) for i in range(10)]
    fwd_avg = statistics.mean(fwd_ms)
    # whole-job work: replicas = one batch per rank, heads = one batch split over the ranks
    total_flops = 4.0 * wl.head_dim * full_heads * wl.batch * nnz
    value = total_flops / (ms_per_step * 1e-3) / 1e12
    attn_tflops = flops / (fwd_avg * 1e-3) / 1e12

    # ---- end to end through the host-buffer entry point (pinned host memory)
    e2e = None
    if not args.no_e2e:
        qh, kh, vh = (t.pin_memory() for t in (q, k, v))
        oh = torch.empty_like(qh).pin_memory()
        plan.forward_host(qh, kh, vh, oh)  # allocates the workspace, warms up
        n_e2e = max(1, min(args.steps, 5))
        if distributed:
            dist.barrier()
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(n_e2e):
            plan.forward_host(qh, kh, vh, oh)
        e1.record(stream)
        torch.cuda.synchronize()
        e2e_ms = e0.elapsed_time(e1) / n_e2e
        if distributed:
            t = torch.tensor([e2e_ms], device="cuda")
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            e2e_ms = float(t.item())
        e2e = {"value": total_flops / (e2e_ms * 1e-3) / 1e12, "unit": "TFLOP/s", "ms_per_step": e2e_ms,
               "h2d_bytes_per_step": 3 * tensor_bytes, "d2h_bytes_per_step": tensor_bytes,
               "api": "hilberta_forward_host (pinned host buffers; per slice of heads: H2D, one launch with entry and exit gathers fused in, D2H; the slices are pipelined over two copy streams)",
               "steps": n_e2e}
        assert torch.isfinite(oh.float()).all()

    # ---- context rows (not part of the metric): dense attention of this build and PyTorch SDPA
    context_rows = None
    if world == 1 and not args.no_context:
        def timed(fn, n=5):
            fn()
            torch.cuda.synchronize()
            a, b_ = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            for _ in range(n):
                fn()
            b_.record(stream)
            torch.cuda.synchronize()
            return a.elapsed_time(b_) / n
        dense_flops = 4.0 * wl.head_dim * wl.heads * wl.batch * wl.S * wl.S
        context_rows = {"dense_gflop": dense_flops / 1e9}
        try:
            n_pad = 1
            while n_pad < max(wl.H, wl.W):
                n_pad *= 2
            dense = hb.Plan(wl.H, wl.W, n_pad * n_pad, 0, 0, wl.n_text)   # one tile, no shared region: every pair kept
            dense.bind_like(qp)
            ms = timed(lambda: dense.forward(qp, kp, vp, op))
            assert dense.status() == 0
            dense.destroy()
            context_rows["dense_this_build"] = {"ms": ms, "tflops": dense_flops / (ms * 1e-3) / 1e12}
        except Exception as e:  # context only
            context_rows["dense_this_build"] = {"error": str(e)[:120]}
        try:
            ms = timed(lambda: torch.nn.functional.scaled_dot_product_attention(qp, kp, vp))
            context_rows["torch_sdpa_dense_bf16"] = {"ms": ms, "tflops": dense_flops / (ms * 1e-3) / 1e12}
        except Exception as e:
            context_rows["torch_sdpa_dense_bf16"] = {"error": str(e)[:120]}
        context_rows["sparse_speedup_vs_dense_this_build"] = (
            context_rows["dense_this_build"]["ms"] / fwd_avg if "ms" in context_rows["dense_this_build"] else None)

    # ---- the whole step as ONE launch: entry and exit gathers fused into the attention kernel
    fused = None
    if world == 1:
        of = torch.empty_like(qd)
        time.sleep(COOL_DOWN_S)
        for _ in range(3):
            plan.forward_fused(qd, kd, vd, of, True, True)
        torch.cuda.synchronize()
        n_f = max(5, min(args.steps, 30))
        fev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n_f)]
        for i, (a, b_) in enumerate(fev):
            f_q, f_k, f_v = sets[i % n_sets][0:3]
            a.record(stream)
            plan.forward_fused(f_q, f_k, f_v, of, True, True)
            b_.record(stream)
        torch.cuda.synchronize()
        assert plan.status() == 0, "device-side wait timed out"
        view = torch.int16 if wl.dtype == "bf16" else torch.int32
        assert torch.equal(of.view(view), od.view(view)), "fused step differs from permute + forward + unpermute"
        fms = sorted(a.elapsed_time(b_) for a, b_ in fev)
        f_med = fms[len(fms) // 2]
        lcf = plan.export(hb.EXPORT_LAUNCH_CLOCK)
        fused = {"ms_per_step_median": f_med, "ms_per_step_min": fms[0],
                 "effective_sm_mhz_last_launch": (1e3 * float(lcf[0]) / float(lcf[1])) if lcf[1] > 0 else None,
                 "useful_tflops": flops / (f_med * 1e-3) / 1e12,
                 "api": "hilberta_forward_fused(in_original=1, out_original=1): q, k, v and out in ORIGINAL order, "
                        "one launch, no permuted copies; bit-identical to the step above"}
        del of

    # ---- backward pass (not part of the metric): dq, dk, dv on the same plan and inputs
    backward = None
    if world == 1 and not args.no_backward and wl.dtype == "bf16":
        lse = torch.empty((wl.batch, wl.heads, wl.S), device="cuda", dtype=torch.float32)
        g = torch.Generator().manual_seed(wl.seed + 7)
        dop = torch.randn(qp.shape, generator=g).to(torch.bfloat16).cuda()
        grads = [torch.empty_like(qp) for _ in range(3)]
        time.sleep(COOL_DOWN_S)
        plan.forward_lse(qp, kp, vp, op, lse)
        for _ in range(3):
            plan.backward(dop, qp, kp, vp, op, lse, *grads)
        torch.cuda.synchronize()
        n_b = max(5, min(args.steps, 30))
        bev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n_b)]
        l0 = hb.launch_count()
        for a, b_ in bev:
            a.record(stream)
            plan.backward(dop, qp, kp, vp, op, lse, *grads)
            b_.record(stream)
        torch.cuda.synchronize()
        assert plan.status() == 0, "device-side wait timed out"
        assert all(torch.isfinite(t.float()).all() for t in grads)
        bms = sorted(a.elapsed_time(b_) for a, b_ in bev)
        b_med = bms[len(bms) // 2]
        bflops = 2.5 * flops          # five contractions of 2 D flops per kept pair
        backward = {
            "ms_per_call_median": b_med, "ms_per_call_min": bms[0],
            "useful_tflops": bflops / (b_med * 1e-3) / 1e12,
            "useful_gflop_per_call": bflops / 1e9,
            "executed_tflops": 1.4 * bflops / (b_med * 1e-3) / 1e12,
            "frac_of_measured_burst_peak": bflops / (b_med * 1e-3) / 1e12 / peaks["bf16_tflops"],
            "launches_per_call": (hb.launch_count() - l0) // n_b,
            "note": "useful = 10 D flops per kept pair (dS, dQ, dK, dV and the recomputed scores); executed = 14 D: "
                    "the dQ and the dK/dV kernels each recompute the scores and dP",
        }
        del dop, grads, lse

    # ---- the same forward with e4m3 operands (not part of the metric): q, k, v rounded to 8-bit floats
    fp8 = None
    if world == 1 and not args.no_fp8 and wl.dtype == "bf16" and wl.head_dim == 128 and not args.groups:
        f8 = torch.float8_e4m3fn
        f_sets = [tuple(t.to(f8) for t in s_[3:6]) for s_ in sets]
        plan8 = hb.Plan(wl.H, wl.W, wl.tile, wl.layer_offset, wl.shared_region, wl.n_text)
        plan8.bind_like(f_sets[0][0])
        o8 = torch.empty_like(op)
        time.sleep(COOL_DOWN_S)
        for i in range(3):
            plan8.forward(*f_sets[i % n_sets], o8)
        torch.cuda.synchronize()
        n_8 = max(5, min(args.steps, 30))
        fev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n_8)]
        for i, (a, b_) in enumerate(fev):
            a.record(stream)
            plan8.forward(*f_sets[i % n_sets], o8)
            b_.record(stream)
        torch.cuda.synchronize()
        assert plan8.status() == 0, "device-side wait timed out"
        assert torch.isfinite(o8.float()).all()
        ms8 = sorted(a.elapsed_time(b_) for a, b_ in fev)
        m8 = ms8[len(ms8) // 2]
        lc8 = plan8.export(hb.EXPORT_LAUNCH_CLOCK)
        fp8 = {"ms_per_call_median": m8, "ms_per_call_min": ms8[0], "useful_tflops": flops / (m8 * 1e-3) / 1e12,
               "effective_sm_mhz_last_launch": (1e3 * float(lc8[0]) / float(lc8[1])) if lc8[1] > 0 else None,
               "speedup_vs_bf16_forward": statistics.median(fwd_ms) / m8,
               "note": "q, k, v and the softmax weights in e4m3 (kind::f8f6f4 MMAs), fp32 softmax and accumulation, "
                       "bf16 output; tolerance rel-L2 4e-2 (weights have three mantissa bits)"}
        plan8.destroy()
        del f_sets, o8

    # ---- sustained: forward launches back to back for >= 2 s, with their own clock record (after the
    # short rows: it runs the GPU into its power cap, and the clock takes seconds to recover)
    sustained = None
    if world == 1 and not args.no_sustained:
        smp = ClockSampler(local)
        n_s = max(50, int(2.2e3 / max(fwd_avg, 1e-3)))
        s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        smp.start()
        s0.record(stream)
        for i in range(n_s):
            a_qp, a_kp, a_vp = sets[i % n_sets][3:6]
            plan.forward(a_qp, a_kp, a_vp, op)
        s1.record(stream)
        torch.cuda.synchronize()
        s_clk = smp.stop()
        s_ms = s0.elapsed_time(s1) / n_s
        lc = plan.export(hb.EXPORT_LAUNCH_CLOCK)
        s_tf = flops / (s_ms * 1e-3) / 1e12
        sustained = {"launches": n_s, "seconds": s0.elapsed_time(s1) * 1e-3, "ms_per_call": s_ms, "useful_tflops": s_tf,
                     "frac_of_measured_sustained_peak": s_tf / peaks["bf16_tflops_sustained"],
                     "frac_of_measured_burst_peak": s_tf / peaks["bf16_tflops"],
                     "clocks": s_clk,
                     "effective_sm_mhz_last_launch": (1e3 * float(lc[0]) / float(lc[1])) if lc[1] > 0 else None}
    # free the main workload's extra buffers before the other sizes are measured
    del sets[1:]
    torch.cuda.empty_cache()

    schedule = None
    if world == 1 and (args.schedule or not args.no_configs):
        schedule = run_schedule57(hb, torch, wl if args.schedule else WORKLOADS["flux1024"], stream, args.steps)

    configs = None
    if world == 1 and not args.no_configs and not args.groups:
        configs = {}
        for name, tiles in (("flux1024", (256, 512, 1024)), ("flux4096", (2048,))):
            for tile in tiles:
                c_wl = WORKLOADS[name].with_(tile=tile, layer_offset=tile // 2)
                configs["%s_tile%d" % (name, tile)] = time_forward_config(hb, torch, c_wl, peaks, stream)

    if rank != 0:
        if distributed:
            dist.destroy_process_group()
        return

    peak = peaks["bf16_tflops"]
    line = {
        "metric": "sparse-attn useful TFLOP/s at %s (Flux shape)" % {"flux1024": "1024^2", "flux2048": "2048^2",
                                                                      "flux4096": "4096^2"}.get(wl.name, wl.name),
        "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step,
        "higher_is_better": True, "scaling": "strong" if shard_heads else "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic", "config": workload_config(wl, world, "heads" if shard_heads else "replicas"),
        "attn_ms_per_call": fwd_avg, "attn_ms_per_call_median": statistics.median(fwd_ms),
        "attn_ms_per_call_min": min(fwd_ms), "attn_useful_tflops": attn_tflops,
        "pct_of_nominal_bf16_peak": 100.0 * attn_tflops / NOMINAL_BF16_TFLOPS,
        "pct_of_measured_burst_peak": 100.0 * attn_tflops / peaks["bf16_tflops"],
        "pct_of_measured_sustained_peak": 100.0 * attn_tflops / peaks["bf16_tflops_sustained"],
        "nnz": nnz, "useful_gflop_per_call": flops / 1e9, "plan_build_ms": plan_ms,
        "permute": {"ms_3_gathers": statistics.mean(perm_ms), "ms_unpermute": statistics.mean(unperm_ms),
                    "gbs_permute": 3 * 2 * tensor_bytes / (statistics.mean(perm_ms) * 1e-3) / 1e9,
                    "gbs_unpermute": 2 * tensor_bytes / (statistics.mean(unperm_ms) * 1e-3) / 1e9,
                    "peak_gbs": peaks["hbm_gbs"], "peak_source": peaks["source"]},
        "roofline": {"kernel": "attn_bf16_kernel", "bound": "tensor", "achieved": attn_tflops, "peak": peak,
                     "unit": "TFLOP/s", "frac": attn_tflops / peak, "peak_source": peaks["source"] + " burst",
                     "frac_of_sustained": attn_tflops / peaks["bf16_tflops_sustained"],
                     "traffic": FORWARD_DRAM_TRAFFIC_BYTES.get(wl.name)},
        "clocks": clocks, "gpu_launches": int(launches), "e2e": e2e, "sustained": sustained, "fused_step": fused, "backward": backward, "fp8_forward": fp8, "schedule57": schedule, "configs": configs,
        "context": {"paper": "A100, Triton kernel vs FlashAttention-2: 2.3x at 1024^2, 4.17x at 2048^2 "
                             "(4.36 ms per call at 2048^2, 16 tiles)", "same_gpu": context_rows},
    }
    if not args.no_cpu_baseline and world == 1 and not args.groups:
        tf, threads, desc, dt = oracle_sample(wl, 15.0)
        line["cpu_baseline"] = {"value": tf, "unit": "TFLOP/s", "cores": threads, "kind": "oracle",
                                "sample": desc, "seconds": dt}
    print(json.dumps(line), flush=True)
    plan.destroy()
    if distributed:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
