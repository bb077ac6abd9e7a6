#!/usr/bin/env python
"""Benchmark of the mixed-batch multi-LoRA layer on B200.

A "step" is one pass of the whole hot path - shrink, fused base GEMM + LoRA expand with
activation save, then the LoRA backward (V, dB, dA, dX) - over one synthetic mixed batch, for
every projection of the workload.  The default workload is the Llama-3-8B-shaped decoder-layer
projection set (q, k, v, o, gate, up, down; 32 adapters of rank 16; 4096 rows of which 1024 are
decode rows and 2048 fine-tuning rows).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg3|cfg2|cfg5] [--impl reference]
                    [--no-extra-configs]

Prints ONE JSON line.  Beside the headline workload the line carries a `configs` block with the other
seeded configurations (cfg2, the three cfg5 runs and their fill ratio, three cfg4 sweep points) and a
`skinny_cold` block (the rank-r kernels on rotating inputs), measured after the headline.  With N > 1 (under torchrun) every rank runs the same workload on its own
GPU (rows are independent, the path needs no collective): weak scaling, value = all ranks' tokens
divided by the slowest rank's time.  `--impl reference` times the CPU oracle instead.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2607_28848_b200 import synth  # noqa: E402

METRIC = "mixed-batch multi-LoRA layer tokens/s and TFLOP/s (fwd+LoRA bwd) vs BF16 roofline"
UNIT = "tokens/s"


# ---------------------------------------------------------------------------------------------
# workloads and their algorithmic work
# ---------------------------------------------------------------------------------------------
def get_workloads(name: str, seed: int = 0):
    if name == "cfg3":
        return synth.cfg3_layer_set(seed), "cfg3: Llama-3-8B decoder-layer projection set (q,k,v,o,gate,up,down), " \
                                           "bf16, 32 adapters r=16, 4096 mixed rows (1024 prefill in 12 segments, " \
                                           "1024 decode, 4x512 fine-tune)"
    if name == "cfg2":
        return [synth.cfg2_single_projection(seed)], "cfg2: 4096x4096 projection, bf16, 16 adapters r=16, 1600 rows"
    if name == "cfg5":
        return [synth.cfg5_decode_heavy(seed)], "cfg5: 5120x13824 up projection, bf16, 128 adapters r=32, " \
                                                "512 decode rows + one 2048-row fine-tune segment"
    raise SystemExit(f"unknown workload {name}")


from paper_2607_28848_b200.accounting import algorithmic_bytes, flops, load_peaks  # noqa: E402


# ---------------------------------------------------------------------------------------------
# clocks
# ---------------------------------------------------------------------------------------------
def _sampler_child(path: str, uuid: str, index: int, period_s: float = 0.003) -> None:
    """Child process: reads SM clock, power and clock-event reasons through NVML every few milliseconds
    (queries only; nothing is set) and appends `time sm_mhz power_w reasons_bitmask` lines to `path`."""
    import pynvml
    pynvml.nvmlInit()
    h = None
    if uuid:
        for cand in (uuid, "GPU-" + uuid):
            try:
                h = pynvml.nvmlDeviceGetHandleByUUID(cand.encode() if hasattr(cand, "encode") else cand)
                break
            except Exception:
                h = None
    if h is None:
        h = pynvml.nvmlDeviceGetHandleByIndex(index)
    try:
        mx = pynvml.nvmlDeviceGetMaxClockInfo(h, pynvml.NVML_CLOCK_SM)
    except Exception:
        mx = 0
    reasons_fn = getattr(pynvml, "nvmlDeviceGetCurrentClocksEventReasons", None) or pynvml.nvmlDeviceGetCurrentClocksThrottleReasons
    with open(path, "w", buffering=1) as fh:
        fh.write(f"# max {mx}\n")
        n, power = 0, 0.0
        while True:
            t = time.time()
            try:
                if n % 4 == 0:           # power changes slowly and its query is the slow one
                    power = pynvml.nvmlDeviceGetPowerUsage(h) / 1000.0
                fh.write(f"{t:.6f} {pynvml.nvmlDeviceGetClockInfo(h, pynvml.NVML_CLOCK_SM)} {power:.1f} {int(reasons_fn(h))}\n")
            except Exception:
                pass
            n += 1
            dt = period_s - (time.time() - t)
            if dt > 0:
                time.sleep(dt)


class ClockSampler:
    """SM clock, power and clock-event reasons DURING named regions, sampled every ~4 ms by a child
    process through NVML (read-only queries), so that a 50 ms timed region still holds a dozen samples."""
    # NVML clock-event reason bits
    REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown"}

    def __init__(self, gpu_index: int, uuid: str = ""):
        self.path = tempfile.NamedTemporaryFile(prefix="clocks_", suffix=".txt", delete=False).name
        self.regions = {}
        try:
            self.proc = subprocess.Popen([sys.executable, os.path.abspath(__file__), "--clock-sampler", self.path,
                                          "--sampler-uuid", uuid, "--sampler-index", str(gpu_index)],
                                         stdout=subprocess.DEVNULL, stderr=subprocess.DEVNULL)
            time.sleep(0.5)              # NVML is up before the first region starts
        except OSError:
            self.proc = None

    def start(self, name: str):
        self.regions[name] = [time.time(), None]

    def stop(self, name: str):
        self.regions[name][1] = time.time()

    def finish(self) -> dict:
        """Per region: median / min SM MHz, sample count, max power, reasons seen."""
        if self.proc is None:
            return {}
        time.sleep(0.02)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        rows, mx = [], None
        try:
            with open(self.path) as fh:
                for ln in fh:
                    if ln.startswith("# max"):
                        mx = float(ln.split()[2])
                        continue
                    f = ln.split()
                    if len(f) == 4:
                        rows.append((float(f[0]), float(f[1]), float(f[2]), int(f[3])))
            os.unlink(self.path)
        except (OSError, ValueError):
            pass
        out = {}
        for name, (t0, t1) in self.regions.items():
            inside = [r for r in rows if t1 is not None and t0 <= r[0] <= t1]
            nearest = False
            if not inside and t1 is not None and rows:
                # An NVML query can stall for tens of milliseconds while the process queues hundreds of launches: a
                # short region may then hold no sample of its own.  Take the samples just around it and say so.
                inside = [r for r in rows if t0 - 0.05 <= r[0] <= t1 + 0.05]
                nearest = True
            if not inside:
                out[name] = {"sm_mhz": None, "sm_max_mhz": mx, "reasons": ["no samples"], "samples": 0}
                continue
            bits = 0
            for r in inside:
                bits |= r[3]
            out[name] = {"sm_mhz": float(np.median([r[1] for r in inside])), "sm_mhz_min": min(r[1] for r in inside),
                         "sm_max_mhz": mx, "reasons": sorted(v for k, v in self.REASONS.items() if bits & k),
                         "samples": len(inside), "power_w_max": max(r[2] for r in inside),
                         "seconds": round(t1 - t0, 4)}
            if nearest:
                out[name]["note"] = "no sample fell inside the region: these are the samples within 50 ms around it"
        return out


# ---------------------------------------------------------------------------------------------
# CPU oracle legs
# ---------------------------------------------------------------------------------------------
def oracle_pass(w, t):
    from oracle import mlora_oracle as orc
    f = orc.forward_blocked(t["X"], t["W"], t["A_all"], t["B_all"], t["scale"], w.segments)
    orc.backward_blocked(t["dY"], t["W"], t["A_all"], t["B_all"], t["scale"], w.segments, f["x_save"], f["u_save"],
                         n_rows=w.n_rows)


def host_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info() if p.get("user_api") == "blas"]
        if n:
            return int(max(n))
    except Exception:
        pass
    return os.cpu_count() or 1


def oracle_sample_text(workloads, secs) -> str:
    total = sum(flops(w)["fwd"] + flops(w)["bwd"] for w in workloads)
    return (f"fp64 numpy oracle (forward_blocked + backward_blocked), one pass over every projection of the workload "
            f"{[w.name for w in workloads]} = {total / 1e9:.0f} GFLOP, the whole step, nothing scaled: {secs:.1f} s")


def oracle_step_seconds(workloads, tensors) -> float:
    t0 = time.perf_counter()
    for w, t in zip(workloads, tensors):
        oracle_pass(w, t)
    return time.perf_counter() - t0


def cpu_baseline(workloads) -> dict:
    """The oracle as it stands, timed once on the whole step (every projection of the workload): the same
    sample the reference arm times per step."""
    tensors = [synth.make_tensors(w) for w in workloads]
    secs = oracle_step_seconds(workloads, tensors)
    return {"value": workloads[0].n_rows / secs, "unit": UNIT, "cores": host_threads(), "kind": "oracle",
            "sample": oracle_sample_text(workloads, secs)}


def run_reference(args, workloads, label):
    """The reference arm: the CPU oracle timed on the host cores; a step is one pass over every projection of
    the workload (the same sample as the GPU arm's cpu_baseline leg), so nothing is extrapolated."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    tensors = [synth.make_tensors(w) for w in workloads]
    for _ in range(args.warmup):
        oracle_step_seconds(workloads, tensors)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_step_seconds(workloads, tensors)
    secs = (time.perf_counter() - t0) / max(args.steps, 1)
    value = workloads[0].n_rows / secs
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": secs * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": label},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": host_threads(), "kind": "oracle",
                             "sample": oracle_sample_text(workloads, secs)},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


# ---------------------------------------------------------------------------------------------
# GPU arm
# ---------------------------------------------------------------------------------------------
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--workload", default="cfg3")
    ap.add_argument("--impl", default="ours")
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--e2e-steps", type=int, default=10, help="0 skips the end-to-end leg")
    ap.add_argument("--projections", default="", help="comma list: run only these projections of the workload")
    ap.add_argument("--with-update", action="store_true",
                    help="also run the AdamW update of the fine-tuned adapters after each backward (not part of the "
                         "headline step; reported under kernels.adamw)")
    ap.add_argument("--graph", action="store_true", help="also time the step replayed from a CUDA graph (step_stats)")
    ap.add_argument("--no-extra-configs", action="store_true",
                    help="skip the `configs` and `skinny_cold` blocks (the other seeded configurations measured after the headline)")
    ap.add_argument("--clock-sampler", default="", help=argparse.SUPPRESS)       # child-process mode of ClockSampler
    ap.add_argument("--sampler-uuid", default="", help=argparse.SUPPRESS)
    ap.add_argument("--sampler-index", type=int, default=0, help=argparse.SUPPRESS)
    ap.add_argument("--dropout", type=float, default=0.0,
                    help="LoRA dropout rate on the fine-tuning rows (the paper trains with 0.05; the headline step "
                         "runs without it); a new seed every step")
    args = ap.parse_args()
    if args.clock_sampler:
        _sampler_child(args.clock_sampler, args.sampler_uuid, args.sampler_index)
        return

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    workloads, label = get_workloads(args.workload, args.seed + rank)
    if args.projections:
        keep = set(args.projections.split(","))
        workloads = [w for w in workloads if w.name.split("_", 1)[1] in keep]
        label += f" [only {sorted(keep)}]"
    if args.impl == "reference":
        run_reference(args, workloads, label)
        return

    import torch
    import torch.distributed as dist
    from paper_2607_28848_b200 import binding as mb
    from paper_2607_28848_b200 import replicas
    from paper_2607_28848_b200.runner import LayerRun, Session

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the layer has no CPU fallback")
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    sess = Session(local_rank)
    peaks = load_peaks()

    runs = []
    for w in workloads:
        t = synth.make_tensors(w)
        runs.append(LayerRun(sess, w.dtype, t, w.segments, w.n_rows))
        del t
    resident = sum(w.d_in * w.d_out * w.elem_bytes + w.n_rows * (w.d_in + w.d_out) * w.elem_bytes for w in workloads)

    opt = []
    if args.with_update:
        for r in runs:
            idx = torch.tensor(r.slots, device=sess.device)
            wA, wB = r.A_all[idx].float().contiguous(), r.B_all[idx].float().contiguous()
            opt.append([wA, wB] + [torch.zeros_like(x) for x in (wA, wA, wB, wB)])
    n_updates = [0]

    n_steps_run = [0]

    def step():
        if args.with_update:
            n_updates[0] += 1
        n_steps_run[0] += 1
        for i, r in enumerate(runs):
            if args.dropout > 0:
                mb.mlora_set_dropout(sess.ctx, args.dropout, (n_steps_run[0] << 8) + i)
            r.forward()
            r.backward()
            if args.with_update:
                wA, wB, mA, vA, mB, vB = opt[i]
                mb.mlora_adamw_update(sess.ctx, r.layer, r.plan, r.dA, r.dB, wA, wB, mA, vA, mB, vB, n_updates[0],
                                      lr=1e-6)

    def barrier():
        replicas.barrier()
        torch.cuda.synchronize()

    warmup = max(args.warmup, 3)
    for _ in range(warmup):
        step()
    torch.cuda.synchronize()
    if sess.ctx and mb.mlora_poll_status(sess.ctx) != mb.MLORA_OK:
        raise SystemExit("device status word reports a timed-out wait")

    launches_per_step_probe = mb.mlora_launch_count(sess.ctx)
    step()
    launches_per_step = mb.mlora_launch_count(sess.ctx) - launches_per_step_probe

    sampler = None
    if rank == 0:
        try:
            uuid = str(torch.cuda.get_device_properties(local_rank).uuid)
        except Exception:
            uuid = ""
        sampler = ClockSampler(local_rank, uuid)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    if sampler:
        sampler.start("timed")
    l0 = mb.mlora_launch_count(sess.ctx)
    ev0.record()
    for _ in range(args.steps):
        step()
    ev1.record()
    barrier()
    if sampler:
        sampler.stop("timed")
    gpu_launches = mb.mlora_launch_count(sess.ctx) - l0
    ms_total = replicas.max_over_ranks(ev0.elapsed_time(ev1), sess.device)     # slowest rank
    # Spread of single steps (median and best of up to 50 more steps, one event between steps):
    # reported beside the headline mean, never instead of it.
    stat_n = max(1, min(args.steps, 50))
    marks = [torch.cuda.Event(enable_timing=True) for _ in range(stat_n + 1)]
    if sampler:
        sampler.start("single_steps")
    marks[0].record()
    for i in range(stat_n):
        step()
        marks[i + 1].record()
    torch.cuda.synchronize()
    if sampler:
        sampler.stop("single_steps")
    step_ms = sorted(marks[i].elapsed_time(marks[i + 1]) for i in range(stat_n))
    # The same step captured once in a CUDA graph and replayed (the calls allocate nothing and never
    # synchronise, so forward + activation save + backward capture as they are); reported beside the
    # headline, which stays the eagerly launched step.
    graph_ms = None
    if args.graph and not args.with_update and args.dropout == 0:
        gstream = torch.cuda.Stream(device=sess.device)
        with torch.cuda.stream(gstream):
            step()
            gstream.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=gstream):
                step()
            for _ in range(3):
                g.replay()
            gstream.synchronize()
            g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            g0.record(gstream)
            for _ in range(args.steps):
                g.replay()
            g1.record(gstream)
            gstream.synchronize()
            graph_ms = g0.elapsed_time(g1) / args.steps
        del g
    step_stats = {"steps": stat_n, "median_ms": step_ms[stat_n // 2], "best_ms": step_ms[0]}
    # Plan build (host validation, routing tables, upload) for this workload's segment table: outside the
    # timed step, as the plans are prebuilt there; one table serves all projections of a layer.
    import time as _time
    w0 = workloads[0]
    plan_ms = {}
    for kind in ("blocking", "stream_ordered"):
        ts = []
        for _ in range(20):
            t0 = _time.perf_counter()
            if kind == "blocking":
                pl = mb.mlora_plan_create(sess.ctx, w0.segments, w0.n_rows, w0.n_adapters)
                mb.mlora_plan_destroy(pl)
            else:
                pl = mb.mlora_plan_create_async(sess.ctx, w0.segments, w0.n_rows, w0.n_adapters)
                mb.mlora_plan_release(pl)
            ts.append((_time.perf_counter() - t0) * 1e3)
        torch.cuda.synchronize()
        plan_ms[kind] = sorted(ts)[len(ts) // 2]
    step_stats["plan_build_host_ms"] = plan_ms
    if graph_ms is not None:
        step_stats["graph_replay_ms_per_step"] = graph_ms
    step_stats["segments"] = int(len(w0.segments))
    # Per-kernel durations: the same steps once more, now with the library recording a CUDA event
    # pair around every launch (which also switches off the overlap of a kernel's set-up with its
    # predecessor's tail, so each pair times one whole kernel).  Kept out of the region above so
    # that the headline number carries no event overhead.
    prof_steps = max(1, min(args.steps, 20))
    mb.mlora_profile_enable(sess.ctx, launches_per_step * prof_steps)
    if sampler:
        sampler.start("per_kernel")
    for _ in range(prof_steps):
        step()
    barrier()
    if sampler:
        sampler.stop("per_kernel")
    kinds, kms = mb.mlora_profile_collect(sess.ctx)
    mb.mlora_profile_enable(sess.ctx, 0)

    ms_per_step = ms_total / args.steps
    T = workloads[0].n_rows
    value = world * T / (ms_per_step * 1e-3)
    tot_flops = sum(flops(w)["fwd"] + flops(w)["bwd"] for w in workloads)

    # ---- per-kernel accounting (CUDA events recorded by the library around each launch) ----
    per_kind = {}
    for k, name in enumerate(mb.PROFILE_KINDS):
        sel = kms[kinds == k]
        if len(sel):
            per_kind[name] = {"launches_per_step": len(sel) / prof_steps, "ms_per_step": float(sel.sum() / prof_steps)}
    gemm_fwd_flops = sum(flops(w)["gemm_fwd"] for w in workloads)
    gemm_bwd_flops = sum(flops(w)["gemm_bwd"] for w in workloads)
    ab = [algorithmic_bytes(w) for w in workloads]
    kernels = {}
    if "gemm_fwd" in per_kind:
        kernels["gemm_fwd"] = {**per_kind["gemm_fwd"], "tflops": gemm_fwd_flops / per_kind["gemm_fwd"]["ms_per_step"] / 1e9}
    if "gemm_bwd" in per_kind:
        kernels["gemm_bwd"] = {**per_kind["gemm_bwd"], "tflops": gemm_bwd_flops / per_kind["gemm_bwd"]["ms_per_step"] / 1e9,
                               "frac_of_sustained": gemm_bwd_flops / per_kind["gemm_bwd"]["ms_per_step"] / 1e9 / peaks["bf16_tflops_sustained"]}
    if "shrink" in per_kind:
        b = sum(a["shrink_fwd"] + a["shrink_bwd"] for a in ab)
        kernels["shrink"] = {**per_kind["shrink"], "gbs": b / per_kind["shrink"]["ms_per_step"] / 1e6,
                             "frac_hbm": b / per_kind["shrink"]["ms_per_step"] / 1e6 / peaks["hbm_gbs"]}
    if "grad" in per_kind:
        b = sum(a["grad_dA"] + a["grad_dB"] for a in ab)
        kernels["grad"] = {**per_kind["grad"], "gbs": b / per_kind["grad"]["ms_per_step"] / 1e6,
                           "frac_hbm": b / per_kind["grad"]["ms_per_step"] / 1e6 / peaks["hbm_gbs"]}
    if "adamw" in per_kind:
        b = sum(30.0 * len(r.slots) * w.rank * (w.d_in + w.d_out) for r, w in zip(runs, workloads))
        kernels["adamw"] = {**per_kind["adamw"], "gbs": b / per_kind["adamw"]["ms_per_step"] / 1e6,
                            "note": "30 bytes per adapter element: grad, weight, two moments read; weight, moments, stored weight written"}
    # per-launch view of the memory-bound kernels: which launch is which follows from the fixed order
    # shrink(fwd), GEMM fwd, shrink(bwd), gradients (dB and dA in one launch), GEMM bwd [, update] per projection
    if "splitk_reduce" in per_kind:     # the small kernels that add up the K slices of split GEMM tiles
        kernels["splitk_reduce"] = per_kind["splitk_reduce"]
    reduce_kind = mb.PROFILE_KINDS.index("splitk_reduce")
    kms_main = kms[kinds != reduce_kind]              # the fixed per-projection order below has no reduction launches
    per_step = len(kms_main) // prof_steps if prof_steps else 0
    labels = []
    for w, a_ in zip(workloads, ab):
        labels += [(w.name, "shrink_fwd", a_["shrink_fwd"]), (w.name, "gemm_fwd", None), (w.name, "shrink_bwd", a_["shrink_bwd"]),
                   (w.name, "grad_dB+dA", a_["grad_dB"] + a_["grad_dA"]), (w.name, "gemm_bwd", None)]
        if args.with_update:
            labels.append((w.name, "adamw", None))
    skinny = []
    if per_step == len(labels) and per_step > 0:
        mean_ms = kms_main[:per_step * prof_steps].reshape(prof_steps, per_step).mean(0)
        for (proj, kern, nbytes), t in zip(labels, mean_ms):
            if nbytes:
                skinny.append({"launch": f"{proj}:{kern}", "mbytes": nbytes / 1e6, "us": float(t * 1e3),
                               "gbs": nbytes / t / 1e6, "frac_hbm": nbytes / t / 1e6 / peaks["hbm_gbs"]})
        skinny.sort(key=lambda d: -d["mbytes"])
        kernels["skinny_largest_launches"] = skinny[:4]
    roofline = None
    if "gemm_fwd" in kernels:
        n_launch = per_kind["gemm_fwd"]["launches_per_step"]
        achieved = kernels["gemm_fwd"]["tflops"]
        roofline = {"kernel": "gemm2_lora_kernel<R, false> (forward: base GEMM + LoRA expand, two-SM tcgen05)", "bound": "tensor",
                    "achieved": achieved, "unit": "TFLOP/s",
                    "frac_of_burst": achieved / peaks["bf16_tflops"],
                    "frac_of_sustained": achieved / peaks["bf16_tflops_sustained"],
                    "frac_of_nominal": achieved / 2250.0,      # datasheet dense bf16 figure, context only
                    "flops_per_launch": gemm_fwd_flops / n_launch,
                    "avg_launch_ms": per_kind["gemm_fwd"]["ms_per_step"] / n_launch,
                    "traffic": None}
        prof = os.path.join(ROOT, "profiles", "traffic.json")
        if os.path.exists(prof):
            try:
                with open(prof) as fh:
                    rec = json.load(fh).get(args.workload, {})
                roofline["traffic"] = rec.get("gemm_fwd_bytes_per_launch")
                roofline["traffic_source"] = ("ncu capture of this kernel recorded in profiles/traffic.json (not measured in this run): "
                                              + str(rec.get("source", "")) + ", build " + str(rec.get("build", "unrecorded")))
            except Exception:
                pass
    # ---- end to end through the public API with host buffers ----
    e2e = None
    if args.e2e_steps > 0 and (rank == 0 or world > 1):
        hx = [r.X.cpu().pin_memory() for r in runs]
        hdy = [r.dY.cpu().pin_memory() for r in runs]
        hy = [torch.empty_like(r.Y, device="cpu").pin_memory() for r in runs]
        hda = [torch.empty_like(r.dA, device="cpu").pin_memory() for r in runs]
        hdb = [torch.empty_like(r.dB, device="cpu").pin_memory() for r in runs]
        hdx = [torch.empty_like(r.dX, device="cpu").pin_memory() for r in runs]
        h2d = sum(t.numel() * t.element_size() for t in hx + hdy)
        d2h = sum(t.numel() * t.element_size() for t in hy + hda + hdb + hdx)

        # Three streams: copies in, compute (the current stream), copies out.  Every step still copies
        # all of its inputs from pinned host memory and all of its results back; the copies of one
        # projection overlap the kernels of its neighbours, ordered by events per projection.
        s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
        cur = torch.cuda.current_stream()
        ev_in = [torch.cuda.Event() for _ in runs]
        ev_comp = [torch.cuda.Event() for _ in runs]
        ev_out = [torch.cuda.Event() for _ in runs]

        def e2e_step():
            for i, r in enumerate(runs):
                with torch.cuda.stream(s_in):
                    s_in.wait_event(ev_comp[i])          # the previous step no longer reads these inputs
                    r.X.copy_(hx[i], non_blocking=True)
                    r.dY.copy_(hdy[i], non_blocking=True)
                    ev_in[i].record(s_in)
                cur.wait_event(ev_in[i])
                cur.wait_event(ev_out[i])                # the previous step's results have left the device
                r.forward()
                r.backward()
                ev_comp[i].record(cur)
                with torch.cuda.stream(s_out):
                    s_out.wait_event(ev_comp[i])
                    hy[i].copy_(r.Y, non_blocking=True)
                    hda[i].copy_(r.dA, non_blocking=True)
                    hdb[i].copy_(r.dB, non_blocking=True)
                    hdx[i].copy_(r.dX, non_blocking=True)
                    ev_out[i].record(s_out)

        def e2e_drain():
            cur.wait_stream(s_in)
            cur.wait_stream(s_out)

        for _ in range(2):
            e2e_step()
        e2e_drain()
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(args.e2e_steps):
            e2e_step()
        e2e_drain()
        e1.record()
        barrier()
        ms_e2e = replicas.max_over_ranks(e0.elapsed_time(e1), sess.device)
        e2e = {"value": world * T * args.e2e_steps / (ms_e2e * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "ms_per_step": ms_e2e / args.e2e_steps, "steps": args.e2e_steps}

    # ---- the other seeded configurations and the skinny kernels cold (rank 0, one GPU) ----
    configs_block, cold_block = None, None
    if rank == 0 and world == 1 and not args.no_extra_configs and not args.projections:
        for r in runs:
            r.close()
        del runs[:]
        torch.cuda.empty_cache()
        configs_block, cold_block = extra_configs(sess, peaks, args.workload)

    clock_regions = sampler.finish() if sampler else {}
    clocks = clock_regions.get("timed")
    status = mb.mlora_poll_status(sess.ctx)
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    if roofline is not None:
        # Which measured peak the kernel is held against follows from the clocks of the pass in which its launches
        # were timed (the per-kernel pass): at (nearly) the full boost clock the comparator is the burst figure, a
        # pass that ran clocked down under the power cap is held against the sustained one.  Both fractions are printed.
        ck = clock_regions.get("per_kernel") or {}
        mhz, mx = ck.get("sm_mhz"), ck.get("sm_max_mhz")
        capped = bool(mhz and mx and mhz < 0.9 * mx and "sw_power_cap" in ck.get("reasons", []))
        roofline["peak"] = peaks["bf16_tflops_sustained"] if capped else peaks["bf16_tflops"]
        roofline["frac"] = roofline["achieved"] / roofline["peak"]
        roofline["peak_source"] = (f"{peaks['source']} {'sustained' if capped else 'burst'} bf16 peak: the per-kernel pass ran at a median "
                                   f"{mhz} MHz of {mx} ({ck.get('seconds')} s, {ck.get('samples')} clock samples, reasons {ck.get('reasons')})")
    step_stats["clocks"] = clock_regions.get("single_steps")
    if clocks and clocks.get("sm_mhz"):
        step_stats["ms_per_step_x_sm_mhz"] = ms_per_step * clocks["sm_mhz"]
        ss = step_stats["clocks"] or {}
        if ss.get("sm_mhz"):
            step_stats["median_ms_x_sm_mhz"] = step_stats["median_ms"] * ss["sm_mhz"]
        step_stats["note"] = ("the timed region comes first and is short; the single steps behind median_ms / best_ms run after it, "
                              "when the board's power controller may have lowered the SM clock (see both clock records: time x MHz "
                              "compares runs at different clocks)")

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": label + (f" + LoRA dropout {args.dropout}" if args.dropout > 0 else ""), "rows_per_step": T, "ft_rows_per_step": workloads[0].ft_rows,
                   "l2_policy": f"inputs larger than L2: one step touches {resident / 1e6:.0f} MB of weights and "
                                f"activations, so nothing survives in the 126 MB L2 from step to step",
                   "parallelism": "replicas (rows are independent; no collective)" if world > 1 else "single GPU"},
        "tflops": tot_flops / (ms_per_step * 1e-3) / 1e12 * 1.0,
        "roofline_whole_step": {"t_roof_ms": tot_flops / (peaks["bf16_tflops"] * 1e12) * 1e3,
                                "frac_of_burst_peak": tot_flops / (peaks["bf16_tflops"] * 1e12) * 1e3 / ms_per_step,
                                "frac_of_sustained_peak": tot_flops / (peaks["bf16_tflops_sustained"] * 1e12) * 1e3 / ms_per_step},
        "clocks": clocks, "e2e": e2e, "gpu_launches": int(gpu_launches), "device_status": int(status),
        "step_stats": step_stats,
        "roofline": roofline, "kernels": kernels,
    }
    if configs_block is not None:
        line["configs"] = configs_block
        line["skinny_cold"] = cold_block
    if not args.no_cpu_baseline and world == 1:
        line["cpu_baseline"] = cpu_baseline(workloads)
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def extra_configs(sess, peaks, headline: str):
    """cfg2, the three cfg5 runs (+ fill ratio) and three cfg4 sweep points: forward + LoRA backward per
    repetition with an L2 flush between repetitions (their inputs are smaller than the L2), median and best
    of 30; then the rank-r kernels cold on their largest instances (rotating copies of the inputs)."""
    import bench_tables as bt

    def entry(w, reps=30):
        med, best = bt.step_time(sess, w, reps)
        fl = flops(w)
        tot = fl["fwd"] + (fl["bwd"] if w.ft_rows else 0.0)
        ab = algorithmic_bytes(w)
        nbytes = ab["gemm_fwd"] + (ab["gemm_bwd"] if w.ft_rows else 0.0)
        t_roof_us = max(tot / (peaks["bf16_tflops"] * 1e12), nbytes / (peaks["hbm_gbs"] * 1e9)) * 1e6
        return {"workload": w.name, "rows": w.n_rows, "ft_rows": w.ft_rows, "median_us": med, "best_us": best,
                "tokens_per_s": w.n_rows / (med * 1e-6), "tflops": tot / (med * 1e-6) / 1e12,
                "t_roof_us": t_roof_us, "frac_of_roofline": t_roof_us / med,
                "roofline_bound": "tensor" if tot / (peaks["bf16_tflops"] * 1e12) >= nbytes / (peaks["hbm_gbs"] * 1e9) else "hbm"}

    out = {"protocol": "forward + LoRA backward per repetition, 256 MB L2 flush between repetitions, CUDA events per repetition, "
                       "median of 30 (best beside it); roofline = slower of FLOPs at the measured burst bf16 peak and each "
                       "tensor once at the measured copy bandwidth"}
    if headline != "cfg2":
        out["cfg2"] = entry(synth.cfg2_single_projection(0))
    if headline != "cfg5":
        c5 = {m: entry(synth.cfg5_decode_heavy(0, m)) for m in ("decode", "finetune", "mixed")}
        c5["fill_ratio_mixed_over_decode_plus_finetune"] = c5["mixed"]["median_us"] / (c5["decode"]["median_us"] + c5["finetune"]["median_us"])
        # the same decode rows ordered by adapter (a layout choice of the caller): a 256-row tile then meets 64 adapters
        # instead of about 110, so the fused expand is 32 instead of 55 extra K-blocks per tile
        c5["decode_sorted_by_adapter"] = entry(synth.cfg5_decode_heavy(0, "decode", sorted_rows=True))
        c5["mixed_sorted_by_adapter"] = entry(synth.cfg5_decode_heavy(0, "mixed", sorted_rows=True))
        out["cfg5"] = c5
    out["cfg4"] = [entry(synth.cfg4_sweep_point(r, n, f), reps=20) for r, n, f in ((16, 8, 0.5), (64, 64, 0.25), (128, 256, 0.5))]
    # the same rank-128 point when the 256 adapters have ranks of their own (8 ... 128, stored zero-padded): a plan that
    # knows them packs the fused expand by rank and reads only the rows a rank needs
    w = synth.cfg4_sweep_point(128, 256, 0.5)
    t = synth.make_tensors(w)
    ranks = [(8, 16, 16, 32, 64, 128)[a % 6] for a in range(w.n_adapters)]
    for a, ra in enumerate(ranks):
        t["A_all"][a, ra:] = 0.0
        t["B_all"][a, ra:] = 0.0
    padded = bt.step_time(sess, w, 20, tensors=t)
    ranked = bt.step_time(sess, w, 20, tensors=t, adapter_rank=ranks)
    out["cfg4_mixed_ranks"] = {"workload": w.name + " with adapter ranks cycling through 8, 16, 16, 32, 64, 128 (stored padded to 128)",
                               "plain_plan_median_us": padded[0], "ranked_plan_median_us": ranked[0],
                               "note": "mlora_plan_create_ranked; not one of the five seeded configurations"}
    cold = {"protocol": "every repetition on another copy of X, dY and the activation buffers (6 copies), one CUDA event pair per launch, "
                        "40 repetitions; bytes = every operand once; fraction of the measured copy bandwidth (median / best)"}
    rows = []
    for w in synth.cfg3_layer_set(0, projections=["gate", "down"]) + [synth.cfg5_decode_heavy(0)]:
        times, nbytes, _rot = bt.cold_skinny(sess, w, 40, 6)
        for k, ts in times.items():
            med, best = float(np.median(ts)), float(np.min(ts))
            rows.append({"launch": f"{w.name}:{k}", "mbytes": nbytes[k] / 1e6, "median_us": med, "best_us": best,
                         "frac_hbm_median": nbytes[k] / med / 1e3 / peaks["hbm_gbs"], "frac_hbm_best": nbytes[k] / best / 1e3 / peaks["hbm_gbs"]})
    cold["launches"] = rows
    return out, cold


if __name__ == "__main__":
    main()
