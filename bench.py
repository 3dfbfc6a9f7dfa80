#!/usr/bin/env python
"""Benchmark of the self-attention hot path (projections -> scores -> softmax -> weighted sum).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c3] [--impl reference]

One "step" is one pass of the whole path over one batch of a seeded synthetic workload
(`paper_2012_01114_b200.inputs.WORKLOADS`).  The default workload is c4, the largest single-GPU one: the masked
attention core at batch 2, 16 heads, n = 8192, d_k = 128, bf16.  Rounds of --steps steps are repeated until the
timed region holds --min-seconds of device time.  Prints ONE JSON line; its `all_workloads` table adds c1, c2, c3, c4
and the twelve points of family c5, each timed with the L2 flushed before every step.

  value        useful TFLOP/s: 2 x (the paper's element-level MAC count for the scheme + the projection
               MACs) / device time, inputs resident in HBM, CUDA events around each step
  e2e          the same metric through psa_attention_host: host buffers in, host buffer out, copies timed
  roofline     dominant kernel, timed by CUDA events recorded inside the library between its kernels
  cpu_baseline the fp64 oracle timed on this machine's cores on a bounded sample of the same workload

With N > 1 (torchrun) every rank runs its own replica of the workload on its own GPU: (batch, head)
units are independent, there is no exchange step, so scaling is weak and the value is the sum over
ranks divided by the slowest rank's time.  `--impl reference` times the oracle alone (rank 0 only).
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "useful attention TFLOP/s (non-skipped FLOPs)"
UNIT = "TFLOP/s"
L2_FLUSH_BYTES = 256 << 20


# dram__bytes_read.sum + dram__bytes_write.sum per launch, from the ncu captures summarised under profiles/
# (attn_persist_kernel_c4_masked_n8192_d128.txt, gemm_and_attn_persist_c3_masked_n1024_d64.txt,
# attn_persist_kernel_c2_full_n512_d64.txt, attn_persist_kernel_c5_n256_full_and_masked_d128.txt).  Each figure is tied to the SHA-256 of the sources of the
# kernel it was measured on; once one of them changes the roofline reports traffic = null.
NCU_TRAFFIC = {
    "sources": {
        "psa_attn_persist.cu": "6faaea0a489bb7cad4f9e6d78e8ed96dd45b2f6e759c65f8d8539c5ae1166c96",
        "psa_softmax.cuh": "d6f464522774d5fa8e06d7bee0caa46cdbc57e830deef1f6ed5d2fd01c6dae71",
        "psa_sched.h": "f58d760c07067dcd12ea1f5d021072901f1247fc43730932f168d76ee1dd69aa",
        "psa_gemm.cu": "aa5a23d2e10a143ef90f2ed14bea1e072da286f79f0fd239b70736824174756c",
        "sm100.cuh": "2cc54c0ff8d920951dbbb97cef53e6b0fc9bd7d43d4002998c5a93069abcd23c"
    },
    "kernel_sources": {
        "attn": ["psa_attn_persist.cu", "psa_softmax.cuh", "psa_sched.h", "sm100.cuh"],
        "proj": ["psa_gemm.cu", "sm100.cuh"]
    },
    "traffic_bytes": {
        "c4": {
            "attn": 590732032
        },
        "c3": {
            "attn": 38193152,
            "proj": 16174080
        },
        "c2": {
            "attn": 19239680,
            "proj": 9854208
        },
        "c5-n256-full": {
            "attn": 1046764800
        },
        "c5-n256-masked": {
            "attn": 1049001984
        }
    }
}


def ncu_traffic(workload, kernel):
    import hashlib
    try:
        for name in NCU_TRAFFIC["kernel_sources"][kernel]:
            with open(os.path.join(ROOT, "paper_2012_01114_b200", "csrc", name), "rb") as f:
                if hashlib.sha256(f.read()).hexdigest() != NCU_TRAFFIC["sources"][name]:
                    return None
        return NCU_TRAFFIC["traffic_bytes"].get(workload, {}).get(kernel)
    except (OSError, KeyError):
        return None


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d.get("bf16_tflops_sustained", d["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


def useful_flops(w, batch=None):
    """2 x MACs the scheme needs at element level (paper Sec. 3.2, 4.2, 5.2) + projection MACs."""
    B = w["batch"] if batch is None else batch
    H, n, D, d = w["heads"], w["n"], w["d_model"], w["d_k"]
    tri = n * (n + 1) // 2
    qk = d * (n * n if w["scheme"] == 0 else tri)
    pv = d * (tri if w["scheme"] == 2 else n * n)
    proj = ((1 if w["scheme"] == 1 else 3) * n * D * H * d) if w["proj"] else 0
    if w.get("wo"):
        proj += n * H * d * D            # output projection of the block workloads
    return {"core": 2.0 * B * H * (qk + pv), "proj": 2.0 * B * proj}


def aggregate(per_rank_flops, max_seconds):
    """Whole-job throughput in TFLOP/s from the sum of the ranks' work and the slowest rank's time."""
    return float(sum(per_rank_flops)) / max_seconds / 1e12


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, index):
        super().__init__(daemon=True)
        self.index, self.samples, self.reasons, self.max_mhz, self._stop_evt = index, [], set(), None, threading.Event()
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def run(self):
        if self.nv is None:
            return
        nv = self.nv
        names = {"hw_slowdown": getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8),
                 "hw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40),
                 "sw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20),
                 "sw_power_cap": getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4)}
        while not self._stop_evt.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                get = getattr(nv, "nvmlDeviceGetCurrentClocksEventReasons", None) or nv.nvmlDeviceGetCurrentClocksThrottleReasons
                r = get(self.h)
                for k, bit in names.items():
                    if r & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            time.sleep(0.001)

    def stop(self):
        self._stop_evt.set()
        self.join(timeout=2)
        med = float(np.median(self.samples)) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


def oracle_sample(w, seconds_budget=20.0):
    """Times the oracle on a bounded sample of workload `w`: whole batch items (projection workloads) or
    whole (batch, head) slices (core-only workloads).  Returns (TFLOP/s, cores, description)."""
    import oracle
    from paper_2012_01114_b200 import inputs
    cores = os.cpu_count() or 1
    name = w["name"]
    if w["proj"]:
        s = inputs.make(name)
        v = s["values"]
        # whole batch items, cycling through the batch, until about half the budget is spent (the batch of the
        # small workloads takes under a second, so it is walked several times)
        done, t0 = 0, time.perf_counter()
        while True:
            b = done % w["batch"]
            if w.get("wo"):
                oracle.attention_block(v["X"][b:b + 1], v["Wq"], v.get("Wk", v["Wq"]), v.get("Wv", v["Wq"]), v["Wo"],
                                       w["heads"], w["scheme"])
            else:
                oracle.attention_layer(v["X"][b:b + 1], v["Wq"], v.get("Wk", v["Wq"]), v.get("Wv", v["Wq"]),
                                       w["heads"], w["scheme"])
            done += 1
            if time.perf_counter() - t0 > seconds_budget / 2:
                break
        dt = time.perf_counter() - t0
        fl = useful_flops(w, batch=done)
        return (fl["core"] + fl["proj"]) / dt / 1e12, cores, "%d batch items (the batch of %d walked cyclically), all heads, projections included (%.1f s)" % (done, w["batch"], dt)
    H, n, d = w["heads"], w["n"], w["d_k"]
    sym = w["scheme"] == 1
    q = inputs.tensor(w["seed"], 4, (1, n, H, d), 1.0, "bf16")[0]
    k = q if sym else inputs.tensor(w["seed"], 5, (1, n, H, d), 1.0, "bf16")[0]
    v = q if sym else inputs.tensor(w["seed"], 6, (1, n, H, d), 1.0, "bf16")[0]
    per_slice = useful_flops(w, batch=1)["core"] / H
    done, t0 = 0, time.perf_counter()
    while done < H:
        oracle.attention_core(q, k, v, w["scheme"], slices=[(0, done)])
        done += 1
        if time.perf_counter() - t0 > seconds_budget / 2:
            break
    dt = time.perf_counter() - t0
    return per_slice * done / dt / 1e12, cores, "%d of %d (batch, head) slices in full (%.1f s)" % (done, w["batch"] * H, dt)


def run_reference(args, w):
    per_step = []
    desc, cores = "", os.cpu_count() or 1
    for i in range(args.warmup + args.steps):
        t0 = time.perf_counter()
        tf, cores, desc = oracle_sample(w, seconds_budget=min(12.0, 2.0 * 150.0 / max(1, args.steps + args.warmup)))
        if i >= args.warmup:
            per_step.append((tf, time.perf_counter() - t0))
    val = float(np.mean([p[0] for p in per_step]))
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": 1e3 * float(np.mean([p[1] for p in per_step])),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": config_of(w, args, None), "gpu_launches": 0,
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def config_of(w, args, flush):
    """`flush`: True / False for the GPU arm's L2 policy, None for the CPU oracle arm."""
    from paper_2012_01114_b200 import inputs
    return {"workload": w["name"], "batch": w["batch"], "heads": w["heads"], "n": w["n"], "d_model": w["d_model"] if w["proj"] else None,
            "d_k": w["d_k"], "scheme": inputs.SCHEME_NAMES[w["scheme"]], "projections": bool(w["proj"]),
            "output_projection": bool(w.get("wo")),
            "parallelism": "replicas x%d (no exchange step)" % args.gpus,
            "l2": "not applicable (CPU oracle)" if flush is None else
                  ("flushed between steps by an untimed %d MiB memset" % (L2_FLUSH_BYTES >> 20)) if flush else
                  "not flushed: the step's inputs and output (%d MB) exceed the 126 MB L2, steps run back to back" % (io_bytes(w) // 1000000)}


def io_bytes(w):
    """Bytes of the tensors one step reads and writes (inputs + output), in the storage type."""
    es = 4 if w["dtype"] == "f32" else 2
    B, H, n, D, d = w["batch"], w["heads"], w["n"], w["d_model"], w["d_k"]
    if w["proj"]:
        nw = 1 if w["scheme"] == 1 else 3
        return es * (B * n * D + nw * D * H * d + B * n * (D if w.get("wo") else H * d) + (H * d * D if w.get("wo") else 0))
    return es * B * n * H * d * ((1 if w["scheme"] == 1 else 3) + 1)


class Prepared:
    """Device tensors and the step closure of one workload.  `shared` lets the c5 family reuse one set of drawn
    Q, K, V values viewed as [65536 / n, n, 16, 128] (the same flat buffer) instead of drawing 400 M numbers per n."""

    def __init__(self, name, torch, psa, inputs, pinned=False, shared=None):
        w = dict(inputs.WORKLOADS[name]); w["name"] = name
        self.w, self.name = w, name
        self.f32 = w["dtype"] == "f32"
        tdtype = torch.float32 if self.f32 else torch.bfloat16
        self.esize = 4 if self.f32 else 2
        H, scheme = w["heads"], w["scheme"]
        self.sym = scheme == psa.SYMMETRIC

        def to_host(arr):
            if self.f32:
                return torch.from_numpy(np.ascontiguousarray(arr, dtype=np.float32))
            return torch.from_numpy(np.ascontiguousarray(arr).view(np.int16)).view(torch.bfloat16)
        self.host = None
        if shared is not None:
            B, n, d = w["batch"], w["n"], w["d_k"]
            self.dev = {k: shared[k].view(B, n, H, d) for k in (("Q",) if self.sym else ("Q", "K", "V"))}
        else:
            up = inputs.make(name)["upload"]
            host = {k: to_host(up[k]) for k in up}
            if pinned:
                host = {k: t.pin_memory() for k, t in host.items()}
                self.host = host
            self.dev = {k: t.cuda() for k, t in host.items()}
        dev = self.dev
        out_cols = w["d_model"] if w.get("wo") else H * w["d_k"]
        self.out = torch.empty((w["batch"], w["n"], out_cols), dtype=tdtype, device="cuda")
        self.out_host = torch.empty(self.out.shape, dtype=tdtype).pin_memory() if pinned else None
        out = self.out
        if w["proj"]:
            layer = psa.psa_attention_f32 if self.f32 else psa.psa_attention
            if w.get("wo"):
                self.step = lambda: psa.psa_attention_block(dev["X"], dev["Wq"], dev.get("Wk"), dev.get("Wv"), dev["Wo"], H, scheme, out=out)
            else:
                self.step = lambda: layer(dev["X"], dev["Wq"], dev.get("Wk"), dev.get("Wv"), H, scheme, out=out)
            self.kernels_per_step = 2 + (1 if self.sym else 0) + (1 if w.get("wo") else 0)
        else:
            self.step = lambda: psa.psa_attention_core(dev["Q"], dev.get("K"), dev.get("V"), scheme, out=out)
            self.kernels_per_step = 2 if self.sym else 1
        fl = useful_flops(w)
        self.flops = fl
        self.flops_step = fl["core"] + fl["proj"]
        # steps of a workload whose tensors exceed L2 need no flush: every step streams them from HBM again
        self.flush = io_bytes(w) <= 2 * (126 << 20)


def more_rounds(total_ms, rounds, min_seconds, max_rounds, dist=None, device="cpu"):
    """Whether the timed region takes another round.  With several ranks the decision is the same on all of them:
    the rank with the least device time so far decides, so that every rank's region reaches `min_seconds`."""
    if dist is not None:
        import torch
        t = torch.tensor([total_ms], dtype=torch.float64, device=device)
        dist.all_reduce(t, op=dist.ReduceOp.MIN)
        total_ms = float(t.item())
    return rounds < max_rounds and total_ms < 1e3 * min_seconds


def timed_region(torch, prep, flushbuf, steps, min_seconds, max_rounds, dist=None):
    """Rounds of `steps` steps until the summed device time reaches `min_seconds` (at least one round).  With a flush
    between steps every step has its own event pair (the flush is outside it); without, one pair brackets a round of
    back-to-back steps.  Returns the per-step milliseconds of every round."""
    per_step_ms = []
    total_ms, rounds = 0.0, 0
    while True:
        if prep.flush:
            ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
            for s, e in ev:
                flushbuf.zero_()
                s.record(); prep.step(); e.record()
            torch.cuda.synchronize()
            ms = sum(s.elapsed_time(e) for s, e in ev)
        else:
            s, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            s.record()
            for _ in range(steps):
                prep.step()
            e.record()
            torch.cuda.synchronize()
            ms = s.elapsed_time(e)
        per_step_ms.append(ms / steps)
        total_ms += ms
        rounds += 1
        if not more_rounds(total_ms, rounds, min_seconds, max_rounds, dist, "cuda"):
            break
    return per_step_ms, total_ms


def kernel_split(torch, psa, prep, flushbuf, steps):
    """Mean per-kernel milliseconds (projection, attention) from CUDA events recorded inside the library, in a pass of
    its own: an event between two kernels keeps the second from being queued behind the first."""
    psa.psa_profile_begin(steps)
    for _ in range(steps):
        if prep.flush:
            flushbuf.zero_()
        prep.step()
    torch.cuda.synchronize()
    proj_ms, attn_ms, calls = psa.psa_profile_end()
    return {"proj": proj_ms / max(calls, 1), "attn": attn_ms / max(calls, 1)}


def quick_point(torch, psa, prep, flushbuf, steps, warmup, peaks):
    """One row of `all_workloads`: L2 flushed before every step, one event pair per step, median."""
    w = prep.w
    for _ in range(warmup):
        flushbuf.zero_(); prep.step()
    torch.cuda.synchronize()
    st, issued = psa.psa_last_issued()
    if st != psa.OK:
        raise RuntimeError("device status %d on %s" % (st, prep.name))
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    for a, b in ev:
        flushbuf.zero_(); a.record(); prep.step(); b.record()
    torch.cuda.synchronize()
    ms = sorted(a.elapsed_time(b) for a, b in ev)
    med = ms[len(ms) // 2]
    full_macs = 2.0 * w["batch"] * w["heads"] * w["d_k"] * w["n"] ** 2
    tf = prep.flops_step / (med * 1e-3) / 1e12
    row = {"workload": prep.name, "n": w["n"], "batch": w["batch"], "d_k": w["d_k"], "scheme": SCHEMES[w["scheme"]],
           "dtype": w["dtype"], "steps": steps, "ms": med, "ms_min": ms[0], "ms_mean": float(np.mean(ms)),
           "useful_tflops": tf, "frac_of_measured_burst_bf16": tf / peaks["bf16_tflops"],
           "algorithmic_gbs": io_bytes(w) / (med * 1e-3) / 1e9,
           "frac_of_measured_hbm": io_bytes(w) / (med * 1e-3) / 1e9 / peaks["hbm_gbs"],
           "issued_fraction_of_full": (issued["qk_macs"] + issued["pv_macs"]) / full_macs,
           "useful_fraction_of_full": (issued["useful_qk_macs"] + issued["useful_pv_macs"]) / full_macs}
    if w["proj"]:
        row["kernel_ms"] = kernel_split(torch, psa, prep, flushbuf, steps)
    return row


SCHEMES = {0: "full", 1: "symmetric", 2: "masked"}


def all_workloads(torch, psa, inputs, flushbuf, steps, peaks, only_c5=False):
    """c1, c2, c3, c4 and the twelve points of family c5 (n x scheme), each timed with the L2 flushed before every step.
    The c5 points share one drawn set of Q, K, V (the numbers of the n = 256 point viewed as [65536 / n, n, 16, 128]):
    timing does not depend on which standard-normal values are in the tensors, and the parity tests use each point's
    own seed."""
    rows = []
    if not only_c5:
        for name in ("c1", "c2", "c3", "c4"):
            prep = Prepared(name, torch, psa, inputs)
            rows.append(quick_point(torch, psa, prep, flushbuf, max(steps, 20) if name != "c4" else steps, 3, peaks))
            del prep
    w0 = inputs.WORKLOADS["c5-n256-full"]
    shape = (w0["batch"], 256, w0["heads"], w0["d_k"])
    shared = {k: torch.from_numpy(inputs.tensor_bits(w0["seed"], t, shape, 1.0).view(np.int16)).cuda().view(torch.bfloat16)
              for k, t in (("Q", 4), ("K", 5), ("V", 6))}
    for n in (256, 1024, 4096, 16384):
        t_full = None
        for scheme in (0, 1, 2):
            prep = Prepared("c5-n%d-%s" % (n, SCHEMES[scheme]), torch, psa, inputs, shared=shared)
            row = quick_point(torch, psa, prep, flushbuf, max(5, min(steps, 10 if n >= 4096 else 20)), 3, peaks)
            if scheme == 0:
                t_full = row["ms"]
            row["time_ratio_full_over_scheme"] = t_full / row["ms"]
            rows.append(row)
            del prep
    return rows


def run_sweep(args):
    import torch
    from paper_2012_01114_b200 import binding as psa, build, inputs
    build.build()
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    peaks = measured_peaks()
    flushbuf = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device="cuda")
    points = all_workloads(torch, psa, inputs, flushbuf, args.steps, peaks, only_c5=True)
    best = max((p for p in points if p["scheme"] == "masked"), key=lambda p: p["useful_tflops"])
    print(json.dumps({"metric": METRIC, "unit": UNIT, "value": best["useful_tflops"], "n_gpus": 1, "dtype": "bf16",
                      "data": "synthetic", "higher_is_better": True,
                      "config": {"workload": "c5 sweep (value = best masked point, n=%d)" % best["n"],
                                 "l2": "flushed between steps by an untimed %d MiB memset" % (L2_FLUSH_BYTES >> 20)},
                      "peaks": peaks, "sweep": points}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="c4", help="headline workload (default: c4, the largest single-GPU one)")
    ap.add_argument("--impl", default="psa", choices=["psa", "reference"])
    ap.add_argument("--min-seconds", type=float, default=1.0,
                    help="rounds of --steps steps are repeated until the timed region holds this much device time")
    ap.add_argument("--sweep", action="store_true", help="time the twelve points of workload family c5 only (one JSON line)")
    ap.add_argument("--no-all", action="store_true", help="skip the all_workloads table (c1-c4 and the c5 family)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer pass (for profiler captures)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "psa" else args.warmup

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    from paper_2012_01114_b200 import inputs
    if args.sweep:
        if rank == 0:
            run_sweep(args)
        return 0
    if args.impl == "reference":
        if rank == 0:
            w = dict(inputs.WORKLOADS[args.workload]); w["name"] = args.workload
            run_reference(args, w)
        return 0

    import torch
    import torch.distributed as dist
    from paper_2012_01114_b200 import binding as psa, build
    build.build()
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    prep = Prepared(args.workload, torch, psa, inputs, pinned=not args.no_e2e)
    w, H, scheme, sym, f32 = prep.w, prep.w["heads"], prep.w["scheme"], prep.sym, prep.f32
    flushbuf = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device="cuda")

    for _ in range(args.warmup):
        if prep.flush:
            flushbuf.zero_()
        prep.step()
    torch.cuda.synchronize()
    st, issued = psa.psa_last_issued()
    if st != psa.OK:
        raise RuntimeError("device status %d after warm-up" % st)

    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    sampler = ClockSampler(local_rank)
    sampler.start()
    t_wall = time.perf_counter()
    per_step_ms, total_ms = timed_region(torch, prep, flushbuf, args.steps, args.min_seconds,
                                         max_rounds=max(1, 20000 // max(1, args.steps)), dist=dist if world > 1 else None)
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    t_wall = time.perf_counter() - t_wall
    clocks = sampler.stop()
    rounds = len(per_step_ms)
    timed_steps = rounds * args.steps
    total_s = total_ms / 1e3
    if world > 1:
        t = torch.tensor([total_s], dtype=torch.float64, device="cuda")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        total_s = float(t.item())
    value = aggregate([prep.flops_step * timed_steps] * world, total_s)

    # per-kernel durations: single-kernel workloads take them from the timed region's own events; the others from
    # events recorded inside the library in a pass of their own
    step_ms_mean = 1e3 * total_s / timed_steps
    if prep.kernels_per_step == 1:
        kern = {"proj": 0.0, "attn": float(np.mean(per_step_ms))}
        kern_from = "the CUDA events of the timed region (one kernel per step)"
    else:
        kern = kernel_split(torch, psa, prep, flushbuf, args.steps)
        kern_from = "in-library CUDA events around each kernel, second pass of the same steps"

    # ---- end to end through the host-buffer entry points (copies inside the timed region)
    e2e = None
    if not args.no_e2e:
        host = prep.host
        if w.get("wo"):
            n_e2e = min(args.steps, 10)
            stream = torch.cuda.current_stream()

            def e2e_step():
                for k in host:
                    prep.dev[k].copy_(host[k], non_blocking=True)
                prep.step()
                prep.out_host.copy_(prep.out, non_blocking=True)
                stream.synchronize()
            api = "pinned copies + psa_attention_block"
        elif w["proj"]:
            n_e2e = min(args.steps, 20)

            def e2e_step():
                psa.psa_attention_host(host["X"], host["Wq"], host.get("Wk"), host.get("Wv"), H, scheme, prep.out_host)
            api = "psa_attention_host"
        else:
            n_e2e = min(args.steps, 10)

            def e2e_step():
                psa.psa_attention_core_host(host["Q"], host.get("K"), host.get("V"), scheme, prep.out_host)
            api = "psa_attention_core_host"
        for _ in range(2):
            e2e_step()
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        t0 = time.perf_counter()
        for _ in range(n_e2e):
            e2e_step()
        e2e_s = time.perf_counter() - t0
        if world > 1:
            t = torch.tensor([e2e_s], dtype=torch.float64, device="cuda")
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            e2e_s = float(t.item())
        e2e = {"value": aggregate([prep.flops_step * n_e2e] * world, e2e_s), "unit": UNIT,
               "h2d_bytes_per_step": int(sum(t.numel() * prep.esize for t in host.values())),
               "d2h_bytes_per_step": int(prep.out_host.numel() * prep.esize), "steps": n_e2e, "api": api}

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return 0

    peaks = measured_peaks()
    fl = prep.flops
    issued_flops = {"proj": 2.0 * issued["proj_macs"], "core": 2.0 * (issued["qk_macs"] + issued["pv_macs"])}
    dominant = "attn" if kern["attn"] >= kern["proj"] else "proj"
    # (the in-library events bracket the input projections and the attention kernel; the output projection of the
    # block workloads runs after them and is left out of the per-kernel figures)
    wo_flops = 2.0 * w["batch"] * w["n"] * H * w["d_k"] * w["d_model"] if w.get("wo") else 0.0
    alg = fl["core"] if dominant == "attn" else fl["proj"] - wo_flops
    achieved = alg / (kern[dominant] * 1e-3) / 1e12 if kern[dominant] > 0 else None
    # a kernel timed inside a region of a second or more runs under the power cap: the sustained peak is its
    # denominator; a region of milliseconds with idle gaps (the flushes) runs at burst clocks
    sustained = total_s >= 0.5 and not prep.flush
    peak = peaks["bf16_tflops_sustained"] if sustained else peaks["bf16_tflops"]
    mhz = clocks.get("sm_mhz") or clocks.get("sm_max_mhz") or 1965.0
    roofline = {"bound": "tensor", "kernel": ("sym_scores_kernel + sym_attn_kernel (symmetric scheme, all passes)" if sym else "attn_persist_kernel (fused scores-softmax-weighted sum)") if dominant == "attn" else "gemm_bf16_kernel (projections)",
                "achieved": achieved, "peak": peak, "unit": "TFLOP/s",
                "frac": (achieved / peak) if achieved else None,
                "peak_source": peaks["source"] + (" sustained bf16 (timed region of %.2f s, steps back to back)" % total_s if sustained else " burst bf16"),
                "frac_of_burst_peak": (achieved / peaks["bf16_tflops"]) if achieved else None,
                "frac_of_sustained_peak": (achieved / peaks["bf16_tflops_sustained"]) if achieved else None,
                "traffic": ncu_traffic(args.workload, dominant), "traffic_unit": "bytes per launch (ncu)",
                "kernel_ms": kern, "kernel_ms_from": kern_from,
                "kernel_ms_x_sm_mhz": {k: v * mhz for k, v in kern.items()},
                "algorithmic_flops": alg, "issued_flops": issued_flops}
    rates = None
    if not f32:
        try:
            rates = psa.psa_measure_pipe_rates()
        except psa.PsaError:
            rates = None
    if dominant == "attn" and kern["attn"] > 0 and not f32:
        # Second ceiling of the attention kernel: one exponential per issued weight on the special-function pipe, at
        # the rate measured on this GPU (results per SM clock per SM) and the SM clock sampled during the timed region.
        sm_count = torch.cuda.get_device_properties(local_rank).multi_processor_count
        per_clk = rates["ex2_per_clk_per_sm"] if rates else 16.0
        xu_peak = per_clk * sm_count * mhz * 1e6
        xu_rate = issued["exps"] / (kern["attn"] * 1e-3)
        roofline["second_ceiling"] = {"bound": "alu", "pipe": "MUFU ex2", "achieved": xu_rate / 1e12, "peak": xu_peak / 1e12,
                                      "unit": "Texp/s", "frac": xu_rate / xu_peak,
                                      "peak_source": "measured" if rates else "nominal",
                                      "peak_from": "%.2f ex2 per clock per SM (%s) x %d SMs x %.0f MHz" % (
                                          per_clk, "psa_measure_pipe_rates" if rates else "nominal", sm_count, mhz)}
    if f32:
        # The fp32 path runs on the CUDA cores and the 64-vector workload is a few microseconds of launch latency:
        # its line reports the bytes it has to move against the measured copy bandwidth.
        nbytes = float(io_bytes(w))
        t_s = (kern["proj"] + kern["attn"]) * 1e-3
        gbs = nbytes / t_s / 1e9 if t_s > 0 else None
        roofline = {"bound": "hbm", "kernel": "fp32 path (launch-latency bound at this size)",
                    "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": (gbs / peaks["hbm_gbs"]) if gbs else None,
                    "peak_source": peaks["source"] + " copy bandwidth", "traffic": None, "traffic_unit": "bytes per launch (ncu)",
                    "kernel_ms": kern, "kernel_ms_from": kern_from,
                    "algorithmic_bytes": nbytes, "issued_flops": issued_flops}
    table = None
    if not args.no_all and world == 1:
        del prep.dev, prep.out
        torch.cuda.empty_cache()
        table = all_workloads(torch, psa, inputs, flushbuf, min(args.steps, 20), peaks)
    cpu = None
    if not args.no_cpu_baseline and world == 1:
        tf, cores, desc = oracle_sample(w)
        cpu = {"value": tf, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc}
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "rounds": rounds, "timed_steps": timed_steps, "timed_region_device_s": total_s,
            "ms_per_step": step_ms_mean, "ms_per_step_median_of_rounds": float(np.median(per_step_ms)),
            "ms_per_step_min_of_rounds": float(np.min(per_step_ms)), "ms_per_step_first_round": per_step_ms[0],
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32" if f32 else "bf16", "data": "synthetic", "config": config_of(w, args, prep.flush), "clocks": clocks, "e2e": e2e,
            "gpu_launches": prep.kernels_per_step * timed_steps, "roofline": roofline, "cpu_baseline": cpu,
            "pct_of_measured_bf16_peak": 100.0 * value / world / peaks["bf16_tflops"],
            "pct_of_measured_sustained_bf16_peak": 100.0 * value / world / peaks["bf16_tflops_sustained"],
            "pct_of_nominal_bf16_peak": 100.0 * value / world / 2250.0,
            "ms_per_step_x_sm_mhz": step_ms_mean * mhz,
            "pipe_rates": rates, "peaks": peaks,
            "skip": {"issued_macs": issued["qk_macs"] + issued["pv_macs"],
                     "useful_macs": issued["useful_qk_macs"] + issued["useful_pv_macs"],
                     "issued_fraction_of_full": (issued["qk_macs"] + issued["pv_macs"]) /
                                                (2.0 * w["batch"] * H * w["d_k"] * w["n"] ** 2)},
            "wall_s_timed_region": t_wall, "all_workloads": table}
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())
