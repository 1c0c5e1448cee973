#!/usr/bin/env python
"""Benchmark of the libcott hot path.

Default workload (the one the headline metric is quoted on): causal cosine attention
forward + backward, bf16 I/O with fp32 state, B=4 H=16 N=4096 d=64, synthetic N(0,1)
tensors.  A step is one cott_fwd followed by one cott_bwd over one batch.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                    [--workload c4|c2|c2-train|c3|c3-train|c5:<N>|decode|c4-bnhd|varlen|varlen-small]

Prints ONE JSON line.  `value` is tokens/s with inputs resident in HBM; `e2e` is the same
metric through the host-buffer entry point (host<->device copies inside the timed region);
`roofline` compares the dominant call with the HBM roofline; `cpu_baseline` times the fp64
oracle on a bounded sample on the host cores.  With N > 1 (torchrun) every rank runs an
independent replica of the workload (heads and batch items are independent: there is no
data-path collective), and the time is the max over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "causal Cottention fwd+bwd tokens/s"
L2_FLUSH_BYTES = 256 << 20  # larger than the 126 MB L2
# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum, one ncu capture) moved per token-head
# by ALL launches of one step of a workload class, keyed by (d, causal, backward included).
# A constant from a committed capture, not a measurement of this run: the JSON line says so.
# Missing key: no capture of that class.
STEP_DRAM_TRAFFIC = {
    (64, True, True): 1563.3,     # C4 step: 409.8 MB over 262 144 token-heads (method's bytes: 1408)
    (64, False, False): 403.5,    # C2 forward: 79.3 MB over 196 608 token-heads (method's bytes: 512;
                                  # a third of the output is still in L2 when the kernel ends)
    (64, False, True): 1160.3,    # C2 forward + backward: 79.3 + 148.8 MB (method's bytes: 1408; the backward's
                                  # second pass over its inputs is served by L2, part of the gradients still there)
}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "source": "fallback"}


WORKLOADS = {
    "c4": dict(name="C4 causal fwd+bwd", B=4, H=16, N=4096, d=64, causal=True, bwd=True),
    "c3": dict(name="C3 causal fwd", B=8, H=12, N=1024, d=64, causal=True, bwd=False),
    # C3 with its backward: one training step of a GPT-2-small attention layer
    "c3-train": dict(name="C3 causal fwd+bwd", B=8, H=12, N=1024, d=64, causal=True, bwd=True),
    "c2": dict(name="C2 bidirectional fwd", B=32, H=12, N=512, d=64, causal=False, bwd=False),
    # the same shape with its backward: one training step of a BERT-base attention layer
    "c2-train": dict(name="C2 bidirectional fwd+bwd", B=32, H=12, N=512, d=64, causal=False, bwd=True),
    # C4 with every tensor stored [B,N,H,d] (what a projection GEMM leaves), read in place
    "c4-bnhd": dict(name="C4 causal fwd+bwd, tensors stored [B,N,H,d]", B=4, H=16, N=4096, d=64, causal=True,
                    bwd=True, layout="bnhd"),
    # packed variable-length batch: 64 sequences of 512..2048 tokens (seeded), no padding rows
    "varlen": dict(name="packed varlen causal fwd+bwd, 64 sequences of 512..2048 tokens", B=64, H=16, N=2048,
                   d=128, causal=True, bwd=True, varlen=True),
    # a quarter of it (0.65 GB of tensors, still several L2s): the case multi-counter profiler captures run on
    "varlen-small": dict(name="packed varlen causal fwd+bwd, 16 sequences of 512..2048 tokens", B=16, H=16, N=2048,
                         d=128, causal=True, bwd=True, varlen=True),
}


def get_workload(spec: str) -> dict:
    if spec in WORKLOADS:
        return dict(WORKLOADS[spec])
    if spec.startswith("c5:"):
        n = int(spec.split(":")[1])
        return dict(name=f"C5 causal fwd N={n}", B=1, H=16, N=n, d=128, causal=True, bwd=False)
    if spec == "decode":
        return dict(name="C5 decode step", B=64, H=16, N=1, d=128, causal=True, bwd=False, decode=True)
    raise SystemExit(f"unknown workload {spec}")


def algorithmic_bytes(w: dict) -> dict:
    """Bytes the method must move per step (bf16 I/O): forward reads q,k,v and writes o
    (4 tensors), backward reads q,k,v,dO and writes dq,dk,dv (7 tensors); a decode step
    reads and writes the fp32 state once."""
    th = w.get("rows", w["B"] * w["N"]) * w["H"] * w["d"] * 2
    if w.get("decode"):
        st = w["B"] * w["H"] * w["d"] * w["d"] * 4
        return {"fwd": 2 * st + 4 * w["B"] * w["H"] * w["d"] * 2, "bwd": 0}
    return {"fwd": 4 * th, "bwd": 7 * th if w["bwd"] else 0}


def roofline_record(w: dict, peaks: dict, kernels_ms: float, kernel: str, fwd_ms: float,
                    bwd_ms: float | None, step_ms: float) -> dict:
    """The `roofline` object of the JSON line.  Bytes are the METHOD's (forward 8d and backward
    14d per token-head in bf16: every tensor of the step once, whatever this implementation
    re-reads); `frac` = those bytes / `kernels_ms` (the time the step's kernel launches take on
    the launching stream) / the copy bandwidth; `calls` holds the same bytes over each whole
    call."""
    ab = algorithmic_bytes(w)
    alg = ab["fwd"] + ab["bwd"]
    d = w["d"]
    per_th = STEP_DRAM_TRAFFIC.get((d, bool(w["causal"]), bool(w.get("bwd"))))
    if w.get("decode") or w.get("varlen"):
        per_th = None
    traffic = per_th * (w.get("rows", w["B"] * w["N"]) * w["H"]) if per_th else None
    achieved = alg / (kernels_ms * 1e-3) / 1e9
    frac_of = lambda nbytes, ms: nbytes / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"]
    rec = {
        "bound": "hbm", "kernel": kernel, "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
        "frac": achieved / peaks["hbm_gbs"], "peak_source": peaks["source"],
        "algorithmic_bytes": alg,
        "algorithmic_bytes_per_token_head": {"fwd": 8 * d, "bwd": 14 * d if w.get("bwd") else 0},
        "ms": kernels_ms, "frac_of_nominal_8TBs": achieved / 8000.0,
        "traffic": traffic,
        "traffic_source": "ncu capture summarised under profiles/ (a constant, not measured in this run)",
        "traffic_over_algorithmic": (traffic / alg) if traffic else None,
        "goal": "causal forward at long N >= 0.60 of the measured copy bandwidth (peak above)",
        "calls": {"fwd": {"ms": fwd_ms, "frac": frac_of(ab["fwd"], fwd_ms)},
                  "step": {"ms": step_ms, "frac": frac_of(alg, step_ms)}},
    }
    if bwd_ms is not None:
        rec["calls"]["bwd"] = {"ms": bwd_ms, "frac": frac_of(ab["bwd"], bwd_ms)}
    return rec


class ClockSampler:
    """Samples SM clock and clock-event (throttle) reasons while the timed region runs.

    Read-only NVML queries from a background thread every 2 ms (the timed region of a default
    run lasts tens of milliseconds); falls back to an `nvidia-smi -lms` child process when the
    NVML binding is missing."""
    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
    PERIOD_S = 0.002

    def __init__(self, gpu_index: int, uuid: str | None = None):
        self.proc = None
        self.thread = None
        self.gpu_index = gpu_index
        self.uuid = uuid
        self.sm, self.bits = [], 0
        self.max_mhz = None
        self._stop = False

    def _nvml_loop(self, nv, handle):
        while not self._stop:
            try:
                self.sm.append(float(nv.nvmlDeviceGetClockInfo(handle, nv.NVML_CLOCK_SM)))
                self.bits |= int(nv.nvmlDeviceGetCurrentClocksEventReasons(handle))
            except Exception:       # a failed read is a missing sample, not a failed run
                pass
            time.sleep(self.PERIOD_S)

    def start(self):
        try:
            import pynvml as nv
            nv.nvmlInit()
            handle = None
            if self.uuid:
                try:
                    handle = nv.nvmlDeviceGetHandleByUUID(self.uuid)
                except Exception:
                    handle = None
            if handle is None:
                handle = nv.nvmlDeviceGetHandleByIndex(self.gpu_index)
            self.max_mhz = float(nv.nvmlDeviceGetMaxClockInfo(handle, nv.NVML_CLOCK_SM))
            self._nv = nv
            import threading
            self.thread = threading.Thread(target=self._nvml_loop, args=(nv, handle), daemon=True)
            self.thread.start()
            return
        except Exception:
            self.thread = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "100",
                 "-i", str(self.gpu_index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self) -> dict:
        if self.thread is not None:
            self._stop = True
            self.thread.join(timeout=2)
            nv = self._nv
            names = (("hw_slowdown", nv.nvmlClocksEventReasonHwSlowdown),
                     ("hw_thermal_slowdown", nv.nvmlClocksEventReasonHwThermalSlowdown),
                     ("sw_thermal_slowdown", nv.nvmlClocksEventReasonSwThermalSlowdown),
                     ("sw_power_cap", nv.nvmlClocksEventReasonSwPowerCap))
            reasons = sorted(n for n, bit in names if self.bits & bit)
            return {"sm_mhz": statistics.median(self.sm) if self.sm else None, "sm_max_mhz": self.max_mhz,
                    "samples": len(self.sm), "source": "nvml, read back to back with 2 ms sleeps", "reasons": reasons}
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        sm, mx, reasons = [], [], set()
        for line in out.strip().splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "source": "nvidia-smi, 100 ms period", "reasons": sorted(reasons)}


def dist_env():
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    return rank, world, local


def max_over_ranks(value: float, world: int) -> float:
    """Max of a per-rank scalar (device time) over all ranks; identity for one rank."""
    if world == 1:
        return value
    import torch
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64, device="cuda" if dist.get_backend() == "nccl" else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_tokens_per_s(tokens_per_rank_step: int, world: int, ms_per_step_max: float) -> float:
    """Whole-job throughput: every rank processes its own replica batch (weak scaling)."""
    return tokens_per_rank_step * world / (ms_per_step_max * 1e-3)


# ----------------------------------------------------------------------------- CPU oracle arm
def oracle_sample_step(w: dict, sample_heads: int, form: str = "quadratic"):
    """Returns (callable running the oracle once on the bounded sample, tokens it covers).
    The sample keeps N and d and takes `sample_heads` heads of one batch item; tokens are
    scaled by the fraction of (b,h) pairs covered."""
    import torch
    import oracle
    from paper_2409_18747_b200 import synth
    H = min(sample_heads, w["H"])
    if w.get("decode"):
        c = synth.make_qkv(1, H, 1, w["d"], torch.bfloat16, 99)
        import numpy as np
        state = np.zeros((1, H, w["d"], w["d"]))
        run = lambda: oracle.decode_step(c["q"][:, :, 0], c["k"][:, :, 0], c["v"][:, :, 0], c["m"], 8192.0, state)
        return run, w["B"] * (H / (w["B"] * w["H"])), f"decode step on {H} of {w['B'] * w['H']} (b,h) states"
    if w["N"] > 4096:
        # long sequences: the definition on evenly spaced rows of one head, about 2e10 flops
        import numpy as np
        c = synth.make_qkv(1, 1, w["N"], w["d"], torch.bfloat16, 99)
        n_rows = max(4, int(2e10 / (w["N"] / 2 * w["d"] * 4)))
        rows = np.linspace(0, w["N"] - 1, n_rows).astype(np.int64)
        run = lambda: oracle.fwd_rows(c["q"], c["k"], c["v"], c["m"], rows, None, w["causal"])
        return run, n_rows / w["H"], (f"fp64 quadratic definition on {n_rows} evenly spaced rows of one head "
                                      f"at N={w['N']}, d={w['d']}")
    c = synth.make_qkv(1, H, w["N"], w["d"], torch.bfloat16, 99, with_do=True)

    recurrent = form == "recurrent" and w["causal"]

    def run():
        if recurrent:
            oracle.fwd_recurrent(c["q"], c["k"], c["v"], c["m"], None)
            if w["bwd"]:
                oracle.bwd_recurrent(c["q"], c["k"], c["v"], c["d_o"], c["m"], None)
            return
        oracle.fwd_quadratic(c["q"], c["k"], c["v"], c["m"], None, w["causal"])
        if w["bwd"]:
            oracle.bwd_quadratic(c["q"], c["k"], c["v"], c["d_o"], c["m"], None, w["causal"])
    frac = H / (w["B"] * w["H"])
    what = "fwd+bwd" if w["bwd"] else "fwd"
    name = "recurrence (Eq. 8, running state)" if recurrent else "quadratic definition"
    return run, w["B"] * w["N"] * frac, (f"fp64 {name} {what} on {H} of {w['B'] * w['H']} (b,h) "
                                         f"pairs at N={w['N']}, d={w['d']}")


def run_reference(args, w):
    rank, world, _ = dist_env()
    if rank != 0:
        return
    import oracle
    # bounded sample: fewer (b,h) pairs per step when more steps are asked for, so the whole
    # run stays within a few minutes (one pair at N=4096, d=64 is about 4 core-seconds)
    n_runs = args.steps + max(1, min(args.warmup, 1))
    heads = max(1, min(16, 48 // max(args.steps, 1)))
    form = "quadratic"
    if w["N"] > 4096:
        heads = 1
    elif n_runs > 60 and w["causal"] and not w.get("decode"):
        # many steps: even one pair per step of the quadratic definition (about 1.6 s) would run
        # for many minutes; the oracle's linear-time recurrence on 16 pairs takes a fraction of that
        form, heads = "recurrent", 16
    run, tokens, what = oracle_sample_step(w, heads, form)
    for _ in range(max(1, min(args.warmup, 1))):
        run()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        run()
    dt = (time.perf_counter() - t0) / args.steps
    value = tokens / dt
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w["name"], "B": w["B"], "H": w["H"], "N": w["N"], "d": w["d"]},
        "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": min(oracle.num_threads(), heads), "kind": "oracle",
                         "sample": what},
        "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ----------------------------------------------------------------------------- GPU arm
def run_ours(args, w):
    import torch
    import paper_2409_18747_b200 as cott
    from paper_2409_18747_b200 import synth

    rank, world, local = dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: libcott has no CPU path")
    torch.cuda.set_device(local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    peaks = load_peaks()
    B, H, N, d = w["B"], w["H"], w["N"], w["d"]
    dev = torch.device("cuda", local)
    g = torch.Generator(device=dev); g.manual_seed(1004 + rank)
    mk = lambda *shape: torch.randn(shape, generator=g, device=dev, dtype=torch.float32).to(torch.bfloat16)
    m = torch.randn((H,), generator=g, device=dev, dtype=torch.float32)
    flush = torch.zeros(L2_FLUSH_BYTES // 4, dtype=torch.int32, device=dev)
    flush_sink = torch.zeros(1, dtype=torch.int32, device=dev)

    def flush_l2(i):
        """Evicts the step's tensors from L2 by writing a buffer twice the size of L2.  The L2
        is then full of dirty lines of that buffer, whose write-back the timed kernels pay for
        as they bring in their own data -- about what a steady-state step pays for evicting
        the outputs of the step before it.  COTT_BENCH_FLUSH=read evicts by reading instead
        (clean lines; the kernels' own output write-back then falls partly outside the timed
        region, which flatters short kernels)."""
        if os.environ.get("COTT_BENCH_FLUSH", "write") == "read":
            torch.amax(flush, dim=0, keepdim=True, out=flush_sink)
        else:
            flush.fill_(i & 0xFF)

    stream = torch.cuda.current_stream()
    dt_code = cott.cott.BF16

    if w.get("decode"):
        q, k, v = mk(B, H, d), mk(B, H, d), mk(B, H, d)
        state = torch.randn((B, H, d, d), generator=g, device=dev, dtype=torch.float32)
        o = torch.empty_like(q)
        fwd_call = lambda: cott.decode_step(q, k, v, state, m, 8192.0, out=o)
        bwd_call = None
        tokens_per_step = B
    elif w.get("varlen"):
        import numpy as np
        lens = np.random.RandomState(2024).randint(N // 4, N + 1, size=B)
        lens[0] = N
        T = int(lens.sum())
        w["rows"] = T
        cu = torch.tensor(np.concatenate([[0], np.cumsum(lens)]), dtype=torch.int32, device=dev)
        q, k, v, d_o = mk(T, H, d), mk(T, H, d), mk(T, H, d), mk(T, H, d)
        o = torch.empty_like(q)
        ws_f = torch.empty(cott.workspace_bytes(cott.cott.OP_FWD, dt_code, B, H, N, d, True), dtype=torch.uint8, device=dev)
        ws_b = torch.empty(cott.workspace_bytes(cott.cott.OP_BWD, dt_code, B, H, N, d, True), dtype=torch.uint8, device=dev)
        fwd_call = lambda: cott.fwd_varlen(q, k, v, m, cu, N, causal=True, out=o, workspace=ws_f)
        bwd_call = lambda: cott.bwd_varlen(q, k, v, d_o, m, cu, N, causal=True, workspace=ws_b)
        tokens_per_step = T
    else:
        if w.get("layout") == "bnhd":
            mk4 = lambda: mk(B, N, H, d).permute(0, 2, 1, 3)     # [B,H,N,d] view of [B,N,H,d] storage
        else:
            mk4 = lambda: mk(B, H, N, d)
        q, k, v = mk4(), mk4(), mk4()
        d_o = mk4() if w["bwd"] else None
        o = torch.empty_like(q)
        ws_f = torch.empty(cott.workspace_bytes(cott.cott.OP_FWD, dt_code, B, H, N, d, w["causal"]),
                           dtype=torch.uint8, device=dev)
        fwd_call = lambda: cott.fwd(q, k, v, m, causal=w["causal"], out=o, workspace=ws_f)
        bwd_call = None
        if w["bwd"]:
            ws_b = torch.empty(cott.workspace_bytes(cott.cott.OP_BWD, dt_code, B, H, N, d, w["causal"]),
                               dtype=torch.uint8, device=dev)
            # (a training step: the backward is given the forward call's workspace, whose partial
            # states it reuses where the plan has any)
            bwd_call = lambda: cott.bwd(q, k, v, d_o, m, causal=w["causal"], workspace=ws_b, fwd_workspace=ws_f)
        tokens_per_step = B * N

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize()

    def timed_steps(n_steps, record):
        """Runs n_steps; returns per-step (fwd_ms, bwd_ms) lists measured with CUDA events on
        the launching stream; L2 is flushed before every step (outside the timed spans)."""
        ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(n_steps)]
        for i in range(n_steps):
            flush_l2(i)
            ev[i][0].record(stream)
            fwd_call()
            ev[i][1].record(stream)
            if bwd_call is not None:
                bwd_call()
            ev[i][2].record(stream)
        torch.cuda.synchronize()
        if not record:
            return [], []
        return ([e[0].elapsed_time(e[1]) for e in ev], [e[1].elapsed_time(e[2]) for e in ev])

    timed_steps(max(args.warmup, 3), record=False)
    try:
        gpu_uuid = "GPU-" + str(torch.cuda.get_device_properties(dev).uuid)
    except Exception:
        gpu_uuid = None
    sampler = ClockSampler(local, gpu_uuid)
    barrier()
    launches0 = cott.cott.launch_count()
    sampler.start()
    fwd_ms, bwd_ms = timed_steps(args.steps, record=True)
    barrier()
    clocks = sampler.stop()
    launches = cott.cott.launch_count() - launches0
    # the same steps without the flush: part of the tensors (all of them, for the small
    # workloads) is then served from L2 -- reported beside the flushed figure, never instead
    ev_u = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
    n_unfl = max(3, min(args.steps, 50))
    for _ in range(5):                       # the GPU has idled for a moment: steps to get back up to speed
        fwd_call()
        if bwd_call is not None:
            bwd_call()
    ev_u[0].record(stream)
    for _ in range(n_unfl):
        fwd_call()
        if bwd_call is not None:
            bwd_call()
    ev_u[1].record(stream)
    torch.cuda.synchronize()
    unflushed_ms = ev_u[0].elapsed_time(ev_u[1]) / n_unfl
    step_ms_local = (sum(fwd_ms) + sum(bwd_ms)) / args.steps
    step_ms = max_over_ranks(step_ms_local, world)
    value = aggregate_tokens_per_s(tokens_per_step, world, step_ms)

    # ---- end to end: host buffers in, host buffers out, through cott_fwd_bwd_host
    e2e = None
    if w.get("bwd") and not w.get("decode") and not w.get("varlen") and not w.get("layout"):
        host_in = [t.cpu().pin_memory() for t in (q, k, v, d_o)]
        host_m = m.cpu().pin_memory()
        host_out = [torch.empty_like(host_in[0]).pin_memory() for _ in range(4)]
        host_dm = torch.empty((H,), dtype=torch.float32).pin_memory()
        arena = None
        n_e2e = max(3, min(args.steps, 10))
        evs = [[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(n_e2e)]
        for it in range(2 + n_e2e):
            if it >= 2:
                evs[it - 2][0].record(stream)
            arena = cott.fwd_bwd_host(*host_in, host_m, *host_out, host_dm, causal=w["causal"], arena=arena)
            if it >= 2:
                evs[it - 2][1].record(stream)
            torch.cuda.synchronize()
        e2e_ms = max_over_ranks(sum(a.elapsed_time(b) for a, b in evs) / n_e2e, world)
        nbytes = q.numel() * 2
        e2e = {"value": aggregate_tokens_per_s(tokens_per_step, world, e2e_ms), "unit": "tokens/s",
               "ms_per_step": e2e_ms, "h2d_bytes_per_step": 4 * nbytes + H * 4,
               "d2h_bytes_per_step": 4 * nbytes + H * 4}

    # ---- dominant kernel alone: a profiling pass records CUDA events around every launch of
    # the tensor-core walk kernels on the launching stream (same launch configuration as the
    # timed steps, L2 flushed before each step)
    prof_ms = []
    if not w.get("decode"):
        n_prof = max(3, min(args.steps, 10))
        cott.cott.profile_enable(256)
        for i in range(n_prof):
            flush_l2(i)
            fwd_call()
            if bwd_call is not None:
                bwd_call()
        torch.cuda.synchronize()
        prof_ms = [ms for _, ms in cott.cott.profile_read()]      # every tensor-core launch of the steps
        cott.cott.profile_enable(0)

    # ---- decode as a loop: 1024 steps back to back with no L2 flush (the 67 MB of state fit
    # in L2, so this can run above the HBM roofline), as plain launches and as one replay of a
    # CUDA graph that captured the same 1024 launches
    loop_detail = {}
    if w.get("decode"):
        n_loop = 1024
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        for _ in range(8):
            fwd_call()
        torch.cuda.synchronize()
        e0.record(stream)
        for _ in range(n_loop):
            fwd_call()
        e1.record(stream)
        torch.cuda.synchronize()
        loop_detail["loop_1024_plain_us_per_step"] = e0.elapsed_time(e1) * 1e3 / n_loop
        cap_stream = torch.cuda.Stream()
        cap_stream.wait_stream(stream)
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=cap_stream):
            for _ in range(n_loop):
                fwd_call()
        graph.replay()
        torch.cuda.synchronize()
        e0.record(stream)
        graph.replay()
        e1.record(stream)
        torch.cuda.synchronize()
        loop_detail["loop_1024_graph_us_per_step"] = e0.elapsed_time(e1) * 1e3 / n_loop
        # ---- blocks of T tokens through cott_fwd_stateful: the state is read and written once
        # per block instead of once per token (L2 flushed before every block)
        for T in (16, 128):
            qb, kb, vb = mk(B, H, T, d), mk(B, H, T, d), mk(B, H, T, d)
            ob = torch.empty_like(qb)
            st_a = state.clone()
            ws_blk = torch.empty(cott.workspace_bytes(cott.cott.OP_FWD, dt_code, B, H, T, d, True),
                                 dtype=torch.uint8, device=dev)
            ts = []
            for i in range(8):
                flush_l2(i)
                e0.record(stream)
                _, st_b = cott.fwd_stateful(qb, kb, vb, m, 8192.0, state_in=st_a, out=ob, workspace=ws_blk)
                e1.record(stream)
                torch.cuda.synchronize()
                ts.append(e0.elapsed_time(e1))
                st_a = st_b
            loop_detail[f"block_T{T}_us_per_token"] = statistics.median(ts[2:]) * 1e3 / T

    if world > 1:
        import torch.distributed as dist
        dist.barrier()
        dist.destroy_process_group()
    if rank != 0:
        return
    ab = algorithmic_bytes(w)
    th = w.get("rows", B * N) * H * d * 2       # bytes of one bf16 tensor of the step
    plan = cott.query_plan(cott.cott.OP_BWD if w.get("bwd") else cott.cott.OP_FWD, dt_code, B, H, max(N, 1), d,
                           w["causal"]) if not w.get("decode") else {"path": 0, "group": 1, "chunk": 1}
    if w.get("varlen"):
        plan = {"path": 1, "chunk": 128, "groups": "the dense plan's for max_seqlen, or finer by the total token count",
                "rows": w["rows"], "padded_rows": B * N}
    # Roofline of the step: the METHOD's bytes (forward: q, k, v in, o out = 8d per token-head;
    # backward: q, k, v, dO in, dq, dk, dv out = 14d; decode: the fp32 state in and out) over the
    # time the step's kernel launches take, measured with CUDA events on the stream they are
    # launched on.  Tensors this implementation reads twice count once.
    alg = ab["fwd"] + ab["bwd"]
    # The kernels of a step overlap (a kernel's prologue runs under its predecessor's tail), so
    # their time is the span of the step on the launching stream in the timed region; the
    # profiling pass, which puts an event pair around every launch and so runs them one at a
    # time, is reported beside it.
    dom_ms = step_ms_local
    alone_ms = None
    if prof_ms:
        n_prof_steps = max(3, min(args.steps, 10))
        alone_ms = sum(prof_ms) / n_prof_steps
        kernel = (f"the {len(prof_ms) // n_prof_steps} tcgen05 launches of one step (d={d}): span on the launching "
                  f"stream in the timed region")
    else:
        kernel = "decode_kernel (fp32 SIMT, two CTAs per (b,h))" if w.get("decode") else "cott_fwd call (fp32 SIMT path)"
    roofline = roofline_record(w, peaks, dom_ms, kernel, statistics.mean(fwd_ms),
                               statistics.mean(bwd_ms) if bwd_call is not None else None, step_ms_local)
    if alone_ms is not None:
        roofline["launches_timed_one_at_a_time_ms"] = alone_ms
        roofline["frac_launches_one_at_a_time"] = alg / (alone_ms * 1e-3) / 1e9 / peaks["hbm_gbs"]
    extra = {"step_ms_unflushed_back_to_back": unflushed_ms}
    extra.update(loop_detail)

    cpu = None
    if world == 1 or rank == 0:
        import oracle
        n_pairs = 16 if N <= 4096 else 1
        run, tokens, what = oracle_sample_step(w, n_pairs)
        t0 = time.perf_counter(); run(); dt = time.perf_counter() - t0
        cpu = {"value": tokens / dt, "unit": "tokens/s", "cores": min(oracle.num_threads(), n_pairs, H),
               "kind": "oracle",
               "sample": what, "seconds": dt}

    line = {
        "metric": METRIC if w.get("bwd") else f"{w['name']} tokens/s", "value": value, "unit": "tokens/s",
        "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": step_ms,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": w["name"], "B": B, "H": H, "N": N, "d": d, "causal": w["causal"],
                   "io": "bf16, fp32 state and accumulators", "parallelism": f"replicas x{world}",
                   "l2": "flushed before every step (256 MB " + os.environ.get("COTT_BENCH_FLUSH", "write") + "); working set also exceeds L2",
                   "plan": plan},
        "roofline": roofline, "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": int(launches), "clocks": clocks,
        "detail": extra,
    }
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c4")
    args = ap.parse_args()
    w = get_workload(args.workload)
    if args.impl == "reference":
        run_reference(args, w)
    else:
        run_ours(args, w)


if __name__ == "__main__":
    main()
