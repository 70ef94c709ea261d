#!/usr/bin/env python
"""Benchmark of the chunkwise delta-rule forward pass (one "step" = one pass of the whole hot path
over one batch of the rank-2 workload: B=2, H=16, L=8192, d_k=d_v=128, r=2, chunk=64, bf16 inputs).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload c2]

Prints ONE JSON line.  `value` is tokens/s (B*L tokens per step, all heads) with inputs resident in
HBM; `e2e` is the same metric through the C-ABI call with pinned HOST buffers (copies timed);
`roofline` describes the dominant kernel; `cpu_baseline` is the fp64 oracle timed on this machine's host
cores.  With --gpus N > 1 (torchrun) every rank runs the same batch on its own GPU (sequences are
independent: no collective on the data path) and the value is the aggregate.
`--impl reference` times the fp64 CPU oracle instead (rank 0 only).
"""
from __future__ import annotations

import argparse
import json
import os
import datetime
import statistics
import subprocess
import sys
import tempfile
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import pf_synth  # noqa: E402

METRIC = "tokens/s, rank-2 generalized DeltaNet fwd, L=8192 H=16 d=128"
UNIT = "tokens/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        return d, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


# ---- algorithmic work (per token-head unless noted); d_k = d_v = d allowed to differ ----------------
def alg_bytes_per_token_head(w) -> int:
    e = 2 if w.dtype == "bf16" else 4
    return e * (w.d_k + w.r * w.d_k + w.r * w.d_v + w.r) + 4 * w.d_v      # read q,k,v,beta once; write O fp32


def flops_per_chunk(w, tri: bool) -> dict:
    """Chunk-form FLOPs by step; `tri` halves the products the causal masks make half empty."""
    C, r, dk, dv = w.chunk, w.r, w.d_k, w.d_v
    n = C * r
    h = 0.5 if tri else 1.0
    return {
        "gram": 2 * n * n * dk * h, "solve": n ** 3 / 3.0, "wu": 2 * n * n * (dk + dv) * h,
        "attn": 2 * C * n * dk * h, "corr": 2 * n * dk * dv, "out": 2 * C * dk * dv + 2 * C * n * dv * h,
        "state": 2 * n * dk * dv,
    }


# Figures from ncu captures of the single-launch kernel, valid only for the kernel sources they were taken on (the
# hash of those sources is stored with them; the commands are in profiles/fused_kernel_c2.md):
#   NCU_TRAFFIC      DRAM bytes (read + write) of one full-size launch: {workload: (hash, bytes)}
#   NCU_TENSOR_PIPE  sm__pipe_tensor_cycles_active (% of peak, elapsed), captured on the half-size case
#                    (--batch 1 --heads 16) under the section-capture size rule: {workload: (hash, percent, case)}
NCU_TRAFFIC = {"c2": ("16732b90a2b7b496", 337161216 + 120871424)}
NCU_TENSOR_PIPE = {"c2": ("16732b90a2b7b496", 15.99, "half-size case B=1 H=16 of c2")}


def kernel_source_hash() -> str:
    import hashlib
    h = hashlib.sha256()
    for name in ("pf_fused.cu", "pf_tc_prims.cuh"):
        with open(os.path.join(ROOT, "paper_2504_00492_b200", "csrc", name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:16]


def ncu_traffic(w):
    ent = NCU_TRAFFIC.get(w.name)
    if not ent or ent[0] != kernel_source_hash():
        return None        # no capture, or the kernel has changed since the counters were taken
    return ent[1]


def ncu_tensor_pipe(w):
    ent = NCU_TENSOR_PIPE.get(w.name)
    if not ent or ent[0] != kernel_source_hash():
        return None, None
    return ent[1], ent[2]


class ClockSampler:
    """nvidia-smi samples of SM clock and throttle reasons while the timed region runs.

    The first query of a process initialises the management library, which can hold up kernel launches for tens
    of milliseconds, so the sampler is started before the warm-up and `wait_first_sample` returns once it is
    past that.  Samples carry a timestamp; the summary uses those inside [t_begin, t_end] (host clock) when
    there are any and says so in `window`, else every sample taken since the warm-up began (the GPU is kept
    busy with the same kernel from then on)."""
    Q = ("timestamp,index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int, period_ms: int = 50):
        self.gpu = gpu_index
        self.period_ms = period_ms
        self.proc = None
        self.path = None

    def start(self):
        try:
            f = tempfile.NamedTemporaryFile("w", suffix=".csv", delete=False)
            self.path = f.name
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.gpu), f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", str(self.period_ms)], stdout=f,
                                         stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def wait_first_sample(self, busy, limit_s: float = 10.0):
        """Calls busy() (which launches GPU work) until the first sample has been written."""
        if self.proc is None:
            return
        t0 = time.time()
        while time.time() - t0 < limit_s:
            busy()
            try:
                if os.path.getsize(self.path) > 0:
                    return
            except OSError:
                return

    @staticmethod
    def _stamp(text: str):
        try:
            return datetime.datetime.strptime(text.strip(), "%Y/%m/%d %H:%M:%S.%f").timestamp()
        except ValueError:
            return None

    def stop(self, t_begin: float = None, t_end: float = None) -> dict:
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0, "window": None}
        if self.proc is None:
            return out
        time.sleep(2.5 * self.period_ms * 1e-3)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        try:
            rows = [l.strip().split(", ") for l in open(self.path) if l.strip()]
            os.unlink(self.path)
        except Exception:
            return out
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        parsed = []
        for r in rows:
            if len(r) < 10:
                continue
            try:
                parsed.append((self._stamp(r[0]), float(r[2]), float(r[3]),
                               [nm for nm, val in zip(names, r[6:10]) if val.strip().lower() == "active"]))
            except ValueError:
                continue
        inside = [x for x in parsed if x[0] is not None and t_begin is not None and t_begin <= x[0] <= t_end]
        use, window = (inside, "timed region") if inside else (parsed, "warm-up and timed region")
        if use:
            out.update(sm_mhz=statistics.median(x[1] for x in use), sm_max_mhz=max(x[2] for x in use),
                       reasons=sorted({nm for x in use for nm in x[3]}), samples=len(use), window=window)
        return out


class Ranks:
    """The multi-process plumbing of a replicated run: one process per GPU, no data-path collective (sequences are
    independent, every rank runs its own replica of the workload on inputs of its own seed).  The only exchanges are
    the barriers around the timed region and the max over ranks of the measured time."""

    def __init__(self, backend: str = "nccl", device: str = "cuda"):
        self.rank, self.world, self.local = dist_env()
        self.device = device
        self.dist = None
        if self.world > 1:
            import torch.distributed as dist
            kw = {"device_id": torch.device("cuda", self.local)} if backend == "nccl" else {}
            dist.init_process_group(backend, **kw)
            self.dist = dist

    def seed(self, base: int) -> int:
        return base + 1000 * self.rank

    def barrier(self):
        if self.dist is not None:
            self.dist.barrier()
        if self.device == "cuda":
            torch.cuda.synchronize()

    def max_over_ranks(self, ms: float) -> float:
        if self.dist is None:
            return ms
        t = torch.tensor([ms], dtype=torch.float64, device=self.device)
        self.dist.all_reduce(t, op=self.dist.ReduceOp.MAX)
        return float(t.item())

    def job_value(self, units_per_rank_step: float, steps: int, ms: float) -> float:
        """Whole-job throughput: what all ranks processed, over the slowest rank's time."""
        return units_per_rank_step * self.world * steps / (self.max_over_ranks(ms) * 1e-3)

    def close(self):
        if self.dist is not None:
            self.dist.destroy_process_group()


def fwd_of(pf, w):
    """The entry point for the workload's input type (workload c0 is fp32, the others bf16)."""
    return pf.pf_deltanet_fwd_f32 if w.dtype == "f32" else pf.pf_deltanet_fwd


def dist_env():
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    return rank, world, local


def oracle_timed(w, sample_heads: int):
    """The oracle as it stands on a bounded sample: the first `sample_heads` (b,h) sequences, full L."""
    import oracle
    B = 1
    sub = w.with_(B=B, H=sample_heads)
    inp = pf_synth.make_inputs(sub)
    t0 = time.perf_counter()
    _, _, threads = oracle.deltanet_fwd(inp.q, inp.k, inp.v, inp.beta, inp.S0, return_threads=True)
    dt = time.perf_counter() - t0
    token_heads_per_s = sub.token_heads / dt
    return token_heads_per_s / w.H, threads, dt      # tokens/s for a model with w.H heads


def run_reference(args, w):
    rank, world, _ = dist_env()
    if rank != 0:
        return
    heads = min(w.B * w.H, 16)
    vals, threads = [], 0
    for i in range(args.warmup + args.steps):
        v, threads, dt = oracle_timed(w, heads)
        if i >= args.warmup:
            vals.append((v, dt))
    tok_s = statistics.mean(v for v, _ in vals)
    ms = statistics.mean(dt for _, dt in vals) * 1e3
    sample = f"{heads} of {w.B * w.H} (b,h) sequences of {w.name}, all L={w.L} tokens, per step"
    line = {
        "impl": "reference", "metric": METRIC, "value": tok_s, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "B": w.B, "H": w.H, "L": w.L, "d_k": w.d_k, "d_v": w.d_v, "r": w.r,
                   "chunk": w.chunk, "sample": sample},
        "cpu_baseline": {"value": tok_s, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": tok_s, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))


class SlicePipeline:
    """End-to-end step over slices of the (b,h) sequences on three streams (copy in, compute, copy out).

    All tensors are [B, H, ...] contiguous, so a run of consecutive (b,h) sequences is one contiguous range; a slice is
    handed to the library as a batch of its own (B = 1, H = sequences in the slice).  Per slice: the copy in waits for
    the previous step's kernel on that slice (its device buffers are reused), the kernel waits for the copy in and for
    the previous copy out of that slice's O, the copy out waits for the kernel."""

    def __init__(self, host, dev, O, Sf, hO, hS, w, forward, n_slices):
        self.w, self.forward = w, forward
        n_seq = w.B * w.H
        per = (n_seq + n_slices - 1) // n_slices
        self.ranges = [(a, min(a + per, n_seq)) for a in range(0, n_seq, per)]
        self.n = len(self.ranges)
        flat = lambda t: None if t is None else t.reshape((n_seq,) + tuple(t.shape[2:]))
        self.h = [flat(t) for t in (host.q, host.k, host.v, host.beta, host.S0)]
        self.d = [flat(t) for t in (dev.q, dev.k, dev.v, dev.beta, dev.S0)]
        self.O, self.Sf, self.hO, self.hS = flat(O), flat(Sf), flat(hO), flat(hS)
        self.s_in, self.s_out = torch.cuda.Stream(), torch.cuda.Stream()
        self.in_done = [torch.cuda.Event() for _ in self.ranges]
        self.k_done = [torch.cuda.Event() for _ in self.ranges]
        self.out_done = [torch.cuda.Event() for _ in self.ranges]
        self.first = True

    def step(self, stream):
        """One pass over all slices; `stream` (the timing stream) does the compute and joins the copy streams."""
        start = torch.cuda.Event()
        start.record(stream)
        self.s_in.wait_event(start)
        self.s_out.wait_event(start)
        for i, (a, b) in enumerate(self.ranges):
            with torch.cuda.stream(self.s_in):
                if not self.first:
                    self.s_in.wait_event(self.k_done[i])
                for hs, ds in zip(self.h, self.d):
                    if hs is not None:
                        ds[a:b].copy_(hs[a:b], non_blocking=True)
                self.in_done[i].record(self.s_in)
            stream.wait_event(self.in_done[i])
            if not self.first:
                stream.wait_event(self.out_done[i])
            sl = lambda t: None if t is None else t[a:b].unsqueeze(0)
            q, k, v, beta, S0 = (sl(t) for t in self.d)
            self.forward(q, k, v, beta, S0, O=sl(self.O), S_final=sl(self.Sf), stream=stream)
            self.k_done[i].record(stream)
            with torch.cuda.stream(self.s_out):
                self.s_out.wait_event(self.k_done[i])
                self.hO[a:b].copy_(self.O[a:b], non_blocking=True)
                self.hS[a:b].copy_(self.Sf[a:b], non_blocking=True)
                self.out_done[i].record(self.s_out)
        stream.wait_event(self.in_done[-1])
        stream.wait_event(self.out_done[-1])
        self.first = False


def kernel_profile(forward, d, steps):
    """Per-kernel device time (ms per launch, averaged) from CUDA events recorded inside the library."""
    from paper_2504_00492_b200 import binding
    lib = binding.lib()
    if not hasattr(lib, "pf_profile_enable"):
        return {}
    import ctypes
    lib.pf_profile_enable(1)
    acc = {}
    for _ in range(steps):
        # two calls back to back, the second one read: its kernels start on a busy GPU, as in the timed region (the
        # library's event list holds the latest call)
        forward(d.q, d.k, d.v, d.beta, d.S0)
        forward(d.q, d.k, d.v, d.beta, d.S0)
        torch.cuda.synchronize()
        n = lib.pf_profile_count()
        call = {}
        for i in range(n):
            name = ctypes.create_string_buffer(64)
            ms = ctypes.c_float(0)
            lib.pf_profile_read(i, name, 64, ctypes.byref(ms))
            call[name.value.decode()] = call.get(name.value.decode(), 0.0) + ms.value     # (a kernel may run more than once per call)
        for k, v in call.items():
            acc.setdefault(k, []).append(v)
    lib.pf_profile_enable(0)
    return {k: statistics.mean(v) for k, v in acc.items()}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=400)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c2", choices=sorted(pf_synth.CONFIGS))
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--batch", type=int, default=0, help="override B of the workload (profiling captures)")
    ap.add_argument("--heads", type=int, default=0, help="override H of the workload (profiling captures)")
    ap.add_argument("--ring-depth", type=int, default=0, help="pf_params.ring_depth (0 = the library's default)")
    ap.add_argument("--segments", type=int, default=0, help="pf_params.segments (0 = the library's default)")
    ap.add_argument("--e2e-slices", type=int, default=8, help="(b,h) slices of the pipelined end-to-end run")
    ap.add_argument("--path", default="auto", choices=["auto", "tc", "tc_split", "simt"],
                    help="pf_params.impl: the kernels to run (auto = what the plain entry point does)")
    ap.add_argument("--wu-builder", type=int, default=0, help="pf_params.wu_builder (fp32 SIMT kernels)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    w = pf_synth.CONFIGS[args.workload]
    if args.batch or args.heads:
        w = w.with_(B=args.batch or w.B, H=args.heads or w.H)
        w = w.with_(name=f"{w.name}[B={w.B},H={w.H}]")

    if args.impl == "reference":
        run_reference(args, w)
        return

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU path)")
    torch.cuda.set_device(dist_env()[2])
    ranks = Ranks("nccl", "cuda")
    rank, world, local = ranks.rank, ranks.world, ranks.local

    import paper_2504_00492_b200 as pf
    peaks, peak_kind = load_peaks()
    options = {}
    if args.ring_depth:
        options["ring_depth"] = args.ring_depth
    if args.segments:
        options["segments"] = args.segments
    if args.path != "auto":
        options["impl"] = args.path
    if args.wu_builder:
        options["wu_builder"] = args.wu_builder
    in_dtype = pf.PF_DTYPE_F32 if w.dtype == "f32" else pf.PF_DTYPE_BF16
    # PF_IMPL_AUTO may evaluate with a shorter chunk than the one asked for (the recurrence's result does not depend
    # on it); the work counts below use the chunk length the kernels ran with.
    chunk_used = pf.pf_select_chunk(w.B, w.H, w.L, w.d_k, w.d_v, w.r, w.chunk, in_dtype, args.path)
    w_eval = w.with_(chunk=chunk_used)

    def forward(q, k, v, beta, S0, O=None, S_final=None, stream=None):
        if options:
            return pf.pf_deltanet_fwd_ex(q, k, v, beta, S0, w.chunk, O=O, S_final=S_final, stream=stream, **options)
        return fwd_of(pf, w)(q, k, v, beta, S0, w.chunk, O=O, S_final=S_final, stream=stream)

    host = pf_synth.make_inputs(w, seed=ranks.seed(w.seed)).pin()
    d = host.to("cuda")
    O = torch.empty(w.B, w.H, w.L, w.d_v, dtype=torch.float32, device="cuda")
    Sf = torch.empty(w.B, w.H, w.d_k, w.d_v, dtype=torch.float32, device="cuda")
    stream = torch.cuda.current_stream()

    def step():
        forward(d.q, d.k, d.v, d.beta, d.S0, O=O, S_final=Sf)

    barrier = ranks.barrier

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        sampler.wait_first_sample(lambda: (step(), torch.cuda.synchronize()))
    for _ in range(args.warmup):
        step()
    launches_per_step = pf.pf_last_launch_count()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
    barrier()
    t_begin = time.time()
    ev[0].record(stream)
    for i in range(args.steps):
        step()
        ev[i + 1].record(stream)
    barrier()
    t_end = time.time()
    clocks = sampler.stop(t_begin, t_end) if rank == 0 else {}
    total_ms = ev[0].elapsed_time(ev[-1])
    per_step = [ev[i].elapsed_time(ev[i + 1]) for i in range(args.steps)]
    total_ms = ranks.max_over_ranks(total_ms)
    tokens_per_step = w.tokens * world
    value = tokens_per_step * args.steps / (total_ms * 1e-3)

    # ---- end to end: pinned host inputs -> device, call, outputs -> pinned host, all timed --------------
    # (a) serial: one copy in, one call, one copy out per step, all on one stream;
    # (b) pipelined: the (b,h) sequences are independent, so the batch is cut into slices and slice i's copy in,
    #     call and copy out run on three streams, chained by events: the copies of one slice overlap the kernel of
    #     another and the two copy directions overlap each other.  The reported e2e value is (b)'s.
    hO = torch.empty(O.shape, dtype=O.dtype).pin_memory()
    hS = torch.empty(Sf.shape, dtype=Sf.dtype).pin_memory()
    e2e_steps = max(3, min(args.steps, 10))

    def e2e_step():
        dd = host.to("cuda", non_blocking=True)
        o, s = forward(dd.q, dd.k, dd.v, dd.beta, dd.S0, O=O, S_final=Sf)
        hO.copy_(o, non_blocking=True)
        hS.copy_(s, non_blocking=True)

    e2e_step()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(e2e_steps):
        e2e_step()
    e1.record(stream)
    barrier()
    e2e_serial_ms = ranks.max_over_ranks(e0.elapsed_time(e1))
    e2e_serial = tokens_per_step * e2e_steps / (e2e_serial_ms * 1e-3)
    h2d = host.nbytes()
    d2h = hO.numel() * 4 + hS.numel() * 4

    pipe = SlicePipeline(host, d, O, Sf, hO, hS, w, forward, max(1, min(args.e2e_slices, w.B * w.H)))
    pipe.step(stream)
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(e2e_steps):
        pipe.step(stream)
    e1.record(stream)
    barrier()
    e2e_ms = ranks.max_over_ranks(e0.elapsed_time(e1))
    e2e_value = tokens_per_step * e2e_steps / (e2e_ms * 1e-3)
    e2e_launches = pf.pf_last_launch_count() * pipe.n

    # ---- per-kernel times and the roofline of the dominant kernel -----------------------------------------
    prof = kernel_profile(forward, d, steps=min(args.steps, 10))
    G = w.B * w.H * ((w.L + chunk_used - 1) // chunk_used)
    th = w.token_heads
    fl_tri = flops_per_chunk(w_eval, tri=True)
    fl_dense = flops_per_chunk(w_eval, tri=False)
    ms_step = total_ms / args.steps
    t_hbm_us = th * alg_bytes_per_token_head(w) / (peaks["hbm_gbs"] * 1e9) * 1e6
    t_flop_us = G * sum(fl_dense[k] for k in fl_dense if k != "solve") / (peaks["bf16_tflops"] * 1e12) * 1e6
    path = {"t_hbm_us": t_hbm_us, "t_flop_dense_us": t_flop_us, "frac": max(t_hbm_us, t_flop_us) / (ms_step * 1e3),
            "peaks": peak_kind, "tflops_dense": G * sum(fl_dense.values()) / (ms_step * 1e-3) / 1e12,
            "tflops_tri": G * sum(fl_tri.values()) / (ms_step * 1e-3) / 1e12,
            "hbm_gbs_algorithmic": th * alg_bytes_per_token_head(w) / (ms_step * 1e-3) / 1e9}
    # which algorithmic steps each kernel covers (triangular-aware FLOPs: the conservative count)
    kernel_steps = {
        "simt_gram": ["gram", "attn"], "simt_solve": ["solve"], "simt_wu": ["wu"], "simt_scan": ["corr", "out", "state"],
        "tc_flow": ["gram", "solve", "wu", "attn"], "tc_scan": ["corr", "out", "state"],
    }
    roofline = None
    if prof:
        top = max(prof, key=prof.get)
        if top == "fused":
            # The single-launch path does everything: its algorithmic traffic is one read of q, k, v, beta and one
            # write of O; at the measured peaks that HBM time exceeds the tensor time of the dense FLOPs, so HBM is
            # the roofline that binds (the tensor figure is printed beside it).
            nbytes = th * alg_bytes_per_token_head(w)
            achieved = nbytes / (prof[top] * 1e-3) / 1e9
            fl_d = G * sum(fl_dense[k] for k in fl_dense if k != "solve")
            roofline = {"bound": "hbm", "kernel": top, "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                        "frac": achieved / peaks["hbm_gbs"], "traffic": ncu_traffic(w), "ms_per_launch": prof[top],
                        "peaks": peak_kind, "bytes_per_launch": nbytes,
                        "tensor": {"tflops_dense": fl_d / (prof[top] * 1e-3) / 1e12, "peak": peaks["bf16_tflops"],
                                   "frac": fl_d / (prof[top] * 1e-3) / 1e12 / peaks["bf16_tflops"],
                                   "pipe_active_pct": ncu_tensor_pipe(w)[0], "pipe_active_from": ncu_tensor_pipe(w)[1]},
                        "kernel_ms": prof}
        else:
            steps_of = kernel_steps.get(top, list(fl_tri))
            fl = G * sum(fl_tri[s] for s in steps_of)
            achieved = fl / (prof[top] * 1e-3) / 1e12
            bound = "alu" if top.startswith("simt") else "tensor"
            # fp32 FFMA peak: 148 SMs x 128 lanes x 2 FLOP x max SM clock
            peak = 148 * 128 * 2 * peaks.get("sm_max_mhz", 1965.0) * 1e6 / 1e12 if bound == "alu" else peaks["bf16_tflops"]
            roofline = {"bound": bound, "kernel": top, "achieved": achieved, "peak": peak, "unit": "TFLOP/s",
                        "frac": achieved / peak, "traffic": None, "ms_per_launch": prof[top], "peaks": peak_kind,
                        "flops_per_launch": fl, "flop_count": "triangular-aware", "kernel_ms": prof}

    if rank == 0:
        cpu = None
        if not args.no_cpu_baseline:
            heads = min(w.B * w.H, 32)
            v, threads, dt = oracle_timed(w, heads)
            cpu = {"value": v, "unit": UNIT, "cores": threads, "kind": "oracle",
                   "sample": f"{heads} of {w.B * w.H} (b,h) sequences of {w.name}, all L={w.L} tokens, {dt:.2f} s wall"}
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16 in / f16 operands / f32 accumulate" if pf.pf_select_impl(
                w.B, w.H, w.L, w.d_k, w.d_v, w.r, w.chunk, in_dtype, args.path) in (2, 4) else "f32",      # PF_IMPL_TC, PF_IMPL_TC_SPLIT
            "data": "synthetic",
            "config": {"workload": w.name, "B": w.B, "H": w.H, "L": w.L, "d_k": w.d_k, "d_v": w.d_v, "r": w.r,
                       "chunk": w.chunk, "chunk_evaluated": chunk_used, "path": args.path, "l2": "inputs+outputs (%.0f MB) larger than L2" % (
                           (host.nbytes() + O.numel() * 4) / 1e6), "parallelism": "replicas" if world > 1 else "1 GPU"},
            "ms_per_step_median": statistics.median(per_step), "ms_per_step_min": min(per_step), "ms_per_step_max": max(per_step),
            "token_heads_per_s": value * w.H,
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "steps": e2e_steps, "ms_per_step": e2e_ms / e2e_steps,
                    "how": "%d (b,h) slices pipelined on 3 streams (copy in, compute, copy out)" % pipe.n,
                    "launches_per_step": e2e_launches,
                    "serial": {"value": e2e_serial, "ms_per_step": e2e_serial_ms / e2e_steps,
                               "how": "one copy in, one call, one copy out per step on one stream"}},
            "gpu_launches": launches_per_step * args.steps, "clocks": clocks, "roofline": roofline,
            "path_roofline": path, "cpu_baseline": cpu,
        }
        print(json.dumps(line))
    ranks.close()


if __name__ == "__main__":
    main()
