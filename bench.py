#!/usr/bin/env python
"""Benchmark of the fused vocabulary projection + cross-entropy path (forward + backward).

One "step" is one pass of the whole hot path over one synthetic batch: vp_ce_forward, then
vp_ce_backward (masked-mean upstream gradient), then vp_ce_mean_loss; for the long-context
workload a step is the whole stream (64 calls, dW accumulated across calls).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

Prints ONE JSON line (rank 0).  `value` is tokens/s with inputs resident in HBM; `e2e` is the
same metric through vp_ce_fwd_bwd_host with pinned HOST activations (copies inside the timed
region).  With N > 1 every rank runs an independent replica on its own batch (the path has no
exchange step on one node: weak scaling, no collective in the data path).
`--impl reference` times the float64 CPU oracle on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import dataclasses
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

METRIC = "fused vocab-proj CE fwd+bwd tokens/s"
NOMINAL_BF16_TFLOPS = 2250.0
FALLBACK_PEAKS = {"bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "hbm_gbs": 6650.0}
# DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) of each kernel kind, from ncu captures of
# launches of the same geometry, keyed by (dtype, d, block_v, T_chunk); other geometries report traffic = null.
NCU_DRAM_BYTES_PER_LAUNCH = {
    ("bf16", 2880, 8192, 16384): {"fwd_strip_fold": 159e6, "bwd_strip_residual": 484e6, "dH_gemm": 926e6,
                                  "dW_gemm": 969e6},
    ("bf16", 7168, 8192, 8192): {"fwd_strip_fold": 692e6, "bwd_strip_residual": 898e6, "dH_gemm": 1147e6,
                                 "dW_gemm": 1141e6},
}
# Token chunk used by the timed launch configuration (a call argument of the library).
BENCH_T_CHUNK = {"tiny": 512, "mid": 4096, "moe120b": 16384, "moe667b": 8192, "longctx": 16384}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return p, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


# --------------------------------------------------------------------------- clocks sampler
class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap,power.draw")

    def __init__(self, index: int):
        self.rows = []
        self.proc = None
        self.index = index

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            parts = [x.strip() for x in line.split(",")]
            if len(parts) >= 6:
                self.rows.append(parts)

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm = [float(r[0]) for r in self.rows if r[0].replace(".", "").isdigit()]
        mx = [float(r[1]) for r in self.rows if r[1].replace(".", "").isdigit()]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = [n for i, n in enumerate(names) if any(r[2 + i].lower().startswith("active") for r in self.rows)]
        watts = []
        for r in self.rows:
            try:
                watts.append(float(r[6]))
            except (IndexError, ValueError):
                pass
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": reasons, "samples": len(sm),
                "power_w_median": statistics.median(watts) if watts else None}


# --------------------------------------------------------------------------- CPU oracle leg
def oracle_sample_rate(w, W_bits, H_bits, labels, n_tokens=1024, W64=None):
    """Times the float64 oracle (as it stands) on the first n tokens of the batch against the whole
    vocabulary.  The oracle works through token slabs of 1024 rows and pays O(V d) per slab for its
    float64 dW accumulation, so one full slab is the smallest sample with the steady-state cost of a
    whole run; smaller samples overstate the per-token cost."""
    from oracle import vpce_oracle as orc
    from synth_inputs import IGNORE_INDEX, bf16_bits_to_f64
    try:
        from threadpoolctl import threadpool_info
        cores = max([p.get("num_threads", 1) for p in threadpool_info()] or [os.cpu_count() or 1])
    except Exception:
        cores = os.cpu_count() or 1
    if W64 is None:
        W64 = bf16_bits_to_f64(W_bits)                    # input preparation, outside the timed call
    n = min(int(n_tokens), w.T)
    t0 = time.perf_counter()
    orc.forward_backward(bf16_bits_to_f64(H_bits[:n]), W64, labels[:n], None, IGNORE_INDEX)
    dt = time.perf_counter() - t0
    return {"value": n / dt, "unit": "tokens/s", "cores": int(cores), "kind": "oracle",
            "sample": f"first {n} of {w.T} tokens of one call against the full vocabulary V={w.V}, d={w.d}: "
                      f"float64 forward+backward by the dense definition, {dt:.1f} s wall clock"}, n, dt


def run_reference(args, w):
    """The reference arm: the oracle on the host cores, bounded sample per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from synth_inputs import make_hidden, make_weights, stream_labels
    W_bits = make_weights(w)
    labels = stream_labels(w)[:w.T]
    H_bits = make_hidden(w, 0)
    steps = max(1, args.steps)
    # one oracle slab (1024 tokens, the sample `cpu_baseline` times as well) per step; only a run of many steps
    # (K + W > 16, i.e. more than about two minutes of oracle time) falls back to half or quarter slabs
    total = steps + args.warmup
    n_step = 1024 if total <= 16 else (512 if total <= 32 else 256)
    from synth_inputs import bf16_bits_to_f64
    W64 = bf16_bits_to_f64(W_bits)
    res, n, dt = None, 0, 0.0
    times = []
    for i in range(args.warmup + steps):
        res, n, dt = oracle_sample_rate(w, W_bits, H_bits, labels, n_tokens=n_step, W64=W64)
        if i >= args.warmup:
            times.append(dt)
    ms = 1e3 * sum(times) / len(times)
    val = n / (ms / 1e3)
    out = {"impl": "reference", "metric": METRIC, "value": val, "unit": "tokens/s", "n_gpus": args.gpus,
           "steps": steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
           "vs_baseline": None, "dtype": "f64", "data": "synthetic",
           "config": {"workload": w.name, "T": w.T, "d": w.d, "V": w.V, "block_v": w.block_v,
                      "note": "float64 CPU oracle, each step a bounded token sample of the workload"},
           "cpu_baseline": {"value": val, "unit": "tokens/s", "cores": res["cores"], "kind": "oracle",
                            "sample": res["sample"]},
           "e2e": {"value": val, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
           "gpu_launches": 0}
    print(json.dumps(out), flush=True)


# --------------------------------------------------------------------------- multi-rank helpers
def rank_workload(w, rank: int):
    """Rank r of a multi-GPU run draws its own batch stream (replicas on distinct data)."""
    return w if rank == 0 else dataclasses.replace(w, seed=w.seed + 1000 * rank)


def max_over_ranks(ms: float, device=None) -> float:
    """MAX over ranks of a duration measured on each rank's device (identity on one rank)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(ms)
    t = torch.tensor([ms], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_tokens_per_s(world: int, tokens_per_rank: int, ms_max: float) -> float:
    """Units all ranks processed divided by the slowest rank's time."""
    return world * tokens_per_rank / (ms_max / 1e3)


# --------------------------------------------------------------------------- cuBLAS yard-stick
def cublas_yardstick(w, T_chunk, dev, seconds=1.0):
    """Context, not product code: torch.matmul (cuBLAS) in bf16 on the three contraction shapes of ONE
    (chunk, shard) meeting of this workload, each run back to back for about `seconds` (so the power cap
    acts on it as it does on the timed step), with operands larger than L2 in total.  It answers what a
    library GEMM reaches on these exact shapes and operand layouts under the same conditions:
      strip    Y  = H_c  W_q^T   [T_chunk x d] . [block_v x d]^T      (both operands K-major)
      dH       dH = G    W_q     [T_chunk x block_v] . [block_v x d]  (B MN-major)
      dW       dW = G^T  H_c     [T_chunk x block_v]^T . [T_chunk x d] (A and B MN-major)
    cuBLAS writes bf16 outputs; it runs no fold / residual epilogue and no fp32 accumulation across shards."""
    import torch
    r, c, d = min(T_chunk, w.T), min(w.block_v, w.V), w.d
    Hc = torch.randn(r, d, device=dev, dtype=torch.bfloat16)
    Wq = torch.randn(c, d, device=dev, dtype=torch.bfloat16) * 0.02
    G = torch.randn(r, c, device=dev, dtype=torch.bfloat16) * 0.01
    Y = torch.empty(r, c, device=dev, dtype=torch.bfloat16)
    dHo = torch.empty(r, d, device=dev, dtype=torch.bfloat16)
    dWo = torch.empty(c, d, device=dev, dtype=torch.bfloat16)
    cases = {"strip": lambda: torch.matmul(Hc, Wq.T, out=Y),
             "dH": lambda: torch.matmul(G, Wq, out=dHo),
             "dW": lambda: torch.matmul(G.T, Hc, out=dWo)}
    flops = 2.0 * r * c * d
    out = {"shape": {"rows": r, "cols": c, "d": d}, "seconds_each": seconds, "unit": "TFLOP/s"}
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for name, fn in cases.items():
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        e0.record(); fn(); e1.record(); torch.cuda.synchronize()
        n = max(5, int(seconds * 1e3 / max(e0.elapsed_time(e1), 1e-3)))
        e0.record()
        for _ in range(n):
            fn()
        e1.record(); torch.cuda.synchronize()
        out[name] = flops * n / (e0.elapsed_time(e1) / 1e3) / 1e12
    # the three in the order of a backward meeting, interleaved, as the step runs them (clocks and power sampled)
    n = max(3, int(2 * seconds * 1e3 / (3 * flops / (out["strip"] * 1e12) * 1e3)))
    sampler = ClockSampler(dev.index or 0)
    sampler.start()
    time.sleep(0.3)
    e0.record()
    for _ in range(n):
        for fn in cases.values():
            fn()
    e1.record(); torch.cuda.synchronize()
    out["interleaved"] = 3 * flops * n / (e0.elapsed_time(e1) / 1e3) / 1e12
    out["interleaved_clocks"] = sampler.stop()
    return out


# --------------------------------------------------------------------------- GPU arm
class Ctx:
    def __init__(self):
        import torch
        self.world = int(os.environ.get("WORLD_SIZE", "1"))
        self.rank = int(os.environ.get("RANK", "0"))
        self.local_rank = int(os.environ.get("LOCAL_RANK", "0"))
        torch.cuda.set_device(self.local_rank)
        self.dev = torch.device("cuda", self.local_rank)
        if self.world > 1:
            import torch.distributed as dist
            dist.init_process_group("nccl", device_id=self.dev)

    def barrier(self):
        import torch
        if self.world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize()

    def close(self):
        if self.world > 1:
            import torch.distributed as dist
            dist.destroy_process_group()


def measure(ctx, w, dtype, steps, warmup, t_chunk=0, with_e2e=True, with_cpu_baseline=True, with_yardstick=False,
            prof_on=True):
    """Times `steps` passes of the whole hot path over workload `w` and returns the result line as a dict
    (rank 0; None on the other ranks)."""
    import torch
    import paper_2609_14306_b200 as vp
    from synth_inputs import IGNORE_INDEX, make_hidden, make_weights, stream_labels
    world, rank, dev = ctx.world, ctx.rank, ctx.dev
    barrier = ctx.barrier

    T_chunk = t_chunk or BENCH_T_CHUNK.get(w.name, w.T_chunk)
    T_chunk = min(T_chunk, -(-w.T // 128) * 128)
    chunks_per_call = -(-w.T // T_chunk)

    # ---- inputs (host, seeded) -> device.  Each rank of a multi-GPU run draws its own batch stream.
    tf32 = dtype == "tf32"
    if tf32:
        from synth_inputs import make_hidden_f32, make_weights_f32
        make_w, make_h = make_weights_f32, make_hidden_f32
        to_dev = lambda a: torch.from_numpy(a).to(dev)
        fwd, bwd, ws_fn = vp.vp_ce_forward_f32, vp.vp_ce_backward_f32, vp.vp_ce_workspace_bytes_f32
    else:
        make_w, make_h = make_weights, make_hidden
        to_dev = lambda bits: torch.from_numpy(bits.view(np.int16)).to(dev).view(torch.bfloat16)
        fwd, bwd, ws_fn = vp.vp_ce_forward, vp.vp_ce_backward, vp.vp_ce_workspace_bytes
    W_bits = make_w(w)
    labels_all = stream_labels(w)
    Wd = to_dev(W_bits)
    if not with_cpu_baseline:
        W_bits = None
    H_host0 = make_h(w, 0) if rank == 0 else None
    Hs, labs = [], []
    for call in range(w.n_calls):
        hb = H_host0 if (call == 0 and rank == 0) else make_h(rank_workload(w, rank), call)
        Hs.append(to_dev(hb))
        labs.append(torch.from_numpy(labels_all[call * w.T:(call + 1) * w.T].copy()).to(dev))
    if not with_cpu_baseline:
        H_host0 = None
    n_valid_total = int((labels_all != IGNORE_INDEX).sum())

    torch.cuda.synchronize()
    resident = torch.cuda.memory_allocated(dev)
    torch.cuda.reset_peak_memory_stats(dev)
    ws_bytes = ws_fn(T_chunk, w.d, w.block_v)
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device=dev)
    loss = [torch.empty(w.T, dtype=torch.float32, device=dev) for _ in range(w.n_calls)]
    lse = [torch.empty(w.T, dtype=torch.float32, device=dev) for _ in range(w.n_calls)]
    dH = [torch.empty(w.T, w.d, dtype=torch.float32 if tf32 else torch.bfloat16, device=dev) for _ in range(w.n_calls)]
    dW = torch.empty(w.V, w.d, dtype=torch.float32, device=dev)
    mean = torch.zeros(1, dtype=torch.float32, device=dev)
    nval = torch.zeros(1, dtype=torch.int32, device=dev)
    dl_stream = None
    if w.n_calls > 1:       # streamed context: the caller supplies 1 / n_valid of the whole stream
        dl_stream = [torch.where(l != IGNORE_INDEX, 1.0 / n_valid_total, 0.0).float() for l in labs]

    step_no = [0]
    fwd_status = [0]

    def step(check_forward_status=False):
        # every step plays another ring rank: the shard order is rotated by the global chunk index
        step_no[0] += 1
        for call in range(w.n_calls):
            base = (call + step_no[0]) * chunks_per_call
            fwd(Hs[call], Wd, labs[call], w.block_v, IGNORE_INDEX, loss[call], lse[call], T_chunk, base, ws)
            if check_forward_status:      # warm-up only: the backward clears the word, so read it in between
                fwd_status[0] |= vp.vp_ce_device_status(ws)
            bwd(Hs[call], Wd, labs[call], lse[call], None if dl_stream is None else dl_stream[call],
                dH[call], dW, w.block_v, IGNORE_INDEX, T_chunk, base, call > 0, ws)
            vp.vp_ce_mean_loss(loss[call], labs[call], w.V, IGNORE_INDEX, mean, nval)

    for i in range(warmup):
        step(check_forward_status=(i == 0))
    barrier()
    assert fwd_status[0] == 0, "device status word set by a forward during warm-up"
    assert vp.vp_ce_device_status(ws) == 0, "device status word set by a backward during warm-up"

    sampler = ClockSampler(ctx.local_rank)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    launches0 = vp.vp_ce_launch_count()
    vp.vp_ce_profile_enable(prof_on)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record()
    for _ in range(steps):
        step()
    e1.record()
    barrier()
    vp.vp_ce_profile_enable(False)
    ms_total = e0.elapsed_time(e1)
    prof = vp.vp_ce_profile_collect() if prof_on else None
    launches = vp.vp_ce_launch_count() - launches0
    clocks = sampler.stop() if rank == 0 else None
    ms_total = max_over_ranks(ms_total, dev)
    ms_step = ms_total / steps
    peak_extra = torch.cuda.max_memory_allocated(dev) - resident
    mean_loss = float(mean.item())
    status = vp.vp_ce_device_status(ws)

    # ---- un-profiled control run (same K) so the event overhead of the profiled region is visible
    ms_step_noprof = None
    if prof_on:
        barrier(); e0.record()
        for _ in range(steps):
            step()
        e1.record(); barrier()
        ms_step_noprof = e0.elapsed_time(e1) / steps

    # ---- end to end through the host-buffer entry point
    e2e = None
    if with_e2e and w.n_calls == 1 and not tf32:
        Hh = torch.empty(w.T, w.d, dtype=torch.bfloat16).pin_memory()
        Hh.copy_(Hs[0].cpu())
        lh = labs[0].cpu().pin_memory()
        loss_h = torch.empty(w.T, dtype=torch.float32).pin_memory()
        dH_h = torch.empty(w.T, w.d, dtype=torch.bfloat16).pin_memory()
        H_stage = torch.empty_like(Hs[0]); lab_stage = torch.empty_like(labs[0])
        def e2e_step():
            vp.vp_ce_fwd_bwd_host(Hh, lh, Wd, loss_h, dH_h, dW, w.block_v, IGNORE_INDEX, T_chunk, 0, False,
                                  H_stage, lab_stage, loss[0], lse[0], dH[0], ws)
        for _ in range(3):
            e2e_step()
        barrier(); e0.record()
        for _ in range(steps):
            e2e_step()
        e1.record(); barrier()
        ms_serial = max_over_ranks(e0.elapsed_time(e1), dev) / steps
        serial_status = vp.vp_ce_device_status(ws)
        mean_serial = float(loss_h[lh != IGNORE_INDEX].double().mean())
        # the same steps through HostStepPipeline: two sets of staging buffers and two copy streams, so that the copies of
        # one step overlap the compute of its neighbours (every step still copies its inputs in and its results out)
        pipe = vp.HostStepPipeline(Wd, dW, w.T, w.d, w.block_v, T_chunk, IGNORE_INDEX, depth=2)
        outs = [(loss_h, dH_h), (torch.empty_like(loss_h).pin_memory(), torch.empty_like(dH_h).pin_memory())]
        for i in range(3):
            pipe.submit(Hh, lh, *outs[i % 2])
        pipe.wait()
        barrier(); e0.record()
        for i in range(steps):
            pipe.submit(Hh, lh, *outs[i % 2])
        pipe.wait()
        e1.record(); barrier()
        ms_e2e = max_over_ranks(e0.elapsed_time(e1), dev) / steps
        e2e = {"value": whole_job_tokens_per_s(world, w.T_stream, ms_e2e), "unit": "tokens/s", "ms_per_step": ms_e2e,
               "h2d_bytes_per_step": w.T * w.d * 2 + w.T * 4, "d2h_bytes_per_step": w.T * 4 + w.T * w.d * 2,
               "api": "HostStepPipeline.submit (pinned host H, labels in; loss, dH out every step; W and dW resident; the "
                      "copies of a step run on side streams beside the neighbouring steps' compute)",
               "mean_loss_host": float(outs[(steps - 1) % 2][0][lh != IGNORE_INDEX].double().mean()),
               "device_status": pipe.device_status(),
               "serial": {"value": whole_job_tokens_per_s(world, w.T_stream, ms_serial), "ms_per_step": ms_serial,
                          "api": "vp_ce_fwd_bwd_host (copy in, compute, copy out, synchronise)",
                          "mean_loss_host": mean_serial, "device_status": serial_status}}
        del Hh, loss_h, dH_h, H_stage, pipe, outs

    if rank != 0:
        return None

    peaks, peak_src = load_peaks()
    if tf32:
        # no TF32 peak is measured on this machine: the measured bf16 peaks times the nominal dense ratio (1.1 / 2.25 PFLOP/s)
        ratio = 1100.0 / NOMINAL_BF16_TFLOPS
        peaks = dict(peaks, bf16_tflops=peaks["bf16_tflops"] * ratio,
                     bf16_tflops_sustained=peaks["bf16_tflops_sustained"] * ratio)
        peak_src += " bf16 peak x nominal tf32/bf16 ratio 0.489"
    tokens = w.T_stream
    value = whole_job_tokens_per_s(world, tokens, ms_step)
    tflops = w.flops / (ms_step / 1e3) / 1e12
    out = {
        "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": world, "steps": steps,
        "warmup": warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": dtype, "data": "synthetic",
        "config": {"workload": w.name, "T": w.T, "calls_per_step": w.n_calls, "d": w.d, "V": w.V,
                   "block_v": w.block_v, "T_chunk": T_chunk, "P": w.P, "ignored_labels": w.n_ignored,
                   "parallelism": "replicas only" if world > 1 else "single GPU",
                   "l2": "inputs larger than L2 (W alone is %.2f GB); no flush" % (w.V * w.d * (4 if tf32 else 2) / 1e9)},
        "tflops_per_gpu": tflops,
        "frac_of_bf16_peak": {"burst_measured": tflops / peaks["bf16_tflops"],
                              "sustained_measured": tflops / peaks["bf16_tflops_sustained"],
                              "nominal_2250": tflops / (1100.0 if tf32 else NOMINAL_BF16_TFLOPS), "source": peak_src},
        "flops_per_step": w.flops,
        "peak_bytes": {"workspace_bytes": ws_bytes, "increment_over_resident_inputs": int(peak_extra),
                       "outputs_bytes": int(w.T_stream * 8 + w.T_stream * w.d * (4 if tf32 else 2) + w.V * w.d * 4),
                       "full_fp32_logits_bytes": w.logits_bytes_fp32,
                       "dense_fwd_bwd_would_hold_bytes": 3 * w.logits_bytes_fp32},
        "mean_loss": mean_loss, "device_status": status,
        "gpu_launches": int(launches),
        "clocks": clocks,
    }
    if ms_step_noprof is not None:
        out["ms_per_step_without_kernel_events"] = ms_step_noprof
    if prof:
        # every kernel kind performs 2*T*V*d flops per step; the dominant one is the slowest in total
        flops_kind = 2.0 * w.T_stream * w.V * w.d * steps
        kinds = {}
        for k, (ms, n) in prof.items():
            if n:
                kinds[k] = {"launches": n, "total_ms": ms, "avg_ms": ms / n,
                            "tflops": flops_kind / (ms / 1e3) / 1e12}
        dom = max(kinds, key=lambda k: kinds[k]["total_ms"])
        ach = kinds[dom]["tflops"]
        traffic = NCU_DRAM_BYTES_PER_LAUNCH.get((dtype, w.d, w.block_v, T_chunk), {})
        # the kernel is timed inside a step loop that runs for about a second under the power cap, so the denominator is
        # the SUSTAINED cuBLAS figure; the burst figure is printed beside it
        out["roofline"] = {"bound": "tensor", "kernel": dom, "achieved": ach, "peak": peaks["bf16_tflops_sustained"],
                           "unit": "TFLOP/s", "frac": ach / peaks["bf16_tflops_sustained"],
                           "peak_kind": "bf16_tflops_sustained (kernel timed inside a long, power-capped step), of " + peak_src,
                           "frac_of_burst": ach / peaks["bf16_tflops"], "burst_peak": peaks["bf16_tflops"],
                           "flops_per_launch": flops_kind / kinds[dom]["launches"],
                           "avg_launch_ms": kinds[dom]["avg_ms"],
                           "traffic": traffic.get(dom),
                           "traffic_unit": "bytes of DRAM per launch (ncu capture of a launch of this geometry)"}
        out["kernels"] = kinds
    if e2e:
        out["e2e"] = e2e
    del ws, loss, lse, dH, dW, Hs
    torch.cuda.empty_cache()
    if with_yardstick and world == 1 and not tf32:
        out["cublas_yardstick"] = cublas_yardstick(w, T_chunk, dev)
    if with_cpu_baseline and world == 1 and not tf32:
        cb, _, _ = oracle_sample_rate(w, W_bits, H_host0, labels_all[:w.T])
        out["cpu_baseline"] = cb
    return out


def link_peaks(dev, nbytes=1 << 30):
    """Measured pinned-memory copy bandwidth of the host link, GB/s: each direction alone and both at once
    (plain cudaMemcpyAsync through torch, best of 3).  The yard-stick the streamed optimizer is measured against."""
    import torch
    h_in = torch.empty(nbytes, dtype=torch.uint8).pin_memory()
    h_out = torch.empty(nbytes, dtype=torch.uint8).pin_memory()
    d_in = torch.empty(nbytes, dtype=torch.uint8, device=dev)
    d_out = torch.empty(nbytes, dtype=torch.uint8, device=dev)
    s1, s2 = torch.cuda.Stream(dev), torch.cuda.Stream(dev)

    def run(h2d, d2h):
        best = 1e30
        for _ in range(3):
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            if h2d:
                with torch.cuda.stream(s1):
                    d_in.copy_(h_in, non_blocking=True)
            if d2h:
                with torch.cuda.stream(s2):
                    h_out.copy_(d_out, non_blocking=True)
            torch.cuda.synchronize()
            best = min(best, time.perf_counter() - t0)
        return nbytes / best / 1e9
    return {"h2d_alone": run(True, False), "d2h_alone": run(False, True), "each_direction_when_both_run": run(True, True)}


def measure_adamw(ctx, n_params, bucket, slots, steps, warmup):
    """OffloadStreamAdamW (the paper's other named GPU kernel): one optimizer step over `n_params` parameters whose fp32
    master weights, moments and gradients live in pinned HOST memory, streamed through `slots` device slots of `bucket`
    parameters.  Bound by the host link: 16 bytes in and 12 bytes out per parameter."""
    import torch
    import paper_2609_14306_b200 as vp
    dev = ctx.dev
    hp = dict(lr=1e-3, beta1=0.9, beta2=0.95, eps=1e-8, weight_decay=0.1)
    g = torch.Generator().manual_seed(7)
    host = [torch.empty(n_params, dtype=torch.float32).pin_memory() for _ in range(4)]      # master, m, v, grad
    chunk = 1 << 24
    for a in range(0, n_params, chunk):                                                     # seeded, synthetic state
        b = min(n_params, a + chunk)
        host[0][a:b] = torch.randn(b - a, generator=g) * 0.02
        host[1][a:b] = torch.randn(b - a, generator=g) * 1e-3
        host[2][a:b] = torch.randn(b - a, generator=g).square_() * 1e-6
        host[3][a:b] = torch.randn(b - a, generator=g) * 1e-2
    sample = [h[: 1 << 22].clone() for h in host]                                           # the CPU leg's inputs (before any step)
    w = torch.empty(n_params, dtype=torch.bfloat16, device=dev)
    staging = torch.empty(vp.osadamw_staging_bytes(bucket, slots), dtype=torch.uint8, device=dev)
    h = vp.osadamw_create(bucket, slots, staging)
    sampler = ClockSampler(ctx.local_rank)
    try:
        t = 0
        for _ in range(warmup):
            t += 1
            vp.osadamw_step(h, *host, w, step=t, **hp)
        vp.osadamw_wait(h)
        sampler.start()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        for _ in range(steps):
            t += 1
            vp.osadamw_step(h, *host, w, step=t, **hp)
        vp.osadamw_wait(h)                       # the host state is complete: this is the end of an optimizer step
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / steps
    finally:
        vp.osadamw_destroy(h)
    clocks = sampler.stop()
    # the update kernel alone on device-resident state (what the pipeline hides behind the copies)
    nk = min(n_params, 1 << 26)
    dstate = [torch.randn(nk, device=dev) * 1e-2 for _ in range(4)]
    dstate[2].square_()
    for _ in range(3):
        vp.osadamw_update_device(*dstate, w[:nk], step=1, **hp)
    torch.cuda.synchronize()
    e0.record()
    for i in range(10):
        vp.osadamw_update_device(*dstate, w[:nk], step=2 + i, **hp)
    e1.record()
    torch.cuda.synchronize()
    k_ms = e0.elapsed_time(e1) / 10
    del dstate, staging, w
    torch.cuda.empty_cache()
    link = link_peaks(dev)
    peaks, peak_src = load_peaks()
    in_gbs = 16.0 * n_params / (ms / 1e3) / 1e9
    # the step cannot be shorter than the larger of: its bytes in over the host-to-device rate, its bytes out over the
    # device-to-host rate, and all its bytes over what the link carries when both directions run
    floor_ms = 1e3 * max(16.0 * n_params / (link["h2d_alone"] * 1e9), 12.0 * n_params / (link["d2h_alone"] * 1e9),
                         28.0 * n_params / (2.0 * link["each_direction_when_both_run"] * 1e9))
    # the oracle as it stands on a bounded sample (float64, one pass over 4 Mi parameters)
    from oracle import adamw_oracle as ao
    t0 = time.perf_counter()
    ao.adamw_step(*(x.numpy() for x in sample), 1, **hp)
    cpu_dt = time.perf_counter() - t0
    return {
        "metric": "OffloadStreamAdamW optimizer step, parameters/s (host-resident fp32 state)", "value": n_params / (ms / 1e3),
        "unit": "parameters/s", "ms_per_step": ms, "steps": steps, "warmup": warmup, "dtype": "f32", "data": "synthetic",
        "higher_is_better": True,
        "config": {"workload": "osadamw", "parameters": n_params, "bucket_params": bucket, "slots": slots,
                   "buckets": -(-n_params // bucket), "staging_bytes": vp.osadamw_staging_bytes(bucket, slots),
                   "host_memory": "pinned", "bytes_in_per_param": 16, "bytes_out_per_param": 12},
        "roofline": {"bound": "host-link", "achieved": in_gbs, "peak": 16.0 * n_params / (floor_ms / 1e3) / 1e9, "unit": "GB/s",
                     "frac": floor_ms / ms, "floor_ms": floor_ms,
                     "peak_kind": "host-to-device GB/s at the shortest possible step: max(bytes in / h2d rate, bytes out / d2h "
                                  "rate, all bytes / both-direction rate), pinned cudaMemcpyAsync rates measured in this process "
                                  "(no such figure is in the measured-peaks file)",
                     "traffic": None, "link_gbs": link, "out_gbs": 12.0 * n_params / (ms / 1e3) / 1e9},
        "update_kernel": {"parameters": nk, "ms": k_ms, "gbs": 30.0 * nk / (k_ms / 1e3) / 1e9,
                          "hbm_peak_gbs": peaks["hbm_gbs"], "frac_of_hbm_peak": 30.0 * nk / (k_ms / 1e3) / 1e9 / peaks["hbm_gbs"],
                          "bytes_per_param": 30, "peak_source": peak_src},
        "cpu_baseline": {"value": sample[0].numel() / cpu_dt, "unit": "parameters/s", "cores": os.cpu_count(), "kind": "oracle",
                         "sample": f"float64 AdamW step over the first {sample[0].numel()} parameters, {cpu_dt:.2f} s wall clock"},
        "clocks": clocks,
    }


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="moe120b")
    ap.add_argument("--t-chunk", type=int, default=0)
    ap.add_argument("--shape", default="", help="custom workload T,d,V,block_v (Gaussian inputs, Zipf labels); "
                                                "for kernel experiments, not a benchmark config")
    ap.add_argument("--dtype", default="bf16", choices=["bf16", "tf32"],
                    help="bf16 inputs (the benchmark's metric) or float32 inputs on TF32 tensor cores (the paper's precision)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-also", action="store_true",
                    help="skip the extra measured blocks (the other target configuration, the paper's shape in TF32)")
    ap.add_argument("--no-yardstick", action="store_true", help="skip the cuBLAS context measurement")
    ap.add_argument("--profile-in-timed-region", type=int, default=1)
    ap.add_argument("--tail-parts", type=int, default=-1,
                    help="A/B knob of the gradient GEMMs' K-split tail (vp_ce_set_tail_parts): -1 library's choice, 0 off")
    ap.add_argument("--adamw", default="", help="measure only the streamed AdamW: parameters,bucket,slots (e.g. 268435456,100000000,2)")
    args = ap.parse_args()

    from synth_inputs import PROFILE_WORKLOADS, WORKLOADS
    if args.shape:
        from synth_inputs import custom_workload
        T_, d_, V_, bv_ = (int(x) for x in args.shape.split(","))
        w = custom_workload("custom", T=T_, d=d_, V=V_, block_v=bv_, T_chunk=args.t_chunk or T_, w_std=0.02,
                            labels="zipf", ignore_frac=0.05, seed=99)
        args.workload = "custom"
    else:
        w = WORKLOADS.get(args.workload) or PROFILE_WORKLOADS[args.workload]
    if args.impl == "reference":
        run_reference(args, w)
        return
    if args.warmup < 3:
        args.warmup = 3

    import paper_2609_14306_b200 as vp
    ctx = Ctx()
    vp.load_library()          # raises if the CUDA library is missing: there is no fallback
    if args.tail_parts != -1:
        vp.vp_ce_set_tail_parts(args.tail_parts)

    if args.adamw:
        n_, b_, s_ = (int(x) for x in args.adamw.split(","))
        if ctx.rank == 0:
            print(json.dumps(measure_adamw(ctx, n_, b_, s_, max(1, args.steps), args.warmup)), flush=True)
        ctx.close()
        return
    prof_on = bool(args.profile_in_timed_region)
    out = measure(ctx, w, args.dtype, args.steps, args.warmup, t_chunk=args.t_chunk, with_e2e=not args.no_e2e,
                  with_cpu_baseline=not args.no_cpu_baseline, with_yardstick=not args.no_yardstick, prof_on=prof_on)
    # The default run also measures, in the same process and through the same code, the OTHER configuration the
    # throughput target is stated on (config 4), the long-context stream (config 5: 64 calls per step, same workspace as
    # config 3), the paper's own benchmark shape in the paper's precision (FP32 inputs on TF32 tensor cores) and the
    # streamed AdamW: fewer steps, no CPU leg.  One GPU only, so that a scaling run stays short.
    if ctx.rank == 0 and ctx.world == 1 and not args.no_also and args.workload == "moe120b" and args.dtype == "bf16":
        k = max(3, min(args.steps, 5))
        out["also"] = [
            measure(ctx, WORKLOADS["moe667b"], "bf16", k, 3, with_e2e=not args.no_e2e, with_cpu_baseline=False,
                    with_yardstick=not args.no_yardstick, prof_on=prof_on),
            measure(ctx, WORKLOADS["longctx"], "bf16", 2, 3, with_e2e=False, with_cpu_baseline=False, prof_on=prof_on),
            measure(ctx, PROFILE_WORKLOADS["papershape"], "tf32", 3, 3, with_e2e=False, with_cpu_baseline=False,
                    prof_on=prof_on),
            measure_adamw(ctx, n_params=1 << 28, bucket=1 << 25, slots=2, steps=3, warmup=2),
        ]
    if ctx.rank == 0:
        print(json.dumps(out), flush=True)
    ctx.close()


if __name__ == "__main__":
    main()
