#!/usr/bin/env python
"""Benchmark of the bidirectional VDA forward pass (one "step" = one whole forward over one synthetic clip).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload 768p] [--impl ours|reference]

N > 1 runs N independent replicas of the workload, one process per GPU -- the layer needs no exchange
between GPUs -- and reports the aggregate tokens/s over the slowest rank's time.  Started as a plain
`python bench.py --gpus N` it launches its own N ranks through torch.distributed.run (rendezvous on
127.0.0.1); started under torch.distributed.run (RANK / WORLD_SIZE in the environment) it is one of the
ranks.  NCCL carries the barrier and two scalar reductions, nothing else.  Rank 0 prints ONE JSON line.
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
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "vda_fwd_tokens_per_s"
UNIT = "tokens/s"
PAPER_CONTEXT = ("paper (context only, whole pipeline on 8xB200): 6.70 s DiT denoising for a 14.3 s 768p clip, "
                 "14.5x over 50-step dense H3, attention >85% of dense denoiser runtime")


# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) per token-head from the ncu captures summarised
# under profiles/ (a 20-frame case of the 768p recipe; traffic grows in proportion to the token-heads a launch
# processes, so it is scaled to the benchmarked workload by that count).
DRAM_BYTES_PER_TOKEN_HEAD = {"gram_tc": 547.5, "readout_tc": 514.4}


# ------------------------------------------------------------------------------------------ helpers
def algorithmic_bytes(w) -> dict:
    """Bytes the method must move per forward: read q, k, v and beta once, write out once."""
    es = 4 if w.dtype == "f32" else 2
    tokh = w.B * w.T * w.F * w.H
    return {
        "gram": tokh * (2 * w.d * es + 4),          # k, v, beta
        "readout": tokh * (2 * w.d * es),           # q in, out out
        "total": tokh * (4 * w.d * es + 4),
    }


def implementation_bytes(w) -> dict:
    """Bytes of the per-frame d x d intermediates that the tensor-core kernels move through HBM/L2 on top of
    the algorithmic bytes, as the kernels are written (each array counted once per pass that streams it):
    statistics fp32 [2d][d] written by the Gram kernel, the A half read by the resolve, the B half read by both
    scans; the inverse as three bf16 parts written once and read by both scans; the two read states (bf16)
    written by the scans and read by the read-out."""
    n = w.B * w.H * w.T
    dd = w.d * w.d
    stats = n * dd * 4 * (2 + 1 + 2)
    inverse = n * dd * 2 * 3 * (1 + 2)
    states = n * dd * 2 * (2 + 2)
    return {"statistics": stats, "inverse_split": inverse, "read_states": states, "total": stats + inverse + states}


def algorithmic_flops(w) -> dict:
    tokh = w.B * w.T * w.F * w.H
    n = w.B * w.H * w.T
    return {"tensor": 6 * tokh * w.d * w.d, "fp32": 6 * n * w.d ** 3}


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            m = json.load(f)
        return {"hbm_gbs": float(m["hbm_gbs"]), "bf16_tflops": float(m["bf16_tflops"]),
                "bf16_tflops_sustained": float(m.get("bf16_tflops_sustained", m["bf16_tflops"])), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int, period_ms: int = 50):
        self.gpu = gpu_index
        self.rows = []
        self.proc = None
        self.period = period_ms

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", str(self.period)],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        threading.Thread(target=self._read, daemon=True).start()

    def _read(self):
        for line in self.proc.stdout:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 9:
                continue
            try:
                if int(parts[0]) != self.gpu:
                    continue
                self.rows.append((time.time(), float(parts[1]), float(parts[2]), parts[5:9]))
            except ValueError:
                continue

    def stop(self):
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except Exception:
                self.proc.kill()

    def summary(self, t0: float, t1: float) -> dict:
        rows = [r for r in self.rows if t0 <= r[0] <= t1 + self.period / 1000.0]
        where = "timed region"
        if not rows:
            rows, where = self.rows, "whole run (timed region shorter than the sampling period)"
        if not rows:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0, "window": "nvidia-smi unavailable"}
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = sorted({names[i] for r in rows for i in range(4) if r[3][i].lower() == "active"})
        return {"sm_mhz": statistics.median(r[1] for r in rows), "sm_max_mhz": max(r[2] for r in rows),
                "reasons": reasons, "samples": len(rows), "window": where}


def physical_gpu_index(local: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local])
        except (ValueError, IndexError):
            return local
    return local


def aggregate_over_ranks(ms_local: float, units_local: int, world: int):
    """Whole-job rate: all ranks' units over the slowest rank's time.  Returns (ms_max, units_total)."""
    if world == 1:
        return ms_local, units_local
    import torch
    import torch.distributed as dist
    dev = "cuda" if dist.get_backend() == "nccl" else "cpu"
    t = torch.tensor([ms_local], dtype=torch.float64, device=dev)
    u = torch.tensor([units_local], dtype=torch.int64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), int(u.item())


# ------------------------------------------------------------------------------------------ CPU baseline
def oracle_sample(w, heads: int, frames: int):
    """A bounded sample of the workload for the CPU oracle: `heads` head slices of batch 0, the first
    `frames` frames of each (every frame costs the same: F tokens, one d x d solve per direction)."""
    from paper_2609_20744_b200 import inputs
    ws = w.scaled(B=1, H=heads, T=frames)
    x = inputs.generate(ws, "cpu")
    return ws, [inputs.head_slice(x, 0, h) for h in range(heads)]


def time_oracle(slices) -> float:
    """Seconds for the oracle, as it stands, over the sampled head slices."""
    from oracle import vda_oracle
    t0 = time.perf_counter()
    for (q, k, v, beta, gate) in slices:
        vda_oracle.vda_slice(q, k, v, beta, gate, 1e-6)
    return time.perf_counter() - t0


def blas_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info() if p.get("user_api") == "blas"]
        if n:
            return int(max(n))
    except Exception:
        pass
    return os.cpu_count() or 1


def plan_sample(w, seconds_per_step: float):
    """Choose (heads, frames) so that one oracle pass costs about `seconds_per_step` on this host."""
    probe_T = min(w.T, 4)
    _, sl = oracle_sample(w, 1, probe_T)
    time_oracle(sl)                                       # page in numpy / BLAS
    per_frame = time_oracle(sl) / probe_T                 # seconds per (head, frame)
    per_head = per_frame * w.T
    if per_head <= seconds_per_step:                      # at most 8 slices: drawing them on the CPU costs time too
        return max(1, min(w.B * w.H, 8, int(seconds_per_step / per_head))), w.T
    return 1, max(2, min(w.T, int(seconds_per_step / per_frame)))


def sample_text(w, heads, frames):
    return (f"{heads} of {w.B * w.H} (batch, head) slices x {frames} of {w.T} frames x {w.F} tokens per step; "
            f"rate scaled by {w.B * w.H * w.T}/{heads * frames} (slices and frames are independent, equal-cost units)")


def cpu_baseline(w, seconds: float = 15.0) -> dict:
    heads, frames = plan_sample(w, seconds)
    _, slices = oracle_sample(w, heads, frames)
    sec = time_oracle(slices)
    full = sec * (w.B * w.H * w.T) / (heads * frames)
    return {"value": w.tokens / full, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
            "sample": sample_text(w, heads, frames), "seconds_sample": sec}


# ------------------------------------------------------------------------------------------ arms
def layer_config(w, n_gpus: int, win: dict) -> dict:
    """The `config` object of a bench line.  Both arms build it here, from the workload and the command line
    alone, so that the two lines of one comparison carry the same object; what is specific to an arm (which
    kernels ran, where the oracle ran) sits beside it under `arm`."""
    big = algorithmic_bytes(w)["total"] > 1e9
    return {"workload": w.name, "B": w.B, "T": w.T, "F": w.F, "H": w.H, "d": w.d, "io_dtype": w.dtype,
            "seed": w.seed, "parallelism": "single GPU" if n_gpus == 1 else f"{n_gpus} independent replicas",
            "l2": "inputs+outputs far larger than the 126 MB L2; no flush" if big
                  else "inputs smaller than L2: numbers are L2-warm",
            "window": win}


def run_reference(args, w, rank: int, world: int):
    """The reference arm is the fp64 oracle on the host cores (rank 0 only).  Every step runs the oracle over a
    bounded sample of the workload; `value` scales the sample's rate to the whole workload (units are independent
    and equal-cost), `ms_per_step` is the time a sampled step really took, and the extrapolated time of a whole
    forward is given beside it under its own key."""
    if rank != 0:
        return
    seconds_total = 60.0                                  # for the whole --steps/--warmup run
    heads, frames = plan_sample(w, seconds_total / max(1, args.steps + args.warmup))
    _, slices = oracle_sample(w, heads, frames)
    for _ in range(args.warmup):
        time_oracle(slices)
    sec = sum(time_oracle(slices) for _ in range(args.steps)) / max(1, args.steps)
    full_ms = sec * (w.B * w.H * w.T) / (heads * frames) * 1e3
    value = w.tokens / (full_ms / 1e3)
    win = dict(chunk=args.chunk, radius=args.radius, anchors=bool(args.anchors))
    cfg = layer_config(w, args.gpus, win)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": cfg, "arm": "fp64 CPU oracle (numpy on BLAS threads) on rank 0's host cores",
        "ms_per_step_is": "measured time of one sampled step (see cpu_baseline.sample)",
        "ms_per_forward_extrapolated": full_ms,
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
                         "sample": sample_text(w, heads, frames)},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def run_ours(args, w, rank: int, local_rank: int, world: int):
    import torch
    from paper_2609_20744_b200 import binding, build, inputs

    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; the VDA library has no CPU fallback")
    if rank == 0:
        build.build()
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
    torch.cuda.set_device(local_rank)
    dev = f"cuda:{local_rank}"
    x = inputs.generate(w, dev)
    flags = {"auto": 0, "frames": binding.VDN_FLAG_SCAN_FRAMEWISE, "chunks": binding.VDN_FLAG_SCAN_CHUNKWISE}[args.scan]
    if args.exact_stats:
        flags |= binding.VDN_FLAG_EXACT_STATS
    if args.fp32_resolve:
        flags |= binding.VDN_FLAG_FP32_RESOLVE
    vda = binding.Vda(w.d, w.dtype, device=local_rank, flags=flags)
    out = torch.empty_like(x["q"])
    stream = torch.cuda.current_stream()
    # the headline configuration is the plain entry point; --chunk/--radius/--anchors time the windowed gather
    win = dict(chunk=args.chunk, radius=args.radius, anchors=bool(args.anchors))

    fw = dict(win)
    if args.q_l2_eps > 0:
        # time the read-out that L2-normalises the queries itself; the generated queries have unit norm already,
        # so the result (and the parity check below) moves by eps only
        fw["q_l2_eps"] = args.q_l2_eps

    def step():
        vda.forward(x["q"], x["k"], x["v"], x["beta"], x["gate"], out=out, **fw)

    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()
    vda.profile(True)                    # per-kernel CUDA events on the launch stream, sums cleared here

    sampler = ClockSampler(physical_gpu_index(local_rank))
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    marks = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]     # per-step times (median, min)
    kt = {}
    t_wall0 = time.time()
    ev0.record(stream)
    marks[0].record(stream)
    for i in range(args.steps):
        step()
        marks[i + 1].record(stream)
    ev1.record(stream)
    torch.cuda.synchronize()
    t_wall1 = time.time()
    if world > 1:
        dist.barrier()
    ms_local = ev0.elapsed_time(ev1) / args.steps
    per_step = [marks[i].elapsed_time(marks[i + 1]) for i in range(args.steps)]
    for name, ms, _n in vda.kernel_times():
        kt[name] = ms                    # per-launch means over the timed region
    vda.profile(False)
    launches = vda.launch_count() * args.steps
    if vda.status() != binding.VDN_OK:
        raise SystemExit("bench.py: device-side status word reports an error")
    clocks = sampler.summary(t_wall0, t_wall1) if rank == 0 else None

    ms_max, tokens_total = aggregate_over_ranks(ms_local, w.tokens, world)
    value = tokens_total / (ms_max / 1e3)

    # ---- parity of this very launch configuration against the fp64 oracle, on sampled (batch, head) slices
    parity = None
    if rank == 0 and not args.skip_cpu:
        from oracle import vda_oracle
        tol = 1e-4 if w.dtype == "f32" else 2e-2
        pairs = [(0, 0), (w.B - 1, w.H - 1)]          # first, last and two seeded (batch, head) slices
        import numpy as _np
        rng = _np.random.default_rng(w.seed + 1234)
        while len(pairs) < min(4, w.B * w.H):
            pr = (int(rng.integers(w.B)), int(rng.integers(w.H)))
            if pr not in pairs:
                pairs.append(pr)
        errs, viol = [], []
        for (b, hh) in pairs:
            qs, ks, vs, bs, gs = inputs.head_slice(x, b, hh)
            ref = vda_oracle.vda_slice(qs, ks, vs, bs, gs, 1e-6, **win)["out"]
            got = out[b, :, :, hh, :].double().cpu().numpy()
            errs.append(vda_oracle.slice_error(got, ref))
            # reported, not gated: elements off by more than tol * (|ref| + rms of the slice)
            rms = float(_np.sqrt(_np.mean(ref * ref)))
            viol.append(int(_np.count_nonzero(_np.abs(got - ref) > tol * (_np.abs(ref) + rms))))
            del qs, ks, vs, ref, got
        parity = {"metric": "max over a (batch, head) slice of |gpu - oracle| / max |oracle|", "slices": pairs,
                  "errors": errs, "tolerance": tol, "ok": bool(max(errs) <= tol),
                  "elements_beyond_tol_times_abs_plus_rms": viol, "elements_per_slice": w.T * w.F * w.d}

    # ---- end to end through the host-buffer entry point (H2D + forward + D2H inside the timed region)
    e2e = None
    try:
        if args.skip_e2e:
            raise RuntimeError("skipped (--skip-e2e)")
        xh = {n: torch.empty(t.shape, dtype=t.dtype, pin_memory=True).copy_(t) for n, t in x.items()}
        outh = torch.empty(out.shape, dtype=out.dtype, pin_memory=True)
        e_steps = max(1, min(args.steps, args.e2e_steps))
        vda.forward_host(xh["q"], xh["k"], xh["v"], xh["beta"], xh["gate"], outh, **fw)
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        ev0.record(stream)
        for _ in range(e_steps):
            vda.forward_host(xh["q"], xh["k"], xh["v"], xh["beta"], xh["gate"], outh, **fw)
        ev1.record(stream)
        torch.cuda.synchronize()
        e_ms, e_tok = aggregate_over_ranks(ev0.elapsed_time(ev1) / e_steps, w.tokens, world)
        h2d = sum(xh[n].numel() * xh[n].element_size() for n in ("q", "k", "v", "beta", "gate"))
        e2e = {"value": e_tok / (e_ms / 1e3), "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": outh.numel() * outh.element_size(), "ms_per_step": e_ms, "steps": e_steps,
               "api": "vdn_vda_forward_host (pinned host buffers)" if win == dict(chunk=1, radius=0, anchors=False)
                      and not args.q_l2_eps else "vdn_vda_forward_host_opt (pinned host buffers)"}
        same = bool(torch.equal(outh, out.cpu()))
        e2e["matches_device_entry_point"] = same
        del xh, outh
    except Exception as exc:  # host memory may be too small for the pinned copies
        e2e = {"value": None, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0,
               "error": f"{type(exc).__name__}: {exc}"}

    # ---- sustained: a loop of at least two seconds after the timed region (clocks settle under load)
    sustained = None
    if args.sustain_s > 0:
        n_loop = max(20, int(args.sustain_s * 1e3 / max(ms_local, 1e-3)) + 1)
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        s_wall0 = time.time()
        ev0.record(stream)
        for _ in range(n_loop):
            step()
        ev1.record(stream)
        torch.cuda.synchronize()
        s_wall1 = time.time()
        s_ms, s_tok = aggregate_over_ranks(ev0.elapsed_time(ev1) / n_loop, w.tokens, world)
        if rank == 0:
            s_clk = sampler.summary(s_wall0, s_wall1)
            sustained = {"ms_per_step": s_ms, "value": s_tok / (s_ms / 1e3), "unit": UNIT, "steps": n_loop,
                         "seconds": s_wall1 - s_wall0, "sm_mhz_median": s_clk["sm_mhz"], "reasons": s_clk["reasons"],
                         "ms_times_sm_mhz": s_ms * s_clk["sm_mhz"] if s_clk["sm_mhz"] else None,
                         "timed_region_ms_times_sm_mhz": ms_max * clocks["sm_mhz"] if clocks and clocks["sm_mhz"] else None}

    if rank != 0:
        return
    sampler.stop()

    peaks = measured_peaks()
    ab = algorithmic_bytes(w)
    fl = algorithmic_flops(w)
    # dominant kernel by time; its algorithmic bytes
    roof = None
    if kt:
        dom = max(kt, key=kt.get)
        kind = "gram" if "gram" in dom else ("readout" if dom == "readout_tc" or dom == "readout_simt" else None)
        per_th = DRAM_BYTES_PER_TOKEN_HEAD.get(dom)
        traffic = per_th * w.B * w.T * w.F * w.H if per_th else None
        if kind is not None:
            achieved = ab[kind] / (kt[dom] / 1e3) / 1e9
            roof = {"bound": "hbm", "kernel": dom, "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                    "frac": achieved / peaks["hbm_gbs"], "traffic": traffic, "peak_source": f"of {peaks['source']}",
                    "kernel_ms": kt[dom], "algorithmic_bytes_per_launch": ab[kind]}
        else:
            # resolve / scan: 2 d^3 (Gauss-Jordan) resp. 2 x 2 d^3 (two directions) fp32-equivalent flops per frame
            work = (2 if "resolve" in dom else 4) * w.B * w.H * w.T * w.d ** 3
            if dom.endswith("_tc"):
                # on the tensor cores every fp32 product is six bf16 partial products (three-way splits of both
                # factors): the fraction is of the bf16 tensor peak, counting those; a chain of T dependent
                # frame steps per (batch, head, direction) bounds the scan long before the peak does
                achieved = 6 * work / (kt[dom] / 1e3) / 1e12
                roof = {"bound": "tensor", "kernel": dom, "achieved": achieved, "peak": peaks["bf16_tflops"],
                        "unit": "TFLOP/s", "frac": achieved / peaks["bf16_tflops"], "traffic": None,
                        "peak_source": f"of {peaks['source']} (bf16 burst); six bf16 partial products per fp32 product",
                        "kernel_ms": kt[dom], "fp32_equivalent_tflops": work / (kt[dom] / 1e3) / 1e12}
            else:
                # plain fp32 kernels: peak = SMs x 128 lanes x 2 flop x max SM clock
                import torch as _t
                prop = _t.cuda.get_device_properties(local_rank)
                peak = prop.multi_processor_count * 128 * 2 * 1.965e9 / 1e12
                achieved = work / (kt[dom] / 1e3) / 1e12
                roof = {"bound": "alu", "kernel": dom, "achieved": achieved, "peak": peak, "unit": "TFLOP/s",
                        "frac": achieved / peak, "traffic": None,
                        "peak_source": f"{prop.multi_processor_count} SMs x 128 fp32 lanes x 2 x 1.965 GHz",
                        "kernel_ms": kt[dom]}
    t_roof_ms = max(ab["total"] / (peaks["hbm_gbs"] * 1e9), fl["tensor"] / (peaks["bf16_tflops_sustained"] * 1e12)) * 1e3
    t_roof_nominal_ms = max(ab["total"] / 8e12, fl["tensor"] / 2.25e15) * 1e3

    base = cpu_baseline(w) if (world == 1 and not args.skip_cpu) else None
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_max, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16 in / f32 accumulate, f32 state" if w.dtype == "bf16" else "f32",
        "data": "synthetic",
        "config": layer_config(w, world, win),
        "arm": "tensor-core kernels" if vda.launch_count() and any("tc" in n for n in kt) else "plain-fp32 kernels",
        "clocks": clocks, "e2e": e2e, "gpu_launches": launches, "parity": parity,
        "roofline": roof,
        "ms_per_step_median": statistics.median(per_step), "ms_per_step_min": min(per_step),
        "layer_roofline": {"t_roof_ms_measured_peaks": t_roof_ms, "frac_of_measured": t_roof_ms / (ms_max / 1.0),
                           "t_roof_ms_nominal": t_roof_nominal_ms, "frac_of_nominal": t_roof_nominal_ms / ms_max,
                           "t_fp32_alu_ms": fl["fp32"] / (148 * 128 * 2 * 1.965e9) * 1e3,
                           "algorithmic_bytes": ab["total"], "tensor_flops": fl["tensor"], "fp32_flops": fl["fp32"],
                           # reported separately, as the per-frame d x d intermediates are not algorithmic bytes
                           "implementation_bytes": implementation_bytes(w) if w.d == 128 and w.dtype == "bf16" else None},
        "kernel_ms": kt, "sustained": sustained,
        "cpu_baseline": base,
        "context": PAPER_CONTEXT,
    }
    print(json.dumps(line), flush=True)


def run_prep(args, w, local_rank: int):
    """--stage prep: the feature preparation in front of the layer (Sec. 2.3), timed on the same shape.  Not part
    of the headline step; one JSON line of the same form, `roofline` against the fp32 pipe that bounds it."""
    import torch
    from paper_2609_20744_b200 import binding, build, inputs

    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; the VDA library has no CPU fallback")
    build.build()
    torch.cuda.set_device(local_rank)
    Y, X = args.grid
    if Y * X != w.F:
        raise SystemExit(f"--grid {Y}x{X} does not give F = {w.F}")
    p = inputs.generate_projected(w, f"cuda:{local_rank}")
    vda = binding.Vda(w.d, w.dtype, device=local_rank)
    outs = tuple(torch.empty_like(p[n]) for n in "qkv")
    stream = torch.cuda.current_stream()

    if args.no_spatial:                  # temporal filter + SiLU + normalisation only (the paper's VDA-Prep)
        p["wk_spatial"] = p["wv_spatial"] = None

    fused_q = args.q_l2_eps > 0          # the queries are left to the read-out

    def step():
        vda.prepare(None if fused_q else p["q"], p["k"], p["v"], p, Y, X, out=(None,) + outs[1:] if fused_q else outs)

    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()
    vda.profile(True)
    sampler = ClockSampler(physical_gpu_index(local_rank))
    sampler.start()
    time.sleep(0.3)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0 = time.time()
    ev0.record(stream)
    for _ in range(args.steps):
        step()
    ev1.record(stream)
    torch.cuda.synchronize()
    t1 = time.time()
    ms = ev0.elapsed_time(ev1) / args.steps
    kt = {n: m for n, m, _ in vda.kernel_times()}
    vda.profile(False)
    clocks = sampler.summary(t0, t1)
    sampler.stop()

    # parity of this launch on a sample the oracle can afford: one head, one output frame in the middle of the
    # clip (the oracle gets the five frames the temporal filter reaches), every token of that frame
    parity = None
    if not args.skip_cpu:
        from oracle import prep_oracle, vda_oracle
        tol = 1e-4 if w.dtype == "f32" else 2e-2
        b, h, tc = w.B - 1, w.H - 1, w.T // 2
        lo, hi = max(0, tc - 2), min(w.T, tc + 3)
        f = lambda t: t.detach().double().cpu().numpy()
        sl = slice(h * w.d, (h + 1) * w.d)
        if args.no_spatial:
            ident = torch.zeros((w.H * w.d, 5, 5)); ident[:, 2, 2] = 1.0
            p["wk_spatial"] = p["wv_spatial"] = ident
        ref = prep_oracle.prepare(f(p["q"][b, lo:hi, :, h]), f(p["k"][b, lo:hi, :, h]), f(p["v"][b, lo:hi, :, h]),
                                  f(p["wk_spatial"][sl]), f(p["wk_temporal"][sl]), f(p["wv_spatial"][sl]),
                                  f(p["wv_temporal"][sl]), Y, X)
        errs = [vda_oracle.slice_error(f(o[b, tc, :, h]), r[tc - lo])
                for o, r in list(zip(outs, ref))[1 if fused_q else 0:]]
        parity = {"metric": "max |gpu - oracle| / max |oracle| over the sampled frame, for q', k', v'",
                  "sample": f"batch {b}, head {h}, frame {tc} (needs frames {lo}..{hi - 1} of the input)",
                  "errors": errs, "tolerance": tol, "ok": bool(max(errs) <= tol)}

    es = 4 if w.dtype == "f32" else 2
    elems = w.B * w.T * w.F * w.H * w.d
    alg_bytes = (4 if fused_q else 6) * elems * es   # (q,) k, v read once and written once
    flops = 2 * elems * 2 * (5 if args.no_spatial else 30)   # K and V: (25 +) 5 fused multiply-adds per element
    prop = torch.cuda.get_device_properties(local_rank)
    alu_peak = prop.multi_processor_count * 128 * 2 * 1.965e9 / 1e12
    peaks = measured_peaks()
    dom = max(kt, key=kt.get) if kt else None
    roof = None
    if dom == "prep_kv_temporal":
        kb = 4 * elems * es                          # k and v read once and written once
        achieved = kb / (kt[dom] / 1e3) / 1e9
        roof = {"bound": "hbm", "kernel": dom, "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": achieved / peaks["hbm_gbs"], "traffic": None, "peak_source": f"of {peaks['source']}",
                "kernel_ms": kt[dom], "algorithmic_bytes_per_launch": kb}
    if dom == "prep_spatial":
        sp_flops = 2 * elems * 2 * 25                # K and V: 25 fused multiply-adds per element
        achieved = sp_flops / (kt[dom] / 1e3) / 1e12
        roof = {"bound": "alu", "kernel": dom, "achieved": achieved, "peak": alu_peak, "unit": "TFLOP/s",
                "frac": achieved / alu_peak, "traffic": None,
                "peak_source": f"{prop.multi_processor_count} SMs x 128 fp32 lanes x 2 x 1.965 GHz",
                "kernel_ms": kt[dom], "hbm_GBps_of_this_kernel": 4 * elems * es / (kt[dom] / 1e3) / 1e9}
    base = None
    if not args.skip_cpu:
        from oracle import prep_oracle
        f = lambda t: t.detach().double().cpu().numpy()
        nfr = min(w.T, 6)
        sl = slice(0, w.d)
        args_o = (f(p["q"][0, :nfr, :, 0]), f(p["k"][0, :nfr, :, 0]), f(p["v"][0, :nfr, :, 0]), f(p["wk_spatial"][sl]),
                  f(p["wk_temporal"][sl]), f(p["wv_spatial"][sl]), f(p["wv_temporal"][sl]), Y, X)
        c0 = time.perf_counter()
        prep_oracle.prepare(*args_o)
        sec = time.perf_counter() - c0
        base = {"value": w.tokens / (sec * w.B * w.H * w.T / nfr), "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
                "sample": f"1 of {w.B * w.H} (batch, head) slices x {nfr} of {w.T} frames; rate scaled by the unit count",
                "seconds_sample": sec}
    line = {
        "metric": "vda_prep_tokens_per_s", "value": w.tokens / (ms / 1e3), "unit": UNIT, "n_gpus": 1, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32 arithmetic on bf16 I/O" if w.dtype == "bf16" else "f32", "data": "synthetic",
        "config": {"workload": w.name, "stage": "prep", "B": w.B, "T": w.T, "F": w.F, "Y": Y, "X": X, "H": w.H, "d": w.d,
                   "io_dtype": w.dtype, "queries": "left to the read-out" if fused_q else "normalised here",
                   "l2": "inputs+outputs far larger than the 126 MB L2; no flush"},
        "clocks": clocks, "gpu_launches": vda.launch_count() * args.steps, "parity": parity, "roofline": roof,
        "stage_roofline": {"t_alu_ms": flops / (alu_peak * 1e12) * 1e3, "t_hbm_ms": alg_bytes / (peaks["hbm_gbs"] * 1e9) * 1e3,
                           "algorithmic_bytes": alg_bytes, "fp32_flops": flops},
        "kernel_ms": kt, "cpu_baseline": base,
        "context": "paper (context only): VDA-Prep 17.1 -> 3.4 ms on B200 at 102 latent frames (Sec. 4.3)",
    }
    print(json.dumps(line), flush=True)


def free_port() -> int:
    import socket
    with socket.socket() as so:
        so.bind(("127.0.0.1", 0))
        return so.getsockname()[1]


def launch_ranks(n: int, argv) -> int:
    """Starts n ranks of this script, one per GPU, through torch.distributed.run on 127.0.0.1 and passes their
    output through (rank 0 prints the JSON line).  Returns the launcher's exit code."""
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(free_port()), os.path.abspath(__file__), *argv]
    return subprocess.call(cmd)


def run_launcher_selftest(args, w, rank: int, world: int):
    """Every rank "measures" (10 + 5 rank) ms over the workload's tokens and the ranks aggregate as the real run
    does -- through gloo on CPU, so that the launch path can be exercised on a machine without GPUs."""
    import torch.distributed as dist
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("gloo")
    try:
        ms, tokens = aggregate_over_ranks(10.0 + 5.0 * rank, w.tokens, world)
        if world > 1:
            dist.barrier()
        if rank == 0:
            print(json.dumps({"metric": METRIC, "value": tokens / (ms / 1e3), "unit": UNIT, "n_gpus": world,
                              "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
                              "scaling": "weak", "vs_baseline": None, "dtype": "none",
                              "data": "launcher self-test: made-up times, no GPU work",
                              "config": layer_config(w, world, dict(chunk=args.chunk, radius=args.radius,
                                                                    anchors=bool(args.anchors))),
                              "gpu_launches": 0}), flush=True)
    finally:
        if world > 1:
            dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="768p")
    ap.add_argument("--e2e-steps", type=int, default=2)
    ap.add_argument("--heads", type=int, default=0, help="override H (smaller cases for profiler captures)")
    ap.add_argument("--frames", type=int, default=0, help="override T (smaller cases for profiler captures)")
    ap.add_argument("--chunk", type=int, default=1, help="frames per temporal chunk of the local window (1 = headline)")
    ap.add_argument("--radius", type=int, default=0, help="chunks on either side inside the local window")
    ap.add_argument("--anchors", type=int, default=0, help="1: first and last frame are boundary anchors")
    ap.add_argument("--scan", default="auto", choices=["auto", "frames", "chunks"],
                    help="scan schedule for chunk >= 2 (frame by frame / chunk-wise / the library's choice)")
    ap.add_argument("--stage", default="layer", choices=["layer", "prep"],
                    help="layer = the headline step; prep = the feature preparation in front of it (1 GPU)")
    ap.add_argument("--grid", type=lambda v: tuple(int(x) for x in v.split("x")), default=(48, 85),
                    help="YxX token grid of a frame for --stage prep (768p: 48x85)")
    ap.add_argument("--no-spatial", action="store_true", help="--stage prep without the 5x5 spatial filter")
    ap.add_argument("--q-l2-eps", type=float, default=0.0,
                    help="> 0: the read-out normalises the queries (vdn_vda_options.q_l2_eps); --stage prep then skips Q")
    ap.add_argument("--exact-stats", action="store_true",
                    help="VDN_FLAG_EXACT_STATS: frame statistics from the exactly weighted keys (not the headline)")
    ap.add_argument("--fp32-resolve", action="store_true",
                    help="VDN_FLAG_FP32_RESOLVE: the inverse from the plain-fp32 Gauss-Jordan kernel (not the headline)")
    ap.add_argument("--sustain-s", type=float, default=2.0,
                    help="seconds of back-to-back forwards after the timed region for the `sustained` block (0 = none)")
    ap.add_argument("--launcher-selftest", action="store_true",
                    help="no GPU work: every rank reports a made-up time through gloo on CPU; checks the self-launch "
                         "and the aggregation end to end (the line says so in `data`)")
    ap.add_argument("--skip-e2e", action="store_true", help="no host-buffer pass (profiler captures)")
    ap.add_argument("--skip-cpu", action="store_true", help="no CPU-oracle timing (profiler captures)")
    args = ap.parse_args()

    from paper_2609_20744_b200 import inputs
    w = inputs.WORKLOADS[args.workload]
    if args.heads > 0:
        w = w.scaled(H=args.heads, name=f"{w.name}_H{args.heads}")
    if args.frames > 0:
        w = w.scaled(T=args.frames, name=f"{w.name}_T{args.frames}")

    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and args.stage != "prep" and args.impl != "reference":
        # a plain `python bench.py --gpus N`: become the launcher of N ranks of this very command
        raise SystemExit(launch_ranks(args.gpus, sys.argv[1:]))

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))

    if args.launcher_selftest:
        run_launcher_selftest(args, w, rank, world)
        return
    if args.impl == "reference":
        run_reference(args, w, rank, world)
        return
    if args.stage == "prep":
        if rank == 0:
            run_prep(args, w, local_rank)
        return
    if world > 1:
        import torch
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        torch.cuda.set_device(local_rank)
        dist.init_process_group("nccl", device_id=torch.device(f"cuda:{local_rank}"))
    try:
        run_ours(args, w, rank, local_rank, world)
    finally:
        if world > 1:
            import torch.distributed as dist
            dist.destroy_process_group()


if __name__ == "__main__":
    main()
