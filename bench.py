#!/usr/bin/env python
"""Benchmark of the top-2 MoE layer on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config c4_2048e] [--impl reference]

One step = one pass of the whole layer (gating GEMM + softmax/top-2, capacity assignment, dispatch,
expert FFN, combine; the training configuration adds the backward pass) over one batch of seeded
synthetic input shaped like the paper's MoE layers.  Prints ONE JSON line for the headline
configuration (MoE(2048E) forward):
  value     tokens/s with every input resident in HBM (CUDA events, max over ranks)
  e2e       tokens/s through gshard_moe_top2_forward_host_async: x, u copied from pinned host memory
            and y, l_aux copied back inside the timed region (expert weights are model state
            and stay on the device)
  roofline  the dominant kernel (the expert FFN): algorithmic bytes or FLOPs per launch / its
            measured duration, against the measured peak of the resource that binds it (HBM copy
            bandwidth, or the bf16 tensor throughput where the FLOPs take longer than the bytes)
  sustained the same step repeated for at least two seconds, with the SM clock seen meanwhile
  configs   the same measurement, shortened, for the other full-size configurations
            (MoE(128E), MoE(512E) skewed, MoE(512E) training step), run after the headline one
  cpu_baseline  the CPU oracle timed on this machine's host cores on a bounded sample
With --impl reference only the oracle runs (rank 0), on the same configuration.
N > 1 runs N independent replicas (weak scaling); --parallelism ep shards groups and experts over
the ranks with an all-to-all before and after the expert FFN instead.
"""
from __future__ import annotations

import argparse
import glob
import json
import math
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "MoE layer tokens/sec at E=2048,M=1024,H=8192 (1 B200); % of layer roofline"
UNIT = "tokens/s"
EXTRA_CONFIGS = ("c2_128e", "c3_512e_skew", "c5_512e_train")


def profile_configs():
    """Small cases that profiler captures run on (a capture must end by itself within minutes, so it
    cannot hold a full-size layer): slices of the full-size layers with the same per-expert shapes."""
    from paper_2006_16668_b200.inputs import MoEConfig
    return {
        # 64 experts of the MoE(2048E) layer: 128 rows per expert, 2.1 GB of expert weights
        "p4_slice": MoEConfig("p4_slice", G=32, S=128, M=1024, H=8192, E=64, C=4, seed=20200636),
        # the MoE(2048E) layer with a thin expert hidden dimension: gating, capacity, dispatch and
        # combine see exactly the full sizes (131072 tokens, 2048 experts), expert weights 0.5 GB
        "p4_routing": MoEConfig("p4_routing", G=32, S=4096, M=1024, H=64, E=2048, C=4, seed=20200637),
        # 16 experts of the MoE(128E) layer (1024 rows per expert, tensor-bound expert GEMMs)
        "p2_slice": MoEConfig("p2_slice", G=16, S=512, M=1024, H=8192, E=16, C=64, seed=20200638),
        # 32 experts of the MoE(512E) training step (256 rows per expert)
        "p5_slice": MoEConfig("p5_slice", G=16, S=256, M=1024, H=8192, E=32, C=16, seed=20200639, backward=True),
    }


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


def max_over_ranks(ms: float, world: int, device) -> float:
    """Device time of the slowest rank (every rank calls this; one all-reduce when world > 1)."""
    if world <= 1:
        return float(ms)
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_throughput(tokens_per_rank: int, world: int, ms_per_step: float) -> float:
    """Whole-job tokens/s: every rank processes tokens_per_rank per step (weak scaling)."""
    return world * tokens_per_rank / (ms_per_step * 1e-3)


def ffn_work(M: int, H: int, E: int, rows_per_expert: int, esize: int):
    """Algorithmic work of the expert FFN (eq. (2) over the fixed [E, G*C, M] buffer): bytes = both
    weight matrices + dispatched inputs + expert outputs, FLOPs = two contractions per slot row."""
    R = E * rows_per_expert
    return 2 * E * M * H * esize + 2 * R * M * esize, 4.0 * R * M * H


def kernel_roofline(nbytes: float, flops: float, ms: float, peaks: dict) -> dict:
    """Roofline record of one kernel: the binding resource is the one whose floor time at the measured
    peak is longer; `achieved` and `peak` are in that resource's unit."""
    t_bytes = nbytes / (peaks["hbm_gbs"] * 1e9)
    t_flops = flops / (peaks["bf16_tflops"] * 1e12)
    if t_flops > t_bytes:
        achieved = flops / (ms * 1e-3) / 1e12
        return {"bound": "tensor", "achieved": achieved, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                "frac": achieved / peaks["bf16_tflops"],
                "frac_of_sustained_peak": achieved / peaks["bf16_tflops_sustained"]}
    achieved = nbytes / (ms * 1e-3) / 1e9
    return {"bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
            "frac": achieved / peaks["hbm_gbs"]}


def layer_work(cfg, esize: int):
    """Algorithmic FLOPs and HBM bytes of one step of the layer (what the method must do, whatever
    the kernels do): gating + expert FFN; expert weights, x, y, wg, u each moved once.  The training
    step adds the backward: four more FFN-sized contractions and three gating-sized ones, the weights
    read once more and their gradients written once, dy read and dx written."""
    _, ffn_flops = ffn_work(cfg.M, cfg.H, cfg.E, cfg.G * cfg.C, esize)
    gate_flops = 2.0 * cfg.N * cfg.M * cfg.E
    flops = gate_flops + ffn_flops
    nbytes = 2 * cfg.E * cfg.M * cfg.H * esize + 2 * cfg.N * cfg.M * esize + cfg.M * cfg.E * esize + cfg.N * 4
    if cfg.backward:
        flops = 4 * gate_flops + 3 * ffn_flops
        nbytes = 2 * nbytes + 2 * cfg.E * cfg.M * cfg.H * esize + 2 * cfg.N * cfg.M * esize
    return flops, nbytes


def load_traffic(kernel: str, M: int, H: int, rows_per_expert: int, E: int):
    """DRAM bytes per launch of `kernel` from the committed ncu capture whose per-expert shape matches
    (profiles/*.traffic.json), scaled by the expert count; None when no capture matches."""
    for path in sorted(glob.glob(os.path.join(ROOT, "profiles", "*.traffic.json"))):
        try:
            rec = json.load(open(path))
        except (OSError, ValueError):
            continue
        if rec.get("kernel") == kernel and (rec.get("M"), rec.get("H"), rec.get("rows_per_expert")) == (
                M, H, rows_per_expert):
            per_expert = (rec["dram_bytes_read"] + rec["dram_bytes_write"]) / float(rec["experts"])
            return per_expert * E
    return None


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons with one looping nvidia-smi while timed regions run."""
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        super().__init__(daemon=True)
        self.index = index
        self.samples = []
        self.times = []          # host time at which each sample arrived
        self.proc = None

    def run(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-i", str(self.index), "-lms", "50"], stdout=subprocess.PIPE, text=True)
            for line in self.proc.stdout:
                parts = [p.strip() for p in line.strip().split(",")]
                if len(parts) >= 6:
                    self.samples.append(parts)
                    self.times.append(time.time())
        except Exception:
            pass

    def wait_first_sample(self, timeout_s=5.0):
        """nvidia-smi needs up to a second to print its first line: wait for it, so that short timed
        regions are sampled too."""
        t0 = time.time()
        while not self.samples and time.time() - t0 < timeout_s and self.is_alive():
            time.sleep(0.02)

    def mark(self) -> int:
        return len(self.samples)

    def stop(self):
        if self.proc is not None:
            self.proc.terminate()          # the exact process started above
        self.join(timeout=3)

    def summary(self, start: int = 0, end=None):
        def num(v):
            try:
                return float(v)
            except ValueError:
                return None
        samples = self.samples[start:end]
        sm = [num(s[0]) for s in samples if num(s[0]) is not None]
        mx = [num(s[1]) for s in samples if num(s[1]) is not None]
        # samples taken while the GPU was busy run well above the idle clock
        busy = [v for v in sm if v > 500.0] or sm
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = [n for i, n in enumerate(names) if any(s[2 + i].lower().startswith("active") for s in samples)]
        return {"sm_mhz": statistics.median(busy) if busy else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": reasons, "samples": len(samples), "samples_under_load": len(busy)}


def oracle_sample(cfg, n_groups=16, n_rows=1200, seed_offset=0):
    """Times the CPU oracle on a bounded sample of the configuration: gating + Algorithm 1 for
    n_groups whole groups, eq. (2)-(3) for n_rows token-expert rows of those groups.  Returns
    (tokens/s of a full layer at that per-token cost, description, threads)."""
    import torch
    from oracle import gshard_oracle as orc
    from paper_2006_16668_b200.inputs import make_inputs

    n_groups = min(n_groups, cfg.G)
    small = cfg.scaled(G=n_groups, seed=cfg.seed + seed_offset)     # groups of the same S, M, E
    inp = make_inputs(small, "cpu", with_experts=False)
    x = inp["x"].float().numpy()
    wg = inp["wg"].float().numpy()
    u = inp["u"].numpy()
    # a few experts' weights drawn with the recipe's scales; rows cycle through them
    gen = torch.Generator().manual_seed(cfg.seed + 99 + seed_offset)
    experts = []
    for _ in range(4):
        wi_e = (torch.randn(cfg.M, cfg.H, generator=gen) * cfg.M ** -0.5).to(cfg.torch_dtype).float().numpy()
        wo_e = (torch.randn(cfg.H, cfg.M, generator=gen) * cfg.H ** -0.5).to(cfg.torch_dtype).float().numpy()
        experts.append((wi_e, wo_e))
    t_gate = 0.0
    kept = 0
    routings = []
    for g in range(n_groups):
        t0 = time.perf_counter()
        _, p = orc.gates(x[g], wg)
        m = orc.mean_gates(p)
        e1, e2, g1, g2, _ = orc.top2(p)
        r = orc.capacity(cfg.E, cfg.C, e1, e2, g1, g2, u[g], m)
        t_gate += time.perf_counter() - t0
        kept += int((r.slot >= 0).sum())
        routings.append(r)
    rows = 0
    t_ffn = 0.0
    s = 0
    while rows < n_rows and s < cfg.S:
        for g in range(n_groups):
            for k in range(2):
                if routings[g].slot[s, k] < 0 or rows >= n_rows:
                    continue
                wi_e, wo_e = experts[rows % len(experts)]
                t1 = time.perf_counter()
                orc.ffn_rows(x[g, s:s + 1], wi_e, wo_e)
                t_ffn += time.perf_counter() - t1
                rows += 1
        s += 1
    kept_per_token = kept / float(n_groups * cfg.S)
    per_token = t_gate / (n_groups * cfg.S) + (t_ffn / max(rows, 1)) * kept_per_token
    desc = (f"gating+Algorithm 1 for {n_groups} groups of {cfg.S} tokens ({t_gate:.2f} s) + eq.(2)-(3) for {rows} "
            f"token-expert rows ({t_ffn:.2f} s); tokens/s extrapolated at {kept_per_token:.2f} kept choices/token")
    return 1.0 / per_token, desc, orc.num_threads()


def run_reference(args, cfg):
    """The reference arm of this tier: the CPU oracle as it stands, on the host cores."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    vals = []
    desc, cores = "", 0
    for i in range(args.warmup + args.steps):
        v, desc, cores = oracle_sample(cfg, n_groups=2, n_rows=64, seed_offset=i)
        if i >= args.warmup:
            vals.append(v)
    value = statistics.mean(vals)
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * cfg.N / value,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": {"workload": cfg.name, "G": cfg.G, "S": cfg.S, "M": cfg.M, "H": cfg.H,
                                            "E": cfg.E, "C": cfg.C},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


class Bench:
    """Everything one configuration needs on the device, and the timed regions over it."""

    def __init__(self, cfg, args, flags, dev, world, rank, sampler):
        import torch
        from paper_2006_16668_b200 import binding as B
        from paper_2006_16668_b200.inputs import make_inputs
        self.torch, self.B = torch, B
        self.cfg, self.args, self.dev, self.world, self.rank, self.sampler = cfg, args, dev, world, rank, sampler
        self.peaks = load_peaks()
        self.inp = make_inputs(cfg.scaled(seed=cfg.seed + rank), dev)     # every replica draws its own batch
        self.shape = B.make_shape(cfg, flags=flags)
        self.ws = B.alloc_workspace(self.shape, host_staging=True, device=dev)
        self.y = torch.empty_like(self.inp["x"])
        self.l_aux = torch.zeros(1, dtype=torch.float32, device=dev)
        self.rt, self.rs = B.alloc_routing(self.shape, device=dev)
        self.stream = torch.cuda.current_stream()
        self.train = cfg.backward
        self.bwd_ev = None
        self.launches = 0
        if self.train:
            self.shape_t = B.make_shape(cfg, flags=flags | B.GSHARD_FLAG_SAVE_FOR_BACKWARD)
            self.ctx = torch.empty(B.gshard_moe_top2_context_bytes(self.shape_t), dtype=torch.uint8, device=dev)
            self.wsb = B.alloc_workspace(self.shape_t, for_backward=True, device=dev)
            self.dx = torch.empty_like(self.inp["x"])
            self.dwg = torch.empty(cfg.M, cfg.E, dtype=torch.float32, device=dev)
            self.dwi = torch.empty_like(self.inp["wi"])
            self.dwo = torch.empty_like(self.inp["wo"])

    def step(self):
        B, inp = self.B, self.inp
        if not self.train:
            B.gshard_moe_top2_forward(self.shape, inp["x"], inp["wg"], inp["wi"], inp["wo"], inp["u"], self.y,
                                      self.l_aux, self.rs, None, self.ws, self.stream)
            self.launches = B.gshard_moe_last_launch_count()
            return
        B.gshard_moe_top2_forward(self.shape_t, inp["x"], inp["wg"], inp["wi"], inp["wo"], inp["u"], self.y,
                                  self.l_aux, self.rs, self.ctx, self.ws, self.stream)
        fwd_launches = B.gshard_moe_last_launch_count()
        if self.bwd_ev is not None:
            self.bwd_ev.record(self.stream)
        B.gshard_moe_top2_backward(self.shape_t, inp["x"], inp["wg"], inp["wi"], inp["wo"], self.ctx, inp["dy"],
                                   self.cfg.k_aux, self.dx, self.dwg, self.dwi, self.dwo, self.wsb, self.stream)
        self.launches = fwd_launches + B.gshard_moe_last_launch_count()

    def barrier(self):
        if self.world > 1:
            import torch.distributed as dist
            dist.barrier()
        self.torch.cuda.synchronize()

    def device_status(self) -> int:
        """Status words of the workspaces used (synchronises): a bounded device-side wait that gave up
        shows here, and such a run has no valid result."""
        st = self.B.gshard_moe_last_device_status(self.ws)
        if st == self.B.GSHARD_OK and self.train:
            st = self.B.gshard_moe_last_device_status(self.wsb)
        return st

    def require_ok(self, where: str):
        st = self.device_status()
        if st != self.B.GSHARD_OK:
            raise SystemExit(f"device status after {where}: {self.B.status_string(st)}")

    # ---- device-resident timed region -------------------------------------------------------------
    def timed(self, steps: int, warmup: int) -> dict:
        torch, B, cfg = self.torch, self.B, self.cfg
        for _ in range(warmup):
            self.step()
        self.barrier()
        self.require_ok("warm-up")
        Ev = lambda: torch.cuda.Event(enable_timing=True)
        ev = [Ev() for _ in range(steps + 1)]
        # event pairs recorded by the library around the expert FFN of each timed step (the dominant
        # kernel); recorded once here so that their handles exist before they are handed over
        ffn_ev = [(Ev(), Ev()) for _ in range(steps)]
        bwd_ev = [Ev() for _ in range(steps)] if self.train else None
        for pair in ffn_ev:
            for e in pair:
                e.record(self.stream)
        self.barrier()
        c0 = self.sampler.mark()
        ev[0].record(self.stream)
        for i in range(steps):
            B.gshard_moe_time_expert_ffn(*ffn_ev[i])
            self.bwd_ev = bwd_ev[i] if self.train else None
            self.step()
            ev[i + 1].record(self.stream)
        self.bwd_ev = None
        self.barrier()
        total_ms = max_over_ranks(ev[0].elapsed_time(ev[-1]), self.world, self.dev)
        time.sleep(0.06)                       # let the 50 ms sampler see the end of the region
        clocks = self.sampler.summary(c0)
        self.require_ok("the timed steps")
        ms_per_step = total_ms / steps
        rec = {"ms_per_step": ms_per_step, "value": aggregate_throughput(cfg.N, self.world, ms_per_step),
               "clocks": clocks, "launches_per_step": self.launches}
        rec["ffn_ms"] = sum(a.elapsed_time(b) for a, b in ffn_ev) / steps
        if self.train:
            rec["backward_ms"] = sum(bwd_ev[i].elapsed_time(ev[i + 1]) for i in range(steps)) / steps
            rec["forward_ms"] = ms_per_step - rec["backward_ms"]
        return rec

    def sustained(self, seconds: float, ms_per_step_hint: float) -> dict:
        """The same step back to back for at least `seconds`: what the layer does once the board has
        settled under its power cap.  ms x MHz makes runs at different clocks comparable, and
        `by_clock` gives the mean step time per band of the SM clock sampled while the step ran (the
        run starts near the maximum clock and sinks), i.e. how the step time depends on the clock."""
        torch = self.torch
        steps = max(10, int(math.ceil(seconds * 1e3 / ms_per_step_hint * 1.1)))
        self.barrier()
        c0 = self.sampler.mark()
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
        t0 = time.time()
        ev[0].record(self.stream)
        for i in range(steps):
            self.step()
            ev[i + 1].record(self.stream)
        self.barrier()
        total_ms = max_over_ranks(ev[0].elapsed_time(ev[-1]), self.world, self.dev)
        time.sleep(0.06)
        clocks = self.sampler.summary(c0)
        self.require_ok("the sustained run")
        ms = total_ms / steps
        # step times against the clock sample nearest in time (the GPU runs the queued steps from t0 on)
        samples = [(t, float(p[0])) for t, p in zip(self.sampler.times[c0:], self.sampler.samples[c0:])
                   if p[0].replace(".", "").isdigit()]
        bands = [(0, 1000), (1000, 1200), (1200, 1400), (1400, 1600), (1600, 1800), (1800, 10000)]
        acc = {b: [] for b in bands}
        done = 0.0
        for i in range(steps):
            step_ms = ev[i].elapsed_time(ev[i + 1])
            mid = t0 + (done + 0.5 * step_ms) * 1e-3
            done += step_ms
            if samples:
                mhz = min(samples, key=lambda s: abs(s[0] - mid))[1]
                for b in bands:
                    if b[0] <= mhz < b[1]:
                        acc[b].append(step_ms)
        by_clock = {f"{b[0]}-{b[1]} MHz" if b[1] < 10000 else f">={b[0]} MHz":
                    {"steps": len(v), "ms_per_step": sum(v) / len(v)} for b, v in acc.items() if v}
        return {"steps": steps, "seconds": total_ms * 1e-3, "ms_per_step": ms,
                "value": aggregate_throughput(self.cfg.N, self.world, ms), "sm_mhz": clocks["sm_mhz"],
                "ms_x_mhz": ms * clocks["sm_mhz"] if clocks["sm_mhz"] else None, "reasons": clocks["reasons"],
                "clock_samples": clocks["samples_under_load"], "by_clock": by_clock}

    # ---- records ------------------------------------------------------------------------------------
    def rooflines(self, rec: dict):
        cfg, peaks, args = self.cfg, self.peaks, self.args
        es = 2 if cfg.dtype == "bf16" else 4
        rows = cfg.G * cfg.C
        ffn_bytes, ffn_flops = ffn_work(cfg.M, cfg.H, cfg.E, rows, es)
        fused = (cfg.dtype == "bf16" and not self.train and
                 (args.fused_ffn or (not args.unfused_ffn and rows <= 128)))
        other_form = bool(args.one_sm_mma or args.two_sm_mma or args.fused_ffn or (args.flags & (512 | 32 | 8)))
        compact = (not self.train and cfg.dtype == "bf16" and not fused and
                   bool((args.flags & 16384) or (rows > 128 and not other_form)))
        one_sm = bool(args.one_sm_mma or (args.flags & 512))
        pairs = rows > 128 and not one_sm
        if fused:
            kernel, label, n_launch = "ffn_group4_kernel", "expert FFN, both GEMMs in 1 launch", 1
        else:
            kernel = "umma2_gemm_kernel" if pairs else "umma_gemm_kernel"
            label, n_launch = "expert FFN, 2 grouped-GEMM launches (sum of both)", 2
            if compact and pairs:
                kernel = "umma2_gemm_kernel + umma_gemm_kernel"
                label = ("expert FFN over compacted slots, 2 grouped GEMMs of 2 launches each (sum of the four): kept "
                         "rows in 256-row tiles on CTA pairs, the remaining 128-row tile on single CTAs")
                n_launch = 4
            elif compact:
                label += ", compacted slots: only row tiles that hold kept rows"
        roof = kernel_roofline(ffn_bytes, ffn_flops, rec["ffn_ms"], peaks)
        roof.update({"kernel": f"{kernel} ({label})", "launches_per_step": n_launch,
                     "launch_ms": rec["ffn_ms"] / min(n_launch, 2),     # per GEMM where a GEMM takes two launches
                     "algorithmic_bytes": ffn_bytes, "algorithmic_flops": ffn_flops,
                     "ffn_tflops": ffn_flops / (rec["ffn_ms"] * 1e-3) / 1e12,
                     "ffn_gbs": ffn_bytes / (rec["ffn_ms"] * 1e-3) / 1e9,
                     "traffic": load_traffic(kernel, cfg.M, cfg.H, rows, cfg.E) if fused else None,
                     "traffic_unit": "bytes per launch (ncu capture of a slice with this per-expert shape, scaled "
                                     "by the expert count)", "peak_source": peaks["source"]})
        flops, nbytes = layer_work(cfg, es)
        t_b = nbytes / (peaks["hbm_gbs"] * 1e9)
        t_f, t_fs = flops / (peaks["bf16_tflops"] * 1e12), flops / (peaks["bf16_tflops_sustained"] * 1e12)
        layer = {"bound": "tensor" if t_f > t_b else "hbm", "t_roof_ms": max(t_f, t_b) * 1e3,
                 "frac": max(t_f, t_b) * 1e3 / rec["ms_per_step"], "flops": flops, "bytes": nbytes,
                 "frac_at_sustained_tensor_peak": max(t_fs, t_b) * 1e3 / rec["ms_per_step"],
                 "peak_source": peaks["source"]}
        return roof, layer

    def end_to_end(self, steps: int, warmup: int):
        """Through the host-buffer entry points: the synchronous call, then the pipelined call with two
        staging slots (copies of step i+1 / i-1 under the kernels of step i); every step copies its own
        x, u in and its own y, l_aux out."""
        torch, B, inp, shape, ws, stream = self.torch, self.B, self.inp, self.shape, self.ws, self.stream
        xh = inp["x"].cpu().pin_memory()
        uh = inp["u"].cpu().pin_memory()
        yh = torch.empty_like(xh).pin_memory()
        lh = torch.zeros(1, dtype=torch.float32).pin_memory()
        for _ in range(2):
            B.gshard_moe_top2_forward_host(shape, xh, inp["wg"], inp["wi"], inp["wo"], uh, yh, lh, None, ws, stream)
        self.barrier()
        h0, h1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        h0.record(stream)
        for _ in range(steps):
            B.gshard_moe_top2_forward_host(shape, xh, inp["wg"], inp["wi"], inp["wo"], uh, yh, lh, None, ws, stream)
        h1.record(stream)
        self.barrier()
        sync_ms = max_over_ranks(h0.elapsed_time(h1), self.world, self.dev) / steps
        self.require_ok("the synchronous host calls")
        nslots = 2
        stg = [torch.empty(B.gshard_moe_top2_host_staging_bytes(shape), dtype=torch.uint8, device=self.dev)
               for _ in range(nslots)]
        yhs = [yh, torch.empty_like(xh).pin_memory()]
        lhs = [lh, torch.zeros(1, dtype=torch.float32).pin_memory()]
        s_in, s_out = torch.cuda.Stream(self.dev), torch.cuda.Stream(self.dev)
        evs = [[torch.cuda.Event() for _ in range(3)] for _ in range(nslots)]
        for k in range(nslots):
            for e in evs[k]:
                e.record(stream)

        def pipelined(i):
            k = i % nslots
            B.gshard_moe_top2_forward_host_async(shape, xh, inp["wg"], inp["wi"], inp["wo"], uh, yhs[k], lhs[k], None,
                                                 ws, stg[k], s_in, stream, s_out, *evs[k])
        for i in range(max(warmup, 3)):
            pipelined(i)
        self.barrier()
        h0.record(s_in)
        for i in range(steps):
            pipelined(i)
        h1.record(s_out)
        self.barrier()
        e2e_ms = max_over_ranks(h0.elapsed_time(h1), self.world, self.dev) / steps
        self.require_ok("the pipelined host calls")
        return {"value": aggregate_throughput(self.cfg.N, self.world, e2e_ms), "unit": UNIT,
                "h2d_bytes_per_step": xh.numel() * xh.element_size() + uh.numel() * 4,
                "d2h_bytes_per_step": yh.numel() * yh.element_size() + 4, "ms_per_step": e2e_ms,
                "call": "gshard_moe_top2_forward_host_async, 2 staging slots, 3 streams",
                "ms_per_step_synchronous_call": sync_ms,
                "note": "expert and gating weights stay resident on the device (model state)"}

    def config_record(self, parallelism: str) -> dict:
        cfg = self.cfg
        stats = self.rt["stats"].cpu().tolist()
        return {"workload": cfg.name, "G": cfg.G, "S": cfg.S, "M": cfg.M, "H": cfg.H, "E": cfg.E, "C": cfg.C,
                "tokens_per_step_per_gpu": cfg.N, "parallelism": parallelism,
                "pass": "forward + backward" if self.train else "forward",
                "l2": "inputs larger than L2 (expert weights are streamed once per step)",
                "slots_filled_frac": stats[4] / float(cfg.E * cfg.G * cfg.C)}


def measure(cfg, args, flags, dev, world, rank, sampler, *, e2e: bool, sustained_s: float) -> dict:
    """All timed regions of one configuration; frees its device memory before returning."""
    import torch
    b = Bench(cfg, args, flags, dev, world, rank, sampler)
    rec = b.timed(args.steps, args.warmup)
    roof, layer = b.rooflines(rec)
    out = {"ms_per_step": rec["ms_per_step"], "value": rec["value"], "roofline": roof, "layer_roofline": layer,
           "clocks": rec["clocks"], "launches_per_step": rec["launches_per_step"],
           "config": b.config_record(f"replicas x{world}")}
    if b.train:
        out["forward_ms"], out["backward_ms"] = rec["forward_ms"], rec["backward_ms"]
    if sustained_s > 0:
        s = b.sustained(sustained_s, rec["ms_per_step"])
        s["layer_roofline_frac"] = layer["t_roof_ms"] / s["ms_per_step"]
        out["sustained"] = s
    out["e2e"] = b.end_to_end(args.steps, args.warmup) if (e2e and not b.train) else None
    out["device_status"] = b.device_status()
    del b
    torch.cuda.empty_cache()
    return out


def measure_dense_ffn(args, dev, sampler, n_tokens=131072, M=1024, H=8192) -> dict:
    """The dense feed-forward sub-layer of the adjacent Transformer layer (section 2.1) at the headline
    batch: y = relu(x . wi) . wo over all tokens, bf16, through gshard_dense_ffn_forward."""
    import torch
    from paper_2006_16668_b200 import binding as B
    peaks = load_peaks()
    gen = torch.Generator(device=dev).manual_seed(20200640)
    x = torch.randn(n_tokens, M, generator=gen, device=dev).bfloat16()
    wi = (torch.randn(M, H, generator=gen, device=dev) * M ** -0.5).bfloat16()
    wo = (torch.randn(H, M, generator=gen, device=dev) * H ** -0.5).bfloat16()
    y = torch.empty_like(x)
    ws = torch.empty(B.gshard_dense_ffn_workspace_bytes(n_tokens, M, H, B.GSHARD_BF16), dtype=torch.uint8, device=dev)
    flops = 4.0 * n_tokens * M * H

    def region(steps):
        torch.cuda.synchronize()
        c0 = sampler.mark()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            B.gshard_dense_ffn_forward(x, wi, wo, y, ws)
        e1.record()
        torch.cuda.synchronize()
        time.sleep(0.06)
        if B.gshard_moe_last_device_status(ws) != B.GSHARD_OK:
            raise SystemExit("dense FFN: device status is not OK")
        return e0.elapsed_time(e1) / steps, sampler.summary(c0)

    for _ in range(args.warmup):
        B.gshard_dense_ffn_forward(x, wi, wo, y, ws)
    ms, clocks = region(args.steps)
    rec = {"workload": f"dense FFN of the adjacent Transformer layer, {n_tokens} x {M} x {H}, bf16",
           "ms_per_step": ms, "value": n_tokens / (ms * 1e-3), "unit": UNIT, "tflops": flops / (ms * 1e-3) / 1e12,
           "bound": "tensor", "frac": flops / (ms * 1e-3) / 1e12 / peaks["bf16_tflops"], "clocks": clocks,
           "launches_per_step": B.gshard_moe_last_launch_count(), "kernel": "umma2_gemm_kernel, 2 launches"}
    if args.sustained_seconds > 0:
        steps = int(math.ceil(args.sustained_seconds * 1e3 / ms * 1.1))
        sms, sclk = region(steps)
        rec["sustained"] = {"steps": steps, "ms_per_step": sms, "tflops": flops / (sms * 1e-3) / 1e12,
                            "frac_of_sustained_peak": flops / (sms * 1e-3) / 1e12 / peaks["bf16_tflops_sustained"],
                            "sm_mhz": sclk["sm_mhz"], "reasons": sclk["reasons"]}
    return rec


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--config", default="c4_2048e")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--parallelism", default="replicas", choices=["replicas", "ep"],
                    help="N > 1: independent replicas, or groups and experts sharded with two all-to-alls")
    ap.add_argument("--ep-comm", default="nccl", choices=["nccl", "torch", "p2p"],
                    help="--parallelism ep: collectives as NCCL calls inside the library, torch.distributed callbacks, "
                         "or no collective: peer stores/loads inside the dispatch and combine kernels")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-extra-configs", action="store_true", help="measure only --config")
    ap.add_argument("--sustained-seconds", type=float, default=2.0, help="0 skips the sustained run")
    ap.add_argument("--one-sm-mma", action="store_true", help="ablation: no grouped GEMM on CTA pairs")
    ap.add_argument("--gate-one-sm", action="store_true", help="ablation: gating GEMM on single CTAs, row-major logits")
    ap.add_argument("--gate-cluster", action="store_true",
                    help="ablation: cluster gating kernel with the mean-gate partial sums fused in")
    ap.add_argument("--gather-dispatch", action="store_true",
                    help="single-launch FFN gathers its rows from x (no dispatch buffer)")
    ap.add_argument("--fused-ffn", action="store_true", help="ablation: force the single-launch expert FFN")
    ap.add_argument("--unfused-ffn", action="store_true", help="ablation: force the two grouped-GEMM launches")
    ap.add_argument("--two-sm-mma", action="store_true", help="ablation: grouped GEMMs on CTA pairs (cta_group::2)")
    ap.add_argument("--flags", type=int, default=0, help="further gshard_moe_shape flag bits, OR-ed in")
    args = ap.parse_args()

    from paper_2006_16668_b200.inputs import CONFIGS
    configs = dict(CONFIGS)
    configs.update(profile_configs())
    cfg = configs[args.config]
    if args.impl == "reference":
        run_reference(args, cfg)
        return

    import torch
    import torch.distributed as dist
    from paper_2006_16668_b200 import binding as B

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the layer has no CPU path")
    torch.cuda.set_device(local_rank)
    p2p_single = world == 1 and args.parallelism == "ep" and args.ep_comm == "p2p"
    if p2p_single:                        # symmetric memory wants a process group even for one rank
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29517")
    if world > 1 or p2p_single:
        dist.init_process_group("nccl", rank=rank, world_size=world, device_id=torch.device("cuda", local_rank))
    dev = torch.device("cuda", local_rank)
    args.warmup = max(args.warmup, 3)
    if args.parallelism == "ep":
        from paper_2006_16668_b200 import ep_bench
        ep_bench.run(args, cfg, dev, world, rank, METRIC, UNIT, ClockSampler(local_rank))
        if dist.is_initialized():
            dist.destroy_process_group()
        return

    flags = ((B.GSHARD_FLAG_FUSED_FFN if args.fused_ffn else 0) |
             (B.GSHARD_FLAG_UNFUSED_FFN if args.unfused_ffn else 0) |
             (B.GSHARD_FLAG_TWO_SM_MMA if args.two_sm_mma else 0) |
             (B.GSHARD_FLAG_GATHER_DISPATCH if args.gather_dispatch else 0) |
             (B.GSHARD_FLAG_GATE_CLUSTER if args.gate_cluster else 0) |
             (B.GSHARD_FLAG_GATE_ONE_SM if args.gate_one_sm else 0) |
             (B.GSHARD_FLAG_ONE_SM_MMA if args.one_sm_mma else 0) | args.flags)

    sampler = ClockSampler(local_rank)
    sampler.start()
    sampler.wait_first_sample()
    main_rec = measure(cfg, args, flags, dev, world, rank, sampler, e2e=not args.no_e2e,
                       sustained_s=args.sustained_seconds)
    clocks = main_rec["clocks"]

    # the other full-size configurations, after the headline one (one GPU; replicas would only repeat them)
    extra = {}
    if world == 1 and not args.no_extra_configs and args.config == "c4_2048e":
        for name in EXTRA_CONFIGS:
            r = measure(configs[name], args, flags, dev, world, rank, sampler, e2e=False,
                        sustained_s=args.sustained_seconds)
            keep = {k: r[k] for k in ("ms_per_step", "value", "layer_roofline", "clocks", "launches_per_step",
                                      "device_status")}
            keep["unit"] = UNIT
            keep["pass"] = r["config"]["pass"]
            keep["slots_filled_frac"] = r["config"]["slots_filled_frac"]
            keep["dominant_kernel"] = {k: r["roofline"][k] for k in ("kernel", "bound", "achieved", "peak", "unit",
                                                                     "frac", "launch_ms", "ffn_tflops", "ffn_gbs")}
            if "frac_of_sustained_peak" in r["roofline"]:
                keep["dominant_kernel"]["frac_of_sustained_peak"] = r["roofline"]["frac_of_sustained_peak"]
            for k in ("forward_ms", "backward_ms", "sustained"):
                if k in r:
                    keep[k] = r[k]
            extra[name] = keep
        extra["dense_ffn"] = measure_dense_ffn(args, dev, sampler)
    sampler.stop()
    clocks["reasons_whole_run"] = sampler.summary()["reasons"]

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        v, desc, cores = oracle_sample(cfg)
        cpu = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc}

    if rank == 0:
        line = {"metric": METRIC, "value": main_rec["value"], "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": main_rec["ms_per_step"], "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": cfg.dtype, "data": "synthetic",
                "config": main_rec["config"], "roofline": main_rec["roofline"],
                "layer_roofline": main_rec["layer_roofline"], "sustained": main_rec.get("sustained"),
                "cpu_baseline": cpu, "e2e": main_rec["e2e"],
                "gpu_launches": main_rec["launches_per_step"] * args.steps, "clocks": clocks,
                "device_status": main_rec["device_status"], "configs": extra or None}
        for k in ("forward_ms", "backward_ms"):
            if k in main_rec:
                line[k] = main_rec[k]
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
