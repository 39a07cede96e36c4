#!/usr/bin/env python
"""Benchmark of the ViTCoP pruning operator chain on B200.

One "step" = one pass of the whole hot path over one batch of a workload: Stage II in one call (redundancy filter =
VIC clustering of the vision features, Algorithm 2; K-norm, Eq. 4; cluster-quota selection, Eq. 5; compaction of
hidden states, K and V) followed by the workload's Stage III steps (K-norm of a fresh K, plain top-k, compaction) on
the shrinking sequence.  The headline workload is the largest one ("c4", long-video shaped); the other four are
measured the same way, with fewer steps, under `other_workloads`.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload c4]

Prints ONE JSON line.  `value` is visual tokens pruned per second with the inputs resident in HBM (CUDA-event time
per step, L2 flushed before every step); `e2e` is the same metric through the public API with pinned HOST buffers,
host<->device copies inside the timed region; `roofline` describes the kernel that takes the largest share of the
step; `cpu_baseline` is the CPU oracle timed on the host cores.  `--impl reference` times that oracle (test
infrastructure) instead of the CUDA path.  `--gpus N` without a torchrun environment starts the N ranks itself.
"""
from __future__ import annotations

import argparse
import dataclasses
import hashlib
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2601_17818_b200 import workloads as W  # noqa: E402

METRIC = "visual_tokens_pruned_per_s"
UNIT = "tokens/s"
HEADLINE = "c4"
ALL_WORKLOADS = ("c0", "c1", "c2", "c3", "c4")
L2_BYTES = 126 << 20
KERNEL_SOURCE = {"knorm_kernel": "knorm.cu", "compact_kernel": "compact.cu", "gram_tc_kernel<rho>": "gram.cu",
                 "gram_tc_kernel<delta>": "gram.cu", "gram_resident_kernel": "gram.cu", "delta_pass_kernel": "delta_pass.cu"}


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            p = json.load(fh)
        return dict(hbm_gbs=float(p["hbm_gbs"]), bf16_tflops=float(p["bf16_tflops"]),
                    bf16_tflops_sustained=float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


def source_sha(name: str) -> str:
    with open(os.path.join(ROOT, "paper_2601_17818_b200", "csrc", name), "rb") as fh:
        return hashlib.sha1(fh.read()).hexdigest()[:12]


def ncu_traffic():
    """DRAM read + write bytes per launch from the committed ncu captures: rows of profiles/dram_traffic.md,
    `| kernel | workload | read bytes | written bytes | sha1[:12] of the kernel's source file at capture |`.
    Not measured by this run; a kernel whose source changed since its capture reports null."""
    out = {}
    path = os.path.join(ROOT, "profiles", "dram_traffic.md")
    if not os.path.exists(path):
        return out
    with open(path) as fh:
        for line in fh:
            cells = [c.strip() for c in line.strip().strip("|").split("|")]
            if len(cells) == 5 and cells[2].isdigit() and cells[3].isdigit():
                out[(cells[0].strip("`"), cells[1])] = (int(cells[2]) + int(cells[3]), cells[4].strip("`"))
    return out


def config_of(w, **extra):
    c = {"workload": w.name, "B": w.B, "Nv": w.Nv, "T": w.T, "H": w.H, "d": w.d, "D": w.D, "Dh": w.Dh,
         "budgets": list(w.budgets), "n_centers": w.n_centers, "d_c": w.d_c, "tau": w.tau,
         "step": "Stage II in one call (vitcop_collaborative_step: redundancy filter, K-norm, cluster-quota selection, "
                 "compaction) at budgets[0], then one Stage III call (vitcop_prune_step: K-norm of a fresh K, plain "
                 "top-k, compaction) per further budget"}
    c.update(extra)
    return c


def caps_of(w):
    """Capacity of the visual span entering each step: Nv, then the previous step's budget."""
    return [w.Nv] + [min(b, w.Nv) for b in w.budgets[:-1]]


# ------------------------------------------------------------------------------------------------ oracle legs
def host_arrays(w, B=None):
    """Seeded inputs of one workload's schedule as numpy arrays (bf16 bit patterns, fp32 positions)."""
    B = w.B if B is None else B
    a = {"feat": W.make_features(w, B=B), "pos": W.make_positions(w)[:B].copy(), "hidden": W.make_hidden(w, B=B)}
    for s, cap in enumerate(caps_of(w)):
        a[f"K{s}"], a[f"V{s}"] = W.make_kv(w, s, cap, B=B)
    return a


def oracle_schedule(w, a):
    """The whole schedule on the CPU oracle for the sequences in `a`; returns the number of visual tokens pruned."""
    import oracle
    B = a["feat"].shape[0]
    pruned = 0
    for b in range(B):
        n_vis, hidden = w.Nv, a["hidden"][b]
        for s, budget in enumerate(w.budgets):
            K, V = a[f"K{s}"][b][:, : w.T + n_vis], a[f"V{s}"][b][:, : w.T + n_vis]
            K, V = np.ascontiguousarray(K), np.ascontiguousarray(V)
            score = oracle.knorm(K[None], w.vis_start, n_vis)[0]
            if s == 0:
                r = oracle.vic(a["feat"][b], a["pos"][b], 0, w.d_c, w.tau, w.n_centers)
                keep, _, _ = oracle.select_quota(score, r["label"], budget)
            else:
                keep = oracle.select_plain(score, budget)
            o = oracle.compact(hidden[: w.T + n_vis], K, V, w.T + n_vis, w.vis_start, n_vis, keep, w.T + len(keep))
            hidden, n_vis = o["hidden"], len(keep)
        pruned += w.Nv - n_vis
    return pruned


def oracle_sample(w, per_step_seconds):
    """A bounded sample of the workload for the CPU oracle: (workload to run, number of sequences, description).

    Sequences are independent, so the sample is the first few of them; a sequence of the long-video workload
    alone costs about a quarter of a minute of pairwise fp64 work, so where even one sequence exceeds the bound it is cut to
    its first 4096 visual tokens (budgets and centre count scaled alike) -- the pairwise work per token then is a
    quarter of the full length's, which the description says."""
    cost = {"c0": 0.02, "c1": 0.02, "c2": 0.6, "c3": 1.0, "c4": 16.0}.get(w.name, 0.05)   # seconds per sequence on 16 cores, roughly
    if cost <= per_step_seconds:
        nseq = int(max(1, min(w.B, per_step_seconds // cost, 4)))
        return w, nseq, f"the first {nseq} of {w.B} sequences of workload {w.name}, whole schedule"
    f = 4096 / w.Nv
    small = dataclasses.replace(w, Nv=4096, budgets=tuple(int(b * f) for b in w.budgets),
                                n_centers=int(np.ceil(w.n_centers * f)))
    return small, 1, (f"1 of {w.B} sequences of workload {w.name} cut to its first 4096 of {w.Nv} visual tokens "
                      f"(budgets {list(small.budgets)}, {small.n_centers} centres), whole schedule; the oracle's "
                      f"pairwise work per token is {w.Nv // 4096}x lower than at full length")


class OracleBench:
    def __init__(self, w, per_step_seconds):
        import oracle
        self.w, self.nseq, self.sample = oracle_sample(w, per_step_seconds)
        self.a = host_arrays(self.w, B=self.nseq)
        oracle.build()
        self.cores = oracle.num_threads()

    def step(self):
        return oracle_schedule(self.w, self.a)

    def run(self, steps, warmup):
        for _ in range(warmup):
            self.step()
        t0 = time.perf_counter()
        pruned = sum(self.step() for _ in range(steps))
        dt = time.perf_counter() - t0
        return pruned / dt, dt / steps

    def run_for(self, seconds):
        t0 = time.perf_counter()
        pruned, steps = 0, 0
        while steps < 1 or time.perf_counter() - t0 < seconds:
            pruned += self.step()
            steps += 1
        dt = time.perf_counter() - t0
        return pruned / dt, dt, steps


def run_reference(args):
    if int(os.environ.get("RANK", "0")) != 0:
        return
    w = W.workload(args.workload)
    ob = OracleBench(w, per_step_seconds=4.0)
    value, sec_per_step = ob.run(args.steps, args.warmup)
    sample = f"each step = {ob.sample} (fp64 CPU oracle, OpenMP over rows)"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": sec_per_step * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": config_of(w),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": ob.cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ------------------------------------------------------------------------------------------------ clocks
class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML (read-only) while the timed region runs."""

    def __init__(self, index: int, period_s: float = 0.002):
        super().__init__(daemon=True)
        self.index, self.period = index, period_s
        self.sm, self.reasons, self.sm_max = [], set(), None
        self._halt = threading.Event()
        self.ok = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.sm_max = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
            self.ok = True
        except Exception:
            self.ok = False

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        names = {
            getattr(nv, "nvmlClocksThrottleReasonHwSlowdown", 0x8): "hw_slowdown",
            getattr(nv, "nvmlClocksThrottleReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
            getattr(nv, "nvmlClocksThrottleReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
            getattr(nv, "nvmlClocksThrottleReasonSwPowerCap", 0x4): "sw_power_cap",
            getattr(nv, "nvmlClocksThrottleReasonHwPowerBrakeSlowdown", 0x80): "hw_power_brake",
        }
        while not self._halt.is_set():
            try:
                self.sm.append(int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                r = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                for bit, name in names.items():
                    if r & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(self.period)

    def stop(self):
        self._halt.set()
        self.join(timeout=2)
        return {"sm_mhz": (float(np.median(self.sm)) if self.sm else None), "sm_max_mhz": self.sm_max,
                "reasons": sorted(self.reasons), "samples": len(self.sm)}


# ------------------------------------------------------------------------------------------------ GPU arm
class Schedule:
    """Device buffers and the API calls of one workload's schedule (one set of inputs and outputs)."""

    IN_KEYS = ("feat", "pos", "hidden")

    def __init__(self, w, torch, vb, dev):
        self.w, self.torch, self.vb = w, torch, vb
        B, n = w.B, w.Nv
        self.caps = caps_of(w)
        self.nsteps = len(w.budgets)
        e = lambda *s, dt=torch.bfloat16: torch.empty(s, dtype=dt, device=dev)
        self.feat, self.pos, self.hidden = e(B, n, w.D), e(B, n, 2, dt=torch.float32), e(B, w.N, w.Dh)
        self.K = [e(B, w.H, w.T + c, w.d) for c in self.caps]
        self.V = [e(B, w.H, w.T + c, w.d) for c in self.caps]
        self.label, self.ncl = e(B, n, dt=torch.int32), e(B, dt=torch.int32)
        self.ncap = [w.T + min(b, c) for b, c in zip(w.budgets, self.caps)]
        self.ho = [e(B, nc, w.Dh) for nc in self.ncap]
        self.Ko = [e(B, w.H, nc, w.d) for nc in self.ncap]
        self.Vo = [e(B, w.H, nc, w.d) for nc in self.ncap]
        self.olen = [e(B, dt=torch.int32) for _ in self.ncap]
        self.nkeep = [e(B, dt=torch.int32) for _ in self.ncap]
        self.kpos = [e(B, nc, dt=torch.int32) for nc in self.ncap]
        self.ws_c = vb.alloc_workspace(vb.OP_COLLAB_STEP, device=dev, B=B, Nv=n, D=w.D)
        self.ws_s = [vb.alloc_workspace(vb.OP_PRUNE_STEP, device=dev, B=B, Nv=c) for c in self.caps]
        self.ws_f = None

    def input_tensors(self):
        d = {k: getattr(self, k) for k in self.IN_KEYS}
        for s in range(self.nsteps):
            d[f"K{s}"], d[f"V{s}"] = self.K[s], self.V[s]
        return d

    def output_tensors(self):
        d = {}
        for s in range(self.nsteps):
            d.update({f"ho{s}": self.ho[s], f"Ko{s}": self.Ko[s], f"Vo{s}": self.Vo[s], f"olen{s}": self.olen[s],
                      f"kpos{s}": self.kpos[s]})
        return d

    def upload(self, host, non_blocking=True):
        for k, t in self.input_tensors().items():
            t.copy_(host[k], non_blocking=non_blocking)

    def stage(self, s):
        w, vb = self.w, self.vb
        if s == 0:
            vb.vitcop_collaborative_step(self.feat, self.pos, self.hidden, self.K[0], self.V[0], w.vis_start,
                                         w.budgets[0], self.ho[0], self.Ko[0], self.Vo[0], self.olen[0], self.label,
                                         self.ncl, self.ws_c, metric=0, d_c=w.d_c, tau=w.tau, n_centers=w.n_centers,
                                         kept_pos=self.kpos[0], n_keep_out=self.nkeep[0])
        else:
            # the lengths the previous step left on the device feed this one directly
            vb.vitcop_prune_step(self.ho[s - 1], self.K[s], self.V[s], w.vis_start, self.nkeep[s - 1], self.caps[s],
                                 w.budgets[s], self.ho[s], self.Ko[s], self.Vo[s], self.olen[s], self.ws_s[s],
                                 kept_pos=self.kpos[s], seq_len=self.olen[s - 1], n_keep_out=self.nkeep[s])

    def run(self):
        for s in range(self.nsteps):
            self.stage(s)

    def plain_step0(self):
        """Step 0 as a Stage III step (plain top-k at budgets[0], no clustering) on the full input."""
        w = self.w
        self.vb.vitcop_prune_step(self.hidden, self.K[0], self.V[0], w.vis_start, w.Nv, w.Nv, w.budgets[0], self.ho[0],
                                  self.Ko[0], self.Vo[0], self.olen[0], self.ws_s[0], kept_pos=self.kpos[0],
                                  n_keep_out=self.nkeep[0])

    def filter_then_prune(self):
        w, vb = self.w, self.vb
        if self.ws_f is None:
            self.ws_f = vb.alloc_workspace(vb.OP_FILTER, device=self.feat.device, B=w.B, Nv=w.Nv, D=w.D)
        vb.vitcop_redundancy_filter(self.feat, self.pos, self.label, self.ncl, self.ws_f, metric=0, d_c=w.d_c, tau=w.tau,
                                    n_centers=w.n_centers)
        vb.vitcop_prune_step(self.hidden, self.K[0], self.V[0], w.vis_start, w.Nv, w.Nv, w.budgets[0], self.ho[0],
                             self.Ko[0], self.Vo[0], self.olen[0], self.ws_s[0], label=self.label,
                             kept_pos=self.kpos[0], n_keep_out=self.nkeep[0])


def pinned_inputs(w, torch):
    a = host_arrays(w)
    out = {}
    for k, v in a.items():
        t = torch.from_numpy(v.view(np.int16)).view(torch.bfloat16) if v.dtype == np.uint16 else torch.from_numpy(v)
        out[k] = t.pin_memory()
    return out


def tiles_within_radius(w):
    """Share of the 128 x 256 tiles of the symmetric half whose row block and column blocks lie within the spatial radius
    of one another (bounding boxes of the blocks' positions, fp32): the tiles the density sweep keeps and the delta pass
    reads.  Computed here from the positions alone."""
    pos = W.make_positions(w).astype(np.float32)
    n, tau2 = w.Nv, np.float32(w.tau) ** 2
    TI, TJ = -(-n // 128), -(-n // 256)
    kept = total = 0
    for b in range(pos.shape[0]):
        lo = np.stack([pos[b, i * 128:(i + 1) * 128].min(0) for i in range(TI)])
        hi = np.stack([pos[b, i * 128:(i + 1) * 128].max(0) for i in range(TI)])
        for tj in range(TJ):
            cl, ch = lo[2 * tj:2 * tj + 2].min(0), hi[2 * tj:2 * tj + 2].max(0)
            rows = min(TI, 2 * tj + 2)
            d = np.maximum(np.float32(0), np.maximum(lo[:rows] - ch, cl - hi[:rows]))
            s2 = d[:, 0] * d[:, 0] + d[:, 1] * d[:, 1]
            kept += int(np.count_nonzero(~(s2 > tau2)))
            total += rows
    return kept / max(total, 1)


def algorithmic_units(w, s, vis_in, kept):
    """Per launch at step s: kernel -> (bound, algorithmic bytes or flop).

    knorm:   reads the visual span of K once (H*d bf16 per token) and writes one fp32 score per token   -> HBM
    compact: reads and writes every surviving row of hidden, K and V once, plus the index arrays          -> HBM
    gram:    one sweep over the symmetric half of the Gram matrix incl. the diagonal, 2*D flop per pair,
             B*n*(n+1)/2 pairs                                                                             -> tensor cores
    vis_in / kept: visual tokens entering / surviving the step, summed over the batch."""
    rows_out = w.B * w.T + kept
    u = {"knorm_kernel": ("hbm", vis_in * (w.H * w.d * 2 + 4)),
         "compact_kernel": ("hbm", 2 * rows_out * (w.Dh + 2 * w.H * w.d) * 2 + rows_out * 4 + w.B * 12 + kept * 4)}
    if s == 0:
        sweep = w.B * w.Nv * (w.Nv + 1) * w.D
        u.update({"gram_resident_kernel": ("tensor", sweep), "gram_tc_kernel<rho>": ("tensor", sweep),
                  "gram_tc_kernel<delta>": ("tensor", sweep),
                  # reads the stored Gram value of every pair of the symmetric half (diagonal included) that sits in
                  # a tile within the spatial radius, once: 4 bytes
                  "delta_pass_kernel": ("hbm", int(w.B * w.Nv * (w.Nv + 1) // 2 * 4 * tiles_within_radius(w))
                                        if w.Nv >= 8192 else 0)})
    return u


class Bench:
    """Measurement of one workload on one device."""

    def __init__(self, w, torch, vb, dev, flush, peaks, replicas):
        self.w, self.torch, self.vb, self.dev, self.flush, self.peaks, self.rep = w, torch, vb, dev, flush, peaks, replicas
        self.host = pinned_inputs(w, torch)
        self.sc = Schedule(w, torch, vb, dev)
        self.sc.upload(self.host, non_blocking=False)
        torch.cuda.synchronize()

    # ---- protocols
    def timed(self, fn, steps, warmup):
        """Per-step CUDA-event times (ms) on the current stream, L2 flushed (512 MiB memset) before every step."""
        torch = self.torch
        for _ in range(warmup):
            self.flush.zero_()
            fn()
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        self.rep.barrier()
        for a, b in evs:
            self.flush.zero_()
            a.record()
            fn()
            b.record()
        self.rep.barrier()
        return np.array([a.elapsed_time(b) for a, b in evs], dtype=np.float64)

    def bracketed(self, fn, reps):
        """{kernel: (launches, total ms)} of `reps` flushed runs of fn, from the library's own CUDA-event brackets
        around each kernel (programmatic overlap between kernels is off while they are on)."""
        for _ in range(2):
            self.flush.zero_()
            fn()
        self.torch.cuda.synchronize()
        self.vb.vitcop_kernel_timing_begin()
        for _ in range(reps):
            self.flush.zero_()
            fn()
        return self.vb.vitcop_kernel_timing_end()

    def back_to_back(self, make_call, bytes_per_copy, reps=5):
        """Microseconds per launch of one API call without event brackets: a CUDA graph of R back-to-back calls on R
        rotating copies of its inputs and outputs (R copies exceed twice the L2, so every launch reads from and
        writes to DRAM), replayed `reps` times between two events; time / (R * reps)."""
        torch = self.torch
        R = int(min(48, max(2, -(-3 * L2_BYTES // max(bytes_per_copy, 1)))))
        calls = [make_call(i) for i in range(R)]
        side = torch.cuda.Stream(device=self.dev)
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            for c in calls:
                c()
            torch.cuda.synchronize()
            with torch.cuda.graph(graph, stream=side):
                for c in calls:
                    c()
        for _ in range(2):
            graph.replay()
        self.flush.zero_()
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0.record()
        for _ in range(reps):
            graph.replay()
        t1.record()
        torch.cuda.synchronize()
        us = t0.elapsed_time(t1) * 1e3 / (R * reps)
        del graph, calls
        return us, R

    # ---- the measurements
    def run(self, steps, warmup, e2e_steps, cpu_seconds, with_clocks, local_rank):
        w, sc, torch, vb, peaks = self.w, self.sc, self.torch, self.vb, self.peaks
        sampler = ClockSampler(local_rank) if with_clocks else None
        if sampler:
            sampler.start()
        t_step = self.timed(sc.run, steps, warmup)
        clocks = sampler.stop() if sampler else None
        nkeep = [t.cpu().numpy() for t in sc.nkeep]
        vis_in = [w.B * w.Nv] + [int(k.sum()) for k in nkeep[:-1]]
        kept = [int(k.sum()) for k in nkeep]
        pruned_per_step = w.B * w.Nv - kept[-1]
        total_ms = self.rep.max_over_ranks(float(t_step.sum()), self.dev)
        value = self.rep.whole_job_rate(pruned_per_step, steps, float(t_step.sum()), self.dev)
        res = {"value": value, "ms_per_step": total_ms / steps, "us_per_step_median": float(np.median(t_step) * 1e3),
               "tokens_pruned_per_step": pruned_per_step, "tokens_kept_after_each_stage": kept, "clocks": clocks}

        # per-stage times of the schedule, and step 0 as a plain Stage III step --------------------------------
        n_kt = max(10, min(steps, 40))
        sched = []
        for s in range(sc.nsteps):
            t = self.timed(lambda s=s: sc.stage(s), n_kt, 3)
            sched.append({"stage": "II (quota, one call)" if s == 0 else "III (plain)", "budget": w.budgets[s],
                          "visual_tokens_in": vis_in[s], "visual_tokens_kept": kept[s],
                          "us_median": float(np.median(t) * 1e3), "us_min": float(t.min() * 1e3)})
        res["schedule"] = sched
        t = self.timed(sc.plain_step0, n_kt, 3)
        res["plain_step0"] = {"budget": w.budgets[0], "us_median": float(np.median(t) * 1e3), "us_min": float(t.min() * 1e3),
                              "tokens_pruned": w.B * (w.Nv - min(w.budgets[0], w.Nv))}
        t = self.timed(sc.filter_then_prune, n_kt, 3)
        res["stage2_as_two_calls_us"] = float(np.median(t) * 1e3)
        sc.run()                                            # leave the buffers as the schedule leaves them
        torch.cuda.synchronize()

        # per-kernel device times, stage by stage ----------------------------------------------------------------
        traffic = ncu_traffic()
        kernels, launches_per_step, dom = {}, 0, None
        for s in range(sc.nsteps):
            pk = self.bracketed(lambda s=s: sc.stage(s), n_kt)
            algo = algorithmic_units(w, s, vis_in[s], kept[s])
            for name, (launches, ms) in pk.items():
                us = ms * 1e3 / max(launches, 1)
                launches_per_step += launches // n_kt
                e = {"launches_per_step": launches // n_kt, "us_per_launch": us, "timing": "event bracket"}
                split = name == "knorm_kernel" and "gram_resident_kernel" in pk
                if split:
                    e["note"] = "covers part of the samples only; the rest is computed inside gram_resident_kernel"
                elif name in algo and us > 0:
                    bound, units = algo[name]
                    e.update(self.roofline_entry(bound, units, us))
                    key = (name, w.name)
                    e["traffic"] = None
                    if s == 0 and key in traffic and traffic[key][1] == source_sha(KERNEL_SOURCE[name]):
                        e["traffic"] = traffic[key][0]
                        e["traffic_source"] = "profiles/dram_traffic.md (ncu capture; not measured by this run)"
                kernels[f"{name}@{s}"] = e
                if dom is None or ms > dom[1]:
                    dom = (f"{name}@{s}", ms)
        res["kernels"] = kernels
        res["gpu_launches_per_step"] = launches_per_step
        tiny = torch.zeros(32, device=self.dev)
        t_br = self.timed(lambda: tiny.zero_(), 20, 3)
        bracket_us = float(np.median(t_br) * 1e3)

        # single-kernel calls without brackets (what matters for kernels of a few tens of microseconds) ---------
        res["isolated"] = self.isolated(vis_in, kept)
        # the roofline of the kernel with the largest share of the step
        d = kernels[dom[0]]
        res["roofline"] = {"kernel": dom[0].split("@")[0], "stage": int(dom[0].split("@")[1]),
                           **{k: d.get(k) for k in ("bound", "achieved", "peak", "unit", "frac", "traffic")},
                           "peak_source": d.get("peak_source"), "us_per_launch": d["us_per_launch"],
                           "timing": d["timing"], "algorithmic_units_per_launch": d.get("algorithmic_units_per_launch"),
                           "share_of_step": dom[1] / sum(v["us_per_launch"] * v["launches_per_step"] * n_kt * 1e-3
                                                         for v in kernels.values()),
                           "event_bracket_overhead_us": bracket_us}

        # K-norm at the source of K: the key projection with the norm in its epilogue (no separate read of K) -------
        res["kproj_knorm"] = self.kproj(res["isolated"]["knorm_kernel"]["us_per_launch"])

        # the operators beside the pruning step: cluster merge (Eq. 6), [CLS] saliency (Eq. 1) ---------------------
        res["beside_the_step"] = self.beside_the_step()

        # end to end through the public API with host buffers --------------------------------------------------
        res["e2e"] = self.e2e(e2e_steps, pruned_per_step)

        # CPU oracle beside it -----------------------------------------------------------------------------------
        res["cpu_baseline"] = None
        if cpu_seconds > 0:
            ob = OracleBench(w, per_step_seconds=max(cpu_seconds, 20.0 if w.name == "c4" else cpu_seconds))
            v, secs, passes = ob.run_for(cpu_seconds)
            res["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": ob.cores, "kind": "oracle",
                                   "sample": f"{ob.sample}, {passes} pass(es) in {secs:.1f} s"}
        return res

    def roofline_entry(self, bound, units, us):
        peaks = self.peaks
        if bound == "hbm":
            ach, peak, unit, src = units / (us * 1e-6) / 1e9, peaks["hbm_gbs"], "GB/s", peaks["source"] + " copy"
        else:
            ach, peak, unit, src = units / (us * 1e-6) / 1e12, peaks["bf16_tflops"], "TFLOP/s", peaks["source"] + " burst"
        return dict(bound=bound, achieved=ach, peak=peak, unit=unit, frac=ach / peak, peak_source=src,
                    algorithmic_units_per_launch=units)

    def isolated(self, vis_in, kept):
        """knorm, the two selections and the compaction as stand-alone calls at step 0's shapes (the selection also at
        the first Stage III shape), by the back-to-back protocol; HBM kernels get their roofline fraction from it."""
        w, sc, torch, vb, dev = self.w, self.sc, self.torch, self.vb, self.dev
        B, n = w.B, w.Nv
        out = {}
        kbytes = B * w.H * w.N * w.d * 2
        R_K = int(min(48, max(2, -(-3 * L2_BYTES // kbytes))))
        Ks = [sc.K[0]] + [sc.K[0].clone() for _ in range(R_K - 1)]
        scores = [torch.empty((B, n), dtype=torch.float32, device=dev) for _ in range(R_K)]
        us, R = self.back_to_back(lambda i: (lambda: vb.vitcop_knorm_score(Ks[i % R_K], w.vis_start, n, scores[i % R_K])),
                                  kbytes)
        units = algorithmic_units(w, 1, B * n, 0)["knorm_kernel"][1]
        out["knorm_kernel"] = {"us_per_launch": us, "copies": R, **self.roofline_entry("hbm", units, us)}
        # selections: kilobytes of input, latency-bound; reported in microseconds
        ws = [vb.alloc_workspace(vb.OP_SELECT, device=dev, B=B, Nv=n) for _ in range(4)]
        kidx = [torch.empty((B, n), dtype=torch.int32, device=dev) for _ in range(4)]
        nk = [torch.empty((B,), dtype=torch.int32, device=dev) for _ in range(4)]
        vb.vitcop_knorm_score(sc.K[0], w.vis_start, n, scores[0])
        us, _ = self.back_to_back(lambda i: (lambda: vb.vitcop_select(scores[0], n, w.budgets[0], kidx[i % 4], nk[i % 4],
                                                                     ws[i % 4], label=sc.label)), 1 << 30)
        out["select_quota_kernel"] = {"us_per_launch": us, "tokens_per_sequence": n, "budget": w.budgets[0]}
        us, _ = self.back_to_back(lambda i: (lambda: vb.vitcop_select(scores[0], n, w.budgets[0], kidx[i % 4], nk[i % 4],
                                                                     ws[i % 4])), 1 << 30)
        out["select_plain_kernel"] = {"us_per_launch": us, "tokens_per_sequence": n, "budget": w.budgets[0]}
        # compaction with the schedule's own keep list of step 0
        vb.vitcop_select(scores[0], n, w.budgets[0], kidx[0], nk[0], ws[0], label=sc.label)
        cbytes = kbytes * 2 + B * w.N * w.Dh * 2
        R_C = int(min(48, max(2, -(-3 * L2_BYTES // cbytes))))
        del Ks
        ins = [(sc.hidden, sc.K[0], sc.V[0])] + [(sc.hidden.clone(), sc.K[0].clone(), sc.V[0].clone())
                                                  for _ in range(R_C - 1)]
        outs = [(sc.ho[0], sc.Ko[0], sc.Vo[0])] + [(torch.empty_like(sc.ho[0]), torch.empty_like(sc.Ko[0]),
                                                     torch.empty_like(sc.Vo[0])) for _ in range(R_C - 1)]
        olen = torch.empty((B,), dtype=torch.int32, device=dev)

        def make(i):
            h, K, V = ins[i % R_C]
            ho, Ko, Vo = outs[i % R_C]
            return lambda: vb.vitcop_compact_kv(h, K, V, w.vis_start, n, kidx[0], nk[0], ho, Ko, Vo, olen)

        us, R = self.back_to_back(make, cbytes)
        units = algorithmic_units(w, 0, B * n, int(nk[0].sum()))["compact_kernel"][1]
        out["compact_kernel"] = {"us_per_launch": us, "copies": R, **self.roofline_entry("hbm", units, us)}
        del ins, outs
        torch.cuda.empty_cache()
        return out

    def beside_the_step(self):
        """Cluster merge (Eq. 6) on Stage II's own labels and keep mask, and [CLS] saliency (Eq. 1) over the workload's
        heads with n + 1 keys, as stand-alone calls by the back-to-back protocol, against the copy bandwidth."""
        w, sc, torch, vb, dev = self.w, self.sc, self.torch, self.vb, self.dev
        B, n = w.B, w.Nv
        out = {}
        # ---- merge: reads the hidden row of every visual token that was not kept, writes one row per cluster
        score = torch.empty((B, n), dtype=torch.float32, device=dev)
        vb.vitcop_knorm_score(sc.K[0], w.vis_start, n, score)
        kidx = torch.empty((B, n), dtype=torch.int32, device=dev)
        nk = torch.empty((B,), dtype=torch.int32, device=dev)
        km = torch.empty((B, n), dtype=torch.uint8, device=dev)
        vb.vitcop_select(score, n, w.budgets[0], kidx, nk, vb.alloc_workspace(vb.OP_SELECT, device=dev, B=B, Nv=n),
                         label=sc.label, keep_mask=km)
        M = w.n_centers
        hbytes = B * w.N * w.Dh * 2
        R = int(min(16, max(2, -(-3 * L2_BYTES // hbytes))))
        hids = [sc.hidden] + [sc.hidden.clone() for _ in range(R - 1)]
        ml = [torch.empty((B, M), dtype=torch.int32, device=dev) for _ in range(R)]
        mc = [torch.empty((B, M), dtype=torch.int32, device=dev) for _ in range(R)]
        nm = [torch.empty((B,), dtype=torch.int32, device=dev) for _ in range(R)]
        mr = [torch.empty((B, M, w.Dh), dtype=torch.bfloat16, device=dev) for _ in range(R)]
        ws = [vb.alloc_workspace(vb.OP_MERGE, device=dev, B=B, Nv=n, N=M) for _ in range(R)]
        us, copies = self.back_to_back(lambda i: (lambda: vb.vitcop_merge_clusters(
            hids[i % R], w.vis_start, n, sc.label, km, ml[i % R], mc[i % R], nm[i % R], ws[i % R], merged=mr[i % R])),
            hbytes)
        merged_rows, dropped = int(nm[0].sum()), B * n - int(nk.sum())
        units = dropped * w.Dh * 2 + merged_rows * (w.Dh * 2 + 8) + B * n * 5
        out["merge_clusters"] = {"us_per_call": us, "copies": copies, "rows_read": dropped, "rows_written": merged_rows,
                                 **self.roofline_entry("hbm", units, us)}
        del hids, mr
        # ---- saliency: reads every key of every head once
        g = torch.Generator(device=dev).manual_seed(1)
        kbytes = B * w.H * (n + 1) * w.d * 2
        R = int(min(48, max(2, -(-3 * L2_BYTES // kbytes))))
        Kc = (torch.randn((B, w.H, n + 1, w.d), device=dev, generator=g)).to(torch.bfloat16)
        Ks = [Kc] + [Kc.clone() for _ in range(R - 1)]
        q = torch.randn((B, w.H, w.d), device=dev, generator=g).to(torch.bfloat16)
        sal = [torch.empty((B, n), dtype=torch.float32, device=dev) for _ in range(R)]
        wss = [vb.alloc_workspace(vb.OP_SALIENCY, device=dev, B=B, H=w.H, N=n + 1) for _ in range(R)]
        us, copies = self.back_to_back(lambda i: (lambda: vb.vitcop_cls_saliency(q, Ks[i % R], w.d ** -0.5, sal[i % R],
                                                                                wss[i % R])), kbytes)
        out["cls_saliency"] = {"us_per_call": us, "copies": copies, "heads": w.H, "keys": n + 1,
                               **self.roofline_entry("hbm", kbytes + B * n * 4, us)}
        del Ks
        torch.cuda.empty_cache()
        return out

    def kproj(self, knorm_us, reps=10, warm=3):
        """vitcop_kproj_knorm at the workload's shapes (layer input -> K of all heads with rotary embedding + Eq. 4 of
        the visual span), against the tensor-core peak; beside it what the stand-alone K-norm of that K costs."""
        w, sc, torch, vb, dev = self.w, self.sc, self.torch, self.vb, self.dev
        g = torch.Generator(device=dev).manual_seed(0)
        Wk = (torch.randn((w.H * w.d, w.Dh), device=dev, generator=g) / w.Dh ** 0.5).to(torch.bfloat16)
        inv = 1.0 / (10000.0 ** (torch.arange(w.d // 2, device=dev) / (w.d // 2)))
        ang = torch.arange(w.N, device=dev)[:, None] * inv[None, :]
        cos, sin = torch.cos(ang).float().contiguous(), torch.sin(ang).float().contiguous()
        K_out = torch.empty((w.B, w.H, w.N, w.d), dtype=torch.bfloat16, device=dev)
        score = torch.empty((w.B, w.Nv), dtype=torch.float32, device=dev)
        ws = vb.alloc_workspace(vb.OP_KPROJ, device=dev, B=w.B, H=w.H, N=w.N, d=w.d)
        fn = lambda: vb.vitcop_kproj_knorm(sc.hidden, Wk, w.H, w.d, K_out, ws, vis_start=w.vis_start, score=score,
                                           rope_cos=cos, rope_sin=sin)
        t = self.timed(fn, reps, warm)
        us = float(np.median(t) * 1e3)
        flop = 2.0 * w.B * w.N * w.Dh * w.H * w.d
        tf = flop / (us * 1e-6) / 1e12
        out = {"us_median": us, "flop": flop, "achieved": tf, "unit": "TFLOP/s", "peak": self.peaks["bf16_tflops"],
               "frac": tf / self.peaks["bf16_tflops"], "peak_source": self.peaks["source"] + " burst",
               "knorm_standalone_us": knorm_us,
               "note": "GEMM [B*N, Dh] x [Dh, H*d] + rotary embedding + bf16 K + Eq. 4 in the epilogue; the stand-alone "
                       "K-norm (knorm_standalone_us, the separate read of K) is what a pruning step saves when K comes "
                       "from this call"}
        del Wk, K_out
        torch.cuda.empty_cache()
        return out

    def e2e(self, steps, pruned_per_step):
        """Every step copies the schedule's inputs from pinned host memory and all its outputs back.  The copies of
        neighbouring steps overlap the way a serving loop would run them: two sets of device buffers, an upload
        stream, the compute stream and a download stream chained by events."""
        w, torch, vb, dev, host = self.w, self.torch, self.vb, self.dev, self.host
        sets = [self.sc, Schedule(w, torch, vb, dev)]
        outs = [{k: torch.empty(t.shape, dtype=t.dtype).pin_memory() for k, t in x.output_tensors().items()} for x in sets]
        s_up, s_down = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
        s_main = torch.cuda.current_stream()

        def go(n):
            ev_in = [torch.cuda.Event() for _ in range(n)]
            ev_done = [torch.cuda.Event() for _ in range(n)]
            ev_out = [torch.cuda.Event() for _ in range(n)]
            t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            self.rep.barrier()
            t0.record(s_main)
            s_up.wait_event(t0)
            for i in range(n):
                x, o = sets[i % 2], outs[i % 2]
                with torch.cuda.stream(s_up):
                    if i >= 2:
                        s_up.wait_event(ev_done[i - 2])        # the step that last read these input buffers
                    x.upload(host)
                    ev_in[i].record(s_up)
                s_main.wait_event(ev_in[i])
                if i >= 2:
                    s_main.wait_event(ev_out[i - 2])           # its outputs have left these output buffers
                x.run()
                ev_done[i].record(s_main)
                with torch.cuda.stream(s_down):
                    s_down.wait_event(ev_done[i])
                    for k, t in x.output_tensors().items():
                        o[k].copy_(t, non_blocking=True)
                    ev_out[i].record(s_down)
            for e in ev_out[-2:]:
                s_main.wait_event(e)
            t1.record(s_main)
            self.rep.barrier()
            return t0.elapsed_time(t1)

        go(2)
        ms = self.rep.max_over_ranks(float(go(steps)), dev)
        h2d = sum(int(v.numel() * v.element_size()) for v in host.values())
        d2h = sum(int(v.numel() * v.element_size()) for v in outs[0].values())
        del sets, outs
        return {"value": self.rep.world() * pruned_per_step * steps / (ms * 1e-3), "unit": UNIT,
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "ms_per_step": ms / steps,
                "protocol": "uploads, compute and downloads of neighbouring steps overlap (3 streams, 2 buffer sets)"}


def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2601_17818_b200 import binding as vb
    from paper_2601_17818_b200 import replicas

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU fallback")
    vb.lib()                                   # fail loudly if the CUDA library is missing
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    peaks = measured_peaks()
    flush = torch.empty(512 << 20, dtype=torch.uint8, device=dev)     # > 4x the 126 MB L2

    w = W.workload(args.workload)
    solo = rank == 0 and world == 1
    if args.profile_run:
        # for a profiler: the schedule of one workload, warm-up + steps, nothing else launched by this library
        b = Bench(w, torch, vb, dev, flush, peaks, replicas)
        for _ in range(args.warmup + args.steps):
            flush.zero_()
            b.sc.run()
        flush.zero_()
        b.kproj(0.0, reps=1, warm=0)                       # the key projection with the K-norm in its epilogue, once
        torch.cuda.synchronize()
        print(json.dumps({"profile_run": w.name, "steps": args.steps, "warmup": args.warmup}))
        return
    head = Bench(w, torch, vb, dev, flush, peaks, replicas).run(
        args.steps, args.warmup, max(5, min(args.steps, 20)),
        args.cpu_seconds if solo and not args.no_cpu_baseline else 0, True, local)
    others = None
    if solo and not args.no_other_workloads:
        others = {}
        for name in ALL_WORKLOADS:
            if name == w.name:
                continue
            wo = W.workload(name)
            b = Bench(wo, torch, vb, dev, flush, peaks, replicas)
            r = b.run(30, 5, 5, 0 if args.no_cpu_baseline else min(args.cpu_seconds, 8.0), False, local)
            r["unit"], r["config"] = UNIT, config_of(wo)
            others[name] = r
            del b
            torch.cuda.empty_cache()

    if rank == 0:
        line = {
            "metric": METRIC, "value": head["value"], "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": head["ms_per_step"], "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": config_of(w, accumulate="f32", tokens_pruned_per_step=head["tokens_pruned_per_step"],
                                tokens_kept_after_each_stage=head["tokens_kept_after_each_stage"],
                                l2="flushed (512 MiB memset) before every timed step", sharding="replicas only"),
            "clocks": head["clocks"], "e2e": head["e2e"], "gpu_launches": head["gpu_launches_per_step"] * args.steps,
            "roofline": head["roofline"], "cpu_baseline": head["cpu_baseline"], "kernels": head["kernels"],
            "isolated": head["isolated"], "kproj_knorm": head["kproj_knorm"],
            "beside_the_step": head["beside_the_step"], "schedule": head["schedule"],
            "plain_step0": head["plain_step0"],
            "stage2_as_two_calls_us": head["stage2_as_two_calls_us"],
            "us_per_step_median": head["us_per_step_median"], "other_workloads": others,
        }
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=HEADLINE, choices=ALL_WORKLOADS)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-other-workloads", action="store_true", help="measure the headline workload only")
    ap.add_argument("--cpu-seconds", type=float, default=10.0, help="length of the CPU-oracle timing leg")
    ap.add_argument("--profile-run", action="store_true",
                    help="only run the workload's schedule (warm-up + steps) and exit: the command a profiler wraps")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.gpus > 1 and "RANK" not in os.environ:
        # invoked plainly: start the N ranks ourselves, one per GPU
        from paper_2601_17818_b200 import replicas
        raise SystemExit(replicas.launch_ranks(args.gpus, [os.path.abspath(__file__)] + sys.argv[1:]))
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
