#!/usr/bin/env python
"""Benchmark of the ViTCoP pruning operator chain on B200.

One "step" = one pass of the whole hot path over one batch of the LLaVA-1.5-shaped batch-16 workload
("c1"): redundancy filter (VIC clustering of the vision features, Algorithm 2) followed by the fused
pruning step (K-norm, Eq. 4 -> cluster-quota selection, Eq. 5 -> compaction of hidden states, K and V).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload c1]

Prints ONE JSON line.  `value` is visual tokens pruned per second with the inputs resident in HBM
(CUDA-event time per step, L2 flushed between steps); `e2e` is the same metric through the public API
with pinned HOST buffers, host<->device copies inside the timed region; `roofline` describes the kernel
that takes the largest share of the step, timed by CUDA events the library records around each of its
kernels; `cpu_baseline` is the CPU oracle timed on the host cores.  `--impl reference` times that oracle
(test infrastructure) instead of the CUDA path.
"""
from __future__ import annotations

import argparse
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

# DRAM bytes (read + write) per launch from the committed ncu captures under profiles/: kernel name ->
# (bytes per launch on the bench workload, sha1 of the kernel's source file when the counters were taken).
# A kernel whose source changed since reports traffic null.
NCU_TRAFFIC = {
    "gram_resident_kernel": (42614784 + 768, "65aadb1353cc"),       # features + the keys of its share of the K-norm
    "knorm_kernel": (51929856 + 19712, "8b9e2bc93897"),             # the samples the resident sweep leaves (11 of 16)
    "compact_kernel": (33756928 + 882432, "9a7b3fc1ee4a"),
}


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


def config_of(w, **extra):
    c = {"workload": w.name, "B": w.B, "Nv": w.Nv, "T": w.T, "H": w.H, "d": w.d, "D": w.D, "Dh": w.Dh,
         "budget": w.budgets[0], "n_centers": w.n_centers, "d_c": w.d_c, "tau": w.tau,
         "mode": "Stage II in one call (vitcop_collaborative_step): redundancy filter (cosine), K-norm, cluster-quota "
                 "selection, compaction"}
    c.update(extra)
    return c


# ------------------------------------------------------------------------------------------------ oracle legs
def oracle_step(w, feat, pos, K, V, hidden, budget):
    """One step of the hot path on the CPU oracle; returns the number of visual tokens pruned."""
    import oracle
    B = feat.shape[0]
    score = oracle.knorm(K, w.vis_start, w.Nv)
    pruned = 0
    for b in range(B):
        r = oracle.vic(feat[b], pos[b], 0, w.d_c, w.tau, w.n_centers)
        keep, _, _ = oracle.select_quota(score[b], r["label"], budget)
        oracle.compact(hidden[b], K[b], V[b], w.N, w.vis_start, w.Nv, keep, w.T + budget)
        pruned += w.Nv - len(keep)
    return pruned


class OracleBench:
    """The CPU oracle on a bounded sample (the first `sample_B` sequences) of the workload."""

    def __init__(self, w, sample_B):
        import oracle
        self.w, self.sample_B = w, sample_B
        self.feat, self.pos = W.make_features(w, B=sample_B), W.make_positions(w)[:sample_B]
        self.K, self.V = W.make_kv(w, 0, w.Nv, B=sample_B)
        self.hidden = W.make_hidden(w, B=sample_B)
        oracle.build()
        self.cores = oracle.num_threads()

    def step(self):
        return oracle_step(self.w, self.feat, self.pos, self.K, self.V, self.hidden, self.w.budgets[0])

    def run(self, steps, warmup):
        for _ in range(warmup):
            self.step()
        t0 = time.perf_counter()
        pruned = sum(self.step() for _ in range(steps))
        dt = time.perf_counter() - t0
        return pruned / dt, dt / steps

    def run_for(self, seconds, warmup=1):
        for _ in range(warmup):
            self.step()
        t0 = time.perf_counter()
        pruned, steps = 0, 0
        while steps < 3 or time.perf_counter() - t0 < seconds:
            pruned += self.step()
            steps += 1
        dt = time.perf_counter() - t0
        return pruned / dt, dt, steps


def run_reference(args):
    if int(os.environ.get("RANK", "0")) != 0:
        return
    w = W.workload(args.workload)
    sample_B = min(w.B, 4)
    ob = OracleBench(w, sample_B)
    value, sec_per_step = ob.run(args.steps, args.warmup)
    sample = (f"each step = the first {sample_B} of {w.B} sequences of workload {w.name}, whole hot path "
              f"(fp64 CPU oracle, OpenMP over rows)")
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
class Step:
    """Device buffers and the two API calls of one hot-path step."""

    def __init__(self, w, torch, vb, dev):
        self.w, self.torch, self.vb = w, torch, vb
        B, n = w.B, w.Nv
        self.budget = w.budgets[0]
        self.Ncap = w.T + self.budget
        e = lambda *s, dt=torch.bfloat16: torch.empty(s, dtype=dt, device=dev)
        self.feat, self.pos = e(B, n, w.D), e(B, n, 2, dt=torch.float32)
        self.K, self.V, self.hidden = e(B, w.H, w.N, w.d), e(B, w.H, w.N, w.d), e(B, w.N, w.Dh)
        self.label, self.ncl = e(B, n, dt=torch.int32), e(B, dt=torch.int32)
        self.ho, self.Ko, self.Vo = e(B, self.Ncap, w.Dh), e(B, w.H, self.Ncap, w.d), e(B, w.H, self.Ncap, w.d)
        self.olen, self.nkeep = e(B, dt=torch.int32), e(B, dt=torch.int32)
        self.kpos = e(B, self.Ncap, dt=torch.int32)
        self.ws_f = vb.alloc_workspace(vb.OP_FILTER, device=dev, B=B, Nv=n, D=w.D)
        self.ws_s = vb.alloc_workspace(vb.OP_PRUNE_STEP, device=dev, B=B, Nv=n)
        self.ws_c = vb.alloc_workspace(vb.OP_COLLAB_STEP, device=dev, B=B, Nv=n, D=w.D)

    def upload(self, host, non_blocking=True):
        for name in ("feat", "pos", "K", "V", "hidden"):
            getattr(self, name).copy_(host[name], non_blocking=non_blocking)

    def filter(self):
        w = self.w
        self.vb.vitcop_redundancy_filter(self.feat, self.pos, self.label, self.ncl, self.ws_f, metric=0, d_c=w.d_c,
                                         tau=w.tau, n_centers=w.n_centers)

    def prune(self):
        w = self.w
        self.vb.vitcop_prune_step(self.hidden, self.K, self.V, w.vis_start, w.Nv, w.Nv, self.budget, self.ho, self.Ko,
                                  self.Vo, self.olen, self.ws_s, label=self.label, kept_pos=self.kpos,
                                  n_keep_out=self.nkeep)

    def run(self):
        """The whole hot path through the one-call Stage II entry point (same results as filter() + prune())."""
        w = self.w
        self.vb.vitcop_collaborative_step(self.feat, self.pos, self.hidden, self.K, self.V, w.vis_start, self.budget,
                                          self.ho, self.Ko, self.Vo, self.olen, self.label, self.ncl, self.ws_c,
                                          metric=0, d_c=w.d_c, tau=w.tau, n_centers=w.n_centers, kept_pos=self.kpos,
                                          n_keep_out=self.nkeep)

    def run_two_calls(self):
        self.filter()
        self.prune()


def kernel_rooflines(w, nk_total, per_kernel, peaks):
    """Roofline entry of every kernel that has one: algorithmic bytes or flops per launch / measured duration.

    knorm:   reads the visual span of K once (B*H*Nv*d bf16) and writes B*Nv fp32 scores            -> HBM
    compact: reads and writes every surviving row of hidden, K and V once, plus the index arrays    -> HBM
    gram:    one sweep over the symmetric half of the Gram matrix incl. the diagonal, 2*D flop per pair,
             B*n*(n+1)/2 pairs                                                                         -> tensor cores
    The remaining kernels (row statistics, rho reduction, centres/labels, selection) move kilobytes and are
    latency-bound; they are reported in microseconds only.
    """
    rows_out = w.B * w.T + nk_total
    sweep = w.B * w.Nv * (w.Nv + 1) * w.D
    algo = {
        "gram_resident_kernel": ("tensor", sweep),      # one pass over the symmetric half serves norms, Eq. 2 and Eq. 3
        "knorm_kernel": ("hbm", w.B * w.H * w.Nv * w.d * 2 + w.B * w.Nv * 4),
        "compact_kernel": ("hbm", 2 * rows_out * (w.Dh + 2 * w.H * w.d) * 2 + rows_out * 4 + w.B * 12 + nk_total * 4),
        "gram_tc_kernel<rho>": ("tensor", w.B * w.Nv * (w.Nv + 1) * w.D),
        "gram_tc_kernel<delta>": ("tensor", w.B * w.Nv * (w.Nv + 1) * w.D),
    }
    src = {"knorm_kernel": "knorm.cu", "compact_kernel": "compact.cu", "gram_tc_kernel<rho>": "gram.cu",
           "gram_tc_kernel<delta>": "gram.cu", "gram_resident_kernel": "gram.cu"}
    out = {}
    for name, (launches, ms) in per_kernel.items():
        us = ms * 1e3 / max(launches, 1)
        e = {"launches": launches, "us_per_launch": us}
        if name == "knorm_kernel" and "gram_resident_kernel" in per_kernel:
            # the step's K-norm is split: some samples inside gram_resident_kernel, the others in this kernel
            e["note"] = "covers part of the samples only; the rest is computed inside gram_resident_kernel"
            if w.name == "c1" and NCU_TRAFFIC[name][1] == source_sha(src[name]):
                e["traffic"] = NCU_TRAFFIC[name][0]
        elif name in algo and us > 0:
            bound, units = algo[name]
            if bound == "hbm":
                ach, peak, unit = units / (us * 1e-6) / 1e9, peaks["hbm_gbs"], "GB/s"
            else:
                ach, peak, unit = units / (us * 1e-6) / 1e12, peaks["bf16_tflops"], "TFLOP/s"
            traffic = None                      # the counters were taken on workload c1 only
            if w.name == "c1" and name in NCU_TRAFFIC and NCU_TRAFFIC[name][1] == source_sha(src[name]):
                traffic = NCU_TRAFFIC[name][0]
            e.update(bound=bound, achieved=ach, peak=peak, unit=unit, frac=ach / peak, traffic=traffic,
                     algorithmic_units_per_launch=units)
        out[name] = e
    return out


def host_inputs(w, torch):
    """Seeded inputs of one workload as pinned host tensors."""
    feat_b, pos = W.make_features(w), W.make_positions(w)
    K_b, V_b = W.make_kv(w, 0, w.Nv)
    hid_b = W.make_hidden(w)
    bf = lambda a: torch.from_numpy(a.view(np.int16)).view(torch.bfloat16).pin_memory()
    return {"feat": bf(feat_b), "pos": torch.from_numpy(pos.copy()).pin_memory(), "K": bf(K_b), "V": bf(V_b),
            "hidden": bf(hid_b)}


def kernel_times(vb, torch, st, flush, reps):
    """Per-kernel (launches, total ms) of `reps` steps, from the library's own CUDA-event brackets."""
    for _ in range(3):
        flush.zero_()
        st.run()
    torch.cuda.synchronize()
    vb.vitcop_kernel_timing_begin()
    for _ in range(reps):
        flush.zero_()
        st.run()
    return vb.vitcop_kernel_timing_end()


def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2601_17818_b200 import binding as vb

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
    w = W.workload(args.workload)
    peaks = measured_peaks()

    # host inputs (pinned) ---------------------------------------------------------------------------
    host = host_inputs(w, torch)
    st = Step(w, torch, vb, dev)
    st.upload(host, non_blocking=False)
    flush = torch.empty(512 << 20, dtype=torch.uint8, device=dev)     # > 4x the 126 MB L2

    from paper_2601_17818_b200 import replicas
    barrier = replicas.barrier

    def timed(fn, steps, warmup):
        """Per-step CUDA-event times (ms) with an L2 flush before every step."""
        for _ in range(warmup):
            flush.zero_()
            fn()
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        barrier()
        for a, b in evs:
            flush.zero_()
            a.record()
            fn()
            b.record()
        barrier()
        return np.array([a.elapsed_time(b) for a, b in evs], dtype=np.float64)

    def max_over_ranks(x):
        return replicas.max_over_ranks(x, dev)

    # whole step, device resident ------------------------------------------------------------------------
    sampler = ClockSampler(local)
    sampler.start()
    t_step = timed(st.run, args.steps, args.warmup)
    clocks = sampler.stop()
    n_keep = st.nkeep.cpu().numpy()
    nk_total = int(n_keep.sum())
    pruned_per_step = int((w.Nv - n_keep).sum())
    total_ms = max_over_ranks(float(t_step.sum()))
    value = replicas.whole_job_rate(pruned_per_step, args.steps, float(t_step.sum()), dev)

    # per-kernel device times: the library brackets each of its kernels with CUDA events on the stream ----
    n_kt = max(10, min(args.steps, 50))
    per_kernel = kernel_times(vb, torch, st, flush, n_kt)
    kernels = kernel_rooflines(w, nk_total, per_kernel, peaks)
    # what a pair of event records adds to a kernel it brackets, measured on an empty-ish kernel: the per-kernel
    # times above (and the roofline fractions computed from them) include it, nothing is subtracted
    tiny = torch.zeros(32, device=dev)
    t_br = timed(lambda: tiny.zero_(), 20, 3)
    bracket_us = float(np.median(t_br) * 1e3)
    launches_per_step = sum(v[0] for v in per_kernel.values()) // n_kt
    dom = max(per_kernel, key=lambda k: per_kernel[k][1])
    roofline = {"kernel": dom}
    roofline.update({k: kernels[dom].get(k) for k in ("bound", "achieved", "peak", "unit", "frac", "traffic")})
    roofline.update(peak_source=peaks["source"] + (" burst" if kernels[dom].get("bound") == "tensor" else " copy"),
                    us_per_launch=kernels[dom]["us_per_launch"],
                    algorithmic_units_per_launch=kernels[dom].get("algorithmic_units_per_launch"),
                    share_of_step=per_kernel[dom][1] / sum(v[1] for v in per_kernel.values()),
                    event_bracket_overhead_us=bracket_us)

    # per-API-call times (same protocol as the step) -----------------------------------------------------------
    score = torch.empty((w.B, w.Nv), dtype=torch.float32, device=dev)
    kidx = torch.empty((w.B, w.Nv), dtype=torch.int32, device=dev)
    ws_sel = vb.alloc_workspace(vb.OP_SELECT, device=dev, B=w.B, Nv=w.Nv)
    stage_fns = {
        "filter_then_prune_step": st.run_two_calls,
        "filter": st.filter,
        "knorm": lambda: vb.vitcop_knorm_score(st.K, w.vis_start, w.Nv, score),
        "select": lambda: vb.vitcop_select(score, w.Nv, st.budget, kidx, st.nkeep, ws_sel, label=st.label),
        "compact": lambda: vb.vitcop_compact_kv(st.hidden, st.K, st.V, w.vis_start, w.Nv, kidx, st.nkeep, st.ho,
                                                st.Ko, st.Vo, st.olen, kept_pos=st.kpos),
        "prune_step": st.prune,
    }
    # the two stages around the core chain: cluster merge (Eq. 6) after the step, Stage I saliency (Eq. 1) before it
    kmask = torch.empty((w.B, w.Nv), dtype=torch.uint8, device=dev)
    vb.vitcop_select(score, w.Nv, st.budget, kidx, st.nkeep, ws_sel, label=st.label, keep_mask=kmask)
    m_lab = torch.empty((w.B, w.n_centers), dtype=torch.int32, device=dev)
    m_cnt, n_mrg = torch.empty_like(m_lab), torch.empty((w.B,), dtype=torch.int32, device=dev)
    m_rows = torch.empty((w.B, w.n_centers, w.Dh), dtype=torch.bfloat16, device=dev)
    vit_H, vit_M, vit_d = 16, 577, 64                   # CLIP ViT-L/14-336: 16 heads of 64, [CLS] + 576 patches
    q_b, Kv_b = W.make_cls_qk(w.seed, w.B, vit_H, vit_M, vit_d)
    q_cls, K_vit = vb.bf16_tensor(q_b, dev), vb.bf16_tensor(Kv_b, dev)
    sal = torch.empty((w.B, vit_M - 1), dtype=torch.float32, device=dev)
    ws_sal = vb.alloc_workspace(vb.OP_SALIENCY, device=dev, B=w.B, H=vit_H, N=vit_M)
    ws_mrg = vb.alloc_workspace(vb.OP_MERGE, device=dev, B=w.B, Nv=w.Nv, N=w.n_centers)
    stage_fns["merge"] = lambda: vb.vitcop_merge_clusters(st.hidden, w.vis_start, w.Nv, st.label, kmask, m_lab, m_cnt,
                                                          n_mrg, ws_mrg, merged=m_rows)
    stage_fns["cls_saliency"] = lambda: vb.vitcop_cls_saliency(q_cls, K_vit, vit_d ** -0.5, sal, ws_sal)
    stage = {}
    for name, fn in stage_fns.items():
        t = timed(fn, n_kt, 3)
        stage[name] = {"us_median": float(np.median(t) * 1e3), "us_min": float(t.min() * 1e3)}
    merged_rows = int(m_cnt.cpu().numpy()[np.arange(w.n_centers)[None, :] < n_mrg.cpu().numpy()[:, None]].sum())
    for name, nbytes in (("merge", (merged_rows + int(n_mrg.sum())) * w.Dh * 2 + w.B * w.Nv * 5),
                         ("cls_saliency", w.B * vit_H * vit_M * vit_d * 2 + w.B * vit_H * vit_M * 8)):
        gbs = nbytes / (stage[name]["us_median"] * 1e-6) / 1e9
        stage[name].update(algorithmic_bytes=nbytes, gbs=gbs, frac_of_measured_hbm=gbs / peaks["hbm_gbs"])

    # end to end through the public API with host buffers ----------------------------------------------------
    # Every step copies its five inputs from pinned host memory and its outputs back.  The copies of neighbouring
    # steps overlap the way a serving loop would run them: two sets of device buffers, an upload stream, the compute
    # stream and a download stream chained by events; step s + 1 uploads while step s computes and step s - 1
    # downloads.  Each step's inputs (270 MB on c1) exceed the L2, so no flush is needed between steps.
    sets = [st, Step(w, torch, vb, dev)]
    outs = [{k: torch.empty(getattr(x, k).shape, dtype=getattr(x, k).dtype).pin_memory()
             for k in ("ho", "Ko", "Vo", "olen", "kpos")} for x in sets]
    s_up, s_down = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
    s_main = torch.cuda.current_stream()

    def e2e_run(steps):
        ev_in = [torch.cuda.Event() for _ in range(steps)]
        ev_done = [torch.cuda.Event() for _ in range(steps)]
        ev_out = [torch.cuda.Event() for _ in range(steps)]
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        t0.record(s_main)
        s_up.wait_event(t0)
        for i in range(steps):
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
                for k in ("ho", "Ko", "Vo", "olen", "kpos"):
                    o[k].copy_(getattr(x, k), non_blocking=True)
                ev_out[i].record(s_down)
        for e in ev_out[-2:]:
            s_main.wait_event(e)
        t1.record(s_main)
        barrier()
        return t0.elapsed_time(t1)

    n_e2e = max(5, min(args.steps, 20))
    e2e_run(3)
    e2e_ms = max_over_ranks(float(e2e_run(n_e2e)))
    h2d = sum(int(v.numel() * v.element_size()) for v in host.values())
    d2h = sum(int(v.numel() * v.element_size()) for v in outs[0].values())
    e2e = {"value": world * pruned_per_step * n_e2e / (e2e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
           "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms / n_e2e,
           "protocol": "uploads, compute and downloads of neighbouring steps overlap (3 streams, 2 buffer sets)"}

    # CPU oracle beside it (rank 0, N = 1 only; bounded sample of about 10 s) ---------------------------------
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        sample_B = min(w.B, 4)
        ob = OracleBench(w, sample_B)
        v, secs, passes = ob.run_for(args.cpu_seconds)
        cpu = {"value": v, "unit": UNIT, "cores": ob.cores, "kind": "oracle",
               "sample": f"the first {sample_B} of {w.B} sequences of workload {w.name}, whole hot path, "
                         f"{passes} passes in {secs:.1f} s"}

    # the larger workloads, same protocol, fewer steps (context for the fractions: c1 is latency-bound) --------
    others = None
    if rank == 0 and world == 1 and not args.no_other_workloads:
        others = {}
        for name in ("c2", "c3", "c4"):
            wo = W.workload(name)
            so = Step(wo, torch, vb, dev)
            so.upload(host_inputs(wo, torch), non_blocking=False)
            t = timed(so.run, 20, 3)
            nko = so.nkeep.cpu().numpy()
            pk = kernel_times(vb, torch, so, flush, 10)
            ks = kernel_rooflines(wo, int(nko.sum()), pk, peaks)
            others[name] = {"us_per_step_median": float(np.median(t) * 1e3),
                            "value": float((wo.Nv - nko).sum() / (np.median(t) * 1e-3)), "unit": UNIT,
                            "config": config_of(wo),
                            "kernels": {k: {a: v[a] for a in ("us_per_launch", "bound", "achieved", "unit", "frac")
                                            if a in v} for k, v in ks.items()}}
            del so
            torch.cuda.empty_cache()

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": total_ms / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": config_of(w, accumulate="f32", tokens_pruned_per_step=pruned_per_step,
                                tokens_kept_per_step=nk_total,
                                l2="flushed (512 MiB memset) before every timed step", sharding="replicas only"),
            "clocks": clocks, "e2e": e2e, "gpu_launches": launches_per_step * args.steps,
            "roofline": roofline, "cpu_baseline": cpu, "kernels": kernels, "stages": stage,
            "other_workloads": others,
            "us_per_step_median": float(np.median(t_step) * 1e3),
        }
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c1")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-other-workloads", action="store_true", help="skip the c2-c4 summary (N = 1 only)")
    ap.add_argument("--cpu-seconds", type=float, default=10.0, help="length of the CPU-oracle timing leg")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
