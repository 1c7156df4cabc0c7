#!/usr/bin/env python
"""Benchmark of the dKV-Cache denoising step on B200.

A "step" is one denoising step of the whole hot path (policy + compaction,
embedding gather, every layer, vocabulary head, confidence selection).  The
default workload is the LLaDA-8B-shaped configuration: 32 layers, d=4096,
32x128 heads, FFN 12288, vocab 126464, batch 1, prompt 256 + 256 generated in
blocks of 32, one token per step, dKV-Cache-Decode with a refresh every 8
steps.  Synthetic seeded weights and prompt (there are no trained weights or
datasets here).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Prints ONE JSON line.  With --gpus N > 1 (under torchrun) every rank runs an
independent replica (sequences are independent: no data-path collective);
the value is the sum of the ranks' tokens over the slowest rank's time.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

WORKLOADS = {
    # name: (shape fn, batch, prompt, gen, block, k, policy kind, interval, window)
    "llada8b_decode": dict(shape="llada", batch=1, prompt=256, gen=256, block=32, k=1, policy="decode",
                           interval=8, window=0),
    "llada8b_nocache": dict(shape="llada", batch=1, prompt=256, gen=256, block=32, k=1, policy="none",
                            interval=0, window=0),
    "dream7b_pd": dict(shape="dream", batch=4, prompt=512, gen=256, block=256, k=2, policy="pd", interval=16,
                       window=0),
    "llada8b_greedy": dict(shape="llada", batch=1, prompt=128, gen=1024, block=1024, k=1, policy="greedy",
                           interval=2, window=4),
    # the comparison runs of the same shape (prompt 128, generation 1024, no blocks, one token per step)
    "llada8b_long_nocache": dict(shape="llada", batch=1, prompt=128, gen=1024, block=1024, k=1, policy="none",
                                 interval=0, window=0),
    "llada8b_long_decode": dict(shape="llada", batch=1, prompt=128, gen=1024, block=1024, k=1, policy="decode",
                                interval=8, window=0),
    # depth-truncated copy of the default workload (a few GB on the device): the case ncu captures
    "llada8b_decode_2layers": dict(shape="llada", layers=2, batch=1, prompt=256, gen=256, block=32, k=1,
                                   policy="decode", interval=8, window=0),
    "tiny_decode": dict(shape="tiny", batch=1, prompt=32, gen=32, block=32, k=1, policy="decode", interval=8,
                        window=0),
}


# DRAM traffic (read + write) per launch of the projection GEMMs: a RECORDED constant from the ncu capture
# summarised in profiles/k_gemm_tc_llada8b_decode_2layers.md (256 active rows; per launch, independent of
# depth), not measured by this run.
NCU_GEMM_TRAFFIC = {"gemm_qkv": 106.8e6, "gemm_o": 41.4e6, "gemm_gateup": 206.8e6, "gemm_down": 114.7e6}
NCU_GEMM_TRAFFIC_SOURCE = "ncu capture summarised in profiles/k_gemm_tc_llada8b_decode_2layers.md (recorded constant)"


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return dict(hbm=d["hbm_gbs"], tf_burst=d["bf16_tflops"], tf_sust=d["bf16_tflops_sustained"], src="measured")
    return dict(hbm=6650.0, tf_burst=1590.0, tf_sust=1400.0, src="fallback")


def reduce_max(value: float, world: int, device="cuda") -> float:
    """Max over ranks (the slowest replica decides the job's time)."""
    if world <= 1:
        return float(value)
    import torch
    import torch.distributed as dist
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput(tokens_per_rank: int, world: int, ms_local: float, device="cuda"):
    """Whole-job tokens/s of `world` independent replicas: all ranks' tokens over the slowest rank's time."""
    ms = reduce_max(ms_local, world, device)
    return tokens_per_rank * world / (ms * 1e-3), ms


class ClockSampler:
    """nvidia-smi clocks and throttle reasons while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.rows, self.proc, self.index = [], None, index

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "100", "-i", str(self.index)], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
            self.thr = threading.Thread(target=self._read, daemon=True)
            self.thr.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            self.proc.kill()
        sm, mx, reasons, pw = [], [], set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0])); mx.append(float(r[1])); pw.append(float(r[2]))
            except Exception:
                continue
            for n, v in zip(names, r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w_max": max(pw) if pw else None, "samples": len(sm), "reasons": sorted(reasons)}


def step_costs(ms, wl, rows, full_rows):
    """Algorithmic cost of one step with `rows` active rows in total (all sequences) whose queries attend
    `full_rows` slots per sequence: weight bytes (every projection matrix and the head once: the per-step
    figure of the hot-path table), K/V slot bytes, flops."""
    d, L = ms.d_model, full_rows
    w_bytes = 2.0 * (ms.n_layers * ms.params_per_layer() + ms.vocab * d)
    kv_bytes = 2.0 * 2 * wl["batch"] * L * ms.d_kv * ms.n_layers
    head_rows = min(wl["block"], wl["gen"]) * wl["batch"]
    flops = 2.0 * rows * ms.n_layers * ms.params_per_layer() + 4.0 * rows * L * ms.d_q * ms.n_layers + \
        2.0 * head_rows * ms.vocab * d
    return w_bytes, kv_bytes, flops


def shape_of(wl):
    from paper_2505_15781_b200 import synth
    ms = {"llada": synth.llada_shape, "dream": synth.dream_shape, "tiny": synth.tiny_shape}[wl["shape"]]()
    return ms.with_layers(wl["layers"]) if "layers" in wl else ms


# --------------------------------------------------------------------------
# our arm
# --------------------------------------------------------------------------

class Job:
    """One replica of the workload on the current device."""

    def __init__(self, wl, seed=0, order=None, model=None):
        """order: [T, batch, k] device tensor of positions to unmask (a recorded or predefined order; required
        for Greedy, optional replay for the other policies).  model: reuse a built model of the same shape."""
        import torch
        from paper_2505_15781_b200 import binding as B
        from paper_2505_15781_b200 import synth
        self.torch, self.B, self.synth, self.wl = torch, B, synth, wl
        ms = shape_of(wl)
        self.ms = ms
        bf16 = wl["shape"] != "tiny"
        self.dtype = "bf16" if bf16 else "f32"
        if model is None:
            w = synth.make_weights(ms, seed, "bfloat16" if bf16 else "float32", "cuda")
            model = B.dkv_model_create(ms, w, B.DKV_BF16 if bf16 else B.DKV_F32)
            del w
        self.model = model
        kind = {"decode": B.DKV_POLICY_DECODE, "none": B.DKV_POLICY_NONE, "pd": B.DKV_POLICY_PD,
                "prefill": B.DKV_POLICY_PREFILL, "greedy": B.DKV_POLICY_GREEDY}[wl["policy"]]
        self.policy = B.make_policy(kind, wl["interval"], 1, wl["window"], B.DKV_CENTER_PREV,
                                    max_head_rows=wl["block"], max_k=wl["k"])
        self.P, self.G, self.k, self.batch = wl["prompt"], wl["gen"], wl["k"], wl["batch"]
        self.L = self.P + self.G
        self.T = self.G // self.k
        prompts = synth.make_prompt(self.batch, self.P, ms.vocab - 1, seed)
        x0, m0 = synth.initial_state(prompts, self.G, ms.mask_id)
        self.x0, self.m0 = torch.from_numpy(x0).cuda(), torch.from_numpy(m0).cuda()
        self.x, self.m = self.x0.clone(), self.m0.clone()
        self.order = order
        if wl["policy"] == "greedy" and order is None:
            self.order = torch.from_numpy(synth.random_order(self.batch, self.P, self.G, self.k, seed)).cuda()
        need = B.dkv_cache_bytes(self.model, self.batch, self.L, self.policy)
        self.arena = torch.empty(need + 256, dtype=torch.uint8, device="cuda")
        self.cache = None
        self.pos = self.T          # forces a (re)start
        self.launches = 0

    def restart(self):
        if self.cache is not None:
            self.launches += self.B.dkv_get_stats(self.cache).kernel_launches
        self.cache = self.B.dkv_init_cache(self.model, self.batch, self.L, self.P, self.policy, arena=self.arena)
        self.x.copy_(self.x0)
        self.m.copy_(self.m0)
        self.pos = 0

    def total_launches(self):
        return self.launches + (self.B.dkv_get_stats(self.cache).kernel_launches if self.cache else 0)

    def record_order(self):
        """One whole generation; returns the positions it unmasked, [T, batch, k] on the device."""
        self.restart()
        chosen = self.torch.full((self.T, self.batch, self.k), -1, dtype=self.torch.int32, device="cuda")
        self.B.dkv_generate(self.cache, self.x, self.m, self.order, self.k, self.wl["block"], 0, chosen)
        self.torch.cuda.synchronize()
        self.pos = self.T
        return chosen

    def run_steps(self, n, profile_cb=None):
        """n consecutive denoising steps on the device (generations wrap)."""
        done = 0
        while done < n:
            if self.pos >= self.T:
                self.restart()
            chunk = min(n - done, self.T - self.pos)
            if profile_cb is None:
                self.B.dkv_generate(self.cache, self.x, self.m, self.order, self.k, self.wl["block"], chunk)
                self.pos += chunk
                done += chunk
            else:
                for _ in range(chunk):
                    self.B.dkv_generate(self.cache, self.x, self.m, self.order, self.k, self.wl["block"], 1)
                    profile_cb(self.pos)
                    self.pos += 1
                    done += 1

    def active_rows(self, s):
        """Rows one sequence recomputes at 0-based step s (the host-side bound the library is given)."""
        pol = self.wl["policy"]
        if pol == "none" or s == 0:
            return self.L
        if pol == "prefill" or (pol == "pd" and self.is_refresh(s)):
            return self.G
        if self.is_refresh(s):
            return self.L
        if pol == "greedy":
            return min(self.L, self.k * (self.wl["window"] + 2))
        return min(self.L, self.G - s * self.k + self.k)

    def is_refresh(self, s):
        pol, N = self.wl["policy"], self.wl["interval"]
        if pol == "none" or s == 0:
            return True
        if pol == "prefill":
            return False
        return N > 0 and s % N == 0


def run_ours(args, rank, world):
    import torch
    import torch.distributed as dist
    from paper_2505_15781_b200 import binding as B
    dev = int(os.environ.get("LOCAL_RANK", 0))
    torch.cuda.set_device(dev)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", dev))
    wl = WORKLOADS[args.workload]
    job = Job(wl, seed=rank)
    K, W = args.steps, max(args.warmup, 3)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ------------------------------------------------ device-resident timing
    # A step's cost depends on where in the generation it falls (the active set shrinks, every N-th
    # step is a full one).  K = one generation (the default) times all of it; a shorter run times the K
    # steps in the MIDDLE of a generation, reached by untimed steps, so that it stays representative.
    first = max(0, (job.T - K) // 2) if K < job.T else 0
    job.run_steps(W)
    job.restart()
    job.run_steps(first)
    barrier()
    l0 = job.total_launches()
    sampler = ClockSampler(dev)
    sampler.start()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    job.run_steps(K)
    ev1.record()
    barrier()
    ms = ev0.elapsed_time(ev1)
    clocks = sampler.stop()
    launches = job.total_launches() - l0
    status = B.dkv_status(job.cache)
    value, ms = job_throughput(K * job.k * job.batch, world, ms)

    # ------------------------------------------------ end to end (host buffers)
    job.restart()
    xh = torch.empty(job.batch, job.L, dtype=torch.int32).pin_memory()
    mh = torch.empty(job.batch, job.L, dtype=torch.uint8).pin_memory()
    ch = torch.empty(job.batch, job.k, dtype=torch.int32).pin_memory()
    oh = job.order.cpu().pin_memory() if job.order is not None else None
    e2e_K = min(K, job.T)

    def e2e_pass(n, begin=0):
        xh.copy_(job.x0.cpu()); mh.copy_(job.m0.cpu())
        job.restart()
        t0 = time.perf_counter()
        for s in range(begin + n):
            if s == begin:
                torch.cuda.synchronize()
                t0 = time.perf_counter()
            blk = s // (wl["block"] // job.k)
            lo = job.P + blk * wl["block"]
            B.dkv_step_host(job.cache, xh, mh, oh[s] if oh is not None else None, job.k, lo, lo + wl["block"],
                            job.G - s * job.k, ch)
        return time.perf_counter() - t0
    e2e_pass(min(3, e2e_K))
    barrier()
    e2e_s = e2e_pass(e2e_K, first)
    e2e_s = reduce_max(e2e_s, world)
    BL = job.batch * job.L
    e2e = {"value": e2e_K * job.k * job.batch * world / e2e_s, "unit": "tokens/s", "steps": e2e_K,
           "ms_per_step": e2e_s * 1e3 / e2e_K, "h2d_bytes_per_step": BL * 5 + (job.batch * job.k * 4 if oh is not None else 0),
           "d2h_bytes_per_step": BL * 5 + job.batch * job.k * 4}

    # ------------------------------------------------ per-kernel pass (events around every launch)
    pk = peaks()
    roofline, roofline_tensor, roofline_attn, classes = None, None, None, {}
    if rank == 0:
        n_prof = min(K, job.T)

        def profile_pass():
            """Events around every launch of steps first .. first + n_prof - 1, by step kind and kernel class."""
            job.restart()
            job.run_steps(first)
            torch.cuda.synchronize()
            B.dkv_profile_enable(job.cache, True)
            res = {"cached": {}, "refresh": {}}

            def cb(s):
                bucket = res["refresh" if job.is_refresh(s) else "cached"]
                for e in B.dkv_profile_read(job.cache):
                    a = bucket.setdefault(e["name"], dict(launches=0, ms=0.0, bytes=0.0, flops=0.0))
                    for key in ("launches", "ms", "bytes", "flops"):
                        a[key] += e[key]
            job.run_steps(n_prof, profile_cb=cb)
            B.dkv_profile_enable(job.cache, False)
            return res
        agg = profile_pass()
        # The same pass with the row tails as kernels of their own (DKV_FUSE_TAILS=0 is read when a handle
        # is created): the GEMM launches then hold the projection alone, which is what a per-launch
        # weight-streaming fraction should be read against; the tails show up as row-kernel classes.
        os.environ["DKV_FUSE_TAILS"] = "0"
        try:
            agg_plain = profile_pass()
        finally:
            del os.environ["DKV_FUSE_TAILS"]
            job.restart()
        ms_shape = job.ms

        # weight bytes of one launch of each GEMM class (the hot-path table's per-unit figure: 2 K N)
        d_, f_ = ms_shape.d_model, ms_shape.d_ffn
        w_bytes = {"gemm_qkv": 2.0 * (ms_shape.d_q + 2 * ms_shape.d_kv) * d_, "gemm_o": 2.0 * d_ * ms_shape.d_q,
                   "gemm_gateup": 2.0 * 2 * f_ * d_, "gemm_down": 2.0 * d_ * f_, "gemm_head": 2.0 * ms_shape.vocab * d_}

        def gemm_sum(bucket):
            tot = dict(launches=0, ms=0.0, bytes=0.0, flops=0.0, weight_bytes=0.0)
            for name, a in bucket.items():
                if name.startswith("gemm_"):
                    for key in ("launches", "ms", "bytes", "flops"):
                        tot[key] += a[key]
                    tot["weight_bytes"] += a["launches"] * w_bytes[name]
            return tot
        gc, gr = gemm_sum(agg["cached"]), gemm_sum(agg["refresh"])
        traffic = None
        if wl["shape"] == "llada":
            cls = [(n, a["launches"]) for n, a in agg["cached"].items() if n in NCU_GEMM_TRAFFIC and a["launches"]]
            if cls:
                traffic = sum(NCU_GEMM_TRAFFIC[n] * c for n, c in cls) / sum(c for _, c in cls)
        if gc["launches"]:
            ach = gc["weight_bytes"] / (gc["ms"] * 1e-3) / 1e9
            ach_full = gc["bytes"] / (gc["ms"] * 1e-3) / 1e9
            roofline = {"bound": "hbm",
                        "kernel": "k_gemm_tc / k_gemm_tc2 (tcgen05 projection GEMMs with their fused row tails: split-K "
                                  "reduction, residual, norm statistics, RoPE, K/V scatter, SwiGLU, head statistics), "
                                  "launches of the cached steps",
                        "achieved": ach, "peak": pk["hbm"], "unit": "GB/s", "frac": ach / pk["hbm"],
                        "bytes": "weights only (2 K N per launch)",
                        "peak_source": f"of {pk['src']}", "peak_nominal": 7700.0, "frac_of_nominal": ach / 7700.0,
                        "with_rows_and_outputs": {"achieved": ach_full, "frac": ach_full / pk["hbm"],
                                                  "bytes": "weights + row operands + results"},
                        "traffic": traffic, "traffic_source": NCU_GEMM_TRAFFIC_SOURCE,
                        "launches": gc["launches"], "avg_launch_us": gc["ms"] * 1e3 / gc["launches"],
                        "algorithmic_bytes_per_launch": gc["weight_bytes"] / gc["launches"]}
            gp = gemm_sum(agg_plain["cached"])
            if gp["launches"]:
                rows_ms = sum(a["ms"] for n, a in agg_plain["cached"].items() if n in ("resid_norm", "qkv_rope_scatter", "swiglu"))
                tot_plain = sum(a["ms"] for a in agg_plain["cached"].values())
                tot_fused = sum(a["ms"] for a in agg["cached"].values())
                ach_p = gp["weight_bytes"] / (gp["ms"] * 1e-3) / 1e9
                roofline["row_tails_as_kernels"] = {
                    "achieved": ach_p, "frac": ach_p / pk["hbm"], "avg_launch_us": gp["ms"] * 1e3 / gp["launches"],
                    "row_kernel_share_of_cached_steps": rows_ms / tot_plain if tot_plain else None,
                    "cached_steps_event_ms": {"tails_fused": tot_fused, "tails_as_kernels": tot_plain},
                    "what": "the same steps with DKV_FUSE_TAILS=0: GEMM launches hold the projection alone (weights "
                            "only / launch time), the split-K reduction, residual, norm statistics, RoPE and scatter "
                            "run as row kernels"}
        if gr["launches"]:
            ach = gr["flops"] / (gr["ms"] * 1e-3) / 1e12
            roofline_tensor = {"bound": "tensor", "kernel": "k_gemm_tc / k_gemm_tc2, launches of the refresh steps "
                                                            "(each timed alone between events: burst peak)",
                               "achieved": ach, "peak": pk["tf_burst"], "unit": "TFLOP/s", "frac": ach / pk["tf_burst"],
                               "peak_source": f"of {pk['src']} (burst)", "frac_of_sustained": ach / pk["tf_sust"],
                               "peak_nominal": 2250.0, "frac_of_nominal": ach / 2250.0, "launches": gr["launches"],
                               "avg_launch_us": gr["ms"] * 1e3 / gr["launches"]}
            if roofline is None:
                roofline = dict(roofline_tensor, traffic=None)
        # attention against both rooflines, from the same event pass (all steps)
        att = dict(launches=0, ms=0.0, bytes=0.0, flops=0.0)
        for bucket in agg.values():
            if "attention" in bucket:
                for key in att:
                    att[key] += bucket["attention"][key]
        if att["launches"]:
            tf = att["flops"] / (att["ms"] * 1e-3) / 1e12
            gb = att["bytes"] / (att["ms"] * 1e-3) / 1e9
            roofline_attn = {"kernel": "k_attn_tc (tcgen05 attention over the slot cache)", "launches": att["launches"],
                             "avg_launch_us": att["ms"] * 1e3 / att["launches"], "TFLOP/s": tf,
                             "frac_of_tensor_peak": tf / pk["tf_burst"], "GB/s": gb, "frac_of_hbm_peak": gb / pk["hbm"],
                             "note": "launches of this size are latency-bound (few CTAs, few slot tiles each)"}
        # Whole-window figure: roofline time of the timed steps (each step the slower of its flops at the
        # sustained tensor peak and its weight + K/V bytes at the HBM peak) over the measured time.
        t_roof = 0.0
        for s_i in range(first, first + K):
            si = s_i % job.T
            rows = job.batch * job.active_rows(si)
            wb, kvb, fl = step_costs(ms_shape, wl, rows, job.L)
            t_roof += max(fl / (pk["tf_sust"] * 1e12), (wb + kvb) / (pk["hbm"] * 1e9))
        if roofline is not None:
            roofline["whole_window"] = {"roofline_ms": t_roof * 1e3, "measured_ms": ms, "frac": t_roof * 1e3 / ms,
                                        "how": "sum over the timed steps of max(flops / sustained tensor peak, "
                                               "(weight + K/V bytes) / HBM peak), over the device time of the region"}
        for bname, bucket in agg.items():
            tot = sum(a["ms"] for a in bucket.values()) or 1.0
            classes[bname] = {n: {"launches": a["launches"], "ms": round(a["ms"], 3), "share": round(a["ms"] / tot, 4)}
                              for n, a in sorted(bucket.items(), key=lambda kv: -kv[1]["ms"]) if a["launches"]}

    out = None
    if rank == 0:
        st = B.dkv_get_stats(job.cache)
        out = {
            "metric": "generated tokens/s (dKV-Cache denoising steps, whole hot path)",
            "value": value, "unit": "tokens/s", "n_gpus": world, "steps": K, "warmup": W,
            "ms_per_step": ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16 weights as fp16, fp16 operands, fp32 accumulate" if job.dtype == "bf16" else "f32",
            "data": "synthetic",
            "config": {"workload": args.workload, **{k: v for k, v in wl.items()}},
            "timed_steps": f"steps {first}..{first + K - 1} of the {job.T}-step generation",
            "l2": "inputs larger than L2: every step streams all weights (16 GB) once",
            "replicas": "independent replica per GPU, no collective on the data path",
            "memory": {"arena_bytes": int(job.arena.numel()), "kv_slot_bytes": int(st.cache_bytes)},
            "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches), "device_status": status,
            "roofline": roofline, "roofline_refresh_steps": roofline_tensor, "roofline_attention": roofline_attn,
            "kernel_classes": classes,
        }
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    return out


# --------------------------------------------------------------------------
# CPU oracle legs
# --------------------------------------------------------------------------

def oracle_stepper(wl, n_layers, seed=0):
    """The oracle's sampler on a depth-truncated model of the workload's shape."""
    import torch
    from oracle import dkv_oracle as O
    from paper_2505_15781_b200 import synth
    ms = shape_of(wl).with_layers(n_layers)
    dev = "cuda" if torch.cuda.is_available() else "cpu"
    bf16 = wl["shape"] != "tiny"
    w = synth.make_weights(ms, seed, "bfloat16" if bf16 else "float32", dev)
    W = synth.weights_to_numpy(w, np.float32)
    del w
    model = O.Model(ms.n_layers, ms.d_model, ms.n_q_heads, ms.n_kv_heads, ms.head_dim, ms.d_ffn, ms.vocab, ms.mask_id,
                    ms.rope_theta, ms.rms_eps)
    kind = {"decode": O.POLICY_DECODE, "none": O.POLICY_NONE, "pd": O.POLICY_PD, "prefill": O.POLICY_PREFILL,
            "greedy": O.POLICY_GREEDY}[wl["policy"]]
    pol = O.Policy(kind, wl["interval"], 1, wl["window"])
    prompt = synth.make_prompt(wl["batch"], wl["prompt"], ms.vocab - 1, seed)[0]
    order = synth.random_order(wl["batch"], wl["prompt"], wl["gen"], wl["k"], seed)[:, 0, :] if kind == O.POLICY_GREEDY else None
    return O.Sampler(model, W, prompt, wl["gen"], wl["k"], pol, wl["block"], order, form="slots", dtype=np.float32)


def oracle_time_steps(wl, n_steps, budget_s):
    """Time the oracle on one sequence: per step, a 1-layer and a 0-layer model
    are stepped; full depth is extrapolated as t0 + n_layers * (t1 - t0)."""
    full_layers = shape_of(wl).n_layers
    s1, s0 = oracle_stepper(wl, 1), oracle_stepper(wl, 0)
    per_step, t_begin = [], time.perf_counter()
    for i in range(n_steps):
        a = time.perf_counter(); s1.step(); b = time.perf_counter(); s0.step(); c = time.perf_counter()
        t1, t0 = b - a, c - b
        per_step.append(t0 + full_layers * max(t1 - t0, 0.0))
        if time.perf_counter() - t_begin > budget_s:
            break
    return per_step


def cpu_baseline(wl, budget_s=25.0):
    per = oracle_time_steps(wl, 4, budget_s)
    n = len(per)
    return {"value": n * wl["k"] / sum(per), "unit": "tokens/s", "cores": os.cpu_count(), "kind": "oracle",
            "sample": f"steps 1-{n} of the workload, one sequence (1 full step + {n - 1} cached), numpy fp32; "
                      f"a 1-layer and a 0-layer model are timed and the layer time is scaled to full depth "
                      f"(extrapolated)"}


def run_reference(args, rank, world):
    if rank != 0:
        return None
    wl = WORKLOADS[args.workload]
    K = args.steps
    T = wl["gen"] // wl["k"]
    t_wall = time.perf_counter()
    per = oracle_time_steps(wl, min(K, T), budget_s=200.0)
    t_wall = time.perf_counter() - t_wall
    n = len(per)
    total = sum(per)
    val = n * wl["k"] / total
    return {"impl": "reference", "metric": "generated tokens/s (dKV-Cache denoising steps, whole hot path)",
            "value": val, "unit": "tokens/s", "n_gpus": world, "steps": K, "warmup": args.warmup,
            "ms_per_step": total * 1e3 / n, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic", "config": {"workload": args.workload, **wl},
            "extrapolated": True, "sample_wall_s": t_wall,
            "note": "ms_per_step is the full-depth step time extrapolated from a 1-layer and a 0-layer model "
                    "(t0 + n_layers * (t1 - t0)); sample_wall_s is what this run actually spent stepping them",
            "cpu_baseline": {"value": val, "unit": "tokens/s", "cores": os.cpu_count(), "kind": "oracle",
                             "sample": f"first {n} of {K} steps, one sequence; per step a 1-layer and a 0-layer model "
                                       f"are timed and the layer time scaled to full depth (extrapolated)"},
            "e2e": {"value": val, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}


def timed_generation_steps(job, steps):
    """Device time of `steps` consecutive steps from the middle of a generation (all of it when steps >= T)."""
    import torch
    steps = min(steps, job.T)
    first = (job.T - steps) // 2
    job.run_steps(3)
    job.restart()
    job.run_steps(first)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    job.run_steps(steps)
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1), steps, first


def run_order_comparison(args):
    """The long-generation comparison (prompt 128, generation 1024, no blocks, one token per step): the
    no-cache run picks its positions by confidence; that order is recorded and REPLAYED by dKV-Cache-Decode
    (refresh every 8 steps) and dKV-Cache-Greedy (window 4, refresh every 2 / every 8 / never), so that all
    runs traverse one decoding order (Sec. 3.4: Greedy needs the position before the forward pass).
    One JSON line per run; tokens/s over a whole generation unless --steps is smaller."""
    import torch
    from paper_2505_15781_b200 import binding as B
    torch.cuda.set_device(0)
    base = WORKLOADS["llada8b_long_nocache"]
    ref = Job(base)
    order = ref.record_order()
    rows = []
    for name, pol, interval, window in (("no-cache", "none", 0, 0), ("decode N=8", "decode", 8, 0),
                                        ("greedy N=2 w=4", "greedy", 2, 4), ("greedy N=8 w=4", "greedy", 8, 4),
                                        ("greedy no refresh w=4", "greedy", 0, 4)):
        wl = dict(base, policy=pol, interval=interval, window=window)
        job = Job(wl, order=order, model=ref.model)
        ms, steps, first = timed_generation_steps(job, args.steps)
        st = B.dkv_get_stats(job.cache)
        assert B.dkv_status(job.cache) == 0
        row = {"sweep": "order_comparison", "run": name, "prompt": wl["prompt"], "gen": wl["gen"], "steps": steps,
               "first_step": first, "order": "recorded from the no-cache confidence run, replayed",
               "tokens_per_s": steps * job.k * job.batch / (ms * 1e-3), "ms_per_step": ms / steps,
               "cache_ratio": st.cache_ratio, "kv_slot_bytes": int(st.cache_bytes), "arena_bytes": int(job.arena.numel())}
        rows.append(row)
        row["speedup_vs_nocache"] = row["tokens_per_s"] / rows[0]["tokens_per_s"]
        print(json.dumps(row), flush=True)
        del job
        torch.cuda.empty_cache()


def run_length_sweep(args):
    """Speed and memory against decode length and prefill length (the paper's memory-and-speed study,
    Sec. 4.3): generation length x prompt length for no-cache, Decode N=8, Greedy N=2 and N=8 (window 4,
    seeded random order), LLaDA-8B-shaped, batch 1, one token per step.  Each point times --steps steps
    from the middle of its generation.  One JSON line per point."""
    import torch
    from paper_2505_15781_b200 import binding as B
    from paper_2505_15781_b200 import synth
    torch.cuda.set_device(0)
    ms_shape = synth.llada_shape()
    w = synth.make_weights(ms_shape, 0, "bfloat16", "cuda")
    model = B.dkv_model_create(ms_shape, w, B.DKV_BF16)
    del w
    for gen in [int(v) for v in args.sweep_gens.split(",")]:
        for prompt in [int(v) for v in args.sweep_prompts.split(",")]:
            row = {"sweep": "length", "gen": gen, "prompt": prompt}
            for name, pol, interval, window in (("none", "none", 0, 0), ("decode8", "decode", 8, 0),
                                                ("greedy2", "greedy", 2, 4), ("greedy8", "greedy", 8, 4)):
                wl = dict(shape="llada", batch=1, prompt=prompt, gen=gen, block=gen, k=1, policy=pol,
                          interval=interval, window=window)
                job = Job(wl, model=model)
                ms, steps, first = timed_generation_steps(job, args.steps)
                st = B.dkv_get_stats(job.cache)
                assert B.dkv_status(job.cache) == 0
                row[name] = {"tokens_per_s": steps / (ms * 1e-3), "ms_per_step": ms / steps,
                             "kv_slot_gb": st.cache_bytes / 1e9, "arena_gb": job.arena.numel() / 1e9}
                del job
                torch.cuda.empty_cache()
            for name in ("decode8", "greedy2", "greedy8"):
                row[name]["speedup"] = row[name]["tokens_per_s"] / row["none"]["tokens_per_s"]
            print(json.dumps(row), flush=True)


def run_batch_sweep(args):
    """Decode vs no-cache over batch sizes (the paper's batch-size study, App. D: LLaDA, prefill 100):
    prints one JSON line per point.  Not the benchmark contract line."""
    import torch
    torch.cuda.set_device(0)
    for batch in [int(b) for b in args.sweep_batches.split(",")]:
        row = {"sweep": "batch", "batch": batch, "prompt": 100, "gen": 128, "block": 32, "k": 1}
        for policy, interval in (("none", 0), ("decode", 8)):
            wl = dict(shape="llada", batch=batch, prompt=100, gen=128, block=32, k=1, policy=policy,
                      interval=interval, window=0)
            job = Job(wl)
            job.run_steps(8)
            job.restart()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            steps = min(args.steps, job.T)
            e0.record()
            job.run_steps(steps)
            e1.record()
            torch.cuda.synchronize()
            ms = e0.elapsed_time(e1)
            row[policy] = {"tokens_per_s": steps * batch / (ms * 1e-3), "ms_per_step": ms / steps,
                           "arena_gb": job.arena.numel() / 1e9}
            del job
            torch.cuda.empty_cache()
        row["speedup"] = row["decode"]["tokens_per_s"] / row["none"]["tokens_per_s"]
        print(json.dumps(row), flush=True)


LAYER_CLASSES = ("gemm_qkv", "qkv_rope_scatter", "attention", "gemm_o", "resid_norm", "gemm_gateup", "swiglu", "gemm_down")


def run_layer_sweep(args):
    """Single LLaDA-8B-shaped layer: total length x active-row fraction x batch, active rows drawn
    uniformly at random from a seed.  One JSON line per point with, per kernel class of the layer,
    time, GB/s and TFLOP/s, and the layer's fraction of its roofline (the slower of flops at the
    measured bf16 peak and algorithmic bytes at the measured HBM bandwidth) and of the full-recompute
    layer's time.  Points whose arena or work exceed the bounds are skipped and say so."""
    import numpy as np
    import torch
    from paper_2505_15781_b200 import binding as B
    from paper_2505_15781_b200 import synth
    torch.cuda.set_device(0)
    pk = peaks()
    ms = synth.llada_shape(1)
    w = synth.make_weights(ms, 0, "bfloat16", "cuda")
    model = B.dkv_model_create(ms, w, B.DKV_BF16)
    del w
    fracs = [("100%", 1.0), ("50%", 0.5), ("12.5%", 0.125), ("1 row", 0.0)]
    for batch in [int(b) for b in args.sweep_batches.split(",")]:
        for L in [int(v) for v in args.sweep_lengths.split(",")]:
            full_ms = None
            for label, frac in fracs:
                n_act = max(1, int(round(frac * L)))
                R = batch * n_act
                flops = 2.0 * R * 2 * (ms.d_model * (3 * ms.d_model) + ms.d_model * ms.d_model + 3 * ms.d_model * ms.d_ffn) / 2
                flops += 4.0 * R * L * ms.n_q_heads * ms.head_dim
                row = {"sweep": "layer", "batch": batch, "L": L, "active": label, "rows": R}
                pol = B.make_policy(B.DKV_POLICY_DECODE, 0, delay=0, max_head_rows=1)
                need = B.dkv_cache_bytes(model, batch, L, pol)
                if need > args.sweep_max_gb * 1e9 or flops > args.sweep_max_pflop * 1e15:
                    row["skipped"] = f"arena {need / 1e9:.1f} GB, {flops / 1e15:.2f} PFLOP per step: above the sweep's bounds"
                    print(json.dumps(row), flush=True)
                    continue
                arena = torch.empty(need + 256, dtype=torch.uint8, device="cuda")
                cache = B.dkv_init_cache(model, batch, L, 0, pol, arena=arena)
                rng = np.random.Generator(np.random.PCG64(L * 131 + batch))
                x = torch.from_numpy(rng.integers(0, ms.vocab - 1, size=(batch, L)).astype(np.int32)).cuda()
                conf = torch.empty(batch, L, device="cuda")
                pred = torch.empty(batch, L, dtype=torch.int32, device="cuda")

                def mask_for(step):
                    m = np.zeros((batch, L), np.uint8)
                    for b in range(batch):   # position L-1 is always active: it is the one head row
                        idx = synth.random_active_set(L - 1, n_act - 1, seed=step * 1000 + b) if n_act > 1 else []
                        m[b, idx] = 1
                        m[b, L - 1] = 1
                    return torch.from_numpy(m).cuda()
                # step 1 is always a full step (it fills every slot); then two untimed and two profiled steps
                B.dkv_step(cache, x, torch.ones(batch, L, dtype=torch.uint8, device="cuda"), None, 1, L - 1, L, L, conf, pred)
                masks = [mask_for(i) for i in range(4)]
                for i in range(2):
                    B.dkv_step(cache, x, masks[i], None, 1, L - 1, L, n_act, conf, pred)
                torch.cuda.synchronize()
                B.dkv_profile_enable(cache, True)
                agg = {}
                for i in range(2, 4):
                    B.dkv_step(cache, x, masks[i], None, 1, L - 1, L, n_act, conf, pred)
                    for e in B.dkv_profile_read(cache):
                        a = agg.setdefault(e["name"], dict(launches=0, ms=0.0, bytes=0.0, flops=0.0))
                        for key in a:
                            a[key] += e[key]
                B.dkv_profile_enable(cache, False)
                assert B.dkv_status(cache) == 0
                layer_ms = sum(agg[c]["ms"] for c in LAYER_CLASSES if c in agg) / 2
                lb = sum(agg[c]["bytes"] for c in LAYER_CLASSES if c in agg) / 2
                lf = sum(agg[c]["flops"] for c in LAYER_CLASSES if c in agg) / 2
                # algorithmic bytes of the layer: its weights once, the K/V slots of every sequence once
                alg_bytes = 2.0 * (4 * ms.d_model * ms.d_model + 3 * ms.d_model * ms.d_ffn) + \
                    2.0 * 2 * batch * L * ms.n_kv_heads * ms.head_dim
                bound_ms = max(flops / (pk["tf_sust"] * 1e12), alg_bytes / (pk["hbm"] * 1e9)) * 1e3
                row.update(layer_ms=layer_ms, roofline_ms=bound_ms, roofline_frac=bound_ms / layer_ms,
                           bound="tensor" if flops / (pk["tf_sust"] * 1e12) > alg_bytes / (pk["hbm"] * 1e9) else "hbm",
                           kernels={c: {"ms": agg[c]["ms"] / 2, "GB/s": agg[c]["bytes"] / agg[c]["ms"] / 1e6 if agg[c]["ms"] else 0.0,
                                        "TFLOP/s": agg[c]["flops"] / agg[c]["ms"] / 1e9 if agg[c]["ms"] else 0.0}
                                    for c in LAYER_CLASSES if c in agg})
                if label == "100%":
                    full_ms = layer_ms
                if full_ms:
                    row["vs_full_recompute"] = full_ms / layer_ms
                print(json.dumps(row), flush=True)
                del cache, arena
                torch.cuda.empty_cache()


def run_stream_sweep(args):
    """The memory side of a weight-streaming launch alone (`dkv_op_stream_probe`: bulk copies into a ring
    of shared-memory stages, no arithmetic): 201 MB (the gate/up matrix of an LLaDA-shaped layer) of
    unique bytes per launch, with and without bytes that every CTA re-reads from L2, over the number of
    CTAs and the ring depth.  One JSON line per point: time per launch (eight launches back to back
    between two events, each on another L2-cold window) and TB/s."""
    import torch
    from paper_2505_15781_b200 import binding as B
    torch.cuda.set_device(0)
    total = 201 << 20
    big = torch.ones(1 << 30, dtype=torch.uint8, device="cuda")          # four disjoint 256 MB windows: cold in L2
    small = torch.ones(1179648, dtype=torch.uint8, device="cuda")        # 144 rows x 4096 x 2 bytes
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    for ctas in (74, 96, 128, 148):
        for b_kb in (0, 9, 18):
            for stages in (3, 4, 6):
                if (32 + b_kb) * stages > 216:
                    continue
                def launch(r):
                    win = big[(r % 4) * (256 << 20):(r % 4) * (256 << 20) + total]
                    B.dkv_op_stream_probe(win, small if b_kb else None, ctas, 32 << 10, b_kb << 10, stages, status)
                ts = []
                for rep in range(4):      # rep 0 is the warm-up; 8 launches back to back between two events
                    torch.cuda.synchronize()
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    e0.record()
                    for r in range(8):
                        launch(r)
                    e1.record()
                    torch.cuda.synchronize()
                    if rep:
                        ts.append(e0.elapsed_time(e1) * 1e-3 / 8)
                t = sum(ts) / len(ts)
                moved = total // ctas // (32 << 10) * (32 << 10) * ctas
                reread = total // ctas // (32 << 10) * (b_kb << 10) * ctas
                print(json.dumps({"sweep": "stream", "ctas": ctas, "streamed_kb_per_stage": 32, "reread_kb_per_stage": b_kb,
                                  "stages": stages, "launch_us": round(t * 1e6, 1), "best_us": round(min(ts) * 1e6, 1),
                                  "streamed_TBps": round(moved / t / 1e12, 2),
                                  "streamed_plus_reread_TBps": round((moved + reread) / t / 1e12, 2),
                                  "status": int(status.item())}), flush=True)


def run_attention_sweep(args):
    """The attention kernel alone (`dkv_op_attention`, fp16, head_dim 128) over (rows, slots, batch,
    query heads, KV heads) cases: time, TFLOP/s (4*rows*slots*d_q), GB/s of slots + queries + outputs."""
    import torch
    from paper_2505_15781_b200 import binding as B
    torch.cuda.set_device(0)
    cases = [tuple(int(v) for v in c.split("x")) for c in args.attn_cases.split(",")]
    for rows, L, batch, hq, hkv in cases:
        dh = 128
        g = torch.Generator(device="cuda").manual_seed(rows + L)
        q = torch.randn(batch * rows, hq, dh, device="cuda", dtype=torch.float16, generator=g)
        k = torch.randn(batch, hkv, L, dh, device="cuda", dtype=torch.float16, generator=g)
        v = torch.randn(batch, hkv, L, dh, device="cuda", dtype=torch.float16, generator=g)
        o = torch.zeros_like(q)
        row_off = torch.arange(0, batch + 1, dtype=torch.int32, device="cuda") * rows
        for _ in range(3):
            B.dkv_op_attention(q, k, v, o, row_off, batch, rows, L, hq, hkv, dh, B.DKV_F16)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(args.steps):
            B.dkv_op_attention(q, k, v, o, row_off, batch, rows, L, hq, hkv, dh, B.DKV_F16)
        e1.record()
        torch.cuda.synchronize()
        us = e0.elapsed_time(e1) * 1e3 / args.steps
        flops = 4.0 * batch * rows * L * hq * dh
        nbytes = 2.0 * 2 * batch * hkv * L * dh + 2 * 2.0 * batch * rows * hq * dh
        print(json.dumps({"sweep": "attention", "rows": rows, "slots": L, "batch": batch, "q_heads": hq, "kv_heads": hkv,
                          "us": us, "TFLOP/s": flops / us / 1e6, "GB/s": nbytes / us / 1e3}), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=256)
    ap.add_argument("--warmup", type=int, default=256)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llada8b_decode", choices=sorted(WORKLOADS))
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--sweep", default="", choices=["", "batch", "layer", "attention", "order", "length", "stream"])
    ap.add_argument("--sweep-gens", default="128,256,512,1024")
    ap.add_argument("--sweep-prompts", default="0,128,512,2048")
    ap.add_argument("--attn-cases", default="254x512x1x32x32,512x512x1x32x32,1024x1024x8x32x32,4096x4096x1x32x32,"
                                            "8192x8192x1x32x32,1024x8192x1x32x32,1x8192x32x32x32,8x1152x1x32x32,768x768x4x28x4",
                    help="rows x slots x batch x query heads x KV heads, comma separated")
    ap.add_argument("--sweep-batches", default="")
    ap.add_argument("--sweep-lengths", default="1024,2048,4096,8192")
    ap.add_argument("--sweep-max-gb", type=float, default=60.0)
    ap.add_argument("--sweep-max-pflop", type=float, default=1.5)
    args = ap.parse_args()
    if args.sweep == "batch":
        args.sweep_batches = args.sweep_batches or "1,2,4,8,16,32,64"
        run_batch_sweep(args)
        return
    if args.sweep == "stream":
        run_stream_sweep(args)
        return
    if args.sweep == "attention":
        args.steps = min(args.steps, 10)
        run_attention_sweep(args)
        return
    if args.sweep == "order":
        run_order_comparison(args)
        return
    if args.sweep == "length":
        args.steps = min(args.steps, 64)
        run_length_sweep(args)
        return
    if args.sweep == "layer":
        args.sweep_batches = args.sweep_batches or "1,8,32"
        run_layer_sweep(args)
        return
    rank = int(os.environ.get("RANK", 0))
    world = int(os.environ.get("WORLD_SIZE", 1))
    if args.impl == "reference":
        out = run_reference(args, rank, world)
        if out is not None:
            print(json.dumps(out))
        return
    out = run_ours(args, rank, world)
    if rank == 0:
        if world == 1 and not args.no_cpu_baseline:
            out["cpu_baseline"] = cpu_baseline(WORKLOADS[args.workload])
        print(json.dumps(out))


if __name__ == "__main__":
    main()
