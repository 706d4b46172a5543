#!/usr/bin/env python
"""Benchmark of the hierarchical fine-tuning (HiFT) step on B200.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

One "step" = one hift_step: full forward, backward truncated at the active group, fused
group-local optimizer, optimizer-state paging.  Default workload: the LLaMA-7B-shaped causal LM
(32 blocks, d 4096, 32 heads, SwiGLU 11008, vocab 32000, batch 4 x seq 512, bf16 with fp32
master, one block per group plus embedding and head groups, bottom2up, AdamW with inactive-group
state in pinned host memory).  Prints ONE JSON line on rank 0.

N > 1 runs N independent replicas by default (one process per GPU, no data-path collective: the
step has no exchange inside it on one GPU); --parallel dp trains one model data-parallel with an
all-reduce of the active group's gradient, chunk by chunk behind the backward pass; --parallel zero1 also splits the
optimizer state over the ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

import synth

WORKLOADS = {
    "llama7b": synth.config_llama_7b,
    "gpt2large": synth.config_gpt2_large,
    "roberta": synth.config_roberta_base,
    "tiny": synth.config_tiny_fp32,
}


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d.get("bf16_tflops_sustained", d["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "200"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            if len(r) < 6:
                continue
            try:
                sm.append(float(r[0]))
                mx = float(r[1])
            except ValueError:
                continue
            for n, v in zip(names, r[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": mx, "reasons": sorted(reasons),
                "samples": len(sm)}


# ---------------------------------------------------------------------------- CPU oracle leg
def oracle_sample(cfg, gcfg, ocfg, max_blocks=1):
    """Times the fp64 oracle, as it stands, on a bounded sample of the workload: the same widths,
    vocabulary, batch and sequence length, but only `max_blocks` transformer blocks; one step that
    trains the top block (forward, backward through head and block, update).  Returns
    (seconds, sample description, flops of the sample step, threads used)."""
    from oracle import hift_oracle as O
    nb = min(max_blocks, cfg.n_blocks)
    big = cfg.d_model >= 2048
    # at 7B widths the vocabulary matrices alone are 2 x 131 M fp64 values: sample one block with a
    # 1024-entry vocabulary and one sequence, and scale by flops
    small = cfg.scaled(n_blocks=nb, batch=1 if big else cfg.batch, vocab=1024 if big else cfg.vocab)
    g = synth.GroupCfg(layers_per_group=1, split_emb_head=0, order=synth.ORDER_BOTTOM2UP)
    p0 = synth.init_params(small, 0)
    orc = O.HiFTOracle(small, g, ocfg, p0)
    orc.t = nb                                   # group nb = the top block
    tok, lab = synth.batch_for(small, 0, 0)
    t0 = time.perf_counter()
    orc.step(tok, lab)
    dt = time.perf_counter() - t0
    T, d, f, V = small.tokens_per_step, cfg.d_model, cfg.d_ffn, small.vocab
    ffn = 3 if cfg.arch == synth.ARCH_LLAMA else 2
    blk = 2.0 * T * (4 * d * d + ffn * d * f) + 4.0 * T * cfg.seq * d * (0.5 if cfg.causal else 1.0)
    head = 2.0 * T * d * V if cfg.arch != synth.ARCH_POSTLN_ENC else 0.0
    flops = nb * blk + head + head + 2.0 * blk    # forward, head dX, top block dX + dW
    try:
        threads = len(os.sched_getaffinity(0))
    except Exception:
        threads = os.cpu_count() or 1
    desc = (f"fp64 oracle, one step training the top block of a {nb}-block model of the same widths "
            f"(d={d}, f={f}, vocab {V} of {cfg.vocab}, batch {small.batch} of {cfg.batch} x seq {cfg.seq}); "
            f"full-model figure extrapolated by flops")
    return dt, desc, flops, threads


def mean_step_flops(cfg, groups):
    """Algorithmic flops of a HiFT step averaged over one cycle of groups (GEMM + attention)."""
    T, d, f, V, L = cfg.tokens_per_step, cfg.d_model, cfg.d_ffn, cfg.vocab, cfg.n_blocks
    ffn = 3 if cfg.arch == synth.ARCH_LLAMA else 2
    blk_lin = 2.0 * T * (4 * d * d + ffn * d * f)
    blk_att = 4.0 * T * cfg.seq * d * (0.5 if cfg.causal else 1.0)
    head = 2.0 * T * d * V if cfg.arch != synth.ARCH_POSTLN_ENC else 0.0
    fwd = L * (blk_lin + blk_att) + head
    tot = 0.0
    for lo, hi in groups:
        fl = fwd
        if lo <= L:                                       # something below the head is trained
            fl += head                                    # head dX
        head_w = (hi == L + 1 and not cfg.tie_head) or (lo == 0 and cfg.tie_head)
        if head_w:
            fl += head                                    # head dW
        if hi == L + 1 and lo == L + 1 and not head_w:
            fl += head                                    # dX still needed for the final norm's gain
        for u in range(max(lo, 1), L + 1):
            fl += blk_lin + 2.5 * blk_att                 # dX through this block
            if u <= hi:
                fl += blk_lin                             # dW inside the group
        tot += fl
    return tot / len(groups)


# ---------------------------------------------------------------------------- main legs
def run_reference(args, cfg, gcfg, ocfg):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    # --steps K --warmup W as for the other arm, each step one bounded sample of the workload; the run is kept to about
    # two and a half minutes: once the first sample has shown what a step costs, W and K are cut to what fits (the line reports
    # the steps that ran and the steps that were asked for).  --steps-ref / --warmup-ref > 0 override K and W.
    K_req = args.steps_ref if args.steps_ref > 0 else args.steps
    W_req = args.warmup_ref if args.steps_ref > 0 else args.warmup
    budget_s = 150.0
    t_start = time.perf_counter()
    dt, desc, flops, threads = oracle_sample(cfg, gcfg, ocfg)
    fit = max(1, int((budget_s - (time.perf_counter() - t_start)) / max(dt, 1e-3)))
    W_run = min(W_req, max(0, fit - 1), 1 if fit < W_req + K_req else W_req)
    K_run = max(1, min(K_req, fit + 1 - W_run))
    times = [dt]
    for _ in range(W_run + K_run - 1):
        dt, desc, flops, threads = oracle_sample(cfg, gcfg, ocfg)
        times.append(dt)
    times = times[W_run:]
    dt = float(np.mean(times))
    groups = [(g[0], g[-1]) for g in __import__("oracle.hift_oracle", fromlist=["x"]).build_groups(
        cfg.n_units, gcfg.layers_per_group, gcfg.split_emb_head)]
    full = mean_step_flops(cfg, groups)
    value = cfg.tokens_per_step / (dt * full / flops)
    line = {
        "impl": "reference", "metric": "HiFT step tokens/s", "value": value, "unit": "tokens/s",
        "n_gpus": args.gpus, "steps": K_run, "warmup": W_run, "steps_requested": K_req, "warmup_requested": W_req,
        "ms_per_step": dt * full / flops * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": args.workload, "note": "CPU oracle on a bounded sample, extrapolated by flops"},
        "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": threads, "kind": "oracle", "sample": desc},
        "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))


def group_plan(k, K, W):
    """Groups of the W warm-up steps and the K timed steps of one leg.  K a multiple of k: whole cycles of
    the group ids 0 .. k-1 in ascending order; otherwise K group ids spread evenly over the cycle, both ends
    (embedding group 0 and head group k-1) included.  The warm-up trains the tail of the same list, so the
    paging ring is in its steady state when the clock starts.  Every leg uses this one list."""
    if K % k == 0:
        sel = [i % k for i in range(K)]
        kind = f"{K // k} whole cycle(s), groups 0..{k - 1} in ascending order"
    else:
        sel = [int(round(i * (k - 1) / max(K - 1, 1))) for i in range(K)]
        kind = f"{K} groups spread evenly over the cycle of {k} (both ends included)"
    rot = [sel[(j - W) % K] for j in range(K)]        # step j of a leg trains rot[j % K]
    return sel, rot, kind


def pcie_ceiling(n_bytes=2 << 30, reps=3):
    """Plain pinned-memory copies of n_bytes on two streams: host-to-device alone, device-to-host alone, both
    at once (GB/s per direction), timed with CUDA events.  The ceiling of the optimizer-state paging."""
    import torch
    h_in = torch.empty(n_bytes, dtype=torch.uint8).pin_memory()
    h_out = torch.empty(n_bytes, dtype=torch.uint8).pin_memory()
    h_in.fill_(1)
    d_in = torch.empty(n_bytes, dtype=torch.uint8, device="cuda")
    d_out = torch.ones(n_bytes, dtype=torch.uint8, device="cuda")
    s_up, s_dn = torch.cuda.Stream(), torch.cuda.Stream()

    def run(up, dn):
        ev = []
        for st, on, fn in ((s_up, up, lambda: d_in.copy_(h_in, non_blocking=True)),
                           (s_dn, dn, lambda: h_out.copy_(d_out, non_blocking=True))):
            if not on:
                continue
            with torch.cuda.stream(st):
                fn()                                   # warm-up
        torch.cuda.synchronize()
        for st, on, fn in ((s_up, up, lambda: d_in.copy_(h_in, non_blocking=True)),
                           (s_dn, dn, lambda: h_out.copy_(d_out, non_blocking=True))):
            if not on:
                continue
            with torch.cuda.stream(st):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                for _ in range(reps):
                    fn()
                e1.record()
                ev.append((e0, e1))
        torch.cuda.synchronize()
        return [n_bytes * reps / (a.elapsed_time(b) * 1e-3) / 1e9 for a, b in ev]

    up = run(True, False)[0]
    dn = run(False, True)[0]
    both = run(True, True)
    del h_in, h_out, d_in, d_out
    torch.cuda.empty_cache()
    return {"h2d_alone_gbs": round(up, 1), "d2h_alone_gbs": round(dn, 1),
            "both_h2d_gbs": round(both[0], 1), "both_d2h_gbs": round(both[1], 1),
            "bytes_per_copy": n_bytes, "how": "pinned host memory, one copy stream per direction, CUDA events"}


def standalone_kernels(cfg, peaks, launches=20):
    """The short kernels of a step (tens of microseconds: norms, attention), each launched `launches` times
    back to back on its own through the single-kernel entry points, at the workload's shapes, over buffer
    sets that rotate so that consecutive launches do not find their inputs in L2.  An event bracket around a
    single such launch inside the step would read several microseconds too long."""
    import torch
    from paper_2401_15207_b200 import binding as B
    if cfg.dtype != 1:
        return {}
    T, d, H, S, Bt = cfg.tokens_per_step, cfg.d_model, cfg.n_heads, cfg.seq, cfg.batch
    dh = d // H
    kind = 1 if cfg.arch == synth.ARCH_LLAMA else 0
    bf = torch.bfloat16
    out = {}

    def timed(fn, nsets):
        for i in range(3):
            fn(i % nsets)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        torch.cuda._sleep(2_000_000)                 # about a millisecond: the launches below queue up behind it, so the
        e0.record()                                  # host's per-call cost stays out of the measurement
        for i in range(launches):
            fn(i % nsets)
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) * 1e3 / launches          # microseconds per launch

    def entry(name, us, work, tensor, note):
        ach = work / (us * 1e-6) / (1e12 if tensor else 1e9)
        pk = peaks["bf16_tflops_sustained"] if tensor else peaks["hbm_gbs"]
        out[name] = {"avg_us": round(us, 2), "achieved": round(ach, 1), "unit": "TFLOP/s" if tensor else "GB/s",
                     "bound": "tensor" if tensor else "hbm", "frac": round(ach / pk, 3), "what": note,
                     "method": f"standalone loop, {launches} queued launches, CUDA events, rotating buffers"}

    # norms: fp32 stream in, bf16 operand out (forward); bf16 dy + fp32 x + fp32 add in, fp32 + bf16 dx out (backward)
    nsets = max(2, int(200e6 // (T * d * 6)) + 1)
    xs = [torch.randn(T, d, device="cuda") for _ in range(nsets)]
    ys = [torch.empty(T, d, device="cuda", dtype=bf) for _ in range(nsets)]
    stats = [torch.empty(2 * T, device="cuda") for _ in range(nsets)]
    gain = torch.ones(d, device="cuda", dtype=bf)
    bias = torch.zeros(d, device="cuda", dtype=bf) if kind == 0 else None
    us = timed(lambda i: B.k_norm_fwd(1, kind, T, d, cfg.norm_eps, xs[i], gain, bias, ys[i], stats[i]), nsets)
    entry("norm_fwd", us, T * d * 6.0, False, f"[{T}, {d}] fp32 in, bf16 out")
    dxs = [torch.empty(T, d, device="cuda") for _ in range(nsets)]
    us = timed(lambda i: B.k_norm_bwd(1, kind, T, d, ys[i], xs[i], stats[i], gain, xs[(i + 1) % nsets], dxs[i], None, None, None), nsets)
    entry("norm_bwd_dx", us, T * d * 14.0, False, f"[{T}, {d}] bf16 dy, fp32 x and residual gradient in, fp32 out")
    del xs, ys, dxs
    if dh in (64, 128):
        nsets = max(2, int(200e6 // (T * d * 8)) + 1)
        qkv = [torch.randn(T, 3 * d, device="cuda").to(bf) for _ in range(nsets)]
        o = [torch.empty(T, d, device="cuda", dtype=bf) for _ in range(nsets)]
        lse = [torch.empty(Bt * H * S, device="cuda") for _ in range(nsets)]
        fl = 4.0 * Bt * H * S * S * dh * (0.5 if cfg.causal else 1.0)
        us = timed(lambda i: B.k_attention_fwd(1, Bt, S, H, dh, cfg.causal, qkv[i], o[i], lse[i]), nsets)
        entry("attn_fwd", us, fl, True, f"batch {Bt} x seq {S} x {H} heads x {dh}, causal={cfg.causal}")
        do = [torch.randn(T, d, device="cuda").to(bf) for _ in range(nsets)]
        dqkv = [torch.empty(T, 3 * d, device="cuda", dtype=bf) for _ in range(nsets)]
        dsum = torch.empty(T * H, device="cuda")
        us = timed(lambda i: B.k_attention_bwd(1, Bt, S, H, dh, cfg.causal, qkv[i], o[i], lse[i], do[i], dqkv[i], dsum), nsets)
        entry("attn_bwd", us, 2.5 * fl, True, "same shape; dsum + dK/dV + dQ launches together")
    torch.cuda.empty_cache()
    return out


def run_ours(args, cfg, gcfg, ocfg):
    import torch
    import torch.distributed as dist
    from paper_2401_15207_b200 import HiFT, dist_util

    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    ocfg = synth.OptCfg(**{**ocfg.__dict__, "prefetch_groups": args.prefetch, "offload_state": args.offload,
                           "recompute": args.recompute,
                           "shard_rank": rank if args.parallel == "zero1" else 0,
                           "shard_world": world if args.parallel == "zero1" else 0})
    peaks = measured_peaks()
    pcie = None
    if rank == 0 and world == 1 and ocfg.offload_state and not args.no_pcie:
        pcie = pcie_ceiling()
    h = HiFT(cfg, gcfg, ocfg)
    h.init_synthetic(dist_util.rank_seed(1234, rank), cfg.init_std)
    k = h.num_groups()
    K, W = args.steps, args.warmup
    sel, rot, plan_kind = group_plan(k, K, W)
    host = [synth.batch_for(cfg, dist_util.rank_seed(77, rank), t) for t in range(W + K)]
    # the end-to-end leg copies its inputs from pinned host memory: numpy views of pinned tensors (kept alive here)
    pinned_keep = [tuple(torch.from_numpy(np.ascontiguousarray(x, dtype=np.int32)).pin_memory() for x in pair) for pair in host]
    host = [tuple(t.numpy() for t in pair) for pair in pinned_keep]
    dev = [(torch.from_numpy(a).cuda(), torch.from_numpy(b).cuda()) for a, b in host]
    groups = [h.group_units(g) for g in range(k)]

    step_dev, step_host = h.step, h.step_host
    if args.parallel in ("dp", "zero1"):
        dp_step = dist_util.data_parallel_step if args.parallel == "dp" else dist_util.data_parallel_step_sharded
        step_dev = lambda tok, lab: dp_step(h, tok, lab)
        # end to end in this mode: pageable host batch -> device inside the timed call, then the same step
        step_host = lambda tok, lab: step_dev(torch.from_numpy(tok).cuda(), torch.from_numpy(lab).cuda())

    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    paged = []

    def leg(step_fn, batches):
        """W warm-up steps, then K timed steps, on the groups of group_plan: the same ones in every leg."""
        h.force_sequence(rot)
        for t in range(W):
            step_fn(*batches[t])
        trained, step_ms, launches, last = [], [], 0, 0.0
        paged.clear()
        barrier()
        e0.record()
        for t in range(W, W + K):
            trained.append(h.active_group())
            t_host = time.perf_counter()
            last = step_fn(*batches[t])              # returns when the step's loss is on the host
            step_ms.append(round((time.perf_counter() - t_host) * 1e3, 2))
            launches += h.last_step_launches()
            paged.append(h.last_step_paging()[1])    # bytes written back = this group's paged state
        e1.record()
        barrier()
        return e0.elapsed_time(e1), trained, step_ms, launches, last

    # ---- device-resident leg, timed twice over the same K steps: once plain (the reported value) and once
    #      with every kernel launch bracketed by CUDA events on the launching stream (time shares per class,
    #      and the roofline figures of the long kernels; the brackets cost a few per cent)
    sampler = ClockSampler(local)
    sampler.start()
    ms, trained, step_ms, launches, _ = leg(step_dev, dev)
    assert trained == sel
    ms_prof = 0.0
    if not args.skip_profiled:
        h.profile_enable(True)
        ms_prof, trained_prof, _, _, _ = leg(step_dev, dev)
        assert trained_prof == sel
    prof = h.profile()
    h.profile_enable(False)
    clocks = sampler.stop()
    paging = h.last_step_paging()
    timeline = h.last_step_timeline()

    # ---- end-to-end leg: host buffers, copies inside the call
    last_loss = 0.0
    ms_e2e = float("nan")
    if not args.skip_e2e:
        ms_e2e, trained_e2e, _, _, last_loss = leg(step_host, host)
        assert trained_e2e == sel
    h.force_sequence([])

    ms, ms_e2e = dist_util.max_over_ranks([ms, ms_e2e], device="cuda")
    tokens = cfg.tokens_per_step * K * world
    value = tokens / (ms * 1e-3)
    e2e_value = tokens / (ms_e2e * 1e-3)
    peak_hbm = h.peak_hbm_bytes()
    pinned = h.pinned_host_bytes()
    h.close()
    alone = {}
    if rank == 0 and world == 1 and not args.skip_profiled:
        alone = standalone_kernels(cfg, peaks)
    full_ref = None
    if world == 1 and not args.no_full_param_reference and not args.full_param and not args.skip_e2e:
        try:
            full_ref = run_full_param_reference(cfg, ocfg)
        except Exception as e:                      # e.g. not enough HBM for 16 B/param
            full_ref = {"unavailable": str(e)[:200]}

    if rank == 0:
        default_llama = args.workload == "llama7b" and not args.full_param and not args.recompute
        g = {c: prof[c] for c in ("gemm_fwd", "gemm_dx", "gemm_dw")}
        g_launch = sum(v["launches"] for v in g.values())
        g_ms = sum(v["ms"] for v in g.values())
        g_fl = sum(v["work"] for v in g.values())
        achieved = g_fl / (g_ms * 1e-3) / 1e12 if g_ms > 0 else 0.0
        peak = peaks["bf16_tflops_sustained"] if cfg.dtype == 1 else None
        roof = {"kernel": "linear-layer GEMMs (forward, dX, dW)", "bound": "tensor" if cfg.dtype == 1 else "alu",
                "achieved": achieved, "peak": peak, "unit": "TFLOP/s",
                "frac": (achieved / peak) if peak else None,
                "traffic": NCU_GEMM_TRAFFIC["bytes_per_launch"] if default_llama else None,
                "traffic_unit": "bytes per launch",
                "traffic_note": NCU_GEMM_TRAFFIC["note"] if default_llama else
                                "DRAM counters were taken on the llama7b workload only",
                "peak_source": f"bf16 dense sustained, {peaks['source']}",
                "launches": g_launch, "avg_launch_ms": g_ms / max(g_launch, 1),
                "profiled_ms_per_step": ms_prof / K,
                "by_form": {c: {"launches": v["launches"], "ms": v["ms"],
                                "tflops": v["work"] / (v["ms"] * 1e-3) / 1e12 if v["ms"] > 0 else 0.0}
                            for c, v in g.items()}}
        kernel_share = {c: round(v["ms"], 3) for c, v in prof.items()}
        # Every kernel class against its own roofline.  Classes whose launches last hundreds of microseconds
        # are measured inside the step (one event bracket per launch); for the short ones (norms, attention)
        # a bracket adds several microseconds per launch, so their roofline figure comes from the standalone
        # loop and the in-step bracketed time is kept as `in_step_bracketed_us` (an upper bound).
        per_kernel = {}
        for cname, v in prof.items():
            if v["launches"] == 0 or v["ms"] <= 0:
                continue
            tensor = cname.startswith("gemm") or cname.startswith("attn")
            ach = v["work"] / (v["ms"] * 1e-3) / (1e12 if tensor else 1e9)
            pk = (peaks["bf16_tflops_sustained"] if cfg.dtype == 1 else None) if tensor else peaks["hbm_gbs"]
            avg_us = 1e3 * v["ms"] / v["launches"]
            per_kernel[cname] = {"launches": v["launches"], "ms": round(v["ms"], 3), "avg_us": round(avg_us, 2),
                                 "achieved": round(ach, 1), "unit": "TFLOP/s" if tensor else "GB/s",
                                 "bound": "tensor" if tensor else "hbm",
                                 "frac": round(ach / pk, 3) if pk else None,
                                 "method": "in-step event bracket per launch" +
                                           (" (short launches: time is an upper bound, frac a lower bound)" if avg_us < 50 else "")}
        for name, v in alone.items():
            per_kernel[name + "_alone"] = v
        opt = prof["optimizer"]
        opt_gbs = opt["work"] / (opt["ms"] * 1e-3) / 1e9 if opt["ms"] > 0 else 0.0
        cpu = None
        if world == 1 and not args.no_cpu_baseline:
            dt, desc, flops, threads = oracle_sample(cfg, gcfg, ocfg)
            full = mean_step_flops(cfg, groups)
            cpu = {"value": cfg.tokens_per_step / (dt * full / flops), "unit": "tokens/s", "cores": threads,
                   "kind": "oracle", "sample": desc, "sample_seconds": dt}
        if pcie is not None:
            tl = timeline
            if tl[1] == tl[1] and tl[0] == tl[0] and tl[1] > tl[0]:
                pcie["in_step_h2d_gbs"] = round(paging[1] / ((tl[1] - tl[0]) * 1e-3) / 1e9, 1)
            if tl[5] == tl[5] and tl[5] > tl[4]:
                pcie["in_step_d2h_gbs"] = round(paging[1] / ((tl[5] - tl[4]) * 1e-3) / 1e9, 1)
            pcie["paged_bytes_per_step_each_way"] = int(np.mean(paged)) if paged else 0
            pcie["floor_ms_per_step"] = round(pcie["paged_bytes_per_step_each_way"] /
                                              (min(pcie["both_h2d_gbs"], pcie["both_d2h_gbs"]) * 1e9) * 1e3, 2)
        line = {
            "metric": "HiFT step tokens/s", "value": value, "unit": "tokens/s", "n_gpus": world,
            "steps": K, "warmup": W, "ms_per_step": ms / K, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16" if cfg.dtype == 1 else "f32", "data": "synthetic",
            "config": {"workload": args.workload, "global_batch": cfg.batch * world, "seq_len": cfg.seq,
                       "groups": k, "groups_timed": plan_kind + "; the warm-up trains the tail of the same list; "
                       "the plain, the event-bracketed and the end-to-end leg train the same groups",
                       "groups_trained": trained, "ms_by_step": step_ms,
                       "optimizer": ["adamw", "adagrad", "sgdm", "sgd", "adafactor"][ocfg.kind],
                       "offload_state": ocfg.offload_state, "prefetch_groups": ocfg.prefetch_groups, "recompute": ocfg.recompute,
                       "parallelism": (("%s%d" % (args.parallel, world)) if args.parallel != "replicas" else "replicas") if world > 1 else "single",
                       "l2_policy": "inputs larger than L2 (weights + activations of a step exceed 126 MB)"},
            "cycle_mean_ms": round(float(np.mean(step_ms)), 3),
            "peak_hbm_gb": peak_hbm / 1e9, "pinned_host_gb": pinned / 1e9,
            "paging_bytes_last_step": {"h2d_issued": paging[0], "d2h": paging[1]},
            "paging_timeline_ms": dict(zip(["h2d_begin", "h2d_end", "opt_wait_begin", "opt_wait_end", "d2h_begin",
                                            "d2h_end"], [None if x != x else round(x, 2) for x in timeline])),
            "pcie": pcie,
            "e2e": {"value": e2e_value, "unit": "tokens/s",
                    "h2d_bytes_per_step": int(host[0][0].nbytes + host[0][1].nbytes) + (int(np.mean(paged)) if paged else 0),
                    "d2h_bytes_per_step": 4 + (int(np.mean(paged)) if paged else 0), "ms_per_step": ms_e2e / K, "last_loss": last_loss},
            "gpu_launches": int(launches),
            "roofline": roof,
            "optimizer_gbs": opt_gbs, "optimizer_frac_of_hbm": opt_gbs / peaks["hbm_gbs"],
            "kernel_ms": kernel_share,
            "kernels": per_kernel,
            "clocks": clocks,
            "full_param_reference": full_ref,
            "cpu_baseline": cpu,
        }
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def linear_shapes(cfg):
    """(name, form, M, N, K, launches per step in which one block group is active) of the plain linear-layer products of
    one transformer block at the workload's sizes, in hift_k_linear's convention (form 0 forward y[M,N], 1 dX [M,K] from
    dy[M,N], 2 dW [N,K])."""
    T, d, f = cfg.tokens_per_step, cfg.d_model, cfg.d_ffn
    fa = 2 * f if cfg.arch == synth.ARCH_LLAMA else f
    layers = [("qkv", 3 * d, d), ("attn_out", d, d), ("ffn_up", fa, d), ("ffn_down", d, f)]
    out = []
    for name, n, k in layers:
        for form, tag in ((0, "fwd"), (1, "dx"), (2, "dw")):
            out.append((f"{name}_{tag}", form, T, n, k))
    return out


def run_micro(args, cfg):
    """A few launches of single kernels at the workload's shapes through the single-kernel entry points: what an
    `ncu` capture of one kernel is taken on (a few GB on the device, a handful of launches), and a quick timing of
    each shape on its own (CUDA events over `--launches` back-to-back launches behind a queue-filling spin)."""
    import torch
    from paper_2401_15207_b200 import binding as B
    peaks = measured_peaks()
    bf = torch.bfloat16
    rows = []
    n_l = args.launches

    def timed(fn):
        fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda._sleep(2_000_000)                    # launches queue up behind it: the host is out of the timing
        e0.record()
        for _ in range(n_l):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) * 1e3 / n_l

    if args.micro == "gemm":
        for name, form, M, N, K in linear_shapes(cfg):
            if args.only and args.only not in name:
                continue
            x = torch.randn(M, K, device="cuda").to(bf)
            w = (torch.randn(N, K, device="cuda") * 0.02).to(bf)
            dy = torch.randn(M, N, device="cuda").to(bf)
            if form == 0:
                out = torch.empty(M, N, device="cuda", dtype=bf)
                fn = lambda: B.k_linear(0, 1, M, N, K, x, w, out, path=2)
            elif form == 1:
                out = torch.empty(M, K, device="cuda", dtype=bf)
                fn = lambda: B.k_linear(1, 1, M, N, K, dy, w, out, path=2)
            else:
                out = torch.empty(N, K, device="cuda", dtype=torch.float32)
                fn = lambda: B.k_linear(2, 1, M, N, K, dy, x, out, path=2)
            us = timed(fn)
            fl = 2.0 * M * N * K
            algo = 2.0 * (M * K + N * K + M * N) if form != 2 else 2.0 * (M * N + M * K) + 4.0 * N * K
            rows.append({"shape": name, "form": form, "M": M, "N": N, "K": K, "us": round(us, 2),
                         "tflops": round(fl / (us * 1e-6) / 1e12, 1),
                         "frac_of_burst_peak": round(fl / (us * 1e-6) / 1e12 / peaks["bf16_tflops"], 3),
                         "algorithmic_bytes": int(algo)})
            del x, w, dy, out
    elif args.micro == "step":
        # A three-block model of the workload's width: with the middle block as the active group, one step holds every
        # kind of launch of the full-depth step (a frozen block below the group: forward only; the active block; a
        # block above it: forward and dX; the head) on a few GB, so its GEMM launches can be captured one by one and
        # scaled to the full depth by the number of blocks of each kind.
        import dataclasses
        from paper_2401_15207_b200 import HiFT
        small = dataclasses.replace(cfg, n_blocks=3)
        _, gcfg, ocfg = WORKLOADS[args.workload]()
        h = HiFT(small, gcfg, ocfg)
        try:
            h.init_synthetic(1234, small.init_std)
            mid = [g for g in range(h.num_groups()) if h.group_units(g)[0] == 2][0]    # units: embedding 0, blocks 1..3
            h.force_sequence([mid])
            tok, lab = (torch.from_numpy(a).cuda() for a in synth.batch_for(small, 77, 0))
            h.profile_enable(True)
            for _ in range(n_l):
                loss = h.step(tok, lab)
            prof = h.profile()
            rows = [dict(kernel=k, launches=v["launches"] // n_l, ms_per_step=round(v["ms"] / n_l, 4))
                    for k, v in prof.items() if v["launches"]]
            rows.append({"active_group": mid, "units": list(h.group_units(mid)), "loss": loss,
                         "peak_hbm_gb": round(h.peak_hbm_bytes() / 1e9, 2)})
        finally:
            h.close()
    elif args.micro == "sdpa":
        # Context for the attention numbers: the vendor kernels behind torch's scaled_dot_product_attention (cuDNN and
        # flash back ends) at the workload's attention shape, timed like this library's kernels beside them.  Nothing
        # else in this repository calls them.
        import torch.nn.functional as F
        from torch.nn.attention import sdpa_kernel, SDPBackend
        Bt, S, H, dh, causal = cfg.batch, cfg.seq, cfg.n_heads, cfg.d_model // cfg.n_heads, bool(cfg.causal)
        d = H * dh
        T = Bt * S
        qkv = torch.randn(T, 3 * d, device="cuda").to(bf)
        o = torch.empty(T, d, device="cuda", dtype=bf)
        lse = torch.empty(Bt * H * S, device="cuda")
        do = torch.randn(T, d, device="cuda").to(bf)
        dqkv = torch.empty(T, 3 * d, device="cuda", dtype=bf)
        dsum = torch.empty(T * H, device="cuda")
        fl = 4.0 * Bt * H * S * S * dh * (0.5 if causal else 1.0)
        us_f = timed(lambda: B.k_attention_fwd(1, Bt, S, H, dh, int(causal), qkv, o, lse))
        us_b = timed(lambda: B.k_attention_bwd(1, Bt, S, H, dh, int(causal), qkv, o, lse, do, dqkv, dsum))
        rows.append({"impl": "this library", "fwd_us": round(us_f, 2), "bwd_us": round(us_b, 2),
                     "fwd_tflops": round(fl / us_f / 1e6, 1), "bwd_tflops": round(2.5 * fl / us_b / 1e6, 1)})
        q, k, v = (torch.randn(Bt, H, S, dh, device="cuda", dtype=bf, requires_grad=True) for _ in range(3))
        for name, be in (("torch sdpa, cuDNN back end", SDPBackend.CUDNN_ATTENTION), ("torch sdpa, flash back end", SDPBackend.FLASH_ATTENTION)):
            try:
                with sdpa_kernel(be):
                    with torch.no_grad():
                        us_f = timed(lambda: F.scaled_dot_product_attention(q, k, v, is_causal=causal))
                    out = F.scaled_dot_product_attention(q, k, v, is_causal=causal)
                    g = torch.randn_like(out)
                    # autograd.grad: no accumulation kernels into .grad beside the backward kernel itself
                    us_b = timed(lambda: torch.autograd.grad(out, (q, k, v), g, retain_graph=True))
                rows.append({"impl": name, "fwd_us": round(us_f, 2), "bwd_us": round(us_b, 2),
                             "fwd_tflops": round(fl / us_f / 1e6, 1), "bwd_tflops": round(2.5 * fl / us_b / 1e6, 1)})
            except Exception as e:
                rows.append({"impl": name, "unavailable": str(e)[:160]})
        rows.append({"shape": f"batch {Bt} x seq {S} x {H} heads x {dh}, causal={int(causal)}", "flops_fwd": fl})
    else:
        rows = [dict(kernel=k, **v) for k, v in standalone_kernels(cfg, peaks, launches=n_l).items()]
    print(json.dumps({"micro": args.micro, "workload": args.workload, "launches": n_l,
                      "peak_tflops_burst": peaks["bf16_tflops"], "rows": rows}))


def run_full_param_reference(cfg, ocfg, steps=4, warmup=3):
    """The same model trained the ordinary way: one group holding every unit (k = 1), all master
    weights and optimizer state resident on the GPU, full backward.  Returns tokens/s and peak HBM."""
    import torch
    from paper_2401_15207_b200 import HiFT
    g = synth.GroupCfg(layers_per_group=cfg.n_units, split_emb_head=0, order=synth.ORDER_BOTTOM2UP)
    o = synth.OptCfg(**{**ocfg.__dict__, "offload_state": 0, "prefetch_groups": 0})
    h = HiFT(cfg, g, o)
    try:
        h.init_synthetic(99, cfg.init_std)
        dev = [tuple(torch.from_numpy(a).cuda() for a in synth.batch_for(cfg, 55, t)) for t in range(warmup + steps)]
        for t in range(warmup):
            h.step(*dev[t])
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        for t in range(warmup, warmup + steps):
            h.step(*dev[t])
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / steps
        return {"tokens_per_s": cfg.tokens_per_step / (ms * 1e-3), "ms_per_step": ms,
                "peak_hbm_gb": h.peak_hbm_bytes() / 1e9, "steps": steps}
    finally:
        h.close()


def run_sweep_optimizer(args):
    """Group-local fused optimizer over flat buffers of 2^20 .. 2^30 elements (bf16 param, fp32
    master/state, gradients N(0, 1e-3)): achieved algorithmic GB/s against the measured HBM peak."""
    import torch
    from paper_2401_15207_b200 import opt_step
    peaks = measured_peaks()
    rows = []
    for kind, name, bpe in ((0, "adamw", 30), (1, "adagrad", 22), (2, "sgdm", 22)):      # fp32-master form of hift_opt_step
        for lg in range(20, 31):
            n = 1 << lg
            # rotate over enough buffer sets to exceed L2 (126 MB) between visits
            sets = max(1, min(8, int(200e6 // (n * bpe)) + 1))
            bufs = []
            for _ in range(sets):
                master = torch.randn(n, device="cuda") * 0.02
                grad = torch.randn(n, device="cuda") * 1e-3
                bufs.append((torch.zeros(n, dtype=torch.bfloat16, device="cuda"), master, grad,
                             torch.zeros(n, device="cuda"), torch.zeros(n, device="cuda")))
            iters = max(5, min(200, int(2e9 // (n * bpe))))
            for i in range(3):
                p, m, g, a, b = bufs[i % sets]
                opt_step(kind, n, p, m, g, a, b, lr=1e-3, eps=1e-8 if kind != 1 else 1e-10, tau=1)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            e0.record()
            for i in range(iters):
                p, m, g, a, b = bufs[i % sets]
                opt_step(kind, n, p, m, g, a, b, lr=1e-3, eps=1e-8 if kind != 1 else 1e-10, tau=2 + i)
            e1.record()
            torch.cuda.synchronize()
            us = e0.elapsed_time(e1) * 1e3 / iters
            gbs = n * bpe / (us * 1e-6) / 1e9
            rows.append({"optimizer": name, "log2_n": lg, "us": round(us, 2), "gbs": round(gbs, 1),
                         "frac_of_hbm": round(gbs / peaks["hbm_gbs"], 3),
                         "l2_resident": bool(n * bpe * sets < 126e6)})
            del bufs
            torch.cuda.empty_cache()
    # the CPU side of the same table: the oracle's update functions (numpy, fp64), as they stand, on 2^20 .. 2^26
    # elements; bytes counted as for the GPU (the arrays the update reads and writes, at the oracle's 8 bytes each)
    from oracle import hift_oracle as O
    cpu_rows = []
    for kind, name, arrays in ((0, "adamw", 7), (1, "adagrad", 5), (2, "sgdm", 5)):
        for lg in range(20, 27, 2):
            n = 1 << lg
            master, grad, s0, s1 = (x.astype(np.float64) for x in synth.flat_optimizer_inputs(n, seed=lg, warm=True))
            s0 = np.abs(s0)
            reps = max(1, min(5, (1 << 24) // n))
            t0 = time.perf_counter()
            for r in range(reps):
                if kind == 0:
                    master, s0, s1 = O.adamw_update(master, grad, s0, s1, 1e-3, 0.9, 0.999, 1e-8, 0.01, 2 + r)
                elif kind == 1:
                    master, s0 = O.adagrad_update(master, grad, s0, 1e-2, 1e-10)
                else:
                    master, s0 = O.sgdm_update(master, grad, s0, 1e-3, 0.9)
            dt = (time.perf_counter() - t0) / reps
            cpu_rows.append({"optimizer": name, "log2_n": lg, "ms": round(dt * 1e3, 2), "elements_per_s": round(n / dt / 1e6, 1),
                             "gbs": round(n * 8 * arrays / dt / 1e9, 2)})
    try:
        threads = len(os.sched_getaffinity(0))
    except Exception:
        threads = os.cpu_count() or 1
    print(json.dumps({"sweep": "optimizer", "unit": "GB/s", "hbm_peak_gbs": peaks["hbm_gbs"],
                      "peak_source": peaks["source"], "rows": rows,
                      "cpu_oracle": {"kind": "oracle (numpy fp64 update functions as they stand)", "cores": threads,
                                     "elements_per_s_unit": "M elements/s", "rows": cpu_rows}}))


def run_sweep_depth(args):
    """GPT-2-large-shaped config with block-group g = 0..17 forced active (plus the embedding and head
    groups): step time and dX / dW GEMM throughput versus the depth at which the backward pass stops."""
    import torch
    from paper_2401_15207_b200 import HiFT
    cfg, gcfg, ocfg = synth.config_gpt2_large(synth.OPT_SGDM)
    ocfg = synth.OptCfg(**{**ocfg.__dict__, "prefetch_groups": 1})
    h = HiFT(cfg, gcfg, ocfg)
    h.init_synthetic(5, cfg.init_std)
    dev = [tuple(torch.from_numpy(a).cuda() for a in synth.batch_for(cfg, 5, t)) for t in range(4)]
    peaks = measured_peaks()
    rows = []
    for g in range(h.num_groups()):
        h.force_group(g)
        for t in range(3):
            h.step(*dev[t])
        h.profile_enable(True)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        for t in range(4):
            h.step(*dev[t])
        e1.record()
        torch.cuda.synchronize()
        prof = h.profile()
        h.profile_enable(False)
        lo, hi = h.group_units(g)
        tf = lambda c: prof[c]["work"] / (prof[c]["ms"] * 1e-3) / 1e12 if prof[c]["ms"] > 0 else 0.0
        label = "embedding" if hi == 0 else ("head" if lo == cfg.n_blocks + 1 else f"blocks {lo - 1}-{hi - 1}")
        rows.append({"group": g, "units": label, "ms_per_step": round(e0.elapsed_time(e1) / 4, 3),
                     "dx_tflops": round(tf("gemm_dx"), 1), "dw_tflops": round(tf("gemm_dw"), 1),
                     "dx_frac_of_peak": round(tf("gemm_dx") / peaks["bf16_tflops_sustained"], 3),
                     "dw_frac_of_peak": round(tf("gemm_dw") / peaks["bf16_tflops_sustained"], 3),
                     "dx_launches": prof["gemm_dx"]["launches"] // 4, "dw_launches": prof["gemm_dw"]["launches"] // 4})
    h.close()
    print(json.dumps({"sweep": "depth", "workload": "gpt2large", "peak_tflops": peaks["bf16_tflops_sustained"],
                      "rows": rows}))


# dram__bytes_read.sum + dram__bytes_write.sum of the tensor-core GEMM launches of one llama7b step (the step that
# trains block 4: 129 forward, 113 dX, 4 dW launches).  Taken with ncu on `--micro step` (the same model with three
# blocks, a few GB: one frozen block, the active block, one block above it and the head) and scaled to 32 blocks by the
# number of blocks of each kind; the whole step is timed with CUDA events only.  Retake it after a change to the GEMM.
NCU_GEMM_TRAFFIC = {
    "bytes_per_launch": 53.214e9 / 246,
    "note": "ncu on a three-block model of the same width, every GEMM launch of one step, scaled to 32 blocks by block "
            "kind: 53.21 GB over the 246 GEMM launches of the step that trains block 4 = 216.3 MB per launch, against "
            "205.1 MB of operands and results per launch (1.05)",
}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=34)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llama7b", choices=sorted(WORKLOADS))
    ap.add_argument("--parallel", default="replicas", choices=["replicas", "dp", "zero1"],
                    help="N > 1: independent replicas (default); dp: one model, data parallel, the active group's gradient "
                         "all-reduced chunk by chunk behind the backward pass; zero1: the same with the optimizer state (and its "
                         "paging) split over the ranks: gradient pieces reduced to their owners, updated parameter pieces broadcast")
    ap.add_argument("--prefetch", type=int, default=3,
                    help="state slots beyond the first (0 paper order, 1 upload at step start, 2-3 uploads one or two steps ahead)")
    ap.add_argument("--no-pcie", action="store_true", help="leave out the pinned-memcpy ceiling measurement")
    ap.add_argument("--offload", type=int, default=1)
    ap.add_argument("--recompute", type=int, default=0,
                    help="1: frozen blocks above the group keep only their input and are recomputed in the backward pass "
                         "(less HBM, one more forward of those blocks)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--full-param", action="store_true",
                    help="one group holding every unit, state resident: the ordinary full-parameter step")
    ap.add_argument("--skip-e2e", action="store_true", help="profiling runs: leave out the end-to-end leg")
    ap.add_argument("--skip-profiled", action="store_true", help="profiling runs: leave out the event-bracketed pass")
    ap.add_argument("--no-full-param-reference", action="store_true",
                    help="leave out the k = 1 full-parameter step of the same model (needs ~132 GB at the 7B shape)")
    ap.add_argument("--sweep", default=None, choices=["optimizer", "depth"],
                    help="kernel sweeps instead of the step benchmark")
    ap.add_argument("--micro", default=None, choices=["gemm", "kernels", "step", "sdpa"],
                    help="single kernels at the workload's shapes, a few launches each (small enough for an ncu capture)")
    ap.add_argument("--launches", type=int, default=3)
    ap.add_argument("--only", default=None, help="--micro gemm: only shapes whose name contains this")
    ap.add_argument("--steps-ref", type=int, default=0, help="--impl reference: overrides --steps / --warmup when > 0")
    ap.add_argument("--warmup-ref", type=int, default=0)
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if args.sweep == "optimizer":
        return run_sweep_optimizer(args)
    if args.sweep == "depth":
        return run_sweep_depth(args)
    cfg, gcfg, ocfg = WORKLOADS[args.workload]()
    if args.micro:
        return run_micro(args, cfg)
    if args.full_param:
        gcfg = synth.GroupCfg(layers_per_group=cfg.n_units, split_emb_head=0, order=synth.ORDER_BOTTOM2UP)
        args.offload, args.prefetch = 0, 0
    if args.impl == "reference":
        run_reference(args, cfg, gcfg, ocfg)
    else:
        run_ours(args, cfg, gcfg, ocfg)


if __name__ == "__main__":
    main()
