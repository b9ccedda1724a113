#!/usr/bin/env python
"""Benchmark of the RAP decode hot path on B200: decode tokens/s and the attention scan's
achieved HBM bandwidth on a synthetic, seeded, 8B-shaped stack (rho = 0.7, 32K-token cache).

One step = every layer's rap_qkv_rope_append + rap_decode_attn for one batch of new tokens.
`value` is timed with inputs resident in HBM; `e2e` goes through rap_decode_step_host with
pinned host inputs and outputs.  `--impl reference` times the CPU oracle on a bounded sample.
Prints ONE JSON line on rank 0.
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

from paper_2602_02599_b200 import synth  # noqa: E402

METRIC = "decode_tokens_per_s"
UNIT = "tokens/s"
T_PREFILL_TAIL = 256     # last cached positions of every sequence are written by the real append path


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return float(p["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def load_traffic(workload):
    """(DRAM bytes per attention-scan launch, where the figure comes from) from the committed ncu summary, if it
    lists this workload.  The counters are not taken in this run: the file holds one capture on a cut-down launch,
    scaled to the full launch by the number of (sequence, KV head) units."""
    path = os.path.join(ROOT, "profiles", "attn_decode_traffic.txt")
    if os.path.exists(path):
        source = "ncu capture on a cut-down launch, scaled by units (profiles/attn_decode_traffic.txt)"
        for line in open(path):
            if line.startswith("# source:"):
                source = line[len("# source:"):].strip()
            f = line.split()
            if len(f) == 2 and f[0] == workload:
                return float(f[1]), source
    return None, None


class ClockSampler(threading.Thread):
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        super().__init__(daemon=True)
        self.index, self.rows, self.proc = index, [], None

    def run(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            for line in self.proc.stdout:
                self.rows.append([c.strip() for c in line.split(",")])
        except Exception:
            pass

    def stop(self):
        if self.proc is not None:
            self.proc.terminate()
        self.join(timeout=2)
        sm = [float(r[0]) for r in self.rows if r and r[0].replace(".", "").isdigit()]
        mx = [float(r[1]) for r in self.rows if len(r) > 1 and r[1].replace(".", "").isdigit()]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = [n for i, n in enumerate(names) if any(len(r) > 3 + i and r[3 + i] == "Active" for r in self.rows)]
        busy = [s for s in sm if s > 0]
        return {"sm_mhz": float(np.median(busy)) if busy else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": reasons, "samples": len(sm)}


def build_stack(w, torch, seed_offset=0, new_rows=64):
    """Allocate the stack (cache capacity: the workload's context plus room for new_rows decode steps), build
    tables, upload weights and fill the caches (synthetic, seeded)."""
    from paper_2602_02599_b200.stack import DecodeStack
    st = DecodeStack(w, max_rows=max(w.batch, 2048), s_cap=((w.seq + max(64, new_rows) + 7) // 8) * 8)
    ks, vs = synth.draw_scores(w)
    st.build_tables(ks, vs)
    st.fill_synthetic(w.seed + seed_offset, tail=T_PREFILL_TAIL)
    torch.cuda.synchronize()
    return st


def max_over_ranks(values, device, world):
    """Element-wise maximum of per-rank timings (every rank gets the result): replicas share nothing
    on the data path, the only exchange of a multi-GPU run is this one reduction of clock readings."""
    import torch
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if world > 1:
        import torch.distributed as dist
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def aggregate_throughput(per_rank_batch, world, ms_per_step):
    """Whole-job tokens/s of `world` independent replicas that each decode per_rank_batch tokens per step."""
    return world * per_rank_batch / (ms_per_step * 1e-3)


def pick_workload(args):
    """The named workload, optionally cut down (--layers/--batch/--seq) for profiler-sized runs."""
    from dataclasses import replace
    w = synth.CONFIGS[args.workload]
    over = {k: v for k, v in (("n_layers", args.layers), ("batch", args.batch), ("seq", args.seq)) if v}
    return replace(w, name=w.name + "-cut", **over) if over else w


def attn_bytes(w, length):
    return w.batch * w.n_kv_heads * length * (2 * w.n_pairs + w.n_vch) * w.elem_bytes


def workload_string(w):
    return (f"{w.name}: L={w.n_layers} hidden={w.hidden} Hq/Hkv={w.n_q_heads}/{w.n_kv_heads} D={w.head_dim} "
            f"rho={w.rho} P={w.n_pairs} dv={w.n_vch} B={w.batch} S={w.seq}")


def time_decode_steps(st, w, torch, K, W, first_len, x_all, barrier=None, profile=True):
    """W warm-up steps, then K timed steps of rap_decode_step (CUDA events on the launching stream, a
    synchronize on both sides).  profile: CUDA events around every rap_decode_attn launch of the timed steps; an
    event between two launches keeps them from overlapping (inside a step the library lets a projection start
    while the attention launch before it drains), so the step time of a profiled pass is an upper bound and the
    headline value comes from a pass without them.
    Returns ms per step, ms per attention launch, ms per layer for the rest, and the launches counted."""
    L = w.n_layers
    barrier = barrier or torch.cuda.synchronize
    st.seq_len.fill_(first_len)
    for i in range(W):
        st.decode_step(x_all[i % len(x_all)], first_len + i, advance=1)
    barrier()
    launches0 = st.ctx.rap_kernel_launch_count()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if profile:
        st.ctx.rap_profile_attn(K * L)
    t0.record()
    for i in range(K):
        st.decode_step(x_all[(W + i) % len(x_all)], first_len + W + i, advance=1)
    t1.record()
    barrier()
    launches = st.ctx.rap_kernel_launch_count() - launches0
    ms_total = t0.elapsed_time(t1)
    attn_sum, attn_calls = None, K * L
    if profile:
        attn_sum, attn_calls = st.ctx.rap_profile_attn_read()
        st.ctx.rap_profile_attn(0)
        assert attn_calls == K * L, (attn_calls, K * L)
    code, detail = st.ctx.rap_get_last_device_status()
    assert code == 0, f"device status {code} detail {detail}"
    mean_len = first_len + W + (K + 1) / 2.0
    return {"ms_total": ms_total, "ms_step": ms_total / K, "attn_ms": attn_sum / attn_calls if profile else None,
            "rest_ms": (ms_total - attn_sum) / attn_calls if profile else None, "launches": int(launches),
            "mean_len": mean_len}


def time_workload(st, w, torch, K, W, x_all, barrier=None):
    """Two passes over the same K + W steps: the first without events inside the steps gives the step time, the
    second with events around every attention launch gives the per-launch times (it rewrites the rows the first
    pass appended)."""
    r = time_decode_steps(st, w, torch, K, W, w.seq, x_all, barrier, profile=False)
    rp = time_decode_steps(st, w, torch, K, W, w.seq, x_all, barrier, profile=True)
    r["attn_ms"], r["rest_ms_serialized"] = rp["attn_ms"], rp["rest_ms"]
    r["rest_ms"] = r["ms_step"] / w.n_layers - rp["attn_ms"]
    r["ms_step_profiled"] = rp["ms_step"]
    return r


def summarize(w, r, peak):
    """One workload's numbers in the shape the extra keys of the bench line use."""
    alg = attn_bytes(w, r["mean_len"])
    gbps = alg / (r["attn_ms"] * 1e-3) / 1e9
    step_bytes = w.n_layers * (alg + w.hidden * w.n_out * w.elem_bytes)
    return {"workload": workload_string(w), "tokens_per_s": w.batch / (r["ms_step"] * 1e-3), "ms_per_step": r["ms_step"],
            "attn_ms_per_layer": r["attn_ms"], "rest_ms_per_layer": r["rest_ms"],
            "rest_ms_per_layer_serialized": r.get("rest_ms_serialized"), "attn_gbps": gbps,
            "frac": gbps / peak, "frac_of_nominal_8000": gbps / 8000.0,
            "step_gbps": step_bytes / (r["ms_step"] * 1e-3) / 1e9,
            "tokens_per_s_at_70pct_of_nominal": w.batch / (step_bytes / 5600e9)}


def run_ours(args):
    import torch
    import torch.distributed as dist
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device(f"cuda:{local}"))
    w = pick_workload(args)
    L, B, K, W = w.n_layers, w.batch, args.steps, args.warmup
    n_steps = K + W
    st = build_stack(w, torch, seed_offset=rank, new_rows=2 * n_steps + 16)
    if args.attn_variant:
        st.ctx.rap_set_attn_variant(args.attn_variant)
    cut = bool(args.attn_variant or args.layers or args.batch or args.seq)
    extras = args.extras and world == 1 and not cut and args.workload == "8b"
    assert w.seq + 2 * n_steps + 8 < st.s_cap, "cache capacity too small for this many steps"
    dev = st.device
    # per-step inputs, resident in HBM before the timed region
    xg = torch.Generator(device=dev).manual_seed(w.seed + 17 + rank)
    x_all = torch.empty((n_steps, L, B, w.hidden), dtype=st.dt, device=dev).normal_(0.0, 1.0, generator=xg)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(local)
    sampler.start()
    time.sleep(0.3)
    # one C call per step: every layer's projection + RoPE + append, then the attention; the library
    # advances seq_len on the device
    r = time_decode_steps(st, w, torch, K, W, w.seq, x_all, barrier, profile=False)
    clocks = sampler.stop()
    # per-launch times of the attention scan: the same steps again with CUDA events around every launch
    rp = time_decode_steps(st, w, torch, K, W, w.seq, x_all, barrier, profile=True)
    ms_total, launches = r["ms_total"], r["launches"]
    attn_ms = rp["attn_ms"]
    proj_ms = r["ms_step"] / L - attn_ms          # what a layer costs beyond its attention launch, in the step as timed

    # ---- end to end through the host-buffer entry point ------------------------------------
    ev = lambda: torch.cuda.Event(enable_timing=True)
    hx = [torch.empty((L, B, w.hidden), dtype=st.dt).pin_memory() for _ in range(2)]
    for h in hx:
        h.copy_(x_all[0].cpu())
    h_out = torch.empty((L, st.out_stride), dtype=torch.float32).pin_memory()
    e2e_steps = K
    e2e_warm = 3
    for i in range(e2e_warm):
        st.decode_step_host(hx[i & 1], h_out, w.seq + n_steps + i, advance=1)
    barrier()
    e0 = time.perf_counter()
    d0, d1 = ev(), ev()
    d0.record()
    for i in range(e2e_steps):
        st.decode_step_host(hx[i & 1], h_out, w.seq + n_steps + e2e_warm + i, advance=1)
    d1.record()
    barrier()
    e2e_ms = max(d0.elapsed_time(d1), (time.perf_counter() - e0) * 1e3) / e2e_steps

    ms_total, e2e_ms = max_over_ranks([ms_total, e2e_ms], dev, world)
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return
    ms_step = ms_total / K
    peak, peak_kind = load_peaks()
    alg = attn_bytes(w, rp["mean_len"])
    achieved = alg / (attn_ms * 1e-3) / 1e9
    traffic, traffic_source = (None, None) if cut else load_traffic(args.workload)
    line = {
        "metric": METRIC, "value": aggregate_throughput(B, world, ms_step), "unit": UNIT, "n_gpus": world, "steps": K,
        "warmup": W, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16" if w.dtype == "bf16" else "f32", "data": "synthetic",
        "config": {"workload": workload_string(w),
                   "per_gpu_batch": B, "global_batch": world * B, "context": w.seq,
                   "l2": "inputs larger than L2 (%.1f GB of KV cache per step)" % (L * alg / 1e9),
                   "parallelism": "replicas" if world > 1 else "single"},
        "clocks": clocks, "gpu_launches": int(launches),
        "e2e": {"value": aggregate_throughput(B, world, e2e_ms), "unit": UNIT, "steps": e2e_steps, "warmup": e2e_warm,
                "h2d_bytes_per_step": int(hx[0].numel() * hx[0].element_size()),
                "d2h_bytes_per_step": int(h_out.numel() * 4)},
        "roofline": {"bound": "hbm", "kernel": "rap_decode_attn (attn_mma_kernel: split-KV scan with the merge of the splits fused in)"
                     if not args.attn_variant else "rap_decode_attn (forced tier %d)" % args.attn_variant,
                     "achieved": achieved,
                     "peak": peak, "peak_source": peak_kind + " copy bandwidth (read + write); a read-only stream can exceed it",
                     "unit": "GB/s", "frac": achieved / peak,
                     "frac_of_nominal_8000": achieved / 8000.0, "bytes_per_launch": alg, "ms_per_launch": attn_ms,
                     "traffic": traffic, "traffic_source": traffic_source},
        "kernels": {"attn_ms_per_layer": attn_ms, "rest_ms_per_layer": proj_ms,
                    "rest_ms_per_layer_serialized": rp["rest_ms"], "ms_per_step_with_events": rp["ms_step"],
                    "note": "attention launches timed in a second pass over the same steps with CUDA events around each "
                            "launch; events keep consecutive kernels from overlapping, so that pass is slower than the "
                            "step time `value` is taken from"},
    }
    if achieved > peak:
        line["roofline"]["note"] = ("achieved exceeds the measured copy figure: that figure is a read+write copy, this kernel only "
                                    "reads; judge it by frac_of_nominal_8000")
    if extras:
        # the scan on the plain FP32 pipes (no tensor-core instruction), same workload and protocol
        st.ctx.rap_set_attn_variant(3)
        k2 = min(K, 5)
        r3 = time_workload(st, w, torch, k2, 3, x_all)      # rewrites the rows the first passes appended
        st.ctx.rap_set_attn_variant(0)
        line["fp32_pipe_scan"] = dict(summarize(w, r3, peak), steps=k2, warmup=3, kernel="attn_scan_kernel (forced tier 3)")
    if args.cpu_baseline:
        line["cpu_baseline"] = cpu_baseline(w, st, torch)
    if extras:
        st.close()
        del st, x_all
        torch.cuda.empty_cache()
        line["other_workloads"] = other_workloads(torch, min(K, 10), peak)
        line["sweep"] = sweep_rows(torch, min(K, 10), 3, peak)
        line["quantised_cache"] = q8_rows(torch, min(K, 10), 3, peak)
        line["quantised_cache_step"] = q8_step(torch, "8b", min(K, 10), 3)
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def other_workloads(torch, K, peak):
    """The 3B- and 14B-shaped workloads through the same protocol as the headline (whole decode steps)."""
    rows = []
    for name in ("3b", "14b"):
        w = synth.CONFIGS[name]
        st = build_stack(w, torch, new_rows=K + 8)
        xg = torch.Generator(device=st.device).manual_seed(w.seed + 17)
        x_all = torch.empty((K + 3, w.n_layers, w.batch, w.hidden), dtype=st.dt, device=st.device).normal_(0.0, 1.0, generator=xg)
        r = time_workload(st, w, torch, K, 3, x_all)
        rows.append(dict(summarize(w, r, peak), steps=K, warmup=3))
        st.close()
        del st, x_all
        torch.cuda.empty_cache()
    return rows


class CoreMeter:
    """Cores that actually worked inside the `with` blocks: process CPU time over wall time."""

    def __init__(self):
        self.cpu, self.wall = 0.0, 0.0

    def __enter__(self):
        t = os.times()
        self._c, self._w = t.user + t.system, time.perf_counter()

    def __exit__(self, *exc):
        t = os.times()
        self.cpu += t.user + t.system - self._c
        self.wall += time.perf_counter() - self._w

    def cores(self):
        return max(1, int(round(self.cpu / self.wall))) if self.wall > 0 else 1


def cpu_baseline(w, st, torch, budget_s=15.0):
    """The oracle, as it stands, on the host cores: full-length scans of sampled (layer, b, kv-head)
    units plus one layer's projection, extrapolated linearly to a whole step."""
    from oracle import rap_oracle as O
    rng = np.random.default_rng(123)
    L, B, Hkv, Hq, G = w.n_layers, w.batch, w.n_kv_heads, w.n_q_heads, w.group
    n = w.seq + 1
    torch.cuda.synchronize()
    busy = CoreMeter()
    times, t_start = [], time.perf_counter()
    while time.perf_counter() - t_start < budget_s and len(times) < 256:
        l, b, h = int(rng.integers(L)), int(rng.integers(B)), int(rng.integers(Hkv))
        K = st.k_cache[l][b, h, :n].to(torch.float64).cpu().numpy()[None, None]
        V = st.v_cache[l][b, h, :n].to(torch.float64).cpu().numpy()[None, None]
        q = rng.standard_normal((1, G, K.shape[-1]))
        t = time.perf_counter()
        with busy:
            O.decode_attn(q, K, V, [n], w.head_dim)
        times.append(time.perf_counter() - t)
    x = O.round_storage(synth.draw_hidden(w, 0, 0, B), w.dtype)
    wq = st.w_qkv[0].to(torch.float64).cpu().numpy()
    inv = st.inv_freq[0].cpu().numpy()
    t = time.perf_counter()
    with busy:
        O.qkv_rope(x, wq, None, np.full(B, w.seq), inv, Hq, Hkv, w.n_pairs, w.n_vch)
    t_proj = time.perf_counter() - t
    t_step = float(np.mean(times)) * L * B * Hkv + L * t_proj
    return {"value": B / t_step, "unit": UNIT, "cores": busy.cores(), "cores_available": os.cpu_count(), "kind": "oracle",
            "sample": f"{len(times)} of {L * B * Hkv} (layer, sequence, kv-head) full-length scans + 1 of {L} layer "
                      f"projections, one after the other (the NumPy routines decide how many threads work: `cores` is "
                      f"process CPU time / wall time over the timed calls), extrapolated linearly to one step"}


def run_reference(args):
    """Reference arm: the CPU oracle on host cores, each step a bounded sample of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import rap_oracle as O
    w = pick_workload(args)
    busy = CoreMeter()
    L, B, Hkv, Hq, G = w.n_layers, w.batch, w.n_kv_heads, w.n_q_heads, w.group
    n = w.seq + 1
    units_per_step = 8
    rng = np.random.default_rng(w.seed)
    sigma = float(np.sqrt(w.hidden) * 0.02)
    wq = O.round_storage(synth.draw_packed_weights(w, 0), w.dtype)
    ks, vs = synth.draw_scores(synth.scaled_down(w, n_layers=1, batch=1, seq=8))
    tabs = O.build_tables(ks, vs, [w.n_pairs], [w.n_vch], w.head_dim, w.rope_theta, w.pairing)

    def sample_step(i):
        t_units = 0.0
        for u in range(units_per_step):
            K = O.round_storage(synth.draw_cache_rows(w, 0, i, u, n, 2 * w.n_pairs, 0), w.dtype)[None, None]
            V = O.round_storage(synth.draw_cache_rows(w, 0, i, u, n, w.n_vch, 1), w.dtype)[None, None]
            q = O.round_storage(rng.standard_normal((1, G, 2 * w.n_pairs)) * sigma, w.dtype)
            t = time.perf_counter()
            with busy:
                O.decode_attn(q, K, V, [n], w.head_dim)
            t_units += time.perf_counter() - t
        x = O.round_storage(synth.draw_hidden(w, 0, i, B), w.dtype)
        t = time.perf_counter()
        with busy:
            O.qkv_rope(x, wq, None, np.full(B, w.seq), tabs["inv_freq"][0], Hq, Hkv, w.n_pairs, w.n_vch)
        t_proj = time.perf_counter() - t
        return t_units / units_per_step * L * B * Hkv + L * t_proj

    for i in range(args.warmup):
        sample_step(i)
    est = [sample_step(args.warmup + i) for i in range(args.steps)]
    t_step = float(np.mean(est))
    val = B / t_step
    sample = (f"per step: {units_per_step} of {L * B * Hkv} (layer, sequence, kv-head) full-length scans + 1 of {L} "
              f"layer projections on synthetic rows, one after the other (`cores` is process CPU time / wall time over "
              f"the timed calls), extrapolated linearly to the whole step")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": int(os.environ.get("WORLD_SIZE", "1")),
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": t_step * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": workload_string(w), "per_gpu_batch": B, "global_batch": B, "context": w.seq,
                   "l2": "inputs larger than L2 (%.1f GB of KV cache per step)" % (L * attn_bytes(w, w.seq + args.warmup + (args.steps + 1) / 2.0) / 1e9),
                   "parallelism": "single"},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": busy.cores(), "cores_available": os.cpu_count(), "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }), flush=True)


def sweep_rows(torch, steps, warmup, peak):
    """Retain-ratio sweep on the 8B shape (batch 16, 16384-token cache, two layers resident): time of
    rap_decode_attn per layer at each rho against the same kernel at rho = 1 (dense), and against the
    low-rank comparator at equal cached dims (latent K of width 2P rebuilt and rotated every call).  Beside the
    comparator's time stands its own bound: reading the latents and V and writing and re-reading the rebuilt
    full-width K at the measured copy bandwidth."""
    from dataclasses import replace
    from paper_2602_02599_b200.stack import DecodeStack
    rows, dense_ms = [], None
    for rho in sorted(synth.SWEEP_COUNTS, reverse=True):
        w = replace(synth.sweep_workload(rho), n_layers=2)
        st = DecodeStack(w)
        st.build_tables(*synth.draw_scores(w))
        g = torch.Generator(device=st.device).manual_seed(w.seed)
        sigma = float(np.sqrt(w.hidden) * 0.02)
        for l in range(2):
            st.k_cache[l].normal_(0.0, sigma, generator=g)
            st.v_cache[l].normal_(0.0, sigma, generator=g)
        n = w.seq + 1
        q = torch.empty((w.batch, w.n_q_heads, 2 * w.n_pairs), dtype=st.dt, device=st.device).normal_(0, sigma, generator=g)
        qf = torch.empty((w.batch, w.n_q_heads, w.head_dim), dtype=st.dt, device=st.device).normal_(0, sigma, generator=g)
        bk = torch.from_numpy(synth.draw_lowrank_factor(w, 0, 2 * w.n_pairs)).to(st.device).to(st.dt).contiguous()
        dl = torch.full((w.batch,), n, dtype=torch.int32, device=st.device)
        out = torch.empty((w.batch, w.n_q_heads, w.n_vch), dtype=torch.float32, device=st.device)

        def timed(fn):
            for i in range(warmup):
                fn(i & 1)
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for i in range(steps):
                fn(i & 1)          # alternate the two layers: 2 x ~1 GB of cache, larger than L2
            e1.record()
            torch.cuda.synchronize()
            return e0.elapsed_time(e1) / steps

        rap_ms = timed(lambda l: st.decode_attn(l, q, dl, n))
        low_ms = timed(lambda l: st.ctx.rap_lowrank_decode_attn(w.batch, 2 * w.n_pairs, w.n_vch, qf, st.k_cache[l], bk,
                                                                st.v_cache[l], st.s_cap, dl, n, 0, out))
        code, detail = st.ctx.rap_get_last_device_status()
        assert code == 0, (code, detail)
        if rho == 1.0:
            dense_ms = rap_ms
        by = attn_bytes(w, n)
        units = w.batch * w.n_kv_heads * n * w.elem_bytes
        low_bytes = units * (2 * w.n_pairs + 2 * w.head_dim + w.n_vch)
        low_bound_ms = low_bytes / (peak * 1e9) * 1e3
        rows.append({"rho": rho, "P": w.n_pairs, "dv": w.n_vch, "kv_bytes_per_layer": by, "rap_attn_ms": rap_ms,
                     "rap_GBps": by / rap_ms / 1e6, "rap_frac": by / rap_ms / 1e6 / peak,
                     "rap_frac_of_nominal_8000": by / rap_ms / 1e6 / 8000.0, "rap_vs_dense": rap_ms / dense_ms,
                     "bytes_vs_dense": (2 * w.n_pairs + w.n_vch) / 256.0, "lowrank_attn_ms": low_ms,
                     "lowrank_vs_dense": low_ms / dense_ms, "lowrank_bound_ms": low_bound_ms,
                     "lowrank_bound_vs_dense": low_bound_ms / dense_ms, "lowrank_frac_of_its_bound": low_bound_ms / low_ms})
        st.close()
        del st, q, qf, bk, out
        torch.cuda.empty_cache()
    return rows


def q8_step(torch, name, K, W):
    """Whole decode steps over quantised caches (rap_decode_step_q8: per layer the projection, the quantising append
    and the attention over the quantised cache) on a named workload at full size: tokens/s.  The caches are made
    layer by layer from synthetic bf16 rows by rap_quantize_rows."""
    from paper_2602_02599_b200 import binding
    from paper_2602_02599_b200.stack import DecodeStack
    w = synth.CONFIGS[name]
    st = DecodeStack(w, max_rows=max(w.batch, 32), s_cap=((w.seq + 64 + 7) // 8) * 8, alloc_cache=False)
    st.build_tables(*synth.draw_scores(w))
    g = torch.Generator(device=st.device).manual_seed(w.seed)
    sigma = float(np.sqrt(w.hidden) * 0.02)
    kb, vb = binding.rap_q8_row_bytes(2 * w.n_pairs), binding.rap_q8_row_bytes(w.n_vch)
    n_rows = w.batch * w.n_kv_heads * st.s_cap
    k8, v8 = [], []
    tk = torch.empty((n_rows, 2 * w.n_pairs), dtype=st.dt, device=st.device)
    tv = torch.empty((n_rows, w.n_vch), dtype=st.dt, device=st.device)
    for l in range(w.n_layers):
        st.set_packed_weights(l, synth.draw_packed_weights(w, l))
        tk.normal_(0.0, sigma, generator=g)
        tv.normal_(0.0, sigma, generator=g)
        k8.append(torch.empty((n_rows, kb), dtype=torch.uint8, device=st.device))
        v8.append(torch.empty((n_rows, vb), dtype=torch.uint8, device=st.device))
        st.ctx.rap_quantize_rows(binding.RAP_BF16, n_rows, 2 * w.n_pairs, tk, k8[l])
        st.ctx.rap_quantize_rows(binding.RAP_BF16, n_rows, w.n_vch, tv, v8[l])
    del tk, tv
    x_all = torch.empty((K + W, w.n_layers, w.batch, w.hidden), dtype=st.dt, device=st.device).normal_(0.0, 1.0, generator=g)
    wq, k8p, v8p = binding.ptr_array(st.w_qkv), binding.ptr_array(k8), binding.ptr_array(v8)
    st.seq_len.fill_(w.seq)

    def step(i):
        st.ctx.rap_decode_step_q8(w.batch, x_all[i], wq, None, st.inv_freq, k8p, v8p, st.s_cap, st.seq_len, w.seq + i, 0,
                                  st.q_scratch, st.out, st.out_stride, 1)

    for i in range(W):
        step(i)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(K):
        step(W + i)
    e1.record()
    torch.cuda.synchronize()
    code, detail = st.ctx.rap_get_last_device_status()
    assert code == 0, (code, detail)
    ms = e0.elapsed_time(e1) / K
    st.close()
    del st, k8, v8, x_all
    torch.cuda.empty_cache()
    return {"workload": workload_string(w), "tokens_per_s": w.batch / (ms * 1e-3), "ms_per_step": ms, "steps": K, "warmup": W,
            "kv_bytes_per_step": w.n_layers * w.batch * w.n_kv_heads * (w.seq + W + (K + 1) / 2.0) * (kb + vb)}


def q8_rows(torch, steps, warmup, peak, names=("3b", "8b", "14b"), batch=0):
    """Composition with 8-bit cache quantisation: rap_decode_attn_q8 against rap_decode_attn on the shaped workloads
    (full batch and context, two layers resident and alternated so that the caches are larger than L2).  The
    quantised caches are made from the same synthetic bf16 rows by rap_quantize_rows.  Algorithmic bytes of the
    quantised scan: B * H_kv * len * (row bytes of K + row bytes of V), scales and padding included."""
    from dataclasses import replace
    from paper_2602_02599_b200 import binding
    from paper_2602_02599_b200.stack import DecodeStack
    rows = []
    for name in names:
        w = replace(synth.CONFIGS[name], n_layers=2)
        if batch:
            w = replace(w, batch=batch, name=w.name + "-cut")
        st = DecodeStack(w)
        st.build_tables(*synth.draw_scores(w))
        g = torch.Generator(device=st.device).manual_seed(w.seed)
        sigma = float(np.sqrt(w.hidden) * 0.02)
        kb, vb = binding.rap_q8_row_bytes(2 * w.n_pairs), binding.rap_q8_row_bytes(w.n_vch)
        n_rows = w.batch * w.n_kv_heads * st.s_cap
        k8, v8 = [], []
        for l in range(2):
            st.k_cache[l].normal_(0.0, sigma, generator=g)
            st.v_cache[l].normal_(0.0, sigma, generator=g)
            k8.append(torch.empty((n_rows, kb), dtype=torch.uint8, device=st.device))
            v8.append(torch.empty((n_rows, vb), dtype=torch.uint8, device=st.device))
            st.ctx.rap_quantize_rows(binding.RAP_BF16, n_rows, 2 * w.n_pairs, st.k_cache[l], k8[l])
            st.ctx.rap_quantize_rows(binding.RAP_BF16, n_rows, w.n_vch, st.v_cache[l], v8[l])
        n = w.seq + 1
        q = torch.empty((w.batch, w.n_q_heads, 2 * w.n_pairs), dtype=st.dt, device=st.device).normal_(0, sigma, generator=g)
        dl = torch.full((w.batch,), n, dtype=torch.int32, device=st.device)
        out = torch.empty((w.batch, w.n_q_heads, w.n_vch), dtype=torch.float32, device=st.device)

        def timed(fn):
            for i in range(warmup):
                fn(i & 1)
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for i in range(steps):
                fn(i & 1)
            e1.record()
            torch.cuda.synchronize()
            return e0.elapsed_time(e1) / steps

        ms16 = timed(lambda l: st.decode_attn(l, q, dl, n))
        ms8 = timed(lambda l: st.ctx.rap_decode_attn_q8(l, w.batch, q, k8[l], v8[l], st.s_cap, dl, n, 0, out))
        code, detail = st.ctx.rap_get_last_device_status()
        assert code == 0, (code, detail)
        by16 = attn_bytes(w, n)
        by8 = w.batch * w.n_kv_heads * n * (kb + vb)
        dense = w.batch * w.n_kv_heads * n * 2 * w.head_dim * w.elem_bytes
        rows.append({"workload": workload_string(w), "bf16_attn_ms": ms16, "q8_attn_ms": ms8, "q8_speedup": ms16 / ms8,
                     "q8_bytes_per_layer": by8, "q8_bytes_vs_bf16": by8 / by16, "q8_bytes_vs_unpruned_bf16": by8 / dense,
                     "q8_GBps": by8 / ms8 / 1e6, "q8_frac": by8 / ms8 / 1e6 / peak, "q8_frac_of_nominal_8000": by8 / ms8 / 1e6 / 8000.0,
                     "steps": steps, "warmup": warmup})
        st.close()
        del st, k8, v8, q, out
        torch.cuda.empty_cache()
    return rows


def run_q8(args):
    """--q8: the quantised-cache rows alone (optionally one workload, optionally a cut batch for profiler runs)."""
    import torch
    torch.cuda.set_device(0)
    peak, _ = load_peaks()
    names = (args.workload,) if args.workload in ("3b", "14b") or args.batch else ("3b", "8b", "14b")
    rows = q8_rows(torch, args.steps, args.warmup, peak, names=names, batch=args.batch)
    line = {"metric": "quantised_cache_attention", "unit": "ms", "n_gpus": 1, "steps": args.steps,
            "warmup": args.warmup, "dtype": "int8 codes, fp16 MMA, fp32 accumulate", "data": "synthetic",
            "higher_is_better": False, "quantised_cache": rows}
    if not args.batch:
        line["quantised_cache_step"] = q8_step(torch, args.workload if args.workload in ("3b", "8b", "14b") else "8b", args.steps, args.warmup)
    print(json.dumps(line), flush=True)


def run_sweep(args):
    import torch
    torch.cuda.set_device(0)
    peak, _ = load_peaks()
    rows = sweep_rows(torch, args.steps, args.warmup, peak)
    print(json.dumps({"metric": "attention_cost_ratio_vs_dense", "unit": "ratio", "n_gpus": 1, "steps": args.steps,
                      "warmup": args.warmup, "dtype": "bf16", "data": "synthetic", "higher_is_better": False,
                      "config": {"workload": "sweep on the 8B shape: 32q/8kv heads, D=128, B=16, S=16384, 2 layers resident"},
                      "sweep": rows}), flush=True)


def run_prefill(args):
    """rap_prefill_attn (causal block attention on the reduced dims) on the 8B head shapes of the retain-ratio
    sweep: time per call, TFLOP/s on the causal flops B H_q T (T + 1) (2P + d_v'), and the fraction of the measured
    dense bf16 peak.  --prefill-case B:T picks the size (default 2:4096 and 1:16384); --attn-variant 1 times the
    warp-level mma.sync kernel instead of the tcgen05 one."""
    import torch
    from dataclasses import replace
    from paper_2602_02599_b200.stack import DecodeStack
    torch.cuda.set_device(0)
    peak = None
    pp = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(pp):
        peak = json.load(open(pp)).get("bf16_tflops")
    cases = [tuple(int(v) for v in c.split(":")) for c in (args.prefill_case.split(",") if args.prefill_case else ["2:4096", "1:16384"])]
    rows = []
    for B, T in cases:
        dense_ms = None
        for rho in sorted(synth.SWEEP_COUNTS, reverse=True):
            w = replace(synth.sweep_workload(rho), n_layers=1, batch=B, seq=T)
            st = DecodeStack(w, s_cap=T + 8)
            st.build_tables(*synth.draw_scores(w))
            if args.attn_variant:
                st.ctx.rap_set_attn_variant(args.attn_variant)
            g = torch.Generator(device=st.device).manual_seed(w.seed)
            sigma = float(np.sqrt(w.hidden) * 0.02)
            st.k_cache[0].normal_(0.0, sigma, generator=g)
            st.v_cache[0].normal_(0.0, sigma, generator=g)
            q = torch.empty((B, T, w.n_q_heads, 2 * w.n_pairs), dtype=st.dt, device=st.device).normal_(0, sigma, generator=g)
            ds = torch.zeros(B, dtype=torch.int32, device=st.device)
            out = torch.empty((B, T, w.n_q_heads, w.n_vch), dtype=torch.float32, device=st.device)
            call = lambda: st.ctx.rap_prefill_attn(0, B, T, q, st.k_cache[0], st.v_cache[0], st.s_cap, ds, 0, out)
            for _ in range(args.warmup):
                call()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(args.steps):
                call()
            e1.record()
            torch.cuda.synchronize()
            ms = e0.elapsed_time(e1) / args.steps
            code, detail = st.ctx.rap_get_last_device_status()
            assert code == 0, (code, detail)
            if rho == 1.0:
                dense_ms = ms
            flops = B * w.n_q_heads * T * (T + 1) * (2 * w.n_pairs + w.n_vch)
            tf = flops / ms / 1e9
            rows.append({"rho": rho, "P": w.n_pairs, "dv": w.n_vch, "B": B, "T": T, "ms": ms, "TFLOPs": tf,
                         "frac_of_measured_bf16_peak": tf / peak if peak else None, "time_vs_dense": ms / dense_ms})
            st.close()
            del st, q, out
            torch.cuda.empty_cache()
    print(json.dumps({"metric": "prefill_attention_tflops", "unit": "TFLOP/s", "n_gpus": 1, "steps": args.steps,
                      "warmup": args.warmup, "dtype": "bf16", "data": "synthetic", "higher_is_better": True,
                      "config": {"workload": "rap_prefill_attn on the 8B head shapes (32q/8kv heads, D=128), start = 0"},
                      "roofline": {"bound": "tensor", "peak": peak, "peak_source": "measured" if peak else None, "unit": "TFLOP/s"},
                      "prefill": rows}), flush=True)


def replica_launch_command(n, argv):
    """`bench.py --gpus N` started without a launcher: the command that starts N replica processes of this
    script, one per GPU, on this node (rendezvous on 127.0.0.1 at a free port)."""
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
            "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + list(argv)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="8b", choices=sorted(synth.CONFIGS))
    ap.add_argument("--no-cpu-baseline", dest="cpu_baseline", action="store_false")
    ap.add_argument("--layers", type=int, default=0, help="cut the workload to this many layers (profiling)")
    ap.add_argument("--batch", type=int, default=0, help="cut the workload to this batch (profiling)")
    ap.add_argument("--seq", type=int, default=0, help="cut the workload to this context (profiling)")
    ap.add_argument("--attn-variant", type=int, default=0,
                    help="force a kernel tier of rap_decode_attn (profiling; 3 = the FP32-pipe scan)")
    ap.add_argument("--prefill", action="store_true", help="time rap_prefill_attn on the sweep's head shapes")
    ap.add_argument("--prefill-case", default="", help="B:T[,B:T...] for --prefill")
    ap.add_argument("--sweep", action="store_true", help="retain-ratio sweep with the dense and low-rank comparators")
    ap.add_argument("--q8", action="store_true", help="rap_decode_attn_q8 against rap_decode_attn on the shaped workloads")
    ap.add_argument("--no-extras", dest="extras", action="store_false",
                    help="headline measurement only (skip the other workloads, the sweep and the FP32-pipe scan)")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(subprocess.call(replica_launch_command(args.gpus, sys.argv[1:])))
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3
    if int(os.environ.get("WORLD_SIZE", "1")) > 1:
        args.cpu_baseline = False
    if args.impl == "reference":
        run_reference(args)
    elif args.q8:
        run_q8(args)
    elif args.sweep:
        run_sweep(args)
    elif args.prefill:
        run_prefill(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
