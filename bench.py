"""Benchmark of the MoQAE hot path: one step = route (once per routing-sharing group) ->
quantise+pack (every layer) -> decode attention (every layer) on a synthetic Llama-shaped
workload.  Prints ONE JSON line (rank 0).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg4|cfg2|cfg3]
    python bench.py --impl reference ...      # the CPU oracle on a bounded sample

The headline `value` is the decode-attention effective HBM bandwidth: bytes the method must
move in the decode phase (packed KV + scale/zero + tail + q + split partials + out) divided by
the device time of that phase, measured with CUDA events inside the timed steps.  N > 1 runs
independent replicas (the path has no exchange step): value = sum of all ranks' bytes / max
time.
"""
from __future__ import annotations

import argparse
import dataclasses
import datetime
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

L2_BYTES = 126 * 1024 * 1024

# dram__bytes_read.sum + dram__bytes_write.sum of ONE decode_mma_kernel launch (one cfg4 layer at full
# context, realised mix 57.7/31.4/6.4/4.5), from the ncu capture summarised in
# profiles/decode_mma_kernel_cfg4.txt: 617.81 MB + 5.65 MB against 619.0 MB of algorithmic bytes.
# Reported only for the workload and launch shape it was taken on.
NCU_DECODE_TRAFFIC = {"cfg4": 623457536}


def read_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            p = json.load(f)
        return float(p["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples taken while the timed region runs.  The tool
    needs a few hundred ms to produce its first line, so it is started before the warm-up and only
    the samples whose time stamps fall between begin() and end() are used."""
    Q = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None
        self.t_begin = self.t_end = None

    def begin(self):
        self.t_begin = datetime.datetime.now()

    def end(self):
        self.t_end = datetime.datetime.now()

    def start(self):
        try:
            self.p = subprocess.Popen(["nvidia-smi", "-i", str(self.gpu), f"--query-gpu={self.Q}",
                                       "--format=csv,noheader,nounits", "-lms", "50"],
                                      stdout=self.f, stderr=subprocess.DEVNULL)
        except Exception:
            self.p = None

    def stop(self):
        """Ends the sampling; returns the summary of the begin()..end() window."""
        if self.p is not None:
            self.p.terminate()
            try:
                self.p.wait(timeout=5)
            except Exception:
                self.p.kill()
            self.f.flush()
            self.f.seek(0)
            self.lines = self.f.read().splitlines()
            try:
                os.unlink(self.f.name)
            except OSError:
                pass
        return self.summary(self.t_begin, self.t_end)

    def summary(self, t_begin, t_end):
        """Median SM clock and the throttle reasons seen between two host time stamps."""
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.p is None:
            return out
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in getattr(self, "lines", []):
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 9:
                continue
            try:
                when = datetime.datetime.strptime(parts[0], "%Y/%m/%d %H:%M:%S.%f")
                if t_begin and t_end and not (t_begin <= when <= t_end):
                    continue
                sm.append(float(parts[1]))
                mx.append(float(parts[2]))
            except ValueError:
                continue
            for n, v in zip(names, parts[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        if sm:
            out = {"sm_mhz": float(np.median(sm)), "sm_max_mhz": float(max(mx)),
                   "reasons": sorted(reasons), "samples": len(sm)}
        return out


# ------------------------------------------------------------------------------------------
# workload set-up on the device
# ------------------------------------------------------------------------------------------
class Job:
    """Device-resident inputs, cache and scratch of one workload."""

    N_DISTINCT = 4      # distinct per-layer K/V inputs; layer l reads input l mod 4 (each > L2)

    def __init__(self, wl, device, seed=1234, context=None, force_map=False, rf=1, overlap=True):
        import torch

        from paper_2506_07533_b200 import binding as mq
        from paper_2506_07533_b200 import synth
        self.torch, self.mq, self.wl, self.device = torch, mq, wl, device
        self.overlap = overlap
        T = self.T = context or wl.context
        B, Hkv, Hq = wl.batch, wl.n_kv_heads, wl.n_q_heads
        self.cfg = mq.make_config(n_layers=wl.n_layers, n_q_heads=Hq, n_kv_heads=Hkv, chunk=wl.chunk,
                                  dtype=wl.dtype, d_in=wl.d_in, max_tokens=T + wl.chunk, batch=B,
                                  rs_group=wl.rs_group, rf_first_chunk=rf, tail_capacity=wl.chunk)
        self.rf = rf
        nd = min(self.N_DISTINCT, wl.n_layers)
        self.kv = [synth.keys_values(B, T, Hkv, 128, wl.dtype, seed + 10 * i, device,
                                     outlier_frac=wl.outlier_frac) for i in range(nd)]
        self.force_map = force_map
        nh = 0 if force_map else min(2, wl.n_groups)
        self.hidden = [synth.hidden_states(B, T, wl.d_in, wl.chunk, wl.dtype, seed + 100 + i, device)
                       for i in range(nh)]
        self.W1, self.W2, self.W3, self.bias = synth.router_weights(wl.d_in, 4, wl.dtype, seed + 7, device,
                                                                    gated=wl.gated_router)
        self.q = synth.normal((wl.n_layers, B, Hq, 128), wl.dtype, seed + 9, device)
        if wl.decode_steps > 1:
            self.k_new = synth.normal((wl.decode_steps, wl.n_layers, B, Hkv, 128), wl.dtype, seed + 11, device)
            self.v_new = synth.normal((wl.decode_steps, wl.n_layers, B, Hkv, 128), wl.dtype, seed + 12, device)
        self.out = torch.zeros((wl.n_layers, B, Hq, 128), dtype=torch.float32, device=device)
        self.ws = torch.zeros(mq.moqae_decode_attn_workspace(self.cfg), dtype=torch.uint8, device=device)
        self.n_splits = self.ws.numel() // (B * Hq * 130 * 4)
        # capacity: room for the calibrated mix with slack, never more than all chunks
        C = T // wl.chunk
        self.cache = None
        self.capacity = [C, C, C, C]
        self.forced = None
        self._calibrate(seed)

    # the router's bias is tuned (with the library's own router) until the chunk mix is within
    # five points of the workload's target; otherwise a seeded multinomial map is forced
    def _calibrate(self, seed):
        torch, mq, wl = self.torch, self.mq, self.wl
        C = self.T // wl.chunk
        probe_cfg = mq.make_config(n_layers=1, n_q_heads=wl.n_q_heads, n_kv_heads=wl.n_kv_heads, chunk=wl.chunk,
                                   dtype=wl.dtype, d_in=wl.d_in, max_tokens=self.T + wl.chunk, batch=wl.batch,
                                   rf_first_chunk=self.rf)
        probe = mq.moqae_cache_bind(probe_cfg, [1, 1, 1, 1], device=self.device)
        target = np.asarray(wl.mix, dtype=np.float64)
        bias = np.zeros(4)
        ok = False
        for it in range(0 if self.force_map else 60):
            self.bias.copy_(torch.tensor(bias, dtype=torch.float32))
            mq.moqae_route(probe_cfg, self.hidden[0], self.T, self.W1, self.W2, self.W3, self.bias, 0, probe)
            cnt = probe.count[0].sum(0).cpu().numpy().astype(np.float64)
            cnt[3] -= wl.batch * self.rf            # frozen first chunks are not the router's choice
            mix = cnt / max(cnt.sum(), 1)
            if np.abs(mix - target).max() <= 0.05:
                ok = True
                break
            step = 0.5 if it < 30 else 0.2
            bias += step * np.clip(np.log((target + 1e-3) / (mix + 1e-3)), -2, 2) * self._logit_scale(probe_cfg, probe)
        self.calibrated = ok
        if not ok:
            from paper_2506_07533_b200 import synth
            self.forced = torch.from_numpy(synth.multinomial_map(wl.batch, C, wl.mix, seed + 5)).to(self.device)
        # size the pools from the realised maps of all groups
        cap = np.ones(4, dtype=np.int64)
        for g in range(wl.n_groups):
            if self.forced is None:
                mq.moqae_route(probe_cfg, self.hidden[g % len(self.hidden)], self.T, self.W1, self.W2, self.W3,
                               self.bias, 0, probe)
                cnt = probe.count[0].cpu().numpy()
            else:
                m = self.forced.cpu().numpy()
                cnt = np.stack([(m == w).sum(1) for w in range(4)], 1)
            cap = np.maximum(cap, cnt.max(0))
        self.capacity = [int(c) for c in cap]
        del probe
        self.cache = mq.moqae_cache_bind(self.cfg, self.capacity, device=self.device)

    def _logit_scale(self, cfg, probe):
        # spread of the logits, estimated once from the vote margins being O(1): use a fixed unit
        return 1.0 if self.wl.gated_router else 0.5

    # ---- phases -------------------------------------------------------------------------
    def route_all(self):
        wl = self.wl
        if self.forced is not None:
            return
        for g in range(wl.n_groups):
            self.mq.moqae_route(self.cfg, self.hidden[g % len(self.hidden)], self.T, self.W1, self.W2, self.W3,
                                self.bias, g, self.cache)

    def quantize_all(self):
        wl = self.wl
        for l in range(wl.n_layers):
            K, V = self.kv[l % len(self.kv)]
            fm = self.forced if (self.forced is not None and l % wl.rs_group == 0) else None
            self.mq.moqae_quantize_kv(self.cfg, K, V, self.T, l, self.cache, forced_map=fm)

    def decode_all(self):
        wl = self.wl
        if wl.decode_steps == 1:
            # the layers' calls read nothing the call before them writes, so each may start while
            # the previous one is still finishing (all but the first, which follows other work)
            for l in range(wl.n_layers):
                flags = self.mq.DECODE_OVERLAP_PREVIOUS if (l > 0 and self.overlap) else 0
                self.mq.moqae_decode_attn_ex(self.cfg, self.q[l], l, self.cache, self.out[l], self.ws, flags=flags)
            return
        # generation loop: every step appends one token per sequence to each layer's 16-bit tail
        # (routing is not re-run) and attends over the grown cache
        if not self.overlap:
            for s in range(wl.decode_steps):
                for l in range(wl.n_layers):
                    self.mq.moqae_append_kv(self.cfg, self.k_new[s, l], self.v_new[s, l], l, self.cache)
                    self.mq.moqae_decode_attn(self.cfg, self.q[l], l, self.cache, self.out[l], self.ws)
            return
        # the same step with the new token's rows handed to the attention call itself: nothing is written
        # to the cache while the layers attend, so their launches can be chained; the appends follow
        for s in range(wl.decode_steps):
            for l in range(wl.n_layers):
                flags = self.mq.DECODE_OVERLAP_PREVIOUS if l > 0 else 0
                self.mq.moqae_decode_attn_step(self.cfg, self.q[l], self.k_new[s, l], self.v_new[s, l], l, self.cache,
                                               self.out[l], self.ws, flags=flags)
            for l in range(wl.n_layers):
                self.mq.moqae_append_kv(self.cfg, self.k_new[s, l], self.v_new[s, l], l, self.cache)

    def counts(self):
        return self.cache.count.cpu().numpy()           # [groups, batch, 4]

    def bytes_per_step(self):
        from paper_2506_07533_b200 import workloads as W
        wl, cnt = self.wl, self.counts()
        tail = self.T % wl.chunk
        route = 0 if self.forced is not None else wl.n_groups * W.route_bytes_per_group(wl, self.T, bool(self.rf))
        quant = sum(W.quantize_bytes_per_layer(cnt[l // wl.rs_group], wl, self.T) for l in range(wl.n_layers))
        dec = 0
        for st in range(wl.decode_steps):
            t_len = tail + (st + 1 if wl.decode_steps > 1 else 0)
            dec += sum(W.decode_bytes_per_layer(cnt[l // wl.rs_group], wl, self.n_splits, t_len)
                       for l in range(wl.n_layers))
        return route, quant, dec

    def launches_per_step(self):
        wl = self.wl
        route = 0 if self.forced is not None else 2 * wl.n_groups        # score+vote, finalise
        quant = 2 * wl.n_layers + (wl.n_groups if self.forced is not None else 0)
        per_decode = 1 + (1 if wl.decode_steps > 1 else 0)                # split-K with fused combine (+ append)
        return route + quant + per_decode * wl.n_layers * wl.decode_steps


def max_over_ranks(values, device, world):
    """Element-wise maximum of `values` over all ranks (replicas share no data: the slowest rank's
    device time is the job's time).  world == 1: the values themselves."""
    import torch
    import torch.distributed as dist
    t = torch.tensor([float(v) for v in values], dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t.cpu()]


def whole_job_gbs(bytes_per_rank, ms, world):
    """Aggregate throughput of `world` replicas that each move `bytes_per_rank` in at most `ms`."""
    return world * bytes_per_rank / (ms * 1e6)


def free_port() -> int:
    import socket
    with socket.socket(socket.AF_INET, socket.SOCK_STREAM) as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def spawn_command(n_ranks: int, argv: list) -> list:
    """Command line that runs this script as `n_ranks` ranks on this node (one per GPU)."""
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n_ranks}",
            "--master-addr", "127.0.0.1", "--master-port", str(free_port()), os.path.abspath(__file__), *argv]


def run_rendezvous_check(args):
    """The multi-rank skeleton of run_ours without a GPU: process group (gloo), barrier, the
    maximum over ranks of stub timings, one JSON line from rank 0."""
    import torch
    import torch.distributed as dist
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if world > 1:
        dist.init_process_group("gloo")
        dist.barrier()
    ms = max_over_ranks([10.0 + rank], torch.device("cpu"), world)[0]
    if rank == 0:
        print(json.dumps({"rendezvous_check": True, "n_gpus": world, "requested_gpus": args.gpus,
                          "ms_max_over_ranks": ms, "value": whole_job_gbs(1e9, ms, world)}), flush=True)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def run_ours(args):
    import torch
    import torch.distributed as dist

    from paper_2506_07533_b200 import build as mqbuild
    from paper_2506_07533_b200 import workloads as W

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device(f"cuda:{local}"))
    torch.cuda.set_device(local)
    device = torch.device(f"cuda:{local}")
    if rank == 0:
        mqbuild.build()
    if world > 1:
        dist.barrier()
    wl = W.WORKLOADS[args.workload]
    if args.layers:
        wl = dataclasses.replace(wl, n_layers=args.layers)
    if args.chunk:
        wl = dataclasses.replace(wl, chunk=args.chunk)
    if args.batch:
        wl = dataclasses.replace(wl, batch=args.batch)
    if args.rs_group:
        wl = dataclasses.replace(wl, rs_group=args.rs_group)
    if args.mix:
        wl = dataclasses.replace(wl, mix=tuple(float(x) for x in args.mix.split(",")))
    job = Job(wl, device, seed=1234 + rank, context=args.context, force_map=bool(args.mix), rf=0 if args.no_rf else 1,
              overlap=not args.no_overlap)
    torch.cuda.synchronize()

    def one_step(ev=None):
        if ev:
            ev[0].record()
        job.route_all()
        if ev:
            ev[1].record()
        job.quantize_all()
        if ev:
            ev[2].record()
        job.decode_all()
        if ev:
            ev[3].record()

    sampler = ClockSampler(local)
    sampler.start()
    for _ in range(args.warmup):
        one_step()
    torch.cuda.synchronize()
    status = job.mq.moqae_poll_status(job.cache)
    if status != 0:
        raise RuntimeError(f"device status {status} after warm-up")
    b_route, b_quant, b_dec = job.bytes_per_step()

    events = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(args.steps)]
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    sampler.begin()
    t0 = torch.cuda.Event(enable_timing=True)
    t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    for s in range(args.steps):
        one_step(events[s])
    t1.record()
    torch.cuda.synchronize()
    sampler.end()
    if world > 1:
        dist.barrier()
    total_ms = t0.elapsed_time(t1)
    ms_route = sum(e[0].elapsed_time(e[1]) for e in events) / args.steps
    ms_quant = sum(e[1].elapsed_time(e[2]) for e in events) / args.steps
    ms_dec = sum(e[2].elapsed_time(e[3]) for e in events) / args.steps
    dec_steps_ms = sorted(e[2].elapsed_time(e[3]) for e in events)          # this rank's decode phase, step by step

    # end to end, right after the timed steps (same power state): the decode calls with the
    # queries coming from and the outputs going to pinned host memory, then the whole step with
    # every input on the host
    t_e2e0 = datetime.datetime.now()
    if args.e2e_steps > 0:
        e2e_dec = measure_e2e_decode(job, max(5, args.e2e_steps), torch)
    else:
        e2e_dec = {"ms": float("nan"), "h2d": 0, "d2h": 0, "steps": 0}
    t_e2e1 = datetime.datetime.now()
    clocks = sampler.stop()
    clocks_e2e = sampler.summary(t_e2e0, t_e2e1)
    if args.e2e_step_steps > 0:
        e2e = measure_e2e(job, args, torch)
    else:
        e2e = {"ms_dec": float("nan"), "ms_step": float("nan"), "h2d": 0, "d2h": 0, "steps": 0}

    total_ms, ms_route, ms_quant, ms_dec, e2e_ms_dec, e2e_ms_step = max_over_ranks(
        [total_ms, ms_route, ms_quant, ms_dec, e2e_dec["ms"], e2e["ms_step"]], device, world)

    if rank == 0:
        peak, peak_kind = read_peaks()
        dec_gbs = whole_job_gbs(b_dec, ms_dec, world)
        per_launch_bytes = b_dec / (wl.n_layers * wl.decode_steps)
        per_launch_ms = ms_dec / (wl.n_layers * wl.decode_steps)
        achieved = per_launch_bytes / (per_launch_ms * 1e6)
        cnt = job.counts().astype(np.float64)
        mix = (cnt.sum((0, 1)) / max(cnt.sum(), 1)).round(4).tolist()
        line = {
            "metric": "decode-attn effective HBM GB/s", "value": round(dec_gbs, 1), "unit": "GB/s",
            "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": round(total_ms / args.steps, 4), "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16" if wl.dtype == 1 else "f16", "data": "synthetic",
            "config": {"workload": f"{wl.name}: L{wl.n_layers} Hq{wl.n_q_heads}/Hkv{wl.n_kv_heads} d128 "
                                   f"B{wl.batch} ctx{job.T} chunk{wl.chunk} rs_group{wl.rs_group}",
                       "step": "route (per sharing group) + quantize_pack (per layer) + decode_attn (per layer)",
                       "expert_mix_realised_2_4_8_16": mix,
                       "mix_source": "router bias calibrated" if job.forced is None else "forced seeded multinomial map",
                       "l2": "working set per phase >> 126 MB L2; no layer is touched twice in a row",
                       "parallelism": "replicas only" if world > 1 else "single GPU",
                       "n_splits": job.n_splits,
                       "decode_launches": ("consecutive layers overlap (programmatic dependent launch)"
                                           + ("; each step attends to the new token's rows directly and appends them after the step"
                                              if wl.decode_steps > 1 else "")
                                           if job.overlap else "serialised")},
            "phase_ms": {"route": round(ms_route, 4), "quantize_pack": round(ms_quant, 4),
                         "decode_attn": round(ms_dec, 4)},
            "decode_ms_per_step": {"mean": round(ms_dec, 4), "median": round(dec_steps_ms[len(dec_steps_ms) // 2], 4),
                                   "min": round(dec_steps_ms[0], 4), "max": round(dec_steps_ms[-1], 4)},
            "context_tokens_per_s": round(world * wl.batch * job.T * wl.decode_steps / (ms_dec * 1e-3), 1),
            "quantize_route_gbs": round(world * (b_route + b_quant) / ((ms_route + ms_quant) * 1e6), 1),
            "bytes_per_step": {"route": b_route, "quantize_pack": b_quant, "decode_attn": b_dec},
            "gpu_launches": job.launches_per_step() * args.steps,
            "clocks": clocks,
            "roofline": {"bound": "hbm", "kernel": "decode_mma_kernel (split-K partials + combine by the last CTA)",
                         "achieved": round(achieved, 1), "peak": peak, "unit": "GB/s",
                         "frac": round(achieved / peak, 4), "peak_source": f"of {peak_kind}",
                         "frac_of_8TBs_spec": round(achieved / 8000.0, 4),
                         "bytes_per_launch": int(per_launch_bytes), "ms_per_launch": round(per_launch_ms, 5),
                         "traffic": args.traffic if args.traffic is not None else
                         (NCU_DECODE_TRAFFIC.get(wl.name) if (args.context is None and args.chunk is None and args.batch is None
                                                              and args.mix is None) else None)},
            "roofline_quantize": {"bound": "hbm", "achieved": round(b_quant / (ms_quant * 1e6), 1), "peak": peak,
                                  "unit": "GB/s", "frac": round(b_quant / (ms_quant * 1e6) / peak, 4)},
            "roofline_route": ({"bound": "hbm", "achieved": round(b_route / (ms_route * 1e6), 1), "peak": peak,
                                "unit": "GB/s", "frac": round(b_route / (ms_route * 1e6) / peak, 4)}
                               if b_route else None),
            "e2e": {"value": round(world * b_dec / (e2e_ms_dec * 1e6), 1), "unit": "GB/s",
                    "h2d_bytes_per_step": e2e_dec["h2d"], "d2h_bytes_per_step": e2e_dec["d2h"],
                    "ms_per_step": round(e2e_ms_dec, 4), "steps": e2e_dec["steps"], "clocks": clocks_e2e,
                    "note": "the metric through the library's calls with host buffers: per step the queries of all "
                            "layers are copied from pinned host memory, the decode calls run, out is read back; "
                            "value = decode bytes of the step / that time"},
            "e2e_step": {"value": round(world * (b_route + b_quant + b_dec) / (e2e_ms_step * 1e6), 1), "unit": "GB/s",
                         "h2d_bytes_per_step": e2e["h2d"], "d2h_bytes_per_step": e2e["d2h"],
                         "ms_per_step": round(e2e_ms_step, 3), "steps": e2e["steps"],
                         "note": "whole step (route + quantise+pack + decode) with hidden states, K, V and q copied "
                                 "from pinned host memory every step and out read back: bound by the host link; "
                                 "value = algorithmic bytes of the whole step / that time"},
        }
        if world == 1 and not args.no_prefill_attn:
            # a second kernel family (tensor-bound) reported beside the headline, never part of it
            try:
                line["prefill_attn"] = measure_prefill_attn(job, torch)
            except Exception as exc:                      # the headline line must not depend on it
                line["prefill_attn"] = {"error": f"{type(exc).__name__}: {exc}"}
        if world == 1 and not args.no_project and job.hidden and wl.d_in % 64 == 0:
            try:
                line["project_quantize"] = measure_project_quantize(job, torch)
            except Exception as exc:
                line["project_quantize"] = {"error": f"{type(exc).__name__}: {exc}"}
        if not args.no_cpu_baseline and world == 1:
            line["cpu_baseline"] = cpu_baseline(wl, budget_s=args.cpu_seconds)
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def measure_project_quantize(job, torch, reps=3):
    """K/V projection fused with quantise+pack (layer 0, the workload's hidden states as the block
    input, random weights): device time of `reps` launches after one warm-up.  Tensor-bound:
    FLOPs = 2 * tokens * d_in * 2 * n_kv_heads * 128; the HBM side (hidden states read once per
    unit row + packed bytes written) is reported beside it."""
    wl, T = job.wl, job.T
    from paper_2506_07533_b200 import synth
    from paper_2506_07533_b200 import workloads as W
    n_out = wl.n_kv_heads * 128
    Wk = synth.normal((n_out, wl.d_in), wl.dtype, 4001, job.device, std=wl.d_in ** -0.5)
    Wv = synth.normal((n_out, wl.d_in), wl.dtype, 4002, job.device, std=wl.d_in ** -0.5)
    hidden = job.hidden[0]
    job.mq.moqae_project_quantize_kv(job.cfg, hidden, Wk, Wv, T, 0, job.cache)
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
    ev[0].record()
    for _ in range(reps):
        job.mq.moqae_project_quantize_kv(job.cfg, hidden, Wk, Wv, T, 0, job.cache)
    ev[1].record()
    torch.cuda.synchronize()
    ms = ev[0].elapsed_time(ev[1]) / reps
    flops = 2.0 * wl.batch * T * wl.d_in * 2 * n_out
    cnt = job.counts()
    hbm = wl.batch * T * wl.d_in * 2 + 2 * n_out * wl.d_in * 2 + W.cache_bytes_per_layer(cnt[0], wl.chunk, wl.n_kv_heads, T % wl.chunk)
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            pk = json.load(f)
        peak, sustained, src = float(pk["bf16_tflops"]), float(pk.get("bf16_tflops_sustained", 0.0)) or None, "of measured"
    except Exception:
        peak, sustained, src = 1590.0, 1400.0, "of fallback"
    hbm_peak, _ = read_peaks()
    tf = flops / (ms * 1e9)
    return {"ms": round(ms, 3), "tflops": round(tf, 1), "bound": "tensor", "peak": peak, "frac": round(tf / peak, 4),
            "peak_sustained": sustained, "frac_of_sustained": round(tf / sustained, 4) if sustained else None,
            "peak_source": src, "flops": flops, "hbm_bytes": int(hbm), "hbm_gbs": round(hbm / (ms * 1e6), 1),
            "hbm_frac": round(hbm / (ms * 1e6) / hbm_peak, 4),
            "saved_bytes_vs_unfused": int(2 * 2 * wl.batch * T * n_out * 2),
            "note": "the 16-bit K/V rows (written by a separate projection, read by quantise+pack) never exist",
            "status": job.mq.moqae_poll_status(job.cache)}


def measure_prefill_attn(job, torch, reps=3):
    """Causal prefill attention of layer 0 over its quantised cache (tensor-core bound): device time of
    `reps` launches after one warm-up; FLOPs = 2 products x 2 x 128 x (T (T + 1) / 2) per query head."""
    wl, T = job.wl, job.T
    q = job.torch.randn(wl.batch, T, wl.n_q_heads, 128, device=job.device, dtype=torch.float32)
    q = q.to(torch.bfloat16 if wl.dtype == 1 else torch.float16)
    out = torch.empty((wl.batch, T, wl.n_q_heads, 128), dtype=torch.float32, device=job.device)
    ws = torch.empty(job.mq.moqae_prefill_attn_workspace(job.cfg, T), dtype=torch.uint8, device=job.device)

    def timed(workspace):
        job.mq.moqae_prefill_attn(job.cfg, q, T, 0, job.cache, out, workspace=workspace)
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
        ev[0].record()
        for _ in range(reps):
            job.mq.moqae_prefill_attn(job.cfg, q, T, 0, job.cache, out, workspace=workspace)
        ev[1].record()
        torch.cuda.synchronize()
        return ev[0].elapsed_time(ev[1]) / reps

    ms_fused = timed(None)          # every CTA expands the packed tiles itself
    ms = timed(ws)                  # the layer expanded once into the fp16 workspace (that pass is timed too)
    flops = 4.0 * 128 * (T * (T + 1) / 2) * wl.n_q_heads * wl.batch
    # burst figure for a launch of a few ms timed alone; the sustained one (cuBLAS under the power
    # cap) is the fair denominator once a launch runs for a good fraction of a second
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            pk = json.load(f)
        peak, sustained, src = float(pk["bf16_tflops"]), float(pk.get("bf16_tflops_sustained", 0.0)) or None, "of measured"
    except Exception:
        peak, sustained, src = 1590.0, 1400.0, "of fallback"
    tf = flops / (ms * 1e9)
    return {"ms": round(ms, 3), "tflops": round(tf, 1), "ms_no_workspace": round(ms_fused, 3),
            "tflops_no_workspace": round(flops / (ms_fused * 1e9), 1), "workspace_bytes": ws.numel(),
            "bound": "tensor", "peak": peak, "frac": round(tf / peak, 4),
            "peak_sustained": sustained, "frac_of_sustained": round(tf / sustained, 4) if sustained else None,
            "peak_source": src, "flops": flops, "status": job.mq.moqae_poll_status(job.cache)}


def measure_e2e_decode(job, steps, torch):
    """The metric end to end through the library's calls with HOST buffers: every step copies the
    queries of all layers from pinned host memory, runs the decode calls and reads `out` back; the
    timed region holds exactly these copies.  Returns ms per step and the bytes copied."""
    h_q = job.q.cpu().pin_memory()
    h_out = torch.empty(job.out.shape, dtype=torch.float32).pin_memory()
    d_q = torch.empty_like(job.q)
    new_tok = []
    if job.wl.decode_steps > 1:                      # the generated tokens' K/V rows also start on the host
        new_tok = [(job.k_new, job.k_new.cpu().pin_memory()), (job.v_new, job.v_new.cpu().pin_memory())]
    h2d = h_q.numel() * 2 + sum(h.numel() * 2 for _, h in new_tok)
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
    saved = job.q
    job.q = d_q
    try:
        for s in range(steps + 2):                   # two warm-up passes
            if s == 2:
                ev[0].record()
            d_q.copy_(h_q, non_blocking=True)
            for d_t, h_t in new_tok:
                d_t.copy_(h_t, non_blocking=True)
            job.decode_all()
            h_out.copy_(job.out, non_blocking=True)
        ev[1].record()
        torch.cuda.synchronize()
    finally:
        job.q = saved
    return {"ms": ev[0].elapsed_time(ev[1]) / steps, "h2d": int(h2d), "d2h": int(h_out.numel() * 4), "steps": steps}


def measure_e2e(job, args, torch):
    """The whole step (route + quantise+pack + decode) with hidden states, K, V and q starting in
    pinned host memory and `out` read back: PCIe-bound by construction."""
    wl = job.wl
    steps = max(1, args.e2e_step_steps)
    h_kv = [(K.cpu().pin_memory(), V.cpu().pin_memory()) for K, V in job.kv]
    h_hidden = [h.cpu().pin_memory() for h in job.hidden]
    h_q = job.q.cpu().pin_memory()
    h_out = torch.empty(job.out.shape, dtype=torch.float32).pin_memory()
    d_K, d_V = torch.empty_like(job.kv[0][0]), torch.empty_like(job.kv[0][1])
    d_h = torch.empty_like(job.hidden[0]) if job.hidden else None
    d_q = torch.empty_like(job.q)
    new_tok = []
    if wl.decode_steps > 1:                          # the generated tokens' K/V rows also start on the host
        new_tok = [(job.k_new, job.k_new.cpu().pin_memory()), (job.v_new, job.v_new.cpu().pin_memory())]
    h2d = 0
    ms_dec, ms_step = 0.0, 0.0
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
    for s in range(steps + 1):                       # first pass is warm-up
        h2d = 0
        ev[0].record()
        if job.forced is None:
            for g in range(wl.n_groups):
                src = h_hidden[g % len(h_hidden)]
                d_h.copy_(src, non_blocking=True)
                h2d += src.numel() * 2
                job.mq.moqae_route(job.cfg, d_h, job.T, job.W1, job.W2, job.W3, job.bias, g, job.cache)
        for l in range(wl.n_layers):
            hk, hv = h_kv[l % len(h_kv)]
            d_K.copy_(hk, non_blocking=True)
            d_V.copy_(hv, non_blocking=True)
            h2d += 2 * hk.numel() * 2
            fm = job.forced if (job.forced is not None and l % wl.rs_group == 0) else None
            job.mq.moqae_quantize_kv(job.cfg, d_K, d_V, job.T, l, job.cache, forced_map=fm)
        ev[1].record()
        d_q.copy_(h_q, non_blocking=True)
        h2d += h_q.numel() * 2
        for d_t, h_t in new_tok:
            d_t.copy_(h_t, non_blocking=True)
            h2d += h_t.numel() * 2
        saved = job.q
        job.q = d_q
        job.decode_all()
        job.q = saved
        h_out.copy_(job.out, non_blocking=True)
        ev[2].record()
        torch.cuda.synchronize()
        if s > 0:
            ms_dec += ev[1].elapsed_time(ev[2])
            ms_step += ev[0].elapsed_time(ev[2])
    return {"ms_dec": ms_dec / steps, "ms_step": ms_step / steps, "h2d": int(h2d),
            "d2h": int(h_out.numel() * 4), "steps": steps}


# ------------------------------------------------------------------------------------------
# CPU oracle, timed as it stands on a bounded sample (reported baseline, not the target)
# ------------------------------------------------------------------------------------------
def oracle_sample(wl, tokens: int, seed=77):
    """One sequence and ONE kv head of one layer over `tokens` context tokens, mixed widths
    at the workload's target mix: quantise+pack, then decode for the head's query group."""
    from oracle import moqae_oracle as O
    from paper_2506_07533_b200 import synth
    from paper_2506_07533_b200 import workloads as W
    G = wl.n_q_heads // wl.n_kv_heads
    C = tokens // wl.chunk
    K, V = synth.keys_values(1, tokens, 1, 128, wl.dtype, seed, "cpu", outlier_channels=(3,))
    q = synth.normal((1, G, 128), wl.dtype, seed + 1, "cpu")
    bmap = synth.multinomial_map(1, C, wl.mix, seed + 2)
    Ku, Vu, qu = synth.to_u16(K), synth.to_u16(V), synth.to_u16(q)
    t0 = time.perf_counter()
    cache = O.quantize_kv(Ku, Vu, wl.dtype, wl.chunk, bmap)
    t1 = time.perf_counter()
    O.decode_attn(qu, wl.dtype, cache, wl.chunk)
    t2 = time.perf_counter()
    cnt = cache["count"]
    kv_bytes = W.cache_bytes_per_layer(cnt, wl.chunk, 1, 0)
    return {"quant_s": t1 - t0, "decode_s": t2 - t1, "decode_bytes": kv_bytes + G * 128 * 6,
            "quant_bytes": tokens * 512 + kv_bytes, "tokens": tokens}


def cpu_baseline(wl, budget_s=20.0):
    """The oracle as it stands on about `budget_s` seconds of work: whole-context (sequence, kv head)
    pairs of one layer, one after the other (quantise+pack, then decode for the head's query group)."""
    import threadpoolctl
    probe = oracle_sample(wl, 4 * wl.chunk)
    per_tok = (probe["quant_s"] + probe["decode_s"]) / probe["tokens"]
    tokens = int(min(wl.context, max(4 * wl.chunk, budget_s / max(per_tok, 1e-9))) // wl.chunk * wl.chunk)
    runs, spent = [], 0.0
    while spent < budget_s and len(runs) < wl.batch * wl.n_kv_heads:
        r = oracle_sample(wl, tokens, seed=77 + len(runs))
        runs.append(r)
        spent += r["quant_s"] + r["decode_s"]
    dec_s = sum(r["decode_s"] for r in runs)
    q_s = sum(r["quant_s"] for r in runs)
    threads = max([p.get("num_threads", 1) for p in threadpoolctl.threadpool_info()] or [1])
    return {"value": round(sum(r["decode_bytes"] for r in runs) / dec_s / 1e9, 5), "unit": "GB/s",
            "cores": int(threads), "kind": "oracle",
            "sample": f"decode attention of {len(runs)} (sequence, kv head) pairs x {tokens} context tokens of one "
                      f"layer of {wl.name} (numpy float64 oracle, {dec_s:.1f} s); their quantise+pack ran at "
                      f"{sum(r['quant_bytes'] for r in runs) / q_s / 1e9:.5f} GB/s ({q_s:.1f} s)",
            "host_cpus": os.cpu_count()}


def run_reference(args):
    """Reference arm: the CPU oracle, as it stands, on a bounded sample of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2506_07533_b200 import workloads as W
    wl = W.WORKLOADS[args.workload]
    tokens = max(wl.chunk * 2, min(wl.context, args.reference_tokens) // wl.chunk * wl.chunk)
    for _ in range(args.warmup):
        oracle_sample(wl, wl.chunk * 2)
    tot_s, tot_b, last = 0.0, 0, None
    for _ in range(args.steps):
        last = oracle_sample(wl, tokens)
        tot_s += last["decode_s"]
        tot_b += last["decode_bytes"]
    import threadpoolctl
    threads = max([p.get("num_threads", 1) for p in threadpoolctl.threadpool_info()] or [1])
    val = tot_b / tot_s / 1e9
    sample = (f"decode attention of 1 sequence x 1 kv head x {tokens} context tokens of {wl.name} per step "
              f"(numpy float64 oracle)")
    line = {"impl": "reference", "metric": "decode-attn effective HBM GB/s", "value": round(val, 5), "unit": "GB/s",
            "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": round(1e3 * tot_s / args.steps, 3), "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": f"{wl.name} (bounded sample: {sample})"},
            "cpu_baseline": {"value": round(val, 5), "unit": "GB/s", "cores": int(threads), "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": round(val, 5), "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg4", choices=["cfg1", "cfg2", "cfg3", "cfg4", "cfg5"])
    ap.add_argument("--context", type=int, default=None, help="override the context length (profiling)")
    ap.add_argument("--layers", type=int, default=None, help="override the layer count (profiling)")
    ap.add_argument("--chunk", type=int, default=None, help="override the chunk size (chunk-size sweep)")
    ap.add_argument("--batch", type=int, default=None, help="override the batch size (context sweeps)")
    ap.add_argument("--rs-group", type=int, default=None, help="override the routing-sharing group size")
    ap.add_argument("--prefill-attn", action="store_true",
                    help="(default at one GPU; kept for old command lines) also time the causal prefill attention of layer 0 over its quantised cache")
    ap.add_argument("--no-prefill-attn", action="store_true", help="skip the prefill-attention measurement")
    ap.add_argument("--no-project", action="store_true", help="skip the fused projection+quantise measurement")
    ap.add_argument("--no-rf", action="store_true", help="switch routing freezing off (chunk 0 is routed too)")
    ap.add_argument("--mix", default=None,
                    help="four comma-separated shares: skip the router and force a seeded multinomial map "
                         "with this 2/4/8/16-bit mix (e.g. 1,0,0,0 = uniform 2-bit)")
    ap.add_argument("--no-overlap", action="store_true",
                    help="serialise the decode launches of consecutive layers (no programmatic dependent launch)")
    ap.add_argument("--e2e-steps", type=int, default=5,
                    help="timed steps of the end-to-end decode measurement (0 skips it; at least 5 otherwise)")
    ap.add_argument("--e2e-step-steps", type=int, default=1,
                    help="timed whole steps with every input copied from the host (0 skips it)")
    ap.add_argument("--rendezvous-check", action="store_true",
                    help="only start the ranks, form the process group on CPU (gloo), exchange stub timings and "
                         "print the line's multi-rank fields: checks the launch path on a box without GPUs")
    ap.add_argument("--cpu-seconds", type=float, default=15.0)
    ap.add_argument("--reference-tokens", type=int, default=32768)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--traffic", type=float, default=None,
                    help="dram bytes per decode launch from an ncu capture (overrides the recorded figure)")
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "ours" and args.context is None and args.layers is None:
        args.warmup = 3
    if args.impl == "reference":
        run_reference(args)
        return
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # started as plain `python bench.py --gpus N`: start the N ranks ourselves, one per GPU
        sys.exit(subprocess.call(spawn_command(args.gpus, sys.argv[1:])))
    if args.rendezvous_check:
        run_rendezvous_check(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
