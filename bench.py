#!/usr/bin/env python
"""Benchmark of the SPAR-K decode hot path on B200.

A "step" is one interleave cycle (N_text + N_speech decode steps) of the workload for all of its
sequences: it contains text steps, early-exit speech steps and full-depth refresh steps that
flush pending positions, i.e. every stage of the path.  `value` is decode tokens per second with
tokens resident on the device; `e2e` is the same loop through sparsk_decode_step_host with host
token buffers and a device->host read of every result.  Prints ONE JSON line on rank 0.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg2_step_b1]
  python bench.py --impl reference ...     # times the CPU oracle on a bounded sample
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
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2603_09215_b200 import synth  # noqa: E402

# DRAM bytes (read + write) per algorithmic byte of the persistent kernel, from its profiler capture
# on a two-layer launch (935.29 MB read + 7.0 MB written against 934.3 MB algorithmic); a launch's
# traffic is its layers' weights and cache, so it grows in proportion to the layer passes and the
# ratio carries over to the full-size launches timed here.
MEGA_DRAM_PER_ALGORITHMIC_BYTE = (935.29 + 7.0) / 934.3

KC = {"qkv": 1, "attn": 2, "oproj": 3, "gateup": 4, "down": 5, "head": 6, "mega": 7, "all": 8}


# --------------------------------------------------------------------------- byte model
def layer_weight_bytes(d):
    qd, kd = d["n_q_heads"] * d["head_dim"], d["n_kv_heads"] * d["head_dim"]
    return 2 * (qd * d["d_model"] + 2 * kd * d["d_model"] + d["d_model"] * qd + 3 * d["d_ffn"] * d["d_model"]
                + 2 * d["d_model"])


def step_bytes(d, depths, mods, lens, pend):
    """Algorithmic HBM bytes of one decode step: each active layer's weights once, each active
    (sequence, layer) pair's KV prefix once plus the rows it appends, each (head, modality)
    slice used once, the embedding rows."""
    L, e = d["n_layers"], d["exit_layer"]
    kvb = 2 * d["n_kv_heads"] * d["head_dim"] * 2
    wl = layer_weight_bytes(d)
    any_full = any(x == L for x in depths) and e < L
    total = wl * e + (wl * (L - e) if any_full else 0)
    for dep, ln, pn in zip(depths, lens, pend):
        total += e * ((ln + 1) * kvb + kvb)
        if dep == L and e < L:
            total += (L - e) * ((ln + 1) * kvb + (pn + 1) * kvb)
    for head, mod in {(dep, m) for dep, m in zip(depths, mods)}:
        rows = d["vocab_speech"] if mod else d["vocab_text"]
        total += rows * d["d_model"] * 2 + d["d_model"] * 2
    total += len(depths) * d["d_model"] * 2
    return total


def step_bytes_dyn(d, depths, mods, lens):
    """The same model for steps whose depths the library decided (confidence-based exit, Sec. V-B):
    layer l's weights once if any sequence ran it, each sequence's KV prefix for the layers it ran,
    and the head slice of every layer consulted: from conf_start up to the layer a confidence step
    left at (the projections that are wasted when the step goes on, Sec. V-C), or the head it
    was read from for a scheduled step."""
    L = d["n_layers"]
    kvb = 2 * d["n_kv_heads"] * d["head_dim"] * 2
    total = layer_weight_bytes(d) * max(depths)
    heads = set()
    for dep, m, ln in zip(depths, mods, lens):
        total += dep * ((ln + 1) * kvb + kvb)
        if (d.get("conf_modalities", 0) >> (1 if m else 0)) & 1:
            heads |= {(l, m) for l in range(d["conf_start"], min(dep, L - 1) + 1)}
        heads.add((dep, m))
    for _, m in heads:
        total += (d["vocab_speech"] if m else d["vocab_text"]) * d["d_model"] * 2 + d["d_model"] * 2
    return total + len(depths) * d["d_model"] * 2


# --------------------------------------------------------------------------- clocks
class ClockSampler:
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, uuid):
        self.uuid, self.lines, self.proc = uuid, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", self.uuid, f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except OSError:
            self.proc = None

    def _read(self):
        for ln in self.proc.stdout:
            self.lines.append(ln.strip())

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, pw, reasons = [], [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1])); pw.append(float(f[2]))
            except ValueError:
                continue
            for nm, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w_max": max(pw) if pw else None, "samples": len(sm), "reasons": sorted(reasons)}


# --------------------------------------------------------------------------- workload
def workload_setup(name, rank, exit_layer=None, period=None):
    wl = dict(synth.WORKLOADS[name])
    if exit_layer is not None:
        wl["exit_layer"] = exit_layer
    if period is not None:
        wl["refresh_period"] = period
    dims = synth.model_dims(wl["shape"], wl["exit_layer"], wl["refresh_period"], wl["refresh_phase"])
    B = wl["batch"]
    prompts = synth.make_prompts(dims, B, wl["prompt"][0], wl["prompt"][1], seed=1 + 1000 * rank,
                                 len_seed=2 + 1000 * rank)
    phi, off = synth.make_phases(B, wl["n_text"], wl["n_speech"], wl["refresh_period"], wl["random_phase"],
                                 seed=3 + 1000 * rank)
    return wl, dims, prompts, phi, off


def cycle_schedule(wl, phi, off, g0, n):
    out = []
    for g in range(g0, g0 + n):
        mc = [synth.interleave(g, wl["n_text"], wl["n_speech"], int(p), int(o)) for p, o in zip(phi, off)]
        out.append((np.array([m for m, _ in mc], np.uint8), np.array([c for _, c in mc], np.int32)))
    return out


class Runner:
    """Drives one library context through decode steps with tokens kept on the device."""

    def __init__(self, dims, gw, wl, prompts, phi, off, total_steps, options=None, synthetic_kv=False, sampling=None,
                 prefill_rows=64):
        import torch
        from paper_2603_09215_b200 import binding
        self.torch = torch
        self.wl, self.dims, self.phi, self.off = wl, dims, phi, off
        B = wl["batch"]
        self.B = B
        K = dims["refresh_period"]
        max_len = max(len(p) for p in prompts) + total_steps + 8
        max_pending = max(K - 1, 1) if dims["exit_layer"] < dims["n_layers"] else 1
        if dims.get("conf_modalities", 0):
            max_pending = max(max_pending, wl["n_speech"] + 1)   # a whole chunk may leave early
        self.last_depths = None
        self.ctx = binding.Sparsk(dims, gw, B, max_len, max_pending, prefill_rows=prefill_rows)
        for k, v in (options or {}).items():
            self.ctx.set_option(k, v)
        # nucleus sampling (Sec. V-A decodes the 28-layer backbone with it): a table of uniform
        # numbers on the device, one row per decode step
        self.sampling = sampling
        if sampling:
            self.uni = torch.from_numpy(synth.make_uniforms(1024 * B, seed=7)).cuda().view(1024, B)
            self.uni_row = 0
        self.slots = list(range(B))
        if synthetic_kv:
            self._fill_synthetic(prompts)
        else:
            self.ctx.prefill(self.slots, [p[:-1] for p in prompts])
        self.tok = [torch.tensor([int(p[-1]) for p in prompts], dtype=torch.int32, device="cuda"),
                    torch.zeros(B, dtype=torch.int32, device="cuda")]
        self.dep = torch.zeros(B, dtype=torch.int32, device="cuda")
        self.host_tok = np.array([int(p[-1]) for p in prompts], np.int32)
        self.g = 0
        self.lens = [len(p) - 1 for p in prompts]
        self.pend = [0] * B
        self.depth_log = []     # (modality, depth) per emitted token
        self.bytes = 0
        self.mega_seen = self.ctx.route_counts()["mega"]
        self.mega_layers = 0    # layer passes that ran inside the persistent kernel
        self.mega_bytes = 0     # their weight and cache bytes

    def _fill_synthetic(self, prompts):
        torch = self.torch
        for s, p in enumerate(prompts):
            n = len(p) - 1
            k, v = synth.synth_kv(self.dims, n, seed=100 + s)
            for layer in range(1, self.dims["n_layers"] + 1):
                kt = torch.from_numpy(k[layer - 1].view(np.int16)).cuda().view(torch.bfloat16).to(torch.float16)
                vt = torch.from_numpy(v[layer - 1].view(np.int16)).cuda().view(torch.bfloat16).to(torch.float16)
                self.ctx.import_kv(s, layer, 0, kt, vt)
            self.ctx.set_len(s, n)
        torch.cuda.synchronize()

    def _account(self, mods, ctrs):
        """Byte model of the step just enqueued, and which of its two passes the library ran in
        the persistent kernel (asked of the library, not re-derived: sparsk_route_counts)."""
        d = self.dims
        L, e, K, r = d["n_layers"], d["exit_layer"], d["refresh_period"], d["refresh_phase"]
        te = d.get("text_exit", 0)

        def depth(m, c):
            if (m == 0 and te == 0) or (m == 1 and te == 2):
                return L
            return L if c % K == r else e
        if d.get("conf_modalities", 0):
            # the library decided the depths: read them back (the step has synchronised already)
            depths = [int(x) for x in (self.last_depths if self.last_depths is not None else self.dep.cpu().numpy())]
            self.bytes += step_bytes_dyn(d, depths, mods, self.lens)
            self.mega_seen = self.ctx.route_counts()["mega"]
            for i, dep in enumerate(depths):
                self.lens[i] += 1
                self.depth_log.append((int(mods[i]), dep))
            return
        depths = [depth(m, c) for m, c in zip(mods, ctrs)]
        self.bytes += step_bytes(d, depths, mods, self.lens, self.pend)
        kvb = 2 * d["n_kv_heads"] * d["head_dim"] * 2
        wl = layer_weight_bytes(d)
        up = [(ln, pn) for dep, ln, pn in zip(depths, self.lens, self.pend) if dep == L and e < L]
        rows_lo, rows_up = len(depths), sum(pn + 1 for _, pn in up)
        mega_now = self.ctx.route_counts()["mega"]
        delta, self.mega_seen = mega_now - self.mega_seen, mega_now
        n_up = (L - e) if up else 0
        # the persistent kernel takes the small passes: if only one of the two ran there, it is
        # the one with fewer rows (the counts differ unless e = L - e)
        lo_in = delta == e + n_up or (delta == e and (n_up != e or rows_lo <= rows_up))
        up_in = n_up and (delta == e + n_up or (delta == n_up and not lo_in))
        if delta and lo_in:
            self.mega_layers += e
            self.mega_bytes += e * (wl + sum((ln + 2) * kvb for ln in self.lens))
        if delta and up_in:
            self.mega_layers += n_up
            self.mega_bytes += n_up * (wl + sum((ln + 1) * kvb + (pn + 1) * kvb for ln, pn in up))
        for i, dep in enumerate(depths):
            self.lens[i] += 1
            self.pend[i] = 0 if dep == L else self.pend[i] + 1
            self.depth_log.append((int(mods[i]), dep))

    def run_cycles(self, n_cycles, host=False):
        cyc = self.wl["n_text"] + self.wl["n_speech"]
        sched = cycle_schedule(self.wl, self.phi, self.off, self.g, n_cycles * cyc)
        if host:
            nt, dp = np.zeros(self.B, np.int32), np.zeros(self.B, np.int32)
            for mods, ctrs in sched:
                self._next_uniforms()
                self.ctx.decode_step_host(self.slots, self.host_tok, mods, ctrs, nt, dp)
                self.last_depths = dp
                self.host_tok[:] = nt
                self._account(mods, ctrs)
        else:
            for mods, ctrs in sched:
                self._next_uniforms()
                self.ctx.decode_step(self.slots, self.tok[0], mods, ctrs, self.tok[1], self.dep)
                self.last_depths = None
                self.tok.reverse()
                self._account(mods, ctrs)
        self.g += n_cycles * cyc
        return n_cycles * cyc * self.B

    def _next_uniforms(self):
        if self.sampling:
            self.ctx.set_sampling(self.sampling[0], self.sampling[1], self.uni[self.uni_row % 1024])
            self.uni_row += 1

    def sync_host_tokens(self):
        self.host_tok[:] = self.tok[0].cpu().numpy()

    def push_host_tokens(self):
        self.tok[0].copy_(self.torch.from_numpy(self.host_tok))


def layer_saving(log, L):
    sp = [dep for m, dep in log if m == 1]
    al = [dep for _, dep in log]
    f = lambda xs: (1 - (sum(xs) / len(xs)) / L) * 100 if xs else 0.0
    return {"speech_mean_depth": sum(sp) / max(1, len(sp)), "speech_saving_pct": f(sp), "all_saving_pct": f(al)}


# --------------------------------------------------------------------------- CPU oracle timing
def oracle_sample(wl, dims, w, prompts, phi, off, n_steps, start_g=0, seqs=1):
    """Times the C oracle, as it stands, for `n_steps` consecutive decode steps of the first
    `seqs` sequences, starting from a cache of the workload's prompt length filled with stand-in
    values (the oracle's cost does not depend on the cache contents)."""
    from oracle import oracle as ora
    from oracle.bruteforce import bf16_to_f64
    n = max(len(p) for p in prompts[:seqs]) - 1
    om = ora.OracleModel(dims, w, max_len=n + n_steps + 2)
    seq = []
    for s in range(seqs):
        sq = om.new_seq(max(1, dims["refresh_period"]))
        k, v = synth.synth_kv(dims, len(prompts[s]) - 1, seed=100 + s)
        for layer in range(1, dims["n_layers"] + 1):
            kf, vf = bf16_to_f64(k[layer - 1]), bf16_to_f64(v[layer - 1])
            for p in range(kf.shape[0]):
                sq.set_kv(layer, p, kf[p], vf[p])
        sq.set_len(len(prompts[s]) - 1)
        seq.append(sq)
    toks = [int(prompts[s][-1]) for s in range(seqs)]
    t0 = time.perf_counter()
    for g in range(start_g, start_g + n_steps):
        for s in range(seqs):
            m, c = synth.interleave(g, wl["n_text"], wl["n_speech"], int(phi[s]), int(off[s]))
            r = seq[s].decode_step(toks[s], m, c, want_logits=False)
            toks[s] = r["token"]
    dt = time.perf_counter() - t0
    return dt, n_steps * seqs


def omp_threads():
    return int(os.environ.get("OMP_NUM_THREADS", os.cpu_count() or 1))


# --------------------------------------------------------------------------- ranks
def max_over_ranks(ms: float, world: int, device: str) -> float:
    """Replicas share nothing on the data path; the only exchange is this one: the job's time is
    the slowest rank's."""
    if world <= 1:
        return ms
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_tokens_per_s(tokens_per_rank: int, ms: float, world: int) -> float:
    """Whole-job throughput of `world` replicas that each emitted tokens_per_rank in ms."""
    return world * tokens_per_rank / (ms / 1e3)


def batch_leg(name, gw, rank, world, W, cycles, opts, sampling, hbm_peak, peak_kind, uuid, timed, with_full):
    """One more workload on the weights already on the device: throughput of the scheduled decoder
    and of full depth, the step's byte-model fraction of the HBM peak, and the dominant GEMM class
    (gate/up) timed launch by launch."""
    wl, dims, prompts, phi, off = workload_setup(name, rank)
    cyc = wl["n_text"] + wl["n_speech"]
    L = dims["n_layers"]
    total_steps = ((W + cycles) * 2 + 8) * cyc
    run = Runner(dims, gw, wl, prompts, phi, off, total_steps, opts, False, sampling)
    run.run_cycles(W)
    sampler = ClockSampler(uuid)
    sampler.start()
    b0 = run.bytes
    ms, ntok, launches = timed(run, cycles)
    clocks = sampler.stop()
    step_b = run.bytes - b0
    ach = step_b / (ms * 1e-3) / 1e9
    out = {"workload": name, "batch_per_gpu": wl["batch"], "prompt_len": list(wl["prompt"]),
           "exit_layer": wl["exit_layer"], "refresh_period": wl["refresh_period"],
           "cache_fill": "real prefill of random prompts", "steps": cycles, "decode_steps_per_step": cyc,
           "value": job_tokens_per_s(ntok, ms, world), "unit": "tokens/s", "ms_per_step": ms / cycles,
           "gpu_launches": int(launches), "clocks": clocks,
           "step_hbm": {"bytes_per_step": step_b / cycles, "achieved_gbs": ach,
                        "frac_of_measured_copy": ach / hbm_peak, "frac_of_nominal_8tbs": ach / 8000.0}}
    d = dims
    run.ctx.set_option("time_kernel", KC["gateup"])
    run.run_cycles(min(cycles, 4))
    kms, kn = run.ctx.kernel_time()
    run.ctx.set_option("time_kernel", 0)
    kbytes = 2 * d["d_ffn"] * d["d_model"] * 2
    if kn:
        g = kbytes / (kms / kn * 1e-3) / 1e9
        out["roofline"] = {"bound": "hbm", "kernel": "gateup", "unit": "GB/s", "peak": hbm_peak, "peak_kind": peak_kind,
                           "achieved": g, "frac": g / hbm_peak, "launches_timed": kn, "avg_launch_us": 1e3 * kms / kn,
                           "bytes_per_launch": kbytes, "traffic": None}
    sav = layer_saving(run.depth_log, L)
    out["layer_saving"] = sav
    out["routes"] = run.ctx.route_counts()
    run.ctx.close()
    del run
    if with_full:
        wl_f = dict(wl, refresh_period=1, refresh_phase=0)
        dims_f = synth.model_dims(wl["shape"], wl["exit_layer"], 1, 0)
        rf = Runner(dims_f, gw, wl_f, prompts, phi, off, total_steps, opts, False, sampling)
        rf.run_cycles(W)
        fb0 = rf.bytes
        ms_f, ntok_f, _ = timed(rf, cycles)
        fb = rf.bytes - fb0
        out["full_depth"] = {"value": job_tokens_per_s(ntok_f, ms_f, world), "unit": "tokens/s",
                             "ms_per_step": ms_f / cycles, "bytes_per_step": fb / cycles,
                             "hbm_frac": fb / (ms_f * 1e-3) / 1e9 / hbm_peak}
        out["reduction"] = {"wall_time_pct": (1 - (ms / cycles) / (ms_f / cycles)) * 100,
                            "byte_model_pct": (1 - step_b / fb) * 100,
                            "layer_saving_all_tokens_pct": sav["all_saving_pct"]}
        rf.ctx.close()
    return out


# --------------------------------------------------------------------------- main
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=40)
    ap.add_argument("--warmup", type=int, default=4)
    ap.add_argument("--impl", default="sparsk", choices=["sparsk", "reference"])
    ap.add_argument("--workload", default="cfg2_step_b1", choices=sorted(synth.WORKLOADS))
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-full-depth", action="store_true")
    ap.add_argument("--no-batch64", action="store_true",
                    help="skip the batch-64 leg (workload cfg3_step_b64) that the default run adds")
    ap.add_argument("--option", action="append", default=[], help="library option name=value")
    ap.add_argument("--time-kernel", default="mega", choices=sorted(KC))
    ap.add_argument("--sampling", default=None, metavar="T,P",
                    help="nucleus sampling with temperature T and top_p P (the paper's 0.7,0.9) instead of the arg max")
    ap.add_argument("--conf", default=None, metavar="START,THRESHOLD",
                    help="decode speech steps with confidence-based exit (Sec. V-B) from layer START with the given "
                         "entropy threshold (the paper: 26,0.1 for the 28-layer backbone, 36,0.5 for the 40-layer one)")
    ap.add_argument("--prefill-rows", type=int, default=64, help="rows per prefill pass (a prompt chunk)")
    ap.add_argument("--exit-layer", type=int, default=None, help="override the workload's exit layer e (sweep cells)")
    ap.add_argument("--period", type=int, default=None, help="override the workload's refresh period K (sweep cells)")
    args = ap.parse_args()
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    W = max(args.warmup, 3)
    wl, dims, prompts, phi, off = workload_setup(args.workload, rank, args.exit_layer, args.period)
    cyc = wl["n_text"] + wl["n_speech"]
    L = dims["n_layers"]
    head_layers = [wl["exit_layer"], L]
    if args.conf:
        c_start, c_thr = args.conf.split(",")
        dims.update(conf_modalities=2, conf_start=int(c_start), conf_threshold=float(c_thr))
        head_layers += list(range(int(c_start), L))
    cfg = {"workload": args.workload, "shape": wl["shape"], "batch_per_gpu": wl["batch"],
           "prompt_len": list(wl["prompt"]), "interleave": f'{wl["n_text"]}:{wl["n_speech"]}',
           "exit_layer": wl["exit_layer"], "refresh_period": wl["refresh_period"],
           "refresh_phase": wl["refresh_phase"], "decode_steps_per_step": cyc,
           "l2": "inputs larger than L2 (all active layers' weights are streamed every decode step)",
           "parallelism": f"replicas x{world}" if world > 1 else "single GPU"}

    if args.impl == "reference":
        if rank != 0:
            return
        w = synth.make_weights(dims, seed=0, head_layers=[wl["exit_layer"], L])
        seqs = min(wl["batch"], 1)
        times, toks = [], 0
        for i in range(W + args.steps):
            dt, n = oracle_sample(wl, dims, w, prompts, phi, off, 1, start_g=i, seqs=seqs)
            if i >= W:
                times.append(dt)
                toks += n
        tot = sum(times)
        val = toks / tot
        base = {"value": val, "unit": "tokens/s", "cores": omp_threads(), "kind": "oracle",
                "sample": f"each step = 1 decode step of 1 sequence at cache length {len(prompts[0]) - 1} "
                          f"(stand-in cache values), walking the interleave cycle"}
        print(json.dumps({"impl": "reference", "metric": "decode_tokens_per_s", "value": val, "unit": "tokens/s",
                          "n_gpus": args.gpus, "steps": args.steps, "warmup": W,
                          "ms_per_step": 1e3 * tot / args.steps, "higher_is_better": True, "scaling": "weak",
                          "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": cfg,
                          "cpu_baseline": base,
                          "e2e": {"value": val, "unit": "tokens/s", "h2d_bytes_per_step": 0,
                                  "d2h_bytes_per_step": 0}}))
        return

    import torch
    from paper_2603_09215_b200 import binding
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    t_setup = time.time()
    w = synth.make_weights(dims, seed=0, head_layers=head_layers)
    gw = binding.upload_weights(w)
    opts = {}
    for o in args.option:
        k, v = o.split("=")
        opts[k] = int(v)
    sampling = tuple(float(x) for x in args.sampling.split(",")) if args.sampling else None
    cfg["decoding"] = f"nucleus T={sampling[0]} top_p={sampling[1]}" if sampling else "greedy (restricted arg max)"
    if args.conf:
        cfg["speech_exit"] = f"confidence-based from layer {dims['conf_start']}, entropy threshold {dims['conf_threshold']}"
    synthetic_kv = max(wl["prompt"]) > 4096      # long prompts: cache contents are stand-ins
    extra = (W + args.steps) * 2 + 8
    total_steps = extra * cyc
    run = Runner(dims, gw, wl, prompts, phi, off, total_steps, opts, synthetic_kv, sampling, args.prefill_rows)
    cfg["cache_fill"] = "stand-in values (imported)" if synthetic_kv else "real prefill of random prompts"
    setup_s = time.time() - t_setup

    def timed(runner, cycles, host=False):
        barrier()
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        l0 = runner.ctx.launch_count()
        ev0.record()
        n = runner.run_cycles(cycles, host=host)
        ev1.record()
        barrier()
        ms = max_over_ranks(ev0.elapsed_time(ev1), world, "cuda")
        return ms, n, runner.ctx.launch_count() - l0

    # ---- SPAR-K schedule, tokens on the device
    run.run_cycles(W)
    torch.cuda.synchronize()
    uuid = str(torch.cuda.get_device_properties(local).uuid)
    uuid = uuid if uuid.startswith("GPU-") else "GPU-" + uuid
    sampler = ClockSampler(uuid)
    sampler.start()
    b0 = run.bytes
    # a profiler started with "--profile-from-start off" sees exactly this timed region
    torch.cuda.profiler.start()
    ms, ntok, launches = timed(run, args.steps)
    torch.cuda.profiler.stop()
    clocks = sampler.stop()
    step_b = (run.bytes - b0)
    value = job_tokens_per_s(ntok, ms, world)
    peaks = {}
    pk_path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(pk_path):
        peaks = json.load(open(pk_path))
    hbm_peak = float(peaks.get("hbm_gbs", 6650.0))
    peak_kind = "measured" if "hbm_gbs" in peaks else "fallback"

    # ---- the same loop through the host-buffer entry point
    run.sync_host_tokens()
    run.run_cycles(1, host=True)
    ms_e2e, ntok_e2e, _ = timed(run, args.steps, host=True)
    run.push_host_tokens()
    B = wl["batch"]
    e2e = {"value": world * ntok_e2e / (ms_e2e / 1e3), "unit": "tokens/s",
           "h2d_bytes_per_step": cyc * (4 * B + 12 * B), "d2h_bytes_per_step": cyc * (8 * B + 4)}

    # ---- dominant kernel, timed live with events around each of its launches
    kname = args.time_kernel
    run.ctx.set_option("time_kernel", KC[kname])
    ml0, mb0 = run.mega_layers, run.mega_bytes
    run.run_cycles(min(args.steps, 8))
    kms, kn = run.ctx.kernel_time()
    classes = None
    if kname == "all":
        n_steps = min(args.steps, 8) * cyc
        classes = {k: {"ms_per_decode_step": v[0] / n_steps, "launches_per_decode_step": v[1] / n_steps}
                   for k, v in run.ctx.kernel_time_by_class().items() if v[1]}
    run.ctx.set_option("time_kernel", 0)
    d = dims
    kbytes = {"gateup": 2 * d["d_ffn"] * d["d_model"] * 2, "down": d["d_ffn"] * d["d_model"] * 2,
              "qkv": (d["n_q_heads"] + 2 * d["n_kv_heads"]) * d["head_dim"] * d["d_model"] * 2,
              "oproj": d["n_q_heads"] * d["head_dim"] * d["d_model"] * 2}.get(kname)
    roof = {"bound": "hbm", "kernel": kname, "unit": "GB/s", "peak": hbm_peak, "peak_kind": peak_kind,
            "traffic": None}
    if kname == "mega" and kn:
        # the persistent kernel: algorithmic bytes of the layer passes it ran (weights of every
        # layer once per pass, cache prefix read and rows appended) over its summed launch time
        lb = run.mega_bytes - mb0
        ach = lb / (kms * 1e-3) / 1e9
        roof.update(achieved=ach, frac=ach / hbm_peak, launches_timed=kn, avg_launch_us=1e3 * kms / kn,
                    bytes_per_launch=lb / kn, traffic=lb / kn * MEGA_DRAM_PER_ALGORITHMIC_BYTE,
                    traffic_source="ncu capture of a two-layer launch, scaled by layer passes",
                    layer_passes=run.mega_layers - ml0,
                    us_per_layer=1e3 * kms / max(1, run.mega_layers - ml0))
    elif kbytes and kn:
        ach = kbytes / (kms / kn * 1e-3) / 1e9
        roof.update(achieved=ach, frac=ach / hbm_peak, launches_timed=kn, avg_launch_us=1e3 * kms / kn,
                    bytes_per_launch=kbytes)
    else:
        roof.update(achieved=None, frac=None)

    # ---- full depth (K = 1) on the same weights
    full = None
    if not args.no_full_depth:
        wl_f = dict(wl, refresh_period=1, refresh_phase=0)
        dims_f = synth.model_dims(wl["shape"], wl["exit_layer"], 1, 0)
        rf = Runner(dims_f, gw, wl_f, prompts, phi, off, total_steps, opts, synthetic_kv, sampling)
        rf.run_cycles(W)
        fb0 = rf.bytes
        ms_f, ntok_f, _ = timed(rf, args.steps)
        full = {"value": world * ntok_f / (ms_f / 1e3), "unit": "tokens/s", "ms_per_step": ms_f / args.steps,
                "bytes_per_step": (rf.bytes - fb0) / args.steps,
                "hbm_frac": ((rf.bytes - fb0) / (ms_f * 1e-3) / 1e9) / hbm_peak}
        rf.ctx.close()

    # ---- the batch-64 half of the metric: workload cfg3_step_b64 on the same weights
    batch64 = None
    if args.workload == "cfg2_step_b1" and not args.no_batch64:
        batch64 = batch_leg("cfg3_step_b64", gw, rank, world, W, min(args.steps, 12), opts, sampling, hbm_peak,
                            peak_kind, uuid, timed, not args.no_full_depth)

    sav = layer_saving(run.depth_log, L)
    out = {"metric": "decode_tokens_per_s", "value": value, "unit": "tokens/s", "n_gpus": world,
           "steps": args.steps, "warmup": W, "ms_per_step": ms / args.steps, "higher_is_better": True,
           "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic", "config": cfg,
           "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches), "roofline": roof,
           "step_hbm": {"bytes_per_step": step_b / args.steps, "achieved_gbs": step_b / (ms * 1e-3) / 1e9,
                        "frac_of_measured_copy": step_b / (ms * 1e-3) / 1e9 / hbm_peak,
                        "frac_of_nominal_8tbs": step_b / (ms * 1e-3) / 1e9 / 8000.0},
           "layer_saving": sav, "setup_s": setup_s}
    if classes:
        out["kernel_classes"] = classes
    if batch64:
        out["batch64"] = batch64
    if full:
        out["full_depth"] = full
        out["reduction"] = {"wall_time_pct": (1 - (ms / args.steps) / full["ms_per_step"]) * 100,
                            "byte_model_pct": (1 - (step_b / args.steps) / full["bytes_per_step"]) * 100,
                            "layer_saving_all_tokens_pct": sav["all_saving_pct"]}
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        seqs = 1
        # about 10-30 s of CPU work: whole interleave cycles, at least one, at most 20 decode steps
        n_cyc = max(1, 20 // cyc)
        dt, n = oracle_sample(wl, dims, w, prompts, phi, off, n_cyc * cyc, start_g=0, seqs=seqs)
        out["cpu_baseline"] = {"value": n / dt, "unit": "tokens/s", "cores": omp_threads(), "kind": "oracle",
                               "sample": f"{n_cyc} interleave cycle(s) ({n_cyc * cyc} decode steps) of 1 sequence at "
                                         f"cache length {len(prompts[0]) - 1} (stand-in cache values), {dt:.1f} s"}
    run.ctx.close()
    if rank == 0:
        print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
