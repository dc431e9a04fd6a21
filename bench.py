#!/usr/bin/env python
"""Benchmark of the latent-KV decode path (lorc_append + lorc_decode_attn per layer).

A "step" is one decode step of the whole layer stack: for every layer, append
the new token's latents for every sequence, then run decode attention over the
latent cache.  Prints ONE JSON line (rank 0).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

With N > 1 (under torchrun) every rank runs its own replica of the workload on
its own GPU (the path shards by sequence, without any exchange); the value is the
number of tokens all ranks decoded divided by the slowest rank's time.
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

METRIC = "LoRC decode-attn tokens/s (latent KV, 8B shape); % of HBM/TC roofline"
UNIT = "tokens/s"


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=64, help="timed decode steps (the 8B configuration decodes 64 tokens after its 4096-token context)")
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="cfg2_8b_progressive")
    ap.add_argument("--layers", type=int, default=0, help="debug: use only the first LAYERS layers")
    ap.add_argument("--debug-fp32", action="store_true", help="time the plain fp32 kernels")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--ref-budget", type=float, default=None,
                    help="--impl reference: seconds of oracle time sampled per step "
                         "(default: 100 s shared by all steps, at most 6 s each)")
    ap.add_argument("--full-rank", action="store_true",
                    help="time the uncompressed reference mode (ordinary KV cache, no latents) instead of the latent path")
    ap.add_argument("--no-graph", action="store_true", help="launch call by call instead of replaying a CUDA graph")
    ap.add_argument("--stages", action="store_true",
                    help="call-by-call launches with per-kernel CUDA events; adds a 'stages' object (ms per step)")
    return ap.parse_args()


# DRAM traffic of one lorc_score_kernel launch, from the ncu capture summarised in
# profiles/attention_kernels_cfg2_layers0-1.md (set to None once the kernel has changed since that capture).  The
# capture is of the layer with rank 928; the read traffic is the latent keys, which grow with rank, batch and
# context, the written traffic the scores, which grow with batch and context only.
SCORE_KERNEL_TRAFFIC = {"read_bytes": 127.69e6, "write_bytes": 8.53e6, "rank": 928, "batch": 16, "context": 4100}


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d.get("bf16_tflops_sustained", d["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


# --------------------------------------------------------------------------- clocks
class ClockSampler:
    """Samples the SM clock and the clock-event (throttle) reasons while the timed region runs.

    Reads only.  NVML is polled from a thread every few milliseconds (the timed region of a decode benchmark lasts
    tens of milliseconds, too short for a freshly started nvidia-smi to report anything); without the NVML module the
    sampler falls back to an nvidia-smi loop."""
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")
    # NVML clock-event reason bits
    BITS = {"sw_power_cap": 0x4, "hw_slowdown": 0x8, "sw_thermal_slowdown": 0x20, "hw_thermal_slowdown": 0x40}

    def __init__(self, index):
        self.index = index
        self.rows = []
        self.proc = None
        self.nvml = None
        self.samples = []          # (sm MHz, reason bit mask)
        self.sm_max = None
        self._stop = False

    def start(self):
        try:
            import pynvml
            pynvml.nvmlInit()
            # NVML numbers devices by PCI order, CUDA_VISIBLE_DEVICES may remap: look the device up by its UUID
            import torch
            uuid = str(torch.cuda.get_device_properties(self.index).uuid)
            handle = None
            for i in range(pynvml.nvmlDeviceGetCount()):
                h = pynvml.nvmlDeviceGetHandleByIndex(i)
                u = pynvml.nvmlDeviceGetUUID(h)
                u = u.decode() if isinstance(u, bytes) else u
                if uuid in u:
                    handle = h
                    break
            if handle is None:
                handle = pynvml.nvmlDeviceGetHandleByIndex(self.index)
            self.nvml, self.handle = pynvml, handle
            self.sm_max = float(pynvml.nvmlDeviceGetMaxClockInfo(handle, pynvml.NVML_CLOCK_SM))
            self.thread = threading.Thread(target=self._poll, daemon=True)
            self.thread.start()
            return
        except Exception:
            self.nvml = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _poll(self):
        nv, h = self.nvml, self.handle
        reasons = getattr(nv, "nvmlDeviceGetCurrentClocksEventReasons", None) or \
            getattr(nv, "nvmlDeviceGetCurrentClocksThrottleReasons", None)
        while not self._stop:
            try:
                mhz = float(nv.nvmlDeviceGetClockInfo(h, nv.NVML_CLOCK_SM))
                mask = int(reasons(h)) if reasons else 0
                self.samples.append((mhz, mask))
            except Exception:
                pass
            time.sleep(0.004)

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append(line.strip())

    def stop(self):
        if self.nvml is not None:
            self._stop = True
            self.thread.join(timeout=2)
            sm = sorted(x[0] for x in self.samples)
            mask = 0
            for x in self.samples:
                mask |= x[1]
            reasons = sorted(k for k, bit in self.BITS.items() if mask & bit)
            return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_min_mhz": sm[0] if sm else None,
                    "sm_max_mhz": self.sm_max, "reasons": reasons, "samples": len(sm), "source": "nvml"}
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            f = [x.strip() for x in r.split(",")]
            if len(f) < 6:
                continue
            try:
                sm.append(float(f[0]))
                mx = float(f[1])
            except ValueError:
                continue
            for nm, val in zip(names, f[2:6]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        sm.sort()
        med = sm[len(sm) // 2] if sm else None
        return {"sm_mhz": med, "sm_max_mhz": mx, "reasons": sorted(reasons), "samples": len(sm), "source": "nvidia-smi"}


# ------------------------------------------------------------------ workload set-up
def algorithmic_counts(shape, ranks, batch, n_ctx):
    """Per decode step over all layers: tensor-eligible FLOPs and latent+factor bytes of
    lorc_decode_attn with every sequence holding n_ctx tokens."""
    n, Hq, dh = shape.n, shape.n_q_heads, shape.d_head
    flops = 0.0
    byts = 0.0
    for r in ranks:
        per_tok = 2.0 * r * n + 2.0 * Hq * dh + 2.0 * Hq * r
        flops += batch * n_ctx * per_tok + batch * 2.0 * Hq * r * dh
        byts += batch * n_ctx * 2.0 * (r + r) + 2.0 * (r + r) * n + 4.0 * batch * Hq * dh
    return flops, byts


class Workload:
    """Factors, prefilled latent caches and per-step inputs of one configuration on one GPU."""

    def __init__(self, L, shape, n_layers, total_steps, device, flags, full_rank=False):
        import torch
        from paper_2410_03111_b200 import host
        from workloads import device as wdev
        self.L, self.shape, self.torch = L, shape, torch
        self.n_layers = n_layers
        self.ranks = shape.ranks[:n_layers]
        b, N = shape.batch, shape.context
        self.batch = b
        self.n_max = ((N + total_steps + 127) // 128) * 128
        self.ctx = L.lorc_create(n_layers, shape.d_model, shape.n_q_heads, shape.n_kv_heads, shape.d_head,
                                 shape.rope_theta, max_pos=self.n_max, flags=flags)
        self.caches, self.keep = [], []
        self.seq_lens = torch.zeros(b, dtype=torch.int32, device=device)
        chunk = 512
        for l in range(n_layers):
            r = self.ranks[l]
            Uk, sk, Vk = wdev.weight_generators(shape.d_model, shape.n, shape.sigma_p, l, "k", device)
            Uv, sv, Vv = wdev.weight_generators(shape.d_model, shape.n, shape.sigma_p, l, "v", device)
            if full_rank:
                # the uncompressed mode takes the dense weights; its cache rows are whole keys and values
                Ak, Av = host.dense_weight(Uk, sk, Vk), host.dense_weight(Uv, sv, Vv)
                Bk = Bv = None
                L.lorc_load_factors(self.ctx, l, L.LORC_MODE_FULL, 0, 0, Ak, None, Av, None)
                r = shape.n
            else:
                Ak, Bk = host.factors_from_svd(Uk, sk, Vk, r)
                Av, Bv = host.factors_from_svd(Uv, sv, Vv, r)
                L.lorc_load_factors(self.ctx, l, L.LORC_MODE_LATENT, r, r, Ak, Bk, Av, Bv)
            k = torch.zeros(b, self.n_max, r, dtype=torch.bfloat16, device=device)
            v = torch.zeros(b, self.n_max, r, dtype=torch.bfloat16, device=device)
            self.keep.append((k, v))
            self.caches.append(L.make_cache(k, v, self.seq_lens, b, self.n_max, seq_stride=self.n_max))
            del Uk, Vk, Uv, Vv, Ak, Bk, Av, Bv
        # prefill through the library's own cache write, in chunks
        done = 0
        while done < N:
            T = min(chunk, N - done)
            self.seq_lens.fill_(done + T)
            for l in range(n_layers):
                x = wdev.hidden_states((b, T, shape.d_model), l, done // chunk, device)
                L.lorc_append(self.ctx, l, self.caches[l], x, T=T)
            done += T
        torch.cuda.synchronize()
        rc = L.lorc_sync_status(self.ctx)
        if rc:
            raise RuntimeError(f"prefill failed: {L.lorc_last_error(self.ctx)}")
        # per-step inputs: a fresh token and a fresh query per layer and step
        self.x = [wdev.hidden_states((total_steps, b, shape.d_model), l, 10 ** 6, device) for l in range(n_layers)]
        self.q = [wdev.queries((total_steps, b, shape.n_q_heads, shape.d_head), l, 0, device, 8.0)
                  for l in range(n_layers)]
        self.out = torch.zeros(n_layers, b, shape.n_q_heads, shape.d_head, dtype=torch.bfloat16, device=device)
        ws_bytes = L.lorc_workspace_bytes(self.ctx, b, self.n_max)
        self.ws = torch.zeros(ws_bytes, dtype=torch.uint8, device=device)
        L.lorc_set_workspace(self.ctx, self.ws)
        self.step_index = 0

    def _layers(self, xs, qs, append=True, attn=True):
        L = self.L
        for l in range(self.n_layers):
            if append:
                L.lorc_append(self.ctx, l, self.caches[l], xs[l], T=1)
            if attn:
                L.lorc_decode_attn(self.ctx, l, self.caches[l], qs[l], self.out[l])

    def step(self):
        """One decode step on the device, launched call by call: all layers, inputs already in HBM."""
        i = self.step_index
        self.seq_lens += 1
        self._layers([x[i] for x in self.x], [q[i] for q in self.q])
        self.step_index += 1

    def capture(self):
        """Capture one decode step (and, separately, the attention calls alone) into CUDA graphs.
        The step's inputs are read from fixed buffers that step_graph() refills before each replay."""
        torch = self.torch
        self.x_cur = torch.stack([x[0] for x in self.x]).contiguous()
        self.q_cur = torch.stack([q[0] for q in self.q]).contiguous()
        self.x_all = torch.stack(self.x).transpose(0, 1).contiguous()      # [steps, L, b, D]
        self.q_all = torch.stack(self.q).transpose(0, 1).contiguous()
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            self.g_attn = torch.cuda.CUDAGraph()
            with torch.cuda.graph(self.g_attn, stream=side):
                self._layers(self.x_cur, self.q_cur, append=False)
            # (work issued during capture is recorded, not executed: the cache does not advance here)
            self.g_step = torch.cuda.CUDAGraph()
            n0 = self.L.lorc_launch_count(self.ctx)
            with torch.cuda.graph(self.g_step, stream=side):
                self.seq_lens += 1
                self._layers(self.x_cur, self.q_cur)
            self.launches_per_step = self.L.lorc_launch_count(self.ctx) - n0
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()

    def step_graph(self):
        i = self.step_index
        self.x_cur.copy_(self.x_all[i])
        self.q_cur.copy_(self.q_all[i])
        self.g_step.replay()
        self.step_index += 1

    def step_host(self, xh, qh, oh):
        """One decode step through the host-buffer entry point (H2D and D2H inside)."""
        L = self.L
        self.seq_lens += 1
        for l in range(self.n_layers):
            L.lorc_decode_step_host(self.ctx, l, self.caches[l], xh[l], qh[l], oh[l])
        self.torch.cuda.current_stream().synchronize()
        self.step_index += 1


# ------------------------------------------------------------------- CPU baseline
def oracle_sample(shape, n_layers, budget_s=15.0, layers=None, n_ctx=None):
    """Time the fp64 oracle on a bounded sample of the workload: whole (layer, sequence)
    units (one new token appended, then decode attention over the full context).
    Returns (seconds per unit-rank, description, threads used, units timed)."""
    import numpy as np
    from oracle import lorc_oracle as O
    from workloads import synth
    try:
        from threadpoolctl import threadpool_info
        threads = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        threads = os.cpu_count() or 1
    N = n_ctx or shape.context
    if layers is None:
        layers = sorted(set([0, n_layers // 2, n_layers - 1]))
    rng = np.random.default_rng(7)
    t_total, r_total, units = 0.0, 0, 0
    used = []
    seq = 0
    # synthetic factors and latents with the workload's shapes, drawn once per layer (values do not affect the
    # timing); the budget counts oracle time only
    inputs = {}
    for l in layers:
        r = shape.ranks[l]
        inputs[l] = [synth.to_bf16_exact(a).astype(np.float64) for a in (
            rng.standard_normal((shape.d_model, r)) / 64, rng.standard_normal((shape.d_model, r)) / 64,
            rng.standard_normal((r, shape.n)) / 32, rng.standard_normal((r, shape.n)) / 32,
            rng.standard_normal((N + 1, r)), rng.standard_normal((N + 1, r)))]
    while t_total < budget_s:
        for l in layers:
            r = shape.ranks[l]
            Ak, Av, Bk, Bv, ck, cv = inputs[l]
            x = synth.hidden_states(1, shape.d_model, l, 5 + seq).astype(np.float64)
            q = synth.queries(1, shape.n_q_heads, shape.d_head, l, seq, 8.0)[0].astype(np.float64)
            t0 = time.perf_counter()
            ck[N] = O.append_latent_bf16(x, Ak)[0]
            cv[N] = O.append_latent_bf16(x, Av)[0]
            O.decode_attn_latent(ck, cv, Bk, Bv, q, shape.n_kv_heads, shape.rope_theta)
            t_total += time.perf_counter() - t0
            r_total += r
            units += 1
            used.append(l)
            if t_total > budget_s:
                break
        seq += 1
    layers = sorted(set(used))
    desc = (f"{units} (layer, sequence) units of {shape.name} ({t_total:.1f} s of oracle time): layers {layers}, "
            f"context {N}+1, append of 1 token + decode attention; scaled to the step by rank "
            f"(time per unit proportional to r_l) and by the batch")
    return t_total / r_total, desc, threads, units


def run_reference(args, shape, n_layers):
    """The oracle as the reference arm: each step times a bounded sample and scales it."""
    vals = []
    per_rank, desc, threads = None, "", 1
    budget = args.ref_budget if args.ref_budget else min(6.0, 100.0 / max(1, args.warmup + args.steps))
    for i in range(args.warmup + args.steps):
        per_rank, desc, threads, units = oracle_sample(shape, n_layers, budget_s=budget,
                                                       layers=[0, n_layers - 1] if n_layers > 1 else [0])
        step_s = per_rank * sum(shape.ranks[:n_layers]) * shape.batch
        if i >= args.warmup:
            vals.append(step_s)
    step_s = sum(vals) / len(vals)
    value = shape.batch / step_s
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": step_s * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": shape.name, "layers": n_layers, "batch": shape.batch, "context": shape.context},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": desc},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# --------------------------------------------------------------------------- ranks
def max_over_ranks(values, dist, device):
    """Element-wise maximum of a list of timings over all ranks (the slowest replica sets the job's time)."""
    import torch
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist is not None:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.tolist()]


def whole_job_rate(batch, steps, world, seconds):
    """Tokens per second of the whole job: every rank decodes `batch` sequences per step (weak scaling)."""
    return batch * steps * world / seconds


# --------------------------------------------------------------------------- main
def main():
    args = parse_args()
    from workloads import synth
    shape = synth.CONFIGS[args.config]
    n_layers = args.layers if args.layers > 0 else shape.n_layers
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))

    if args.impl == "reference":
        if rank == 0:
            run_reference(args, shape, n_layers)
        return 0

    import torch
    import paper_2410_03111_b200 as pkg
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU fallback")
    pkg._build.build()
    L = pkg.load()
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=device)

    peaks = load_peaks()
    flags = L.LORC_FLAG_DEBUG_FP32 if args.debug_fp32 else 0
    if args.stages:
        flags |= L.LORC_FLAG_PROFILE
        args.no_graph = True
    e2e_steps = 0 if args.no_e2e else max(2, min(args.steps, 8))
    total_steps = args.warmup + args.steps + e2e_steps + 4
    wl = Workload(L, shape, n_layers, total_steps, device, flags, full_rank=args.full_rank)
    b = shape.batch

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    use_graph = not args.no_graph
    wl.step()                      # first call of every kernel outside any capture
    torch.cuda.synchronize()
    if use_graph:
        try:
            wl.capture()
        except Exception as exc:   # keep the benchmark alive on the call-by-call path
            sys.stderr.write(f"graph capture failed ({exc}); timing call-by-call launches\n")
            use_graph = False
    do_step = wl.step_graph if use_graph else wl.step
    for _ in range(args.warmup):
        do_step()
    barrier()
    launches0 = L.lorc_launch_count(wl.ctx)
    if args.stages:
        L.lorc_profile_read(wl.ctx)          # drop what set-up and warm-up recorded
    sampler = ClockSampler(local_rank)
    sampler.start()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    n_ctx_start = shape.context + 1 + args.warmup
    ev0.record()
    for _ in range(args.steps):
        do_step()
    ev1.record()
    barrier()
    ms = ev0.elapsed_time(ev1)
    stages = None
    if args.stages:
        stages = {k: {"ms_per_step": v[0] / args.steps, "launches_per_step": v[1] / args.steps}
                  for k, v in L.lorc_profile_read(wl.ctx).items()}
    launches_per_step = wl.launches_per_step if use_graph else (L.lorc_launch_count(wl.ctx) - launches0) / args.steps
    # the attention calls alone (all layers), on the cache as it stands after the timed steps
    ea0, ea1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    attn_reps = max(3, min(args.steps, 16))
    def attn_only():
        if use_graph:
            wl.g_attn.replay()
        else:
            wl._layers(None, [q[0] for q in wl.q], append=False)
    attn_only()
    torch.cuda.synchronize()
    ea0.record()
    for _ in range(attn_reps):
        attn_only()
    ea1.record()
    barrier()
    clocks = sampler.stop()
    attn_ms = ea0.elapsed_time(ea1) / attn_reps * args.steps
    # the dominant kernel alone: the same attention calls again, launched one by one with a CUDA event before and
    # after every kernel on the launching stream (the library's own stage bracketing)
    score_prof = None
    if not args.debug_fp32 and not args.full_rank:
        L.lorc_profile_read(wl.ctx)
        L.lorc_profile_enable(wl.ctx, True)
        prof_reps = max(3, min(args.steps, 8))
        for _ in range(prof_reps):
            wl._layers(None, [q[0] for q in wl.q], append=False)
        torch.cuda.synchronize()
        pr = L.lorc_profile_read(wl.ctx)
        L.lorc_profile_enable(wl.ctx, bool(args.stages))
        if pr["score"][1] > 0:
            score_prof = (pr["score"][0] / pr["score"][1], pr["score"][1] // prof_reps,
                          {k: v[0] / prof_reps for k, v in pr.items()})
    path = L.lorc_last_path(wl.ctx)
    rc = L.lorc_sync_status(wl.ctx)
    if rc:
        raise RuntimeError(f"device status {rc}: {L.lorc_last_error(wl.ctx)}")
    launches = int(round(launches_per_step * args.steps))

    # end-to-end: host buffers in, host buffers out, every step
    e2e = None
    if e2e_steps:
        xh = [torch.empty(b, shape.d_model, dtype=torch.bfloat16).pin_memory() for _ in range(n_layers)]
        qh = [torch.empty(b, shape.n_q_heads, shape.d_head, dtype=torch.bfloat16).pin_memory() for _ in range(n_layers)]
        oh = [torch.empty(b, shape.n_q_heads, shape.d_head, dtype=torch.bfloat16).pin_memory() for _ in range(n_layers)]
        for l in range(n_layers):
            xh[l].copy_(wl.x[l][0])
            qh[l].copy_(wl.q[l][0])
        wl.step_host(xh, qh, oh)            # warm
        barrier()
        t0 = time.perf_counter()
        for _ in range(e2e_steps):
            wl.step_host(xh, qh, oh)
        torch.cuda.synchronize()
        e2e_s = time.perf_counter() - t0
        h2d = n_layers * (xh[0].numel() + qh[0].numel()) * 2
        d2h = n_layers * oh[0].numel() * 2
        e2e = (e2e_s, h2d, d2h)

    ms, attn_ms, e2e_s = max_over_ranks([ms, attn_ms, e2e[0] if e2e else 0.0], dist, device)

    if rank == 0:
        value = whole_job_rate(b, args.steps, world, ms * 1e-3)
        n_ctx_mid = n_ctx_start + args.steps      # context the attention-only pass sees
        flops, byts = algorithmic_counts(shape, wl.ranks, b, n_ctx_mid)
        if args.full_rank:
            # uncompressed mode: scores and PV over whole keys and values, 2 n bf16 numbers read per token
            n, Hq, dh = shape.n, shape.n_q_heads, shape.d_head
            flops = len(wl.ranks) * b * n_ctx_mid * 4.0 * Hq * dh
            byts = len(wl.ranks) * (b * n_ctx_mid * 2.0 * 2.0 * n + 4.0 * b * Hq * dh)
        attn_ms_step = attn_ms / args.steps
        t_tc = flops / (peaks["bf16_tflops_sustained"] * 1e12)
        t_hbm = byts / (peaks["hbm_gbs"] * 1e9)
        achieved = flops / (attn_ms_step * 1e-3) / 1e12
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": shape.name, "layers": n_layers, "batch": b, "context": shape.context,
                       "ranks_mean": sum(wl.ranks) / len(wl.ranks), "l2": "inputs larger than L2 (latent cache %.1f GB)" %
                       (sum(2 * 2 * r for r in wl.ranks) * b * n_ctx_mid / 1e9),
                       "kernel_path": {1: "plain fp32 CUDA-core", 2: "tcgen05", 3: "mma.sync streaming kernel (uncompressed mode)"}.get(path, str(path)),
                       "replicas": world, "launch": "cuda graph per step" if use_graph else "call by call",
                       "mode": "full-rank reference (uncompressed KV cache)" if args.full_rank else "latent"},
            "decode_attn": {"ms_per_step": attn_ms_step, "tokens_per_s": b * world / (attn_ms_step * 1e-3),
                            "roofline_ms": max(t_tc, t_hbm) * 1e3, "frac_of_roofline": max(t_tc, t_hbm) * 1e3 / attn_ms_step,
                            "hbm_gbs": byts / (attn_ms_step * 1e-3) / 1e9},
            "clocks": clocks, "gpu_launches": launches,
        }
        line["decode_attn"].update({"achieved_tflops": achieved, "flops_per_step": flops, "bytes_per_step": byts})
        if score_prof:
            # lorc_score_kernel: key reconstruction C_K.B_K on the tensor cores, RoPE and q.k in its epilogue.
            # Algorithmic FLOPs per launch = batch * context * (2 r_k n + 2 H_q d_h), mean over the layers.
            n, Hq, dh = shape.n, shape.n_q_heads, shape.d_head
            k_flops = sum(b * n_ctx_mid * (2.0 * r * n + 2.0 * Hq * dh) for r in wl.ranks) / len(wl.ranks)
            k_ms = score_prof[0]
            k_ach = k_flops / (k_ms * 1e-3) / 1e12
            mean_r = sum(wl.ranks) / len(wl.ranks)
            traffic = None
            if SCORE_KERNEL_TRAFFIC is not None:
                t = SCORE_KERNEL_TRAFFIC
                scale = b * n_ctx_mid / float(t["batch"] * t["context"])
                traffic = (t["read_bytes"] * mean_r / t["rank"] + t["write_bytes"]) * scale
            line["roofline"] = {"bound": "tensor", "achieved": k_ach, "peak": peaks["bf16_tflops_sustained"],
                                "unit": "TFLOP/s", "frac": k_ach / peaks["bf16_tflops_sustained"], "traffic": traffic,
                                "peak_source": peaks["source"] + " (sustained bf16: the kernel runs inside a long step)",
                                "kernel": "lorc_score_kernel", "launch_ms": k_ms, "launches_per_step": score_prof[1],
                                "flops_per_launch": k_flops,
                                "timing": "CUDA events around every launch, call-by-call pass after the timed steps",
                                "stage_ms_per_step": score_prof[2]}
        else:
            gbs = byts / (attn_ms_step * 1e-3) / 1e9
            line["roofline"] = {"bound": "hbm" if args.full_rank else "alu", "achieved": gbs if args.full_rank else achieved,
                                "peak": peaks["hbm_gbs"] if args.full_rank else None,
                                "unit": "GB/s" if args.full_rank else "TFLOP/s",
                                "frac": gbs / peaks["hbm_gbs"] if args.full_rank else None, "traffic": None,
                                "kernel": "whole lorc_decode_attn (" + {1: "plain fp32 CUDA-core kernels", 3: "mma.sync streaming kernel + merge"}.get(path, str(path)) + ")"}
        if stages:
            line["stages"] = stages
        if e2e:
            line["e2e"] = {"value": b * e2e_steps * world / e2e_s, "unit": UNIT, "h2d_bytes_per_step": e2e[1],
                           "d2h_bytes_per_step": e2e[2], "steps": e2e_steps}
        if not args.no_cpu_baseline and world >= 1:
            per_rank, desc, threads, units = oracle_sample(shape, n_layers)
            step_s = per_rank * sum(wl.ranks) * b
            line["cpu_baseline"] = {"value": b / step_s, "unit": UNIT, "cores": threads, "kind": "oracle",
                                    "sample": desc}
        print(json.dumps(line))
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())
