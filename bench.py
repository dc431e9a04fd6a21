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
    ap.add_argument("--mode", default="decode", choices=["decode", "prefill"],
                    help="prefill: time prompt processing (lorc_append + lorc_prefill_attn per chunk and layer) instead of decode steps")
    ap.add_argument("--chunk", type=int, default=1024, help="--mode prefill: prompt tokens per call")
    ap.add_argument("--rope", default="half", choices=["half", "none"],
                    help="none: layers whose keys take no rotation at attention time (the absorbed score path, HBM-bound)")
    ap.add_argument("--no-full-rank-leg", action="store_true",
                    help="skip the 'full_rank' object (the uncompressed mode timed on the same shape in the same run)")
    ap.add_argument("--no-other-configs", action="store_true",
                    help="skip the 'other_configs' object (attention time of the other configurations, a few steps each)")
    return ap.parse_args()


# DRAM traffic of one lorc_score_kernel launch from an ncu capture of the CURRENT kernel (rank, batch and context of the
# captured launch; the read traffic is the latent keys, which grow with rank, batch and context, the written traffic
# the probability images, which grow with batch and context only).  None: no capture of the current kernel yet.
SCORE_KERNEL_TRAFFIC = {"rank": 928, "batch": 16, "context": 4100, "read_bytes": 123.31e6, "write_bytes": 6.72e6}


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d.get("bf16_tflops_sustained", d["bf16_tflops"]),
                "sustained_sm_mhz": (d.get("clocks_under_load") or {}).get("sm_mhz_median"), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "sustained_sm_mhz": 1300.0,
            "source": "fallback"}


def pick_tensor_peak(peaks, timed_region_s, clocks):
    """Which bf16 peak a tensor-bound fraction is quoted against.  The burst figure unless the evidence says the run
    sat in the regime the sustained figure was measured in: a timed region of at least a second AND a sampled SM
    clock under load within 10 % of the clock the sustained peak was measured at."""
    sm = (clocks or {}).get("sm_mhz")
    ref = peaks.get("sustained_sm_mhz")
    if timed_region_s >= 1.0 and sm and ref and sm <= 1.1 * ref:
        return "sustained", peaks["bf16_tflops_sustained"]
    return "burst", peaks["bf16_tflops"]


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
def algorithmic_counts(shape, ranks, batch, tokens, rope=True):
    """Per decode step over all layers: tensor-eligible FLOPs and latent+factor bytes of
    lorc_decode_attn with `tokens` cached tokens in total over the `batch` sequences.  Without rotation the key
    up-projection is absorbed into the query: 2 H_q r FLOP per token for the scores instead of 2 r n + 2 H_q d_h."""
    n, Hq, dh = shape.n, shape.n_q_heads, shape.d_head
    flops = 0.0
    byts = 0.0
    for r in ranks:
        per_tok = (2.0 * r * n + 2.0 * Hq * dh if rope else 2.0 * Hq * r) + 2.0 * Hq * r
        flops += tokens * per_tok + batch * 2.0 * Hq * r * dh
        byts += tokens * 2.0 * (r + r) + 2.0 * (r + r) * n + 4.0 * batch * Hq * dh
    return flops, byts


def full_rank_counts(shape, n_layers, batch, tokens):
    """The same for the uncompressed mode: scores and PV over whole keys and values, 2 n bf16 numbers read per token."""
    n, Hq, dh = shape.n, shape.n_q_heads, shape.d_head
    return n_layers * tokens * 4.0 * Hq * dh, n_layers * (tokens * 2.0 * 2.0 * n + 4.0 * batch * Hq * dh)


class Workload:
    """Factors, filled latent caches and per-step inputs of one configuration on one GPU."""

    def __init__(self, L, shape, n_layers, total_steps, device, flags, full_rank=False, seeded_cache=False,
                 keep_layers=(), layer_ids=None, rope=True):
        """seeded_cache: fill the caches with seeded synthetic rows instead of running the prompt through
        lorc_append (ragged paged configurations, and the short legs that only time attention).
        keep_layers: layers whose bf16 factors are also kept on the host (for the oracle leg).
        layer_ids: which layers of the configuration to build (default: the first n_layers); layer i of the context
        is layer layer_ids[i] of the configuration (its rank, its seeded weights and inputs)."""
        import torch
        from paper_2410_03111_b200 import host
        from workloads import device as wdev
        from workloads import synth
        self.L, self.shape, self.torch = L, shape, torch
        self.layer_ids = list(layer_ids) if layer_ids is not None else list(range(n_layers))
        n_layers = len(self.layer_ids)
        self.n_layers = n_layers
        self.ranks = [shape.ranks[i] for i in self.layer_ids]
        self.full_rank = full_rank
        b, N = shape.batch, shape.context
        self.batch = b
        lo, hi = shape.ragged
        if hi > 0:
            self.lens0 = [int(x) for x in synth.ragged_lengths(b, lo, hi)]
        else:
            self.lens0 = [N] * b
        self.tokens0 = sum(self.lens0)
        self.n_max = ((max(self.lens0) + total_steps + 127) // 128) * 128
        self.rope = rope
        self.ctx = L.lorc_create(n_layers, shape.d_model, shape.n_q_heads, shape.n_kv_heads, shape.d_head,
                                 shape.rope_theta, max_pos=self.n_max, flags=flags,
                                 rope_style=L.LORC_ROPE_HALF_SPLIT if rope else L.LORC_ROPE_NONE)
        self.caches, self.keep, self.host_factors = [], [], {}
        self.seq_lens = torch.zeros(b, dtype=torch.int32, device=device)
        self.page_table = None
        if shape.paged:
            ps = shape.page_size
            self.max_pages = self.n_max // ps
            pages = [(l + total_steps + ps - 1) // ps for l in self.lens0]
            self.n_pages = sum(pages)
            order = synth.page_order(self.n_pages)
            pt = torch.zeros(b, self.max_pages, dtype=torch.int32)
            k0 = 0
            for s_, np_ in enumerate(pages):
                pt[s_, :np_] = torch.from_numpy(order[k0:k0 + np_].astype("int32"))
                k0 += np_
            self.page_table = pt.to(device)
        chunk = 512
        for l in range(n_layers):
            r = self.ranks[l]
            lid = self.layer_ids[l]
            Uk, sk, Vk = wdev.weight_generators(shape.d_model, shape.n, shape.sigma_p, lid, "k", device)
            Uv, sv, Vv = wdev.weight_generators(shape.d_model, shape.n, shape.sigma_p, lid, "v", device)
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
                if l in keep_layers:
                    self.host_factors[l] = tuple(t.float().cpu().numpy().astype("float64") for t in (Ak, Av, Bk, Bv))
            if shape.paged:
                shp = (self.n_pages, shape.page_size, r)
            else:
                shp = (b, self.n_max, r)
            if seeded_cache:
                k = wdev.latents(shp, shape.sigma_p, lid, "k", device)
                v = wdev.latents(shp, shape.sigma_p, lid, "v", device)
            else:
                k = torch.zeros(*shp, dtype=torch.bfloat16, device=device)
                v = torch.zeros(*shp, dtype=torch.bfloat16, device=device)
            self.keep.append((k, v))
            if shape.paged:
                self.caches.append(L.make_cache(k, v, self.seq_lens, b, self.n_max, page_table=self.page_table,
                                                page_size=shape.page_size, max_pages_per_seq=self.max_pages,
                                                n_pages=self.n_pages))
            else:
                self.caches.append(L.make_cache(k, v, self.seq_lens, b, self.n_max, seq_stride=self.n_max))
            del Uk, Vk, Uv, Vv, Ak, Bk, Av, Bv
        if seeded_cache:
            self.seq_lens.copy_(torch.tensor(self.lens0, dtype=torch.int32))
        else:
            # prefill through the library's own cache write, in chunks
            done = 0
            while done < N:
                T = min(chunk, N - done)
                self.seq_lens.fill_(done + T)
                for l in range(n_layers):
                    x = wdev.hidden_states((b, T, shape.d_model), self.layer_ids[l], done // chunk, device)
                    L.lorc_append(self.ctx, l, self.caches[l], x, T=T)
                done += T
        torch.cuda.synchronize()
        rc = L.lorc_sync_status(self.ctx)
        if rc:
            raise RuntimeError(f"prefill failed: {L.lorc_last_error(self.ctx)}")
        # per-step inputs: a fresh token and a fresh query per layer and step
        self.x = [wdev.hidden_states((total_steps, b, shape.d_model), lid, 10 ** 6, device) for lid in self.layer_ids]
        self.q = [wdev.queries((total_steps, b, shape.n_q_heads, shape.d_head), lid, 0, device, 8.0)
                  for lid in self.layer_ids]
        self.out = torch.zeros(n_layers, b, shape.n_q_heads, shape.d_head, dtype=torch.bfloat16, device=device)
        ws_bytes = L.lorc_workspace_bytes(self.ctx, b, self.n_max)
        self.ws = torch.zeros(ws_bytes, dtype=torch.uint8, device=device)
        L.lorc_set_workspace(self.ctx, self.ws)
        self.step_index = 0

    def close(self):
        """Release the context and every device buffer of this workload."""
        torch = self.torch
        torch.cuda.synchronize()
        self.L.lorc_destroy(self.ctx)
        for name in ("caches", "keep", "x", "q", "out", "ws", "x_cur", "q_cur", "x_all", "q_all", "g_attn", "g_step",
                     "seq_lens", "page_table"):
            if hasattr(self, name):
                setattr(self, name, None)
        torch.cuda.empty_cache()

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
def oracle_leg(wl, shape, layers, budget_s=15.0):
    """The cpu_baseline leg: the fp64 oracle, as it stands, redoes whole (layer, sequence) units of the workload the
    GPU just ran: the append of the last token and decode attention over the sequence's cache rows, read back from
    the device.  It is timed, and because it works on the real inputs its result is also compared with the GPU's
    output for the same unit (the 'parity' object).  Returns (seconds per unit-rank, description, threads, parity)."""
    import numpy as np
    from oracle import lorc_oracle as O
    torch = wl.torch
    L = wl.L
    try:
        from threadpoolctl import threadpool_info
        threads = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        threads = os.cpu_count() or 1
    # one more attention call per sampled layer, so that `out` is known to belong to the query and cache used below
    step = wl.step_index - 1
    for l in layers:
        L.lorc_decode_attn(wl.ctx, l, wl.caches[l], wl.q[l][step], wl.out[l])
    torch.cuda.synchronize()
    lens = [int(v) for v in wl.seq_lens.cpu().tolist()]
    t_total, r_total, units, worst, worst_at = 0.0, 0, 0, 0.0, None
    seq = 0
    while t_total < budget_s and seq < wl.batch:
        for l in layers:
            r = wl.ranks[l]
            Ak, Av, Bk, Bv = wl.host_factors[l]
            n = lens[seq]
            k, v = wl.keep[l]
            if wl.page_table is not None:
                pages = wl.page_table[seq, :(n + shape.page_size - 1) // shape.page_size].long()
                k, v = k[pages].reshape(-1, r)[None], v[pages].reshape(-1, r)[None]
                ck = k[0, :n].float().cpu().numpy().astype(np.float64)
                cv = v[0, :n].float().cpu().numpy().astype(np.float64)
            else:
                ck = k[seq, :n].float().cpu().numpy().astype(np.float64)
                cv = v[seq, :n].float().cpu().numpy().astype(np.float64)
            x = wl.x[l][step][seq:seq + 1].float().cpu().numpy().astype(np.float64)
            q = wl.q[l][step][seq].float().cpu().numpy().astype(np.float64)
            got = wl.out[l][seq].float().cpu().numpy().astype(np.float64)
            t0 = time.perf_counter()
            row_k = O.append_latent_bf16(x, Ak)[0]
            row_v = O.append_latent_bf16(x, Av)[0]
            want = O.decode_attn_latent(ck, cv, Bk, Bv, q, shape.n_kv_heads, shape.rope_theta)
            t_total += time.perf_counter() - t0
            # the cache row the GPU wrote for this token against the oracle's (exactly rounded) one, in bf16 ulps
            ulp = float(np.max(np.abs(np.concatenate([row_k - ck[n - 1], row_v - cv[n - 1]])) /
                               np.maximum(np.abs(np.concatenate([row_k, row_v])) * 2.0 ** -8, 1e-30)))
            err = float(O.rel_l2_rows(got, want))
            if err > worst:
                worst, worst_at = err, (l, seq)
            r_total += r
            units += 1
            if t_total > budget_s:
                break
        seq += 1
    desc = (f"{units} (layer, sequence) units of {shape.name} ({t_total:.1f} s of oracle time): layers {sorted(set(layers))}, "
            f"their real cache rows read back from the device, append of the last token + decode attention; scaled "
            f"to the step by rank (time per unit proportional to r_l) and by the batch")
    parity = {"max_rel_l2_row_error": worst, "tolerance": 1e-2, "units": units, "worst_unit_layer_seq": worst_at,
              "append_last_row_max_err_bf16_ulp": ulp,
              "what": "GPU output vs the fp64 oracle on the sampled units, max over (sequence, head) rows of "
                      "||gpu - oracle||_2 / ||oracle||_2; taken outside the timed region"}
    return t_total / r_total, desc, threads, parity


def oracle_sample(shape, n_layers, budget_s=15.0, layers=None, n_ctx=None):
    """The reference arm's sample: time the fp64 oracle on whole (layer, sequence) units with the workload's shapes
    (one new token appended, then decode attention over the full context), on synthetic inputs drawn on the host.
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
    desc = (f"{units} (layer, sequence) units of {shape.name} ({t_total:.1f} s of oracle time; the time per unit varies "
            f"by a few tens of percent from sample to sample): layers {layers}, "
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
def time_attention(wl, reps, use_graph):
    """Device milliseconds of the attention calls of all layers (one decode step's worth), averaged over reps."""
    torch = wl.torch

    def attn_only():
        if use_graph:
            wl.g_attn.replay()
        else:
            wl._layers(None, [q[0] for q in wl.q], append=False)
    attn_only()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        attn_only()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / reps


def attention_leg(L, shape, device, peaks, full_rank=False, steps=4, warmup=3, n_layers=None, rope=True):
    """A short, separate run of another configuration (or of the uncompressed mode): builds the workload with
    seeded cache rows, replays `steps` whole decode steps and the attention calls alone, and reports times and
    roofline fractions.  Everything of it is released before it returns."""
    import torch
    n_layers = n_layers or shape.n_layers
    wl = Workload(L, shape, n_layers, warmup + steps + 3, device, 0, full_rank=full_rank, seeded_cache=True, rope=rope)
    try:
        wl.step()
        torch.cuda.synchronize()
        wl.capture()
        for _ in range(warmup):
            wl.step_graph()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            wl.step_graph()
        e1.record()
        torch.cuda.synchronize()
        step_ms = e0.elapsed_time(e1) / steps
        attn_ms = time_attention(wl, max(3, steps), True)
        path = L.lorc_last_path(wl.ctx)
        rc = L.lorc_sync_status(wl.ctx)
        if rc:
            raise RuntimeError(f"device status {rc}: {L.lorc_last_error(wl.ctx)}")
        tokens = wl.tokens0 + wl.batch * (1 + warmup + steps)
        if full_rank:
            flops, byts = full_rank_counts(shape, n_layers, wl.batch, tokens)
        else:
            flops, byts = algorithmic_counts(shape, wl.ranks, wl.batch, tokens, rope)
        t_hbm = byts / (peaks["hbm_gbs"] * 1e9) * 1e3
        t_burst = flops / (peaks["bf16_tflops"] * 1e12) * 1e3
        t_sust = flops / (peaks["bf16_tflops_sustained"] * 1e12) * 1e3
        return {
            "workload": shape.name, "layers": n_layers, "batch": wl.batch, "cached_tokens": tokens,
            "mode": "full-rank reference (uncompressed KV cache)" if full_rank else
                    ("latent" if rope else "latent, no rotation at attention time (absorbed scores)"),
            "kernel_path": {1: "plain fp32 CUDA-core", 2: "tcgen05", 3: "mma.sync streaming kernel"}.get(path, str(path)),
            "step_ms": step_ms, "tokens_per_s": wl.batch / (step_ms * 1e-3),
            "attn_ms_per_step": attn_ms, "attn_tokens_per_s": wl.batch / (attn_ms * 1e-3),
            "bytes_per_step": byts, "flops_per_step": flops, "hbm_gbs": byts / (attn_ms * 1e-3) / 1e9,
            "achieved_tflops": flops / (attn_ms * 1e-3) / 1e12,
            "bound": "hbm" if t_hbm >= t_burst else "tensor",
            "frac_of_roofline_burst": max(t_hbm, t_burst) / attn_ms,
            "frac_of_roofline_sustained": max(t_hbm, t_sust) / attn_ms,
            "steps": steps, "cache": "seeded rows",
        }
    finally:
        wl.close()


def prefill_leg(L, shape, device, peaks, n_layers=None, chunk=1024, reps=2):
    """Prompt processing of the configuration: for every layer and every chunk of the prompt, lorc_append of the chunk
    and lorc_prefill_attn of its queries over everything cached so far.  Times the cache writes and the attention
    calls separately (CUDA events around each group of calls) and reports prompt tokens per second and the fraction of
    the bf16 tensor peak each reaches on its algorithmic FLOPs:
      cache write   2 D (r_k + r_v) per token;
      attention     reconstruction of every cached key and value, 2 (r_k + r_v) n per cached token and call, plus
                    4 H_q d_h per (query, visible key) pair for Q K^T and P V."""
    import torch
    from paper_2410_03111_b200 import host
    from workloads import device as wdev
    n_layers = n_layers or shape.n_layers
    b, N = shape.batch, shape.context
    n_max = ((N + 127) // 128) * 128
    ctx = L.lorc_create(n_layers, shape.d_model, shape.n_q_heads, shape.n_kv_heads, shape.d_head, shape.rope_theta,
                        max_pos=n_max, flags=0)
    caches, keep = [], []
    seq_lens = torch.zeros(b, dtype=torch.int32, device=device)
    ranks = shape.ranks[:n_layers]
    for l in range(n_layers):
        r = ranks[l]
        Uk, sk, Vk = wdev.weight_generators(shape.d_model, shape.n, shape.sigma_p, l, "k", device)
        Uv, sv, Vv = wdev.weight_generators(shape.d_model, shape.n, shape.sigma_p, l, "v", device)
        Ak, Bk = host.factors_from_svd(Uk, sk, Vk, r)
        Av, Bv = host.factors_from_svd(Uv, sv, Vv, r)
        L.lorc_load_factors(ctx, l, L.LORC_MODE_LATENT, r, r, Ak, Bk, Av, Bv)
        k = torch.zeros(b, n_max, r, dtype=torch.bfloat16, device=device)
        v = torch.zeros(b, n_max, r, dtype=torch.bfloat16, device=device)
        keep.append((k, v))
        caches.append(L.make_cache(k, v, seq_lens, b, n_max, seq_stride=n_max))
        del Uk, Vk, Uv, Vv, Ak, Bk, Av, Bv
    ws = torch.zeros(L.lorc_prefill_workspace_bytes(ctx, b, n_max, chunk), dtype=torch.uint8, device=device)
    L.lorc_set_workspace(ctx, ws)
    x = wdev.hidden_states((b, chunk, shape.d_model), 0, 1, device)
    q = wdev.queries((b, chunk, shape.n_q_heads, shape.d_head), 0, 0, device, 8.0)
    out = torch.zeros(b, chunk, shape.n_q_heads, shape.d_head, dtype=torch.bfloat16, device=device)
    chunks = [(c0, min(chunk, N - c0)) for c0 in range(0, N, chunk)]
    ev = lambda: torch.cuda.Event(enable_timing=True)
    t_app = t_att = 0.0
    for rep in range(reps + 1):                 # the first pass warms up
        app_ms = att_ms = 0.0
        for (c0, T) in chunks:
            seq_lens.fill_(c0 + T)
            e0, e1, e2 = ev(), ev(), ev()
            e0.record()
            for l in range(n_layers):
                L.lorc_append(ctx, l, caches[l], x[:, :T].contiguous() if T != chunk else x, T=T)
            e1.record()
            for l in range(n_layers):
                L.lorc_prefill_attn(ctx, l, caches[l], q[:, :T].contiguous() if T != chunk else q,
                                    out[:, :T].contiguous() if T != chunk else out, T)
            e2.record()
            torch.cuda.synchronize()
            app_ms += e0.elapsed_time(e1)
            att_ms += e1.elapsed_time(e2)
        if rep > 0:
            t_app += app_ms
            t_att += att_ms
    t_app /= reps
    t_att /= reps
    path = L.lorc_last_path(ctx)
    rc = L.lorc_sync_status(ctx)
    if rc:
        raise RuntimeError(f"device status {rc}: {L.lorc_last_error(ctx)}")
    n, Hq, dh = shape.n, shape.n_q_heads, shape.d_head
    f_app = sum(2.0 * shape.d_model * 2 * r for r in ranks) * b * N
    f_rec = sum(sum(2.0 * 2 * r * n * (c0 + T) for (c0, T) in chunks) for r in ranks) * b
    pairs = sum(T * c0 + T * (T + 1) / 2.0 for (c0, T) in chunks)
    f_att = n_layers * 4.0 * Hq * dh * pairs * b
    L.lorc_destroy(ctx)
    del keep, caches, ws
    torch.cuda.empty_cache()
    res = {
        "workload": shape.name, "layers": n_layers, "batch": b, "prompt_tokens": N, "chunk": chunk,
        "kernel_path": {1: "plain fp32 CUDA-core", 2: "tcgen05"}.get(path, str(path)),
        "append_ms": t_app, "attn_ms": t_att, "prompt_tokens_per_s": b * N / ((t_app + t_att) * 1e-3),
        "append": {"flops": f_app, "achieved_tflops": f_app / (t_app * 1e-3) / 1e12,
                   "frac_of_bf16_burst": f_app / (t_app * 1e-3) / 1e12 / peaks["bf16_tflops"]},
        "attention": {"flops_reconstruction": f_rec, "flops_qk_pv": f_att,
                      "achieved_tflops": (f_rec + f_att) / (t_att * 1e-3) / 1e12,
                      "frac_of_bf16_burst": (f_rec + f_att) / (t_att * 1e-3) / 1e12 / peaks["bf16_tflops"]},
        "timing": "CUDA events around the append calls and around the attention calls of every chunk, all layers",
    }
    return res


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
    if args.mode == "prefill":
        if rank == 0:
            res = prefill_leg(L, shape, device, peaks, n_layers=n_layers, chunk=args.chunk)
            print(json.dumps({"metric": "LoRC prompt processing tokens/s (latent KV); % of bf16 tensor peak",
                              "value": res["prompt_tokens_per_s"], "unit": "tokens/s", "n_gpus": 1, "dtype": "bf16",
                              "data": "synthetic", "higher_is_better": True, "config": {"workload": shape.name},
                              "prefill": res}))
        if dist is not None:
            dist.barrier()
            dist.destroy_process_group()
        return 0
    flags = L.LORC_FLAG_DEBUG_FP32 if args.debug_fp32 else 0
    if args.stages:
        flags |= L.LORC_FLAG_PROFILE
        args.no_graph = True
    e2e_steps = 0 if args.no_e2e else max(2, min(args.steps, 8))
    total_steps = args.warmup + args.steps + e2e_steps + 4
    rope = args.rope == "half"
    do_oracle = (not args.no_cpu_baseline) and rank == 0 and world == 1 and not args.full_rank and rope
    # about ten layers spread over the stack (their ranks span the schedule); every sequence of each is redone
    oracle_layers = sorted(set(round(i * (n_layers - 1) / 9) for i in range(10))) if do_oracle else []
    wl = Workload(L, shape, n_layers, total_steps, device, flags, full_rank=args.full_rank,
                  seeded_cache=bool(shape.paged or shape.ragged[1] > 0), keep_layers=oracle_layers, rope=rope)
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
    ev0.record()
    for _ in range(args.steps):
        do_step()
    ev1.record()
    barrier()
    ms = ev0.elapsed_time(ev1)
    clocks = sampler.stop()
    stages = None
    if args.stages:
        stages = {k: {"ms_per_step": v[0] / args.steps, "launches_per_step": v[1] / args.steps}
                  for k, v in L.lorc_profile_read(wl.ctx).items()}
    launches_per_step = wl.launches_per_step if use_graph else (L.lorc_launch_count(wl.ctx) - launches0) / args.steps
    # the attention calls alone (all layers), on the cache as it stands after the timed steps
    # The attention calls alone, twice.  Under load the power cap pulls the SM clock down within tens of milliseconds,
    # so the state the GPU is in decides the time: one pass runs right after the timed steps (the loaded state), one
    # after a second of idling (the state the burst peak of the roofline was measured in: short bursts from rest).
    attn_reps = max(3, min(args.steps, 16))
    post_sampler = ClockSampler(local_rank)
    post_sampler.start()
    attn_ms_loaded = time_attention(wl, attn_reps, use_graph)
    loaded_clocks = post_sampler.stop()
    barrier()
    time.sleep(1.0)
    rest_sampler = ClockSampler(local_rank)
    rest_sampler.start()
    attn_ms_rested = time_attention(wl, attn_reps, use_graph)
    rested_clocks = rest_sampler.stop()
    barrier()
    # the dominant kernel alone: the same attention calls again, launched one by one with a CUDA event before and
    # after every kernel on the launching stream (the library's own stage bracketing)
    score_prof = None
    if not args.debug_fp32 and not args.full_rank and rope:
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
    tokens_mid = wl.tokens0 + b * (1 + args.warmup + args.steps)      # cached tokens the attention-only pass sees

    # the oracle on the units the GPU just ran: CPU baseline and observed parity (rank 0 of a 1-GPU run only)
    cpu = None
    if do_oracle:
        per_rank, desc, threads, parity = oracle_leg(wl, shape, oracle_layers)
        step_s = per_rank * sum(wl.ranks) * b
        cpu = ({"value": b / step_s, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": desc}, parity)

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

    ms, attn_ms_loaded, attn_ms_rested, e2e_s = max_over_ranks(
        [ms, attn_ms_loaded, attn_ms_rested, e2e[0] if e2e else 0.0], dist, device)
    ranks_used = list(wl.ranks)
    wl.close()

    # the uncompressed mode on the same shape, and the other configurations, a few steps each (1-GPU runs only)
    full_leg, others = None, None
    absorbed_leg = prefill = None
    if rank == 0 and world == 1 and not args.full_rank and not args.debug_fp32 and args.layers == 0 and rope:
        if not args.no_other_configs:
            try:
                absorbed_leg = attention_leg(L, shape, device, peaks, steps=4, rope=False)
            except Exception as exc:
                absorbed_leg = {"error": str(exc)[:200]}
        if not args.no_other_configs:
            try:
                prefill = prefill_leg(L, shape, device, peaks, n_layers=min(4, shape.n_layers), chunk=1024, reps=1)
                # the same prompts in one call per layer: the cached keys and values are reconstructed once, not per chunk
                whole = prefill_leg(L, shape, device, peaks, n_layers=min(4, shape.n_layers), chunk=shape.context, reps=1)
                prefill["one_call_per_prompt"] = {k: whole[k] for k in ("chunk", "append_ms", "attn_ms", "prompt_tokens_per_s",
                                                                        "append", "attention")}
            except Exception as exc:
                prefill = {"error": str(exc)[:200]}
        if not args.no_full_rank_leg:
            try:
                full_leg = attention_leg(L, shape, device, peaks, full_rank=True, steps=4)
            except Exception as exc:
                full_leg = {"error": str(exc)[:200]}
        if not args.no_other_configs:
            others = {}
            for name in ("cfg3_8b_long", "cfg4_70b_progressive", "cfg5_ragged_r256", "cfg5_ragged_r128"):
                if name == shape.name:
                    continue
                try:
                    others[name] = attention_leg(L, synth.CONFIGS[name], device, peaks, steps=4)
                except Exception as exc:
                    others[name] = {"error": str(exc)[:200]}

    if rank == 0:
        value = whole_job_rate(b, args.steps, world, ms * 1e-3)
        if args.full_rank:
            flops, byts = full_rank_counts(shape, n_layers, b, tokens_mid)
        else:
            flops, byts = algorithmic_counts(shape, ranks_used, b, tokens_mid, rope)
        timed_s = ms * 1e-3
        which, tc_peak = pick_tensor_peak(peaks, timed_s, clocks)
        # like against like: the burst peak with the pass taken from rest, the sustained peak with the loaded pass
        attn_ms_step = attn_ms_rested if which == "burst" else attn_ms_loaded
        t_hbm = byts / (peaks["hbm_gbs"] * 1e9)
        t_tc = flops / (tc_peak * 1e12)
        t_burst = flops / (peaks["bf16_tflops"] * 1e12)
        t_sust = flops / (peaks["bf16_tflops_sustained"] * 1e12)
        achieved = flops / (attn_ms_step * 1e-3) / 1e12
        attn_s = attn_ms_step * 1e-3
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": shape.name, "layers": n_layers, "batch": b, "context": shape.context,
                       "ranks_mean": sum(ranks_used) / len(ranks_used), "l2": "inputs larger than L2 (latent cache %.1f GB)" %
                       (sum(2 * 2 * r for r in ranks_used) * tokens_mid / 1e9),
                       "kernel_path": {1: "plain fp32 CUDA-core", 2: "tcgen05", 3: "mma.sync streaming kernel (uncompressed mode)"}.get(path, str(path)),
                       "replicas": world, "launch": "cuda graph per step" if use_graph else "call by call",
                       "mode": "full-rank reference (uncompressed KV cache)" if args.full_rank else
                       ("latent" if rope else "latent, no rotation at attention time (absorbed scores)")},
            "decode_attn": {"ms_per_step": attn_ms_step, "tokens_per_s": b * world / attn_s,
                            "roofline_ms": max(t_tc, t_hbm) * 1e3, "frac_of_roofline": max(t_tc, t_hbm) / attn_s,
                            "frac_burst": max(t_burst, t_hbm) / attn_s, "frac_sustained": max(t_sust, t_hbm) / attn_s,
                            "peak_used": which + " bf16 peak (timed region %.3f s, median SM clock under load %s MHz); "
                            "ms_per_step is the pass %s, see passes" %
                            (timed_s, (clocks or {}).get("sm_mhz"),
                             "taken from rest" if which == "burst" else "taken under load"),
                            "hbm_gbs": byts / attn_s / 1e9},
            "clocks": clocks, "gpu_launches": launches,
        }
        line["decode_attn"].update({"achieved_tflops": achieved, "flops_per_step": flops, "bytes_per_step": byts})
        line["decode_attn"]["passes"] = {
            "what": "%d replays of the attention calls alone, (a) right after the timed steps and (b) after one second "
                    "of idling; ms_per_step is (b) when the burst peak is used, (a) when the sustained peak is" % attn_reps,
            "under_load": {"ms_per_step": attn_ms_loaded, "frac_burst": max(t_burst, t_hbm) / (attn_ms_loaded * 1e-3),
                           "frac_sustained": max(t_sust, t_hbm) / (attn_ms_loaded * 1e-3), "clocks": loaded_clocks},
            "from_rest": {"ms_per_step": attn_ms_rested, "frac_burst": max(t_burst, t_hbm) / (attn_ms_rested * 1e-3),
                          "frac_sustained": max(t_sust, t_hbm) / (attn_ms_rested * 1e-3), "clocks": rested_clocks}}
        pc = rested_clocks if which == "burst" else loaded_clocks
        sm, sm_max = (pc or {}).get("sm_mhz"), (pc or {}).get("sm_max_mhz")
        if sm and sm_max and t_burst >= t_hbm:
            # context, not the headline: the same fraction if the burst peak scaled with the SM clock that was sampled
            # under load (it was measured in a short burst, before the power cap pulls the clock down)
            line["decode_attn"]["frac_burst_at_sampled_clock"] = (t_burst / attn_s) * sm_max / sm
        if score_prof:
            # lorc_score_kernel: key reconstruction C_K.B_K on the tensor cores, RoPE, q.k and the softmax numerators in
            # its epilogue.  Algorithmic FLOPs per launch = cached tokens * (2 r_k n + 2 H_q d_h), mean over the layers.
            n, Hq, dh = shape.n, shape.n_q_heads, shape.d_head
            k_flops = sum(tokens_mid * (2.0 * r * n + 2.0 * Hq * dh) for r in ranks_used) / len(ranks_used)
            k_ms = score_prof[0]
            k_ach = k_flops / (k_ms * 1e-3) / 1e12
            mean_r = sum(ranks_used) / len(ranks_used)
            traffic = None
            if SCORE_KERNEL_TRAFFIC is not None:
                t = SCORE_KERNEL_TRAFFIC
                scale = tokens_mid / float(t["batch"] * t["context"])
                traffic = (t["read_bytes"] * mean_r / t["rank"] + t["write_bytes"]) * scale
            line["roofline"] = {"bound": "tensor", "achieved": k_ach, "peak": tc_peak,
                                "unit": "TFLOP/s", "frac": k_ach / tc_peak,
                                "frac_burst": k_ach / peaks["bf16_tflops"],
                                "frac_sustained": k_ach / peaks["bf16_tflops_sustained"], "traffic": traffic,
                                "peak_source": peaks["source"] + " (" + which + " bf16 peak; see decode_attn.peak_used)",
                                "kernel": "lorc_score_kernel", "launch_ms": k_ms, "launches_per_step": score_prof[1],
                                "flops_per_launch": k_flops,
                                "timing": "CUDA events around every launch, call-by-call pass after the timed steps",
                                "stage_ms_per_step": score_prof[2]}
        else:
            gbs = byts / attn_s / 1e9
            hbm_bound = args.full_rank or not rope
            line["roofline"] = {"bound": "hbm" if hbm_bound else "alu", "achieved": gbs if hbm_bound else achieved,
                                "peak": peaks["hbm_gbs"] if hbm_bound else None,
                                "unit": "GB/s" if hbm_bound else "TFLOP/s",
                                "frac": gbs / peaks["hbm_gbs"] if hbm_bound else None, "traffic": None,
                                "kernel": "whole lorc_decode_attn (" + {1: "plain fp32 CUDA-core kernels", 2: "absorbed score kernel + PV + up-projection", 3: "mma.sync streaming kernel + merge"}.get(path, str(path)) + ")"}
        if stages:
            line["stages"] = stages
        if e2e:
            line["e2e"] = {"value": b * e2e_steps * world / e2e_s, "unit": UNIT, "h2d_bytes_per_step": e2e[1],
                           "d2h_bytes_per_step": e2e[2], "steps": e2e_steps}
        if cpu:
            line["cpu_baseline"], line["parity"] = cpu
        if full_leg is not None:
            line["full_rank"] = full_leg
        if others is not None:
            line["other_configs"] = others
        if absorbed_leg is not None:
            line["no_rotation"] = absorbed_leg
        if prefill is not None:
            line["prefill"] = prefill
        print(json.dumps(line))
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())
