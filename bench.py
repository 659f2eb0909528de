#!/usr/bin/env python
"""Benchmark of the BinaryPC decode step (append + decode_attn) on synthetic long-context workloads.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload 2]

One step = one pass of the per-token hot path over the whole batch of one attention layer: bpc_append
(cache write + Algorithm 2 on the new key) followed by bpc_decode_attn (query hash, code scan, top-k,
gathered softmax attention).  The default workload is the 128K-context configuration (batch 4, 32/8
heads, 128-bit codes, 2 % budget); `--layers` independent layer replicas are visited round-robin so
that the codes and selected rows of a step are not left in L2 by the previous one.

The timed region is ONE CUDA graph holding exactly K steps, bracketed by CUDA events on the launching
stream.  With N > 1 (torchrun) every rank runs its own replica set (the path has no exchange step:
replicas only) and the step time is the maximum over ranks.

--impl reference times the CPU checker (oracle/) on the host cores on a bounded sample of the same
workload; it is a deliberately plain program and only a reported baseline.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

from paper_2608_04405_b200.inputs import CONFIGS, Workload, algorithmic_bytes_per_step  # noqa: F401
from paper_2608_04405_b200 import replicas

METRIC = "sparse decode-attn tokens/s (one attention layer, append + decode_attn per step)"
UNIT = "tokens/s"


def _measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            d = json.load(open(p))
            return dict(hbm_gbs=float(d["hbm_gbs"]), bf16_tflops=float(d["bf16_tflops"]),
                        bf16_tflops_sustained=float(d.get("bf16_tflops_sustained", d["bf16_tflops"])), source="measured")
        except Exception:
            pass
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


# ----------------------------------------------------------------------------- clocks
class ClockSampler:
    """Polls NVML (read-only) for SM clock and clock-event reasons while a region runs."""

    def __init__(self, index: int):
        self.samples = []
        self.reasons = set()
        self.max_mhz = None
        self._stop = threading.Event()
        self._thr = None
        self._h = None
        try:
            import pynvml
            self.nv = pynvml
            pynvml.nvmlInit()
            vis = os.environ.get("CUDA_VISIBLE_DEVICES")
            phys = index
            if vis:
                try:
                    phys = int(vis.split(",")[index])
                except Exception:
                    phys = index
            self._h = pynvml.nvmlDeviceGetHandleByIndex(phys)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self._h = None

    def _loop(self):
        nv = self.nv
        names = {"hw_slowdown": 0x8, "sw_power_cap": 0x4, "hw_thermal_slowdown": 0x40, "sw_thermal_slowdown": 0x20,
                 "hw_power_brake": 0x80}
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM))
                try:
                    r = nv.nvmlDeviceGetCurrentClocksEventReasons(self._h)
                except Exception:
                    r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._h)
                for k, bit in names.items():
                    if r & bit:
                        self.reasons.add(k)
            except Exception:
                break
            time.sleep(0.0005)

    def start(self):
        if self._h is not None:
            self._stop.clear()
            self._thr = threading.Thread(target=self._loop, daemon=True)
            self._thr.start()

    def stop(self):
        if self._thr is not None:
            self._stop.set()
            self._thr.join()
            self._thr = None
        return len(self.samples)

    def summary(self, n_timed: int):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0, "samples_in_timed_region": 0}
        return {"sm_mhz": statistics.median(self.samples), "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples), "samples_in_timed_region": n_timed}


# ----------------------------------------------------------------------------- our arm
class Layer:
    """One attention layer replica: caches, codes, context, per-step inputs (all resident on the device)."""

    def __init__(self, spec, salt, extra_rows, B, fit_ws, interleaved, budget_count=0):
        w = Workload(spec, device="cuda", extra_rows=extra_rows, salt=salt)
        self.w = w
        self.budget_count = budget_count    # > 0: a fixed number of selected keys instead of the spec's fraction
        if interleaved:     # one buffer, K and V rows of a token adjacent (row stride 2*head_dim)
            self.kv_buf, kc, vc = B.interleaved_kv(spec.batch, spec.n_kv_heads, w.n_max, spec.head_dim, spec.torch_dtype)
            kc.copy_(w.k_cache)
            vc.copy_(w.v_cache)
            w.k_cache, w.v_cache = kc, vc
        self.cfg = B.make_config(spec.batch, spec.n_q_heads, spec.n_kv_heads, w.n_max, spec.code_bits, spec.torch_dtype,
                                 kv_row_stride=2 * spec.head_dim if interleaved else 0)
        self.ctx = B.Context(self.cfg)
        self.lens0 = list(w.seq_lens)
        self.ctx.set_seq_lens(self.lens0)
        self.codes = self.ctx.alloc_codes()
        self.k_cache, self.v_cache = w.k_cache, w.v_cache
        self.fit_ms = self.encode_ms = None
        e0, e1, e2 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
        if fit_ws[0] is None or fit_ws[0].numel() < self.ctx.fit_workspace_bytes():
            fit_ws[0] = torch.empty(self.ctx.fit_workspace_bytes(), dtype=torch.uint8, device="cuda")
        e0.record()
        self.ctx.fit(self.k_cache, w.v_star, fit_ws[0])
        e1.record()
        self.ctx.encode_keys(self.k_cache, self.codes)
        e2.record()
        torch.cuda.synchronize()
        self.fit_ms, self.encode_ms = e0.elapsed_time(e1), e1.elapsed_time(e2)
        self.q, self.needles = w.queries(self.lens0)
        self.k_new, self.v_new = w.new_kv(self.lens0)
        self.out = torch.zeros(spec.batch, spec.n_q_heads, spec.head_dim, dtype=torch.float32, device="cuda")

    def reconstruction_error(self, rows=16384):
        """Sanity figure of the prefill side, computed with torch from what the library wrote: ||K - H P_h|| / ||K|| over
        the first keys of unit 0 (H = the cache codes as +-1).  A fitted projection gives well below 1; anything else
        means the fit or the encode went wrong, and the benchmark refuses to time that state."""
        n = min(int(self.lens0[0]), rows)
        _, Ph, _ = self.ctx.get_projection()
        K = self.k_cache[0, 0, :n].float()
        words = self.codes[0, 0, :n]
        nbit = 32 if words.dtype == torch.int32 else 64
        shifts = torch.arange(nbit, device=words.device, dtype=words.dtype)
        bits = ((words.unsqueeze(-1) >> shifts) & 1).reshape(n, -1)[:, :self.w.spec.code_bits]
        Hm = bits.float() * 2.0 - 1.0
        return ((K - Hm @ Ph[0].float()).norm() / K.norm()).item()

    def step(self):
        """One decode step: cache write of the new (k, v) + decode, as the single fused launch."""
        self.ctx.append_decode_attn(self.k_new, self.v_new, self.k_cache, self.v_cache, self.codes, self.q,
                                    budget_ppm=self.w.spec.budget_ppm, budget_count=self.budget_count, out=self.out)

    def make_weighted_twin(self, B):
        """A second context on the same caches, codes and projection that scores with Algorithm 3's sign + seven
        magnitude planes instead of Hamming similarity."""
        spec = self.w.spec
        cfg = B.make_config(spec.batch, spec.n_q_heads, spec.n_kv_heads, self.w.n_max, spec.code_bits, spec.torch_dtype,
                            kv_row_stride=self.cfg.kv_row_stride, score_mode=B.BPC_SCORE_WEIGHTED7)
        self.ctx_w7 = B.Context(cfg)
        P, _, _ = self.ctx.get_projection()
        self.ctx_w7.set_projection(P)
        self.ctx_w7.set_seq_lens(self.lens0)

    def make_eas_twin(self, B, eas_ppm):
        """A context with the error-aware safeguard on the same caches and projection: encode again to record the
        per-key reconstruction errors (the codes come out identical), then build the static hard-to-hash set."""
        spec = self.w.spec
        cfg = B.make_config(spec.batch, spec.n_q_heads, spec.n_kv_heads, self.w.n_max, spec.code_bits, spec.torch_dtype,
                            kv_row_stride=self.cfg.kv_row_stride, eas_ppm=eas_ppm)
        self.ctx_eas = B.Context(cfg)
        P, _, _ = self.ctx.get_projection()
        self.ctx_eas.set_projection(P)
        self.ctx_eas.set_seq_lens(self.lens0)
        self.ctx_eas.encode_keys(self.k_cache, self.codes)
        self.ctx_eas.build_eas()

    def step_eas(self):
        self.ctx_eas.append_decode_attn(self.k_new, self.v_new, self.k_cache, self.v_cache, self.codes, self.q,
                                        budget_ppm=self.w.spec.budget_ppm, out=self.out)

    def step_weighted(self):
        self.ctx_w7.append_decode_attn(self.k_new, self.v_new, self.k_cache, self.v_cache, self.codes, self.q,
                                       budget_ppm=self.w.spec.budget_ppm, out=self.out)

    def step_two_calls(self):
        self.ctx.append(self.k_new, self.v_new, self.k_cache, self.v_cache, self.codes)
        self.ctx.decode_attn(self.q, self.k_cache, self.v_cache, self.codes, budget_ppm=self.w.spec.budget_ppm, out=self.out)


def _graph_of(fn):
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        fn()
    return g


def _time_graph(g, dist_barrier):
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    dist_barrier()
    torch.cuda.synchronize()
    e0.record()
    g.replay()
    e1.record()
    torch.cuda.synchronize()
    dist_barrier()
    return e0.elapsed_time(e1)


def _time_graph_reps(g, dist_barrier, reps, before_each, max_over_ranks=lambda x: x):
    """`reps` timed replays of one graph (each replay is one timed region of exactly K steps; the state is reset
    before each); returns the per-replay times in ms, each the maximum over ranks."""
    out = []
    for _ in range(reps):
        before_each()
        out.append(max_over_ranks(_time_graph(g, dist_barrier)))
    return out


def _roofline(spec, lens_now, ms_step, peaks, traffic=None, traffic_source=None):
    alg = algorithmic_bytes_per_step(spec, lens_now)
    achieved = alg / (ms_step * 1e-3) / 1e9
    return {"bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
            "frac": achieved / peaks["hbm_gbs"], "of": peaks["source"], "traffic": traffic,
            "traffic_source": traffic_source,
            "kernel": "bpc_decode_kernel (fused cache write + decode, one launch per step)",
            "us_per_launch": ms_step * 1e3, "algorithmic_bytes": alg,
            "algorithmic_bytes_formula": "per unit: n*b/8 codes + 2*k*D*esz selected K and V rows + G*D*(esz+4) q and out",
            "frac_of_nominal_8TBs": achieved / 8000.0}


def run_ours(args):
    from paper_2608_04405_b200 import binding as B
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    use_dist = world > 1
    if use_dist:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    def barrier():
        if use_dist:
            dist.barrier()

    def max_over_ranks(x: float) -> float:
        return replicas.max_over_ranks(x, device="cuda")

    spec = CONFIGS[args.workload]
    K, W, L = args.steps, args.warmup, args.layers
    extra = K + W + 128                   # rows every replica can still append (the one-replica leg takes K steps on one)
    fit_ws = [None]
    layers = [Layer(spec, salt=replicas.replica_salt(rank, i), extra_rows=extra, B=B, fit_ws=fit_ws, interleaved=not args.separate_kv)
              for i in range(L)]
    fit_ws[0] = None
    torch.cuda.empty_cache()
    recon = [ly.reconstruction_error() for ly in layers]
    if not all(r < 1.0 for r in recon):
        raise RuntimeError("prefill sanity check failed: ||K - H P_h|| / ||K|| per layer replica = %s" % recon)
    fit_power2_ms = None
    if not args.profile:
        # one more fit of layer 0's keys with two power iterations per bit (the variant of Algorithm 1's component search)
        ly0 = layers[0]
        cfgp = B.make_config(spec.batch, spec.n_q_heads, spec.n_kv_heads, ly0.w.n_max, spec.code_bits, spec.torch_dtype,
                             kv_row_stride=ly0.cfg.kv_row_stride, fit_power_iters=2)
        ctxp = B.Context(cfgp)
        ctxp.set_seq_lens(ly0.lens0)
        wsp = torch.empty(ctxp.fit_workspace_bytes(), dtype=torch.uint8, device="cuda")
        ep0, ep1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ep0.record()
        ctxp.fit(ly0.k_cache, ly0.w.v_star, wsp)
        ep1.record()
        torch.cuda.synchronize()
        fit_power2_ms = ep0.elapsed_time(ep1)
        del ctxp, wsp
        torch.cuda.empty_cache()
    peaks = _measured_peaks()

    def set_lens(offset):
        for ly in layers:
            ly.ctx.set_seq_lens([n + offset for n in ly.lens0])

    # --- warm-up: W eager steps
    for s in range(W):
        layers[s % L].step()
    torch.cuda.synchronize()
    if args.profile:                      # plain eager steps for a profiler to capture; no graphs, no other legs
        if args.profile_leg == "work_items":
            for ly in layers:
                ly.ctx.debug_set_decode_path(2)
            for s in range(W):
                layers[s % L].step()
        if args.profile_leg == "weighted7":
            for ly in layers:
                ly.make_weighted_twin(B)
            for s in range(W):
                layers[s % L].step_weighted()
        for s in range(K):
            ly = layers[(W + s) % L]
            ly.step_weighted() if args.profile_leg == "weighted7" else ly.step()
        torch.cuda.synchronize()
        if rank == 0:
            print(json.dumps({"profile_run": True, "workload": spec.name, "steps": K, "warmup": W, "layer_replicas": L,
                              "cluster_size": layers[0].ctx.get_cluster_size()}))
        return
    per_layer_w = [(W + L - 1 - i) // L for i in range(L)]   # steps each layer has taken so far

    def reset_after_warmup():
        for ly, c in zip(layers, per_layer_w):
            ly.ctx.set_seq_lens([n + c for n in ly.lens0])

    # --- the timed region: ONE graph with exactly K steps
    launches0 = sum(ly.ctx.launch_count() for ly in layers)
    g_steps = _graph_of(lambda: [layers[(W + s) % L].step() for s in range(K)])
    launches_per_region = sum(ly.ctx.launch_count() for ly in layers) - launches0
    reset_after_warmup()
    g_steps.replay()                      # first replay uploads the graph; not timed
    torch.cuda.synchronize()
    reset_after_warmup()
    sampler = ClockSampler(local)
    sampler.start()
    rep_ms = _time_graph_reps(g_steps, barrier, args.reps, reset_after_warmup, max_over_ranks)
    n_timed_samples = sampler.stop()
    ms_total = statistics.median(rep_ms)                   # the reported region: the median of the timed replays
    ms_step = ms_total / K
    # the same steps on ONE layer replica: its codes and rows of the previous step are still (largely) in L2
    def reset_hot():
        layers[0].ctx.set_seq_lens([n + per_layer_w[0] for n in layers[0].lens0])
    reset_hot()
    g_hot = _graph_of(lambda: [layers[0].step() for s in range(K)])
    k_hot = K
    reset_hot()
    g_hot.replay(); torch.cuda.synchronize()
    hot_ms = statistics.median(_time_graph_reps(g_hot, barrier, args.reps, reset_hot)) / k_hot
    reset_after_warmup()

    # --- the same K steps as two launches each (bpc_append, then bpc_decode_attn), for comparison
    reset_after_warmup()
    g_two = _graph_of(lambda: [layers[(W + s) % L].step_two_calls() for s in range(K)])
    reset_after_warmup()
    g_two.replay()
    torch.cuda.synchronize()
    reset_after_warmup()
    ms_two = _time_graph(g_two, barrier) / K
    # --- the decode kernel without a cache write: K decode launches, same round-robin, one graph
    reset_after_warmup()
    g_dec = _graph_of(lambda: [layers[(W + s) % L].ctx.decode_attn(
        layers[(W + s) % L].q, layers[(W + s) % L].k_cache, layers[(W + s) % L].v_cache, layers[(W + s) % L].codes,
        budget_ppm=spec.budget_ppm, out=layers[(W + s) % L].out) for s in range(K)])
    g_dec.replay()
    torch.cuda.synchronize()
    ms_dec = _time_graph(g_dec, barrier) / K
    g_app = _graph_of(lambda: [layers[(W + s) % L].ctx.append(
        layers[(W + s) % L].k_new, layers[(W + s) % L].v_new, layers[(W + s) % L].k_cache, layers[(W + s) % L].v_cache,
        layers[(W + s) % L].codes) for s in range(K)])
    reset_after_warmup()
    g_app.replay()
    torch.cuda.synchronize()
    reset_after_warmup()
    ms_app = _time_graph(g_app, barrier) / K
    # --- the same fused step through the library's second decode kernel ((unit, key range) work items on a persistent
    # grid; opt-in, never chosen by the library itself), for comparison
    ms_items = None
    if spec.dtype == "bf16":
        for ly in layers:
            ly.ctx.debug_set_decode_path(2)
        if all(ly.ctx.uses_work_items() for ly in layers):
            reset_after_warmup()
            for s in range(min(W, 8)):
                layers[(W + s) % L].step()
            torch.cuda.synchronize()
            reset_after_warmup()
            g_items = _graph_of(lambda: [layers[(W + s) % L].step() for s in range(K)])
            reset_after_warmup()
            g_items.replay()
            torch.cuda.synchronize()
            reset_after_warmup()
            ms_items = _time_graph(g_items, barrier) / K
        for ly in layers:
            ly.ctx.debug_set_decode_path(0)                 # back to the library's own choice
        reset_after_warmup()
    # --- the paper's weighted score (sign + 7 magnitude planes) on the same workload
    ms_w7 = None
    if True:
        for ly, c in zip(layers, per_layer_w):
            ly.make_weighted_twin(B)
            ly.ctx_w7.set_seq_lens([n + c for n in ly.lens0])
        for s in range(min(W, 8)):
            layers[(W + s) % L].step_weighted()
        torch.cuda.synchronize()
        for ly, c in zip(layers, per_layer_w):
            ly.ctx_w7.set_seq_lens([n + c for n in ly.lens0])
        g_w7 = _graph_of(lambda: [layers[(W + s) % L].step_weighted() for s in range(K)])
        for ly, c in zip(layers, per_layer_w):
            ly.ctx_w7.set_seq_lens([n + c for n in ly.lens0])
        g_w7.replay()
        torch.cuda.synchronize()
        for ly, c in zip(layers, per_layer_w):
            ly.ctx_w7.set_seq_lens([n + c for n in ly.lens0])
        ms_w7 = _time_graph(g_w7, barrier) / K
    # --- with the error-aware safeguard: 10 % of the budget goes to the static hard-to-hash set
    reset_after_warmup()
    for ly, c in zip(layers, per_layer_w):
        ly.make_eas_twin(B, spec.budget_ppm // 10)
        ly.ctx_eas.set_seq_lens([n + c for n in ly.lens0])
    for s in range(min(W, 8)):
        layers[(W + s) % L].step_eas()
    torch.cuda.synchronize()
    for ly, c in zip(layers, per_layer_w):
        ly.ctx_eas.set_seq_lens([n + c for n in ly.lens0])
    g_eas = _graph_of(lambda: [layers[(W + s) % L].step_eas() for s in range(K)])
    for ly, c in zip(layers, per_layer_w):
        ly.ctx_eas.set_seq_lens([n + c for n in ly.lens0])
    g_eas.replay()
    torch.cuda.synchronize()
    for ly, c in zip(layers, per_layer_w):
        ly.ctx_eas.set_seq_lens([n + c for n in ly.lens0])
    ms_eas = _time_graph(g_eas, barrier) / K
    # clocks under the same load, long enough for NVML to see it
    reset_after_warmup()
    sampler.start()
    t_end = time.time() + 0.6
    while time.time() < t_end:
        g_dec.replay()
        torch.cuda.synchronize()
    sampler.stop()
    clocks = sampler.summary(n_timed_samples)

    # --- end to end through the public API with host buffers: every step copies that step's q, k_new and v_new
    # from pinned host memory (one staging buffer per layer), runs the fused call and reads `out` back to pinned
    # host memory; the host waits for each step's result before it starts the next one.  The three operations of
    # a step are captured once per layer in a CUDA graph (the copies are graph memcpy nodes).
    reset_after_warmup()
    e2e = []
    for ly in layers:
        nq, nk = ly.q.numel(), ly.k_new.numel()
        dev_in = torch.empty(nq + 2 * nk, dtype=ly.q.dtype, device="cuda")
        dev_in[:nq].copy_(ly.q.reshape(-1)); dev_in[nq:nq + nk].copy_(ly.k_new.reshape(-1)); dev_in[nq + nk:].copy_(ly.v_new.reshape(-1))
        host_in = dev_in.cpu().pin_memory()
        host_out = torch.zeros_like(ly.out, device="cpu").pin_memory()
        ly.q, ly.k_new, ly.v_new = dev_in[:nq].view_as(ly.q), dev_in[nq:nq + nk].view_as(ly.k_new), dev_in[nq + nk:].view_as(ly.v_new)

        def one(ly=ly, dev_in=dev_in, host_in=host_in, host_out=host_out):
            dev_in.copy_(host_in, non_blocking=True)
            ly.step()
            host_out.copy_(ly.out, non_blocking=True)
        one()
        torch.cuda.synchronize()
        e2e.append((_graph_of(one), host_in, host_out))
    h2d = e2e[0][1].numel() * e2e[0][1].element_size()
    d2h = e2e[0][2].numel() * 4
    reset_after_warmup()
    for s in range(min(W, 8)):
        e2e[(W + s) % L][0].replay()
        torch.cuda.current_stream().synchronize()
    reset_after_warmup()
    barrier()
    torch.cuda.synchronize()
    ee0, ee1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ee0.record()
    for s in range(K):
        e2e[(W + s) % L][0].replay()
        torch.cuda.current_stream().synchronize()          # the step's result is on the host
    ee1.record()
    torch.cuda.synchronize()
    barrier()
    ms_e2e_copy = max_over_ranks(ee0.elapsed_time(ee1)) / K

    # Variant without copy nodes: the kernel reads q, k_new, v_new straight from the pinned host buffers and writes
    # the output straight into pinned host memory (pinned allocations are device-accessible at their host address under
    # unified addressing; checked below through the runtime before it is relied on).  Same bytes cross the bus per step.
    ms_e2e_zc = None
    try:
        from cuda import cudart
        def _device_visible(t):
            err, attr = cudart.cudaPointerGetAttributes(t.data_ptr())
            return int(err) == 0 and int(attr.devicePointer) == t.data_ptr()
        zc = []
        ok = True
        for ly, (_, host_in, host_out) in zip(layers, e2e):
            nq, nk = ly.q.numel(), ly.k_new.numel()
            hq, hk, hv = host_in[:nq].view_as(ly.q), host_in[nq:nq + nk].view_as(ly.k_new), host_in[nq + nk:].view_as(ly.v_new)
            ok = ok and all(_device_visible(t) for t in (host_in, host_out))
            zc.append((hq, hk, hv, host_out))
        if ok:
            reset_after_warmup()
            def zstep(i):
                ly = layers[i % L]; hq, hk, hv, ho = zc[i % L]
                ly.ctx.append_decode_attn(hk, hv, ly.k_cache, ly.v_cache, ly.codes, hq, budget_ppm=spec.budget_ppm, out=ho)
            graphs = []
            for i in range(L):
                zstep(i); torch.cuda.synchronize()
            reset_after_warmup()
            layers[0].step(); torch.cuda.synchronize()          # same step with device-resident inputs: same bits expected
            if not torch.equal(layers[0].out.cpu(), zc[0][3]):
                raise RuntimeError("zero-copy step differs from the device-resident step")
            reset_after_warmup()
            for i in range(L):
                graphs.append(_graph_of(lambda i=i: zstep(i)))
            reset_after_warmup()
            for s_ in range(min(W, 8)):
                graphs[(W + s_) % L].replay(); torch.cuda.current_stream().synchronize()
            reset_after_warmup()
            barrier(); torch.cuda.synchronize()
            z0, z1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            z0.record()
            for s_ in range(K):
                graphs[(W + s_) % L].replay()
                torch.cuda.current_stream().synchronize()      # the step's result is in host memory
            z1.record()
            torch.cuda.synchronize(); barrier()
            ms_e2e_zc = max_over_ranks(z0.elapsed_time(z1)) / K
    except Exception as ex:                                      # no cuda-python, or pointers not device-visible
        ms_e2e_zc = None
    # bpc.h states that q, k_new, v_new and out may be pinned, device-accessible host memory, so both ways of crossing
    # the bus are the library's public API; the faster one is reported and named
    ms_e2e = ms_e2e_copy if ms_e2e_zc is None else min(ms_e2e_copy, ms_e2e_zc)
    e2e_method = "copy nodes (pinned host <-> device buffers)" if (ms_e2e_zc is None or ms_e2e_copy <= ms_e2e_zc) else \
        "kernel reads q, k_new, v_new from and writes out to pinned host memory"

    # planted-needle recall of the selection (how many of the keys a query was built from are among the selected
    # ones); a property of the synthetic data and of hashing, reported for reference
    reset_after_warmup()
    ly0 = layers[0]
    sel = torch.full((spec.batch * spec.n_kv_heads, ly0.w.n_max), -1, dtype=torch.int32, device="cuda")
    ly0.ctx.decode_attn(ly0.q, ly0.k_cache, ly0.v_cache, ly0.codes, budget_ppm=spec.budget_ppm, out=ly0.out, sel_idx=sel)
    torch.cuda.synchronize()
    hits = total_needles = 0
    for bi in range(spec.batch):
        for hq in range(spec.n_q_heads):
            u = bi * spec.n_kv_heads + hq // spec.group
            chosen = sel[u][sel[u] >= 0].long()
            hits += int(torch.isin(ly0.needles[bi, hq], chosen).sum())
            total_needles += ly0.needles.shape[-1]
    err = sum(ly.ctx.last_device_error() for ly in layers)
    lens_now = [n + per_layer_w[0] for n in layers[0].lens0]
    n_keys = sum(spec.n_kv_heads * n for n in layers[0].lens0)
    enc_ms = statistics.median(ly.encode_ms for ly in layers)
    fit_ms = statistics.median(ly.fit_ms for ly in layers)
    enc_flops = 2.0 * n_keys * spec.head_dim * spec.code_bits
    result = {
        "metric": METRIC, "value": replicas.whole_job_tokens_per_s(spec.batch, world, ms_step), "unit": UNIT, "n_gpus": world,
        "steps": K, "warmup": W, "ms_per_step": ms_step, "us_per_step": ms_step * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": spec.name, "batch": spec.batch, "n_q_heads": spec.n_q_heads, "n_kv_heads": spec.n_kv_heads,
                   "head_dim": spec.head_dim, "context": spec.n_ctx, "code_bits": spec.code_bits,
                   "budget_ppm": spec.budget_ppm, "layer_replicas": L,
                   "l2": "inputs larger than L2: %d layer replicas visited round-robin" % L,
                   "cluster_size": layers[0].ctx.get_cluster_size(), "parallelism": "replicas only",
                   "kv_layout": "separate k/v arrays" if args.separate_kv else "interleaved k|v rows (row stride 2*head_dim)"},
        "clocks": clocks,
        "e2e": {"value": world * spec.batch / (ms_e2e * 1e-3), "unit": UNIT, "us_per_step": ms_e2e * 1e3,
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "method": e2e_method,
                "us_per_step_copy_nodes": ms_e2e_copy * 1e3, "us_per_step_zero_copy": None if ms_e2e_zc is None else ms_e2e_zc * 1e3},
        "gpu_launches": launches_per_region,
        "roofline": _roofline(spec, lens_now, ms_step, peaks,
                              # dram__bytes_read.sum + dram__bytes_write.sum of one launch: not measured by this run, quoted
                              # from the committed profiler capture of this workload
                              traffic=116.5e6 if (args.workload == 2 and not args.separate_kv) else None,
                              traffic_source="ncu capture of one launch, profiles/decode_fused_cfg2_ncu.md (not measured in this run)"
                              if (args.workload == 2 and not args.separate_kv) else None),
        "timing": {"reps": args.reps, "us_per_step_median": ms_step * 1e3, "us_per_step_min": min(rep_ms) / K * 1e3,
                   "us_per_step_max": max(rep_ms) / K * 1e3, "timed_region": "one CUDA graph of exactly K steps; median of reps replays",
                   "us_per_step_one_layer_replica_hot_l2": hot_ms * 1e3},
        "breakdown_us": {"fused_step": ms_step * 1e3, "decode_attn_only": ms_dec * 1e3, "append_only": ms_app * 1e3,
                         "append_then_decode_two_launches": ms_two * 1e3,
                         "fused_step_weighted7_scores": None if ms_w7 is None else ms_w7 * 1e3,
                         "fused_step_work_item_kernel_opt_in": None if ms_items is None else ms_items * 1e3,
                         "fused_step_with_error_aware_safeguard": ms_eas * 1e3},
        "prefill": {"fit_ms": fit_ms, "fit_power2_ms": fit_power2_ms, "encode_ms": enc_ms, "encode_keys_per_s": n_keys / (enc_ms * 1e-3),
                    "encode_gemm_tflops": enc_flops / (enc_ms * 1e-3) / 1e12,
                    "encode_frac_of_bf16_peak": enc_flops / (enc_ms * 1e-3) / 1e12 / peaks["bf16_tflops"],
                    # the encode reads every key row once and writes one code per key
                    "encode_algorithmic_bytes": n_keys * (spec.head_dim * spec.esz + spec.code_bits // 8),
                    "encode_hbm_gbs": n_keys * (spec.head_dim * spec.esz + spec.code_bits // 8) / (enc_ms * 1e-3) / 1e9,
                    "encode_frac_of_hbm_peak": n_keys * (spec.head_dim * spec.esz + spec.code_bits // 8) / (enc_ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
                    "reconstruction_err_over_K_per_layer_replica": recon},
        "device_error_word": err,
        "needle_recall": hits / max(1, total_needles),
        "paper_context": "paper reports up to 3.56x end-to-end decode speed-up over FlashAttention-2 on 8 data-center GPUs "
                         "(HF stack, 64-bit codes); context only, not comparable",
    }
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        result["cpu_baseline"] = cpu_baseline(spec, budget_s=args.cpu_budget)
    if rank == 0:
        print(json.dumps(result))
    if use_dist:
        dist.destroy_process_group()


# ----------------------------------------------------------------------------- every synthetic configuration
def run_all_configs(args):
    """One JSON line per synthetic configuration 0-4 and per point of configuration 3's sweep (code length 64/128/256
    x budget 1/2/5 %): the fused step timed like the headline workload (CUDA graph of K steps over enough layer
    replicas that a step's bytes exceed L2 where they can; median of `reps` replays; clocks sampled under the same
    load), with the roofline fraction of each.  Configurations 4 and 2 also time the weighted (Algorithm 3) score."""
    from paper_2608_04405_b200 import binding as B
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    peaks = _measured_peaks()
    K, W = args.steps, max(args.warmup, 3)
    cases = [(CONFIGS[0], "cfg0"), (CONFIGS[1], "cfg1"), (CONFIGS[2], "cfg2"), (CONFIGS[4], "cfg4")]
    for bits in (64, 128, 256):
        for ppm in (10000, 20000, 50000):
            cases.append((CONFIGS[3].scaled(code_bits=bits, budget_ppm=ppm), "cfg3 b=%d budget=%g%%" % (bits, ppm / 1e4)))
    fit_ws = [None]
    for spec, label in cases:
        lens_guess = [spec.n_ctx if spec.n_ctx_min is None else (spec.n_ctx + spec.n_ctx_min) // 2] * spec.batch
        step_bytes = algorithmic_bytes_per_step(spec, lens_guess)
        L = max(2, min(8, -(-(2 * 126 * 2 ** 20) // max(step_bytes, 1))))
        if step_bytes * 8 < 126 * 2 ** 20:
            L = 2                                  # a step is far smaller than L2: it stays resident whatever the replica count
        extra = K + W + 128
        layers = [Layer(spec, salt=i, extra_rows=extra, B=B, fit_ws=fit_ws, interleaved=True) for i in range(L)]
        per = [(W + L - 1 - i) // L for i in range(L)]

        def reset(layers=layers, per=per, which="ctx"):
            for ly, c in zip(layers, per):
                getattr(ly, which).set_seq_lens([n + c for n in ly.lens0])

        def timed(step_name, which="ctx"):
            reset(which=which)
            for s in range(W):
                getattr(layers[s % L], step_name)()
            torch.cuda.synchronize()
            reset(which=which)
            g = _graph_of(lambda: [getattr(layers[(W + s) % L], step_name)() for s in range(K)])
            reset(which=which)
            g.replay(); torch.cuda.synchronize()
            sampler = ClockSampler(0)
            sampler.start()
            ms = _time_graph_reps(g, lambda: None, args.reps, lambda: reset(which=which))
            n_in = sampler.stop()
            sampler.start()
            t_end = time.time() + 0.3
            while time.time() < t_end:
                reset(which=which)
                g.replay(); torch.cuda.synchronize()
            sampler.stop()
            return ms, sampler.summary(n_in)

        rep_ms, clocks = timed("step")
        ms_step = statistics.median(rep_ms) / K
        lens_now = [n + per[0] for n in layers[0].lens0]
        line = {"metric": METRIC, "value": spec.batch / (ms_step * 1e-3), "unit": UNIT, "n_gpus": 1, "steps": K, "warmup": W,
                "ms_per_step": ms_step, "us_per_step": ms_step * 1e3, "higher_is_better": True, "dtype": spec.dtype,
                "data": "synthetic",
                "config": {"workload": label, "name": spec.name, "batch": spec.batch, "n_q_heads": spec.n_q_heads,
                           "n_kv_heads": spec.n_kv_heads, "context": spec.n_ctx, "context_min": spec.n_ctx_min,
                           "code_bits": spec.code_bits, "budget_ppm": spec.budget_ppm, "layer_replicas": L,
                           "l2": ("%d layer replicas visited round-robin: %.0f MB per round" % (L, L * step_bytes / 1e6))
                                 if L * step_bytes > 126 * 2 ** 20 else "a step's bytes fit L2 (latency-bound configuration)",
                           "cluster_size": layers[0].ctx.get_cluster_size(), "kv_layout": "interleaved k|v rows"},
                "timing": {"reps": args.reps, "us_per_step_min": min(rep_ms) / K * 1e3, "us_per_step_max": max(rep_ms) / K * 1e3},
                "clocks": clocks, "roofline": _roofline(spec, lens_now, ms_step, peaks),
                "prefill_ms_per_layer": {"fit": layers[-1].fit_ms, "encode": layers[-1].encode_ms,
                                         "keys": int(sum(layers[-1].lens0)) * spec.n_kv_heads,
                                         "reconstruction_err_over_K": [ly.reconstruction_error() for ly in layers]},
                "device_error_word": max(ly.ctx.last_device_error() for ly in layers)}
        try:                                       # the paper's own score (sign + 7 magnitude planes) on the same workload
            for ly in layers:
                ly.make_weighted_twin(B)
            w7_ms, _ = timed("step_weighted", which="ctx_w7")
            line["us_per_step_weighted7_scores"] = statistics.median(w7_ms) / K * 1e3
        except Exception as ex:
            line["us_per_step_weighted7_scores"] = None
            line["weighted7_note"] = str(ex)[:100]
        print(json.dumps(line), flush=True)
        layers = None
        torch.cuda.empty_cache()


# ----------------------------------------------------------------------------- paper-scale sweep (second workload)
SWEEP_CASES = [  # (context, batch): 64-bit codes, fixed budgets, 32/8 heads, bf16, as in the paper's latency-vs-context study
    (32768, 1), (32768, 16), (131072, 1), (131072, 3), (131072, 8), (262144, 1), (262144, 4), (1048576, 1), (2097152, 1),
]


def run_sweep(args):
    """Decode-step latency of one layer over contexts and batch sizes with 64-bit codes and fixed budgets of 1024 and
    2048 keys (the paper's own operating points: single-word codes, 1K/2K budgets, latency flat in the context length).
    One JSON line; every case is timed like the main workload (CUDA graph of K fused steps over enough layer replicas that
    a step's bytes exceed L2).  Contexts above the kernel's limit (cluster size 16 x keys per block) are reported as
    unsupported."""
    from paper_2608_04405_b200 import binding as B
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    K, W = args.steps, max(args.warmup, 3)
    rows = []
    fit_ws = [None]
    for n_ctx, batch in SWEEP_CASES:
        spec = CONFIGS[1].scaled(name="sweep_ctx%d_b%d" % (n_ctx, batch), wid=100 + len(rows), batch=batch, n_ctx=n_ctx,
                                 code_bits=64, steps=K, needles=8)
        units = batch * spec.n_kv_heads
        for budget in (1024, 2048):
            step_bytes = units * (n_ctx * 8 + 2 * budget * spec.head_dim * 2)
            L = max(2, min(32, -(-(2 * 126 * 2**20) // step_bytes)))
            extra = ((K + W) // L + 2) * 2 + 64
            try:
                layers = [Layer(spec, salt=i, extra_rows=extra, B=B, fit_ws=fit_ws, interleaved=True, budget_count=budget)
                          for i in range(L)]
            except Exception as e:                                   # e.g. context beyond the kernel's limit
                rows.append({"context": n_ctx, "batch": batch, "budget": budget, "unsupported": str(e)[:120]})
                layers = None
                torch.cuda.empty_cache()
                continue
            for s in range(W):
                layers[s % L].step()
            torch.cuda.synchronize()
            per = [(W + L - 1 - i) // L for i in range(L)]
            for ly, c in zip(layers, per):
                ly.ctx.set_seq_lens([n + c for n in ly.lens0])
            g = _graph_of(lambda: [layers[(W + s) % L].step() for s in range(K)])
            for ly, c in zip(layers, per):
                ly.ctx.set_seq_lens([n + c for n in ly.lens0])
            g.replay()
            torch.cuda.synchronize()
            for ly, c in zip(layers, per):
                ly.ctx.set_seq_lens([n + c for n in ly.lens0])
            ms = _time_graph(g, lambda: None) / K
            err = max(ly.ctx.last_device_error() for ly in layers)
            rows.append({"context": n_ctx, "batch": batch, "budget": budget, "us_per_step": round(ms * 1e3, 2),
                         "cluster_size": layers[0].ctx.get_cluster_size(), "streaming": layers[0].ctx.uses_streaming(), "byte_keys": layers[0].ctx.uses_byte_keys(), "layer_replicas": L,
                         "algorithmic_GBps": round(step_bytes / ms / 1e6, 1), "device_error_word": err})
            layers = None
            g = None
            torch.cuda.empty_cache()
    print(json.dumps({"metric": "decode_step_latency_sweep", "unit": "us_per_step", "dtype": "bf16", "data": "synthetic",
                      "config": {"workload": "paper-scale sweep: 64-bit codes, budgets 1024/2048, 32/8 heads, bf16 K|V interleaved",
                                 "cold_l2": "layer replicas visited round-robin, bytes per step x replicas > 2 x L2"},
                      "steps": K, "warmup": W, "cases": rows}))


# ----------------------------------------------------------------------------- quality yard-sticks
def run_quality(args):
    """Selection quality on the synthetic workload for code lengths 32, 64, 128 and 256: recall of the hash selection with
    respect to the exact-score top-k of every query head (the paper's TOPK (Oracle) baseline), cosine similarity between
    the sparse output and dense attention (the paper's output-similarity table), and recall of the planted needles.
    All three selections and both outputs come from the library (bpc_exact_topk, bpc_decode_attn with the workload's
    budget and with a budget of all keys); torch only intersects index sets and takes the cosine of the outputs."""
    from paper_2608_04405_b200 import binding as B
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    spec0 = CONFIGS[args.workload]
    rows = []
    for bits in (32, 64, 128, 256):
        spec = spec0.scaled(code_bits=bits)
        w = Workload(spec, device="cuda", extra_rows=64)
        cfg = B.make_config(spec.batch, spec.n_q_heads, spec.n_kv_heads, w.n_max, bits, spec.torch_dtype)
        ctx = B.Context(cfg)
        ctx.set_seq_lens(w.seq_lens)
        codes = ctx.alloc_codes()
        ws = torch.empty(ctx.fit_workspace_bytes(), dtype=torch.uint8, device="cuda")
        ctx.fit(w.k_cache, w.v_star, ws)
        del ws
        ctx.encode_keys(w.k_cache, codes)
        q, needles = w.queries(w.seq_lens)
        units = spec.batch * spec.n_kv_heads
        dense = ctx.decode_attn(q, w.k_cache, w.v_cache, codes, budget_ppm=1000000)
        _, tsel, tcnt = ctx.exact_topk(q, w.k_cache, budget_ppm=spec.budget_ppm)
        G = spec.group
        P, _, _ = ctx.get_projection()
        for mode_name, mode in (("hamming", B.BPC_SCORE_HAMMING), ("weighted7", B.BPC_SCORE_WEIGHTED7)):
            mctx = ctx
            if mode != B.BPC_SCORE_HAMMING:     # Algorithm 3's sign + seven magnitude planes, same projection and codes
                try:
                    mctx = B.Context(B.make_config(spec.batch, spec.n_q_heads, spec.n_kv_heads, w.n_max, bits, spec.torch_dtype,
                                                   score_mode=mode))
                except Exception as e:          # scores beyond 16 bits for this code length and group size
                    rows.append({"code_bits": bits, "score_mode": mode_name, "unsupported": str(e)[:100]})
                    continue
                mctx.set_projection(P)
                mctx.set_seq_lens(w.seq_lens)
            hsel = torch.full((units, w.n_max), -1, dtype=torch.int32, device="cuda")
            sparse = mctx.decode_attn(q, w.k_cache, w.v_cache, codes, budget_ppm=spec.budget_ppm, sel_idx=hsel)
            torch.cuda.synchronize()
            rec, nrec = [], []
            for bi in range(spec.batch):
                for hq in range(spec.n_q_heads):
                    u = bi * spec.n_kv_heads + hq // G
                    head = bi * spec.n_q_heads + hq
                    k = int(tcnt[head])
                    mine = hsel[u, :k]
                    rec.append(float(torch.isin(tsel[head, :k], mine).float().mean()))
                    nrec.append(float(torch.isin(needles[bi, hq], mine).float().mean()))
            cos = torch.nn.functional.cosine_similarity(sparse.reshape(-1, spec.head_dim), dense.reshape(-1, spec.head_dim), dim=1)
            rows.append({"code_bits": bits, "score_mode": mode_name, "recall_vs_exact_topk": sum(rec) / len(rec),
                         "cosine_sparse_vs_dense": float(cos.mean()), "cosine_min": float(cos.min()),
                         "needle_recall": sum(nrec) / len(nrec), "device_error_word": mctx.last_device_error()})
        del ctx, mctx, codes, w, hsel, tsel, sparse, dense
        torch.cuda.empty_cache()
    print(json.dumps({"metric": "selection_quality", "data": "synthetic", "dtype": "bf16",
                      "config": {"workload": spec0.name, "budget_ppm": spec0.budget_ppm, "code_bits": [32, 64, 128, 256]},
                      "cases": rows}))


# ----------------------------------------------------------------------------- CPU checker arm
def _oracle_unit_setup(spec, seed_salt=0):
    """One unit of the workload prepared for the checker: keys, values, projection, codes (prefill, untimed)."""
    from oracle import bpc_oracle as O
    one = spec.scaled(batch=1, n_kv_heads=1, n_q_heads=spec.group)
    w = Workload(one, device="cpu", extra_rows=64, salt=seed_salt)
    n = w.seq_lens[0]
    K = w.k_cache[0, 0, :n].double().numpy()
    V = w.v_cache[0, 0, :n].double().numpy()
    sub = K[:: max(1, n // 4096)][:4096]              # projection fitted on a strided sample of the keys
    P, _, _ = O.fit(sub, w.v_star[0].double().numpy())
    Ph = O.to_hash_precision(P, spec.dtype)
    bits, _ = O.encode(K, Ph)
    q, _ = w.queries(w.seq_lens)
    return O, K, V, Ph, bits, q[0].double().numpy()


def cpu_baseline(spec, budget_s=15.0):
    O, K, V, Ph, bits, q = _oracle_unit_setup(spec)
    units_per_step = spec.batch * spec.n_kv_heads
    t0, c0 = time.time(), time.process_time()
    done = 0
    while done < 2 or (time.time() - t0 < budget_s and done < 64):
        O.decode_unit(q, K, V, bits, Ph, spec.budget_ppm)
        done += 1
    wall, cpu = time.time() - t0, time.process_time() - c0
    step_s = wall / done * units_per_step
    return {"value": spec.batch / step_s, "unit": UNIT, "cores": max(1, int(round(cpu / max(wall, 1e-9)))),
            "host_cores": os.cpu_count(), "kind": "oracle",
            "sample": "%d single-unit decode steps (query hash, %d-key score, top-k, attention) of %s timed; "
                      "one step = %d such units, scaled" % (done, K.shape[0], spec.name, units_per_step),
            "us_per_step_scaled": step_s * 1e6}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    spec = CONFIGS[args.workload]
    O, K, V, Ph, bits, q = _oracle_unit_setup(spec)
    units_per_step = spec.batch * spec.n_kv_heads
    for _ in range(min(args.warmup, 3)):
        O.decode_unit(q, K, V, bits, Ph, spec.budget_ppm)
    t0, c0 = time.time(), time.process_time()
    for _ in range(args.steps):
        O.decode_unit(q, K, V, bits, Ph, spec.budget_ppm)
    wall, cpu = time.time() - t0, time.process_time() - c0
    step_s = wall / args.steps * units_per_step
    value = spec.batch / step_s
    world = int(os.environ.get("WORLD_SIZE", "1"))
    sample = ("each step times ONE (sequence, KV head) unit of %s (%d keys) on the host and is scaled by the %d units "
              "of a full step" % (spec.name, K.shape[0], units_per_step))
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": step_s * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": spec.name, "batch": spec.batch, "n_q_heads": spec.n_q_heads, "n_kv_heads": spec.n_kv_heads,
                   "head_dim": spec.head_dim, "context": spec.n_ctx, "code_bits": spec.code_bits,
                   "budget_ppm": spec.budget_ppm},
        "scaled": True, "units_timed": 1, "units_per_step": units_per_step,
        "cpu_baseline": {"value": value, "unit": UNIT, "kind": "oracle", "host_cores": os.cpu_count(),
                         "cores": max(1, int(round(cpu / max(wall, 1e-9)))), "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=128)
    ap.add_argument("--warmup", type=int, default=32)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", type=int, default=2)
    ap.add_argument("--layers", type=int, default=4, help="independent layer replicas visited round-robin (cold L2)")
    ap.add_argument("--reps", type=int, default=5, help="timed replays of the K-step graph (median reported)")
    ap.add_argument("--all-configs", action="store_true", help="one JSON line per synthetic configuration 0-4 and per point of configuration 3's code length x budget sweep")
    ap.add_argument("--cpu-budget", type=float, default=15.0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--separate-kv", action="store_true", help="separate K and V arrays instead of interleaved rows")
    ap.add_argument("--profile", action="store_true", help="warm-up plus K eager steps only (for ncu captures)")
    ap.add_argument("--profile-leg", choices=("fused", "weighted7", "work_items"), default="fused",
                    help="with --profile: the fused step with Hamming scores (default) or with the weighted score")
    ap.add_argument("--sweep", action="store_true", help="second workload: latency over contexts and batch sizes, 64-bit codes, 1K/2K budgets")
    ap.add_argument("--quality", action="store_true", help="selection quality yard-sticks (recall vs exact top-k, cosine vs dense) for 32/64/128/256-bit codes")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if args.impl == "reference":
        run_reference(args)
    elif args.all_configs:
        run_all_configs(args)
    elif args.sweep:
        run_sweep(args)
    elif args.quality:
        run_quality(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
