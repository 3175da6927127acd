#!/usr/bin/env python
"""SP-KV decode benchmark (one JSON line).

A step = one decode token for every sequence of the batch through the whole layer stack: per layer
score + append/evict, then decode attention (the library is the attention path only; there are no
projections or MLPs).  The step is ONE spkv_decode_stack call -- the appends of every layer in one
launch, decode attention of every layer in one persistent launch; --per-layer times it as 2 L calls
(spkv_score_append_evict -> spkv_decode_attention per layer).  Inputs are synthetic and seeded,
shaped like the paper's decode workloads (see paper_2605_14037_b200/synth.py); the cache is
brought to the configured context length with spkv_prefill before timing.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config 2] [--impl reference]

value        whole-job decode tokens/s, inputs resident in HBM, one CUDA-graph replay per step
e2e          the same through spkv_decode_stack_host with pinned HOST buffers (H2D + D2H timed);
             the per-layer spkv_decode_step_host beside it
roofline     decode-attention kernel: algorithmic bytes (kept + window K/V, Q, O) of a step over the
             step time, against the measured HBM copy bandwidth, the nominal 8 TB/s and a read-only
             stream the library measures itself; one per-layer launch timed alone beside it
dense        same library, tau = -inf (every pair kept): the full-cache decode baseline
cpu_baseline the CPU oracle timed on a bounded sample of the same workload
"""
from __future__ import annotations

import argparse
import json
import math
import os
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

CONFIGS = {
    # name: layers, batch, q heads, kv heads, context, beta(a, b) of per-head keep rates
    1: dict(name="config1_1layer_b1_ctx4k", L=1, B=1, Hq=8, Hkv=2, T=4096, beta=None, rate=0.2),
    2: dict(name="config2_llama8b_b16_ctx32k", L=32, B=16, Hq=32, Hkv=8, T=32768, beta=(0.5, 2.0)),
    3: dict(name="config3_llama8b_b4_ctx128k", L=32, B=4, Hq=32, Hkv=8, T=131072, beta=(0.3, 3.0)),
    4: dict(name="config4_ragged_b64_prefill8_decode56", L=32, B=64, Hq=32, Hkv=8, T=65536, beta=(0.5, 2.0),
            t_min=4096, n_prefill=8, chunk=8192),
    5: dict(name="config5_llama70b_b8_ctx64k", L=80, B=8, Hq=64, Hkv=8, T=65536, beta=(0.5, 2.5)),
}
W, D_IN, TAU, CHUNK = 128, 512, 0.5, 8192
CACHE_FLAGS = [1]          # SPKV_FLAG_OVERLAP; --stream-ordered clears it


def peaks():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


class ClockSampler:
    """Samples the SM clock and the throttle reasons every 20 ms while a region runs (NVML,
    read-only queries, from a thread of this process; nvidia-smi every 100 ms if NVML cannot be
    loaded).  Samples carry the time they were taken, so that a part of the region can be looked
    at by itself (`window`)."""

    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")
    REASONS = ((0x8, "hw_slowdown"), (0x40, "hw_thermal_slowdown"), (0x20, "sw_thermal_slowdown"),
               (0x4, "sw_power_cap"))

    def __init__(self, index, period_s=0.02):
        self.index, self.period, self.proc, self.thread = index, period_s, None, None
        self.samples = []          # (perf_counter time, sm MHz, [reasons])
        self.max_mhz = None
        self.result = {"sm_mhz": None, "sm_max_mhz": None, "reasons": []}

    def _nvml_loop(self, nv, handle):
        while not self._stop.is_set():
            try:
                mhz = nv.nvmlDeviceGetClockInfo(handle, nv.NVML_CLOCK_SM)
                try:
                    mask = nv.nvmlDeviceGetCurrentClocksEventReasons(handle)
                except Exception:
                    mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(handle)
                self.samples.append((time.perf_counter(), float(mhz), [n for bit, n in self.REASONS if mask & bit]))
            except Exception:
                pass
            self._stop.wait(self.period)

    def __enter__(self):
        import threading
        self._stop = threading.Event()
        try:
            import pynvml as nv
            nv.nvmlInit()
            # NVML numbers devices like nvidia-smi; CUDA_VISIBLE_DEVICES may renumber CUDA's
            vis = os.environ.get("CUDA_VISIBLE_DEVICES", "")
            idx = self.index
            if vis and all(v.strip().isdigit() for v in vis.split(",")) and self.index < len(vis.split(",")):
                idx = int(vis.split(",")[self.index])
            handle = nv.nvmlDeviceGetHandleByIndex(idx)
            self.max_mhz = float(nv.nvmlDeviceGetMaxClockInfo(handle, nv.NVML_CLOCK_SM))
            self.thread = threading.Thread(target=self._nvml_loop, args=(nv, handle), daemon=True)
            self.thread.start()
        except Exception:
            self.thread = None
            try:
                self.t_start = time.perf_counter()
                self.proc = subprocess.Popen(
                    ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}",
                     "--format=csv,noheader,nounits", "-lms", "100"],
                    stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            except Exception:
                self.proc = None
        return self

    def __exit__(self, *exc):
        if self.thread is not None:
            self._stop.set()
            self.thread.join(timeout=2)
        elif self.proc:
            time.sleep(0.15)
            self.proc.terminate()
            try:
                out, _ = self.proc.communicate(timeout=5)
            except Exception:
                self.proc.kill()
                out = ""
            names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
            lines = [l for l in out.strip().splitlines() if len(l.split(",")) >= 6]
            t_end = time.perf_counter()
            for i, line in enumerate(lines):
                parts = [p.strip() for p in line.split(",")]
                try:
                    mhz, mx = float(parts[0]), float(parts[1])
                except ValueError:
                    continue
                self.max_mhz = mx
                # nvidia-smi prints no time we can align: spread the lines evenly over the region
                t = self.t_start + (t_end - self.t_start) * (i + 0.5) / len(lines)
                self.samples.append((t, mhz, [n for n, v in zip(names, parts[2:6]) if v.lower().startswith("active")]))
        self.result = self.window(None, None)
        self.result["samples_under_load"] = len(self.samples)

    def window(self, t0, t1):
        """Median SM clock and the reasons seen among the samples taken in [t0, t1] (all if None)."""
        sel = [x for x in self.samples if (t0 is None or x[0] >= t0) and (t1 is None or x[0] <= t1)]
        if not sel:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": []}
        mhz = sorted(x[1] for x in sel)
        return {"sm_mhz": mhz[len(mhz) // 2], "sm_max_mhz": self.max_mhz,
                "reasons": sorted({r for x in sel for r in x[2]})}


def median(xs):
    xs = sorted(xs)
    n = len(xs)
    return xs[n // 2] if n % 2 else 0.5 * (xs[n // 2 - 1] + xs[n // 2])


def plan_repeats(first_region_s, min_total_s=2.0, min_repeats=5, max_repeats=200):
    """How often the K-step region is timed: until at least `min_total_s` of device time has been
    measured, never fewer than `min_repeats` regions (and never more than `max_repeats`)."""
    need = int(math.ceil(min_total_s / max(first_region_s, 1e-9)))
    return max(min_repeats, min(max_repeats, need))


def max_over_ranks(x, dist=None, device=None):
    """Largest value of x over the ranks of the job (x itself without a process group)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(x)
    import torch
    t = torch.tensor([float(x)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(units_per_rank, seconds_local, dist=None, device=None):
    """Replicas only: every rank processes `units_per_rank` units; the job's rate is all
    ranks' units over the slowest rank's time."""
    world = dist.get_world_size() if dist is not None and dist.is_initialized() else 1
    return world * units_per_rank / max_over_ranks(seconds_local, dist, device)


def build_workload(spkv, synth, torch, cfg, dev, dense, total_steps, seed=0, tau=None):
    """Creates the cache, per-layer predictors and brings every sequence to context T.
    The predictors are calibrated so that head (l, h) keeps a fraction rates[l, h] at tau = 0.5;
    another `tau` (threshold sweep) moves every head's rate along its Gaussian logit
    distribution, as sweeping the threshold of a trained predictor does."""
    import numpy as np
    L, B, Hq, Hkv, T = cfg["L"], cfg["B"], cfg["Hq"], cfg["Hkv"], cfg["T"]
    rng = np.random.default_rng(seed)
    tau = TAU if tau is None else tau
    tau = -math.inf if dense else tau
    if cfg["beta"] is None:
        rates = np.full((L, Hkv), cfg["rate"])
    else:
        rates = synth.keep_rates(rng, L, Hkv, *cfg["beta"])
    tl = 0.0  # logit-space threshold of tau = 0.5, where the biases are calibrated
    pred_np = []
    for l in range(L):
        Wl = synth.linear_predictor(rng, Hkv, D_IN)
        pred_np.append((Wl, synth.bias_for_keep_rate(Wl, rates[l], tl)))
    if dense:
        eff = np.ones_like(rates)
    elif tau == TAU:
        eff = rates
    else:  # P(w.x + b >= tau_logit) for x ~ N(0, I): Phi((b - tau_logit) / |w|)
        tl_run = math.log(tau / (1.0 - tau)) if 0.0 < tau < 1.0 else (-math.inf if tau <= 0.0 else math.inf)
        eff = np.empty_like(rates)
        for l, (Wl, bl) in enumerate(pred_np):
            norms = np.sqrt((synth.bf16_bits_to_f32(Wl).astype(np.float64) ** 2).sum(axis=1))
            z = (bl.astype(np.float64) - tl_run) / norms
            eff[l] = [0.5 * math.erfc(-float(v) / math.sqrt(2.0)) for v in z]
    t_list = cfg.get("t_list")          # per-sequence contexts (ragged batch), else uniform T
    grow = cfg.get("grow", total_steps)  # pairs every sequence may still receive
    t_final = T + grow
    pages_per_unit = np.ceil(eff * (t_final - W) * 1.03 / 64).astype(np.int64) + 2
    pool_pages = int(pages_per_unit.sum() * B)
    if t_list is not None:
        g_list = np.asarray(cfg.get("grow_list", [grow] * B))
        per_seq = np.ceil(eff[:, None, :] * (np.asarray(t_list) + g_list)[None, :, None] * 1.03 / 64) + 2
        pool_pages = int(per_seq.sum())
    cache = spkv.Cache(n_layers=L, max_seqs=B, n_q_heads=Hq, n_kv_heads=Hkv,
                       max_context=t_final + 64, pool_pages=pool_pages, window=W, tau=tau, device=dev,
                       flags=CACHE_FLAGS[0])   # overlap: attention-only stack, inputs staged before the step
    preds, keep = [], []
    for l in range(L):
        Wl, bl = pred_np[l]
        Wd, bd = spkv.bf16_from_bits(Wl, dev), torch.from_numpy(bl).to(dev)
        preds.append(spkv.make_predictor(Wd, bd))
        keep.append((Wd, bd))
    gen = torch.Generator(device=dev)
    gen.manual_seed(seed)
    # state build: device-generated chunks through score + prefill (state only, no attention)
    kv_pool = [torch.randn((CHUNK, Hkv, 128), generator=gen, device=dev, dtype=torch.float32)
               .to(torch.bfloat16) for _ in range(4)]
    for l in range(L):
        for b in range(B):
            done, T_b = 0, (T if t_list is None else int(t_list[b]))
            while done < T_b:
                c = min(CHUNK, T_b - done)
                x = torch.randn((c, D_IN), generator=gen, device=dev, dtype=torch.float32).to(torch.bfloat16)
                lg = cache.spkv_score(preds[l], x)
                k, v = kv_pool[(l + b + done // CHUNK) % 4][:c], kv_pool[(l + b + 1 + done // CHUNK) % 4][:c]
                cache.spkv_prefill(l, b, k, v, lg)
                done += c
    cache.check()
    return cache, preds, rates, gen


def run_ours(args):
    import numpy as np
    import torch

    from paper_2605_14037_b200 import build as spkv_build
    spkv_build.build()
    from paper_2605_14037_b200 import spkv, synth

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    dev = torch.device(f"cuda:{local}")
    torch.cuda.set_device(dev)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    cfg = dict(CONFIGS[args.config])
    if args.layers > 0:
        cfg["L"] = args.layers
        cfg["name"] += f"_{args.layers}layers_only"
    L, B, Hq, Hkv = cfg["L"], cfg["B"], cfg["Hq"], cfg["Hkv"]
    K, Wm = args.steps, args.warmup
    e2e_steps = min(K, args.e2e_steps)
    roof_steps = min(K, 8)
    # every repeat of the timed region starts from the same checkpoint, so the cache (and the
    # per-step inputs) only have to cover ONE pass over the phases below
    total_steps = Wm + K + 2 * (e2e_steps + 3) + roof_steps + 3 + 1
    hbm_peak, peak_kind = peaks()

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    def max_ranks(x):
        return max_over_ranks(x, dist, dev)

    def measure(dense, tau=None):
        nonlocal L
        cfg_run, L_full = cfg, cfg["L"]
        if dense:
            # dense K/V of the whole stack; when it does not fit in ~140 GB a layer subset is
            # measured and scaled (layers are independent and identical in the dense run)
            dense_bytes = cfg["L"] * B * Hkv * (cfg["T"] + total_steps) * 512
            if dense_bytes > 140e9:
                cfg_run = dict(cfg, L=max(1, int(cfg["L"] * 140e9 / dense_bytes)))
        L = cfg_run["L"]
        try:
            return _measure(dense, cfg_run, L_full, tau)
        finally:
            L = L_full

    def _measure(dense, cfg, L_full, tau):
        cache, preds, rates, gen = build_workload(spkv, synth, torch, cfg, dev, dense, total_steps, tau=tau)
        ids = torch.arange(B, dtype=torch.int32, device=dev)
        n_in = 4  # distinct q/k/v input sets cycled over the steps
        # q, k, v of a step live in one flat buffer (one staging copy per step instead of three)
        nq, nkv = L * B * Hq * 128, L * B * Hkv * 128
        qkv_in = torch.randn((n_in, nq + 2 * nkv), generator=gen, device=dev).to(torch.bfloat16)
        q_in = qkv_in[:, :nq].view(n_in, L, B, Hq, 128)
        k_in = qkv_in[:, nq:nq + nkv].view(n_in, L, B, Hkv, 128)
        v_in = qkv_in[:, nq + nkv:].view(n_in, L, B, Hkv, 128)
        x_all = torch.randn((total_steps, L, B, D_IN), generator=gen, device=dev).to(torch.bfloat16)
        # Every step reads its inputs where they lie in HBM (a fresh x per step and layer, q/k/v from
        # four cycled sets): no staging copies.  One CUDA graph per step number, captured before the
        # timed region; the repeats replay the same step numbers from the same cache checkpoint.
        out = torch.empty((L, B, Hq, 128), dtype=torch.bfloat16, device=dev)
        logits = torch.empty((L, B, Hkv), dtype=torch.float32, device=dev)
        cache.decode_workspace(B)
        step_no = [0]
        graphs = {}

        def layer_calls(step, stream=None, events=None):
            xs, qs, ks, vs = x_all[step], q_in[step % n_in], k_in[step % n_in], v_in[step % n_in]
            # the first launch of a step waits for everything before it on the stream even in overlap
            # mode (the previous step's reads of the cache, a rollback copy)
            if not args.per_layer and events is None:
                # the whole stack in two launches: appends of every layer, one persistent decode kernel
                cache.spkv_decode_stack(preds, ids, xs, qs, ks, vs, out=out, logits_out=logits, stream=stream)
                return
            cache.spkv_note_foreign_work()
            for l in range(L):
                cache.spkv_score_append_evict(l, preds[l], ids, xs[l], ks[l], vs[l],
                                              logits_out=logits[l], stream=stream)
                if events is not None:
                    events[l][0].record()
                cache.spkv_decode_attention(l, ids, qs[l], out=out[l], stream=stream)
                if events is not None:
                    events[l][1].record()

        def capture(first, n):
            """CUDA graphs of steps first ... first + n - 1 (capturing runs nothing)."""
            if args.no_graph:
                return
            step = first
            while step < first + n:
                cnt = min(max(1, args.steps_per_graph), first + n - step)
                if step not in graphs:
                    g = torch.cuda.CUDAGraph()
                    with torch.cuda.graph(g):
                        for j in range(cnt):
                            layer_calls(step + j)
                    graphs[step] = (g, cnt)
                step += graphs[step][1]

        if not args.no_graph:
            side = torch.cuda.Stream(device=dev)
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(side):
                layer_calls(0)                           # warm the lazily loaded kernels
            torch.cuda.current_stream().wait_stream(side)
            torch.cuda.synchronize()
            step_no[0] = 1

        def run_steps(n, events=None):
            """n steps starting at step number step_no[0]."""
            i = 0
            while i < n:
                step = step_no[0] + i
                if step in graphs and events is None and graphs[step][1] <= n - i:
                    graphs[step][0].replay()
                    i += graphs[step][1]
                else:
                    layer_calls(step, events=None if events is None else events[i])
                    i += 1
            step_no[0] += n

        run_steps(Wm)
        cache.check()
        st0 = cache.spkv_cache_stats()
        # The timed region is exactly K steps.  It is timed R times -- until >= 2 s of device time
        # have been measured, at least 5 times -- each time from the same state: the cache is rolled
        # back to a checkpoint taken here (metadata + ring pages; outside the timed region), and the
        # same inputs are replayed.  `value` is the median region.
        ckpt = cache.spkv_cache_checkpoint()
        step_mark = step_no[0]
        capture(step_mark, K)
        torch.cuda.synchronize()
        # settle: the same region replayed untimed until the GPU has been under this load for about a
        # second -- a B200 starts at its maximum clock and drops to what its power limit sustains
        # within the first ~0.5 s; the repeats below then all measure the sustained state
        settle_regions, t_settle = 0, time.perf_counter()
        while args.settle_seconds > 0 and time.perf_counter() - t_settle < args.settle_seconds:
            run_steps(K)
            torch.cuda.synchronize()
            cache.spkv_cache_rollback(ckpt)
            step_no[0] = step_mark
            settle_regions += 1
        regions, marks = [], []
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        st1 = None
        with ClockSampler(local) as clk:
            n_rep = 1
            r = 0
            while r < n_rep:
                if r > 0:
                    cache.spkv_cache_rollback(ckpt)
                    step_no[0] = step_mark
                barrier()
                t_a = time.perf_counter()
                torch.cuda.nvtx.range_push("timed_region")      # lets a profiler pick out the timed launches
                e0.record()
                run_steps(K)
                e1.record()
                torch.cuda.synchronize()
                torch.cuda.nvtx.range_pop()
                t_b = time.perf_counter()
                barrier()
                regions.append(max_ranks(e0.elapsed_time(e1)))
                marks.append((t_a, t_b))
                if r == 0:
                    st1 = cache.spkv_cache_stats()
                    n_rep = int(max_ranks(plan_repeats(regions[0] * 1e-3)))
                r += 1
        ms = median(regions)
        per_rep_clock = [clk.window(a, b)["sm_mhz"] for a, b in marks]
        srt = sorted(regions)
        p10, p90 = srt[len(srt) // 10], srt[len(srt) - 1 - len(srt) // 10]
        repeats = {"n": len(regions), "min": min(regions) / K, "median": ms / K, "max": max(regions) / K,
                   "unit": "ms_per_step", "spread": (max(regions) - min(regions)) / ms,
                   "p10": p10 / K, "p90": p90 / K, "spread_p10_p90": (p90 - p10) / ms,
                   "timed_device_s": sum(regions) * 1e-3,
                   "ms_per_step_each": [round(x / K, 5) for x in regions],
                   "sm_mhz_each": per_rep_clock,
                   # region time x median SM clock: flat if a slow repeat is a clock dip, not if it is contention
                   "ms_x_ghz_each": [round(x / K * c * 1e-3, 5) if c else None for x, c in zip(regions, per_rep_clock)],
                   "settle": {"seconds": args.settle_seconds, "untimed_regions": settle_regions},
                   "how": "each repeat = the same K steps replayed from a checkpoint of the cache "
                          "(spkv_cache_rollback, outside the timed region); value = median; before the first "
                          "repeat the region is replayed untimed until the clocks have settled under load"}
        cache.check()

        # decode-kernel duration, measured with events around every launch (no graph)
        evs = [[(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
                for _ in range(L)] for _ in range(roof_steps)]
        run_steps(3, events=[None] * 3)
        torch.cuda.synchronize()
        run_steps(roof_steps, events=evs)
        torch.cuda.synchronize()
        dec_ms = [a.elapsed_time(b) for row in evs for (a, b) in row]
        st2 = cache.spkv_cache_stats()
        kv_bytes = 0.5 * (st1.bytes_resident + st2.bytes_resident)     # all layers, one step
        qo_bytes = L * B * Hq * 128 * 2 * 2
        launch_bytes = (kv_bytes + qo_bytes) / L
        launch_s = (sum(dec_ms) / len(dec_ms)) * 1e-3

        scale_l = L_full / L          # > 1 only for a dense run on a layer subset
        ms *= scale_l
        for k_ in ("min", "median", "max", "p10", "p90"):
            repeats[k_] *= scale_l
        res = dict(layers_measured=L, ms_per_step=ms / K, tokens_per_s=world * B * K / (ms * 1e-3), repeats=repeats,
                   kv_gb_per_step=scale_l * 0.5 * (st0.bytes_resident + st1.bytes_resident) / 1e9,
                   density=st1.density_cache, launch_bytes=launch_bytes, launch_s=launch_s,
                   clocks=clk.result, graph=bool(graphs))

        # end to end through the host-buffer entry point
        if not dense and e2e_steps > 0 and tau is None:
            pin = lambda t: t.contiguous().cpu().pin_memory()
            hx, hq, hk, hv = pin(x_all[:4]), pin(q_in), pin(k_in), pin(v_in)
            hout = torch.empty((L, B, Hq, 128), dtype=torch.bfloat16).pin_memory()

            def e2e_step(s):      # the whole stack in one call: 4 copies in, 2 L kernels, 1 copy out
                cache.spkv_decode_stack_host(preds, ids, hx[s % 4], hq[s % n_in], hk[s % n_in], hv[s % n_in], hout)
                torch.cuda.current_stream().synchronize()   # the step's result is read on the host
                return float(hout[L - 1, 0, 0, 0])

            def e2e_step_per_layer(s):   # layer by layer (the entry point a model with host inputs per layer uses)
                for l in range(L):
                    cache.spkv_decode_step_host(l, preds[l], ids, hx[s % 4, l], hq[s % n_in, l],
                                                hk[s % n_in, l], hv[s % n_in, l], hout[l])
                cache.spkv_decode_step_host_flush()
                torch.cuda.current_stream().synchronize()
                return float(hout[L - 1, 0, 0, 0])

            def timed(fn):
                for s in range(3):
                    fn(s)
                barrier()
                t0 = time.perf_counter()
                for s in range(e2e_steps):
                    fn(s)
                torch.cuda.synchronize()
                return max_ranks(time.perf_counter() - t0)

            dt_layer = timed(e2e_step_per_layer)
            dt = timed(e2e_step)
            cache.check()
            res["e2e"] = {
                "value": world * B * e2e_steps / dt, "unit": "tokens/s",
                "h2d_bytes_per_step": L * B * (D_IN + Hq * 128 + 2 * Hkv * 128) * 2,
                "d2h_bytes_per_step": L * B * Hq * 128 * 2, "steps": e2e_steps,
                "api": "spkv_decode_stack_host",
                "per_layer_api": {"value": world * B * e2e_steps / dt_layer, "api": "spkv_decode_step_host"}}
        if not dense and tau is None:
            # the read-only ceiling of this GPU, measured by the library's own read stream over
            # the cache arena (larger than L2 for every config but the tiny one)
            res["read_ceiling_gbs"] = spkv.spkv_stream_read(cache.arena)
        cache.close()
        del cache
        torch.cuda.empty_cache()
        return res

    if args.sweep_tau:
        # threshold sweep (the deployment-time density control of the paper's section on
        # controlling sparsity at inference time): one line per tau, same predictors, state rebuilt
        for tau in [float(t) for t in args.sweep_tau.split(",")]:
            r = measure(dense=False, tau=tau)
            if rank == 0:
                ach = r["launch_bytes"] / r["launch_s"] / 1e9
                print(json.dumps({"sweep": "tau", "tau": tau, "workload": cfg["name"], "density": r["density"],
                                  "kv_gb_per_step": r["kv_gb_per_step"], "tokens_per_s": r["tokens_per_s"],
                                  "ms_per_step": r["ms_per_step"], "decode_kernel_gbs": ach,
                                  "frac_of_hbm_peak": ach / hbm_peak, "steps": K, "warmup": Wm,
                                  "clocks": r["clocks"]}), flush=True)
        return
    sp = measure(dense=False)
    dn = measure(dense=True) if args.dense else None

    if rank != 0:
        return
    achieved = sp["launch_bytes"] / sp["launch_s"] / 1e9
    in_step = (sp["kv_gb_per_step"] * 1e9 + L * B * Hq * 512) / (sp["ms_per_step"] * 1e-3) / 1e9
    line = {
        "metric": "SP-KV decode tokens/s at 32K ctx; achieved HBM GB/s vs peak (surviving bytes)",
        "value": sp["tokens_per_s"], "unit": "tokens/s", "n_gpus": world, "steps": K, "warmup": Wm,
        "ms_per_step": sp["ms_per_step"], "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": cfg["name"], "layers": L, "batch": B, "q_heads": Hq, "kv_heads": Hkv,
                   "head_dim": 128, "context": cfg["T"], "window": W, "tau": TAU,
                   "keep_rates": ("beta%s" % (cfg["beta"],) if cfg["beta"] else cfg["rate"]),
                   "density": sp["density"], "kv_gb_per_step": sp["kv_gb_per_step"],
                   "l2": "inputs larger than L2 (K/V read per step >> 126 MB)" if sp["kv_gb_per_step"] > 0.5
                         else "working set smaller than L2: latency-bound case",
                   "cuda_graph": sp["graph"], "steps_per_graph": max(1, args.steps_per_graph),
                   "step_api": "2 L per-layer calls" if args.per_layer else "spkv_decode_stack (2 launches per step)",
                   "launch_overlap": ("SPKV_FLAG_OVERLAP" if CACHE_FLAGS[0] else "off (stream-ordered launches)") if args.per_layer
                                     else "not used (plain stream-ordered launches)", "parallelism": "replicas only" if world > 1 else "single GPU"},
        "clocks": sp["clocks"], "repeats": sp["repeats"],
        "gpu_launches": (2 * L if args.per_layer else 2) * K,
        # One step = one spkv_decode_stack call: the appends of every layer (one launch) and ONE
        # persistent decode kernel over all layers.  `achieved` is the algorithmic bytes of the step
        # over the step time (conservative: the step time also holds the append launch).  With
        # --per-layer the step is 2 L launches that overlap in SPKV_FLAG_OVERLAP mode, and `achieved`
        # is a launch's bytes over the average launch period.  A per-layer decode launch timed alone
        # (events around it, no graph, nothing overlapping) is reported beside it.
        "roofline": {"bound": "hbm", "kernel": "decode_tc_kernel" if args.per_layer else "decode_stack_kernel",
                     "achieved": in_step, "peak": hbm_peak,
                     "unit": "GB/s", "frac": in_step / hbm_peak, "peak_kind": f"of {peak_kind}",
                     "frac_of_nominal_8TBs": in_step / 8000.0,
                     "read_ceiling": {"gbs": sp.get("read_ceiling_gbs"),
                                      "frac": in_step / sp["read_ceiling_gbs"] if sp.get("read_ceiling_gbs") else None,
                                      "how": "spkv_stream_read over the cache arena: 32 KB bulk copies into shared "
                                             "memory, one block per SM, pages handed out by an atomic counter, "
                                             "nothing else (the measured peak above is a copy: half writes)"},
                     "bytes_per_launch": sp["launch_bytes"] * (1 if args.per_layer else L),
                     "bytes_per_layer": sp["launch_bytes"], "us_per_layer": sp["ms_per_step"] * 1e3 / L,
                     "how": "algorithmic K/V, Q, O bytes of a step over the step time measured with CUDA events "
                            "around the timed region (graph replay, append launch included)",
                     "per_layer_launch_alone": {"kernel": "decode_tc_kernel", "achieved": achieved,
                                                "frac": achieved / hbm_peak, "launch_us": sp["launch_s"] * 1e6,
                                                "how": "one layer's spkv_decode_attention launch bracketed by CUDA "
                                                       "events, no graph, nothing overlapping"},
                     "traffic": load_traffic(cfg["name"], sp["launch_bytes"] * (1 if args.per_layer else L))},
        "e2e": sp.get("e2e"),
    }
    if dn is not None:
        dn_ach = dn["launch_bytes"] / dn["launch_s"] / 1e9
        line["dense"] = {"tokens_per_s": dn["tokens_per_s"], "ms_per_step": dn["ms_per_step"],
                         "kv_gb_per_step": dn["kv_gb_per_step"],
                         "in_step_gbs": dn["kv_gb_per_step"] / dn["ms_per_step"] * 1e3,   # K/V bytes of a step over its time
                         "achieved_gbs": dn_ach,                                          # one per-layer launch, timed alone
                         "layers_measured": dn["layers_measured"],
                         "scaled_from_layer_subset": dn["layers_measured"] != L,
                         "frac": dn_ach / hbm_peak,
                         "speedup_spkv_over_dense": sp["tokens_per_s"] / dn["tokens_per_s"],
                         "cache_reduction": dn["kv_gb_per_step"] / sp["kv_gb_per_step"]}
    if world == 1 and not args.no_cpu:
        line["cpu_baseline"] = cpu_baseline(cfg, budget_s=args.cpu_seconds)
    print(json.dumps(line))


def run_config4(args):
    """Ragged serving batch: every step 8 sequences run an 8192-pair prefill chunk (score,
    compaction, tensor-core chunk attention) while 56 sequences decode one token each.  The dense
    K/V of this batch (~292 GB) does not fit one GPU, so the dense same-library comparison runs on
    8 of the 32 layers (layers are independent) and its step time is scaled by 4, flagged as such."""
    import numpy as np
    import torch

    from paper_2605_14037_b200 import build as spkv_build
    spkv_build.build()
    from paper_2605_14037_b200 import spkv, synth
    dev = torch.device("cuda:0")
    torch.cuda.set_device(dev)
    K, Wm = max(1, min(args.steps, 8)), 3
    hbm_peak, peak_kind = peaks()
    ev = lambda: torch.cuda.Event(enable_timing=True)

    def leg(dense, layers):
        cfg = dict(CONFIGS[4])
        if layers > 0:
            cfg["L"] = layers
        L, B, Hq, Hkv, C, NP = cfg["L"], cfg["B"], cfg["Hq"], cfg["Hkv"], cfg["chunk"], cfg["n_prefill"]
        rng = np.random.default_rng(4)
        cfg["t_list"] = rng.integers(cfg["t_min"], cfg["T"] + 1, size=B)
        cfg["grow"] = (K + Wm) * C + 64
        cfg["grow_list"] = [cfg["grow"] if b < NP else K + Wm + 64 for b in range(B)]
        cache, preds, rates, gen = build_workload(spkv, synth, torch, cfg, dev, dense, 0)
        if dense:
            rates = np.ones_like(rates)
        dec_ids = torch.arange(NP, B, dtype=torch.int32, device=dev)          # sequences 8..63 decode
        nd = B - NP
        rnd = lambda *shape: torch.randn(shape, generator=gen, device=dev).to(torch.bfloat16)
        xq, qd, kd, vd = rnd(L, nd, D_IN), rnd(L, nd, Hq, 128), rnd(L, nd, Hkv, 128), rnd(L, nd, Hkv, 128)
        xp, qp, kp, vp = rnd(C, D_IN), rnd(C, Hq, 128), rnd(C, Hkv, 128), rnd(C, Hkv, 128)
        out_d = torch.empty((L, nd, Hq, 128), dtype=torch.bfloat16, device=dev)
        out_p = torch.empty((C, Hq, 128), dtype=torch.bfloat16, device=dev)
        lg_p = torch.empty((C, Hkv), dtype=torch.float32, device=dev)

        def step(timers=None):
            a, b, c_ = ev(), ev(), ev()
            a.record()
            for l in range(L):
                for s in range(NP):                                           # sequences 0..7 prefill
                    cache.spkv_score(preds[l], xp, logits=lg_p)
                    cache.spkv_prefill(l, s, kp, vp, lg_p, q=qp, out=out_p)
            b.record()
            if args.per_layer:
                for l in range(L):
                    cache.spkv_score_append_evict(l, preds[l], dec_ids, xq[l], kd[l], vd[l])
                    cache.spkv_decode_attention(l, dec_ids, qd[l], out=out_d[l])
            else:                                                             # sequences 8..63 decode: all layers, two launches
                cache.spkv_decode_stack(preds, dec_ids, xq, qd, kd, vd, out=out_d)
            c_.record()
            if timers is not None:
                timers.append((a, b, c_))

        for _ in range(Wm):
            step()
        cache.check()
        lens0 = [cache.spkv_read_lengths(l)[0][:NP].astype(np.int64) for l in range(L)]
        torch.cuda.synchronize()
        timers, e0, e1 = [], ev(), ev()
        with ClockSampler(0) as clk:
            torch.cuda.nvtx.range_push("timed_region")      # lets a profiler pick out the timed launches
            e0.record()
            for _ in range(K):
                step(timers)
            e1.record()
            torch.cuda.synchronize()
            torch.cuda.nvtx.range_pop()
        cache.check()
        ms = e0.elapsed_time(e1)
        pre_ms = sum(a.elapsed_time(b) for a, b, _ in timers)
        dec_ms = sum(b.elapsed_time(c_) for _, b, c_ in timers)
        st1 = cache.spkv_cache_stats()
        # Useful prefill flops from the REALISED cache lengths.  A query sees the kept pairs of its unit
        # with position <= t - w, plus the w pairs of its window.  Over the timed region a unit's K * C
        # queries all see the n0 pairs kept before it, and a pair kept during it (n1 - n0 of them, from
        # the lengths read before and after) is seen by the queries that come at least w later -- half
        # of the region's queries on average, the gates being independent of position.
        lens1 = [cache.spkv_read_lengths(l)[0][:NP].astype(np.int64) for l in range(L)]
        keys = 0.0
        for l in range(L):
            n0, n1 = lens0[l].astype(np.float64), lens1[l].astype(np.float64)          # [NP, Hkv]
            keys += float(((n0 + 0.5 * (n1 - n0) + W) * (K * C) * (Hq // Hkv)).sum())
        # decode bytes: kept + window pairs of the 56 decoding sequences (their share of the resident bytes)
        lens_all = np.stack([cache.spkv_read_lengths(l)[0] for l in range(L)]).astype(np.int64)   # [L, B, Hkv]
        dec_bytes = float((lens_all[:, NP:].sum() + L * nd * Hkv * W) * 512 + L * nd * Hq * 512)
        res = dict(L=L, B=B, NP=NP, C=C, nd=nd, ms=ms, pre_ms=pre_ms, dec_ms=dec_ms, clocks=clk.result,
                   pre_tflops=keys * 4 * 128 / (pre_ms * 1e-3) / 1e12, dec_gbs=dec_bytes * K / (dec_ms * 1e-3) / 1e9,
                   density=st1.density_cache, resident_gb=st1.bytes_resident / 1e9, name=cfg["name"])
        cache.close()
        del cache
        torch.cuda.empty_cache()
        return res

    sp = leg(False, args.layers)
    dn = leg(True, 8) if args.dense and args.layers <= 0 else None
    L, B, NP, C, nd, ms = sp["L"], sp["B"], sp["NP"], sp["C"], sp["nd"], sp["ms"]
    tokens = K * (NP * C + nd)
    name = sp["name"] + (f"_{args.layers}layers_only" if args.layers > 0 else "")
    dense = None
    if dn is not None:
        f = L / dn["L"]     # layers are independent: the 8-layer step time scales with the layer count
        dense = {"layers_measured": dn["L"], "scaled_by": f, "ms_per_step": dn["ms"] / K * f,
                 "tokens_per_s": tokens / (dn["ms"] * 1e-3 * f), "resident_gb_measured": dn["resident_gb"],
                 "decode": {"ms_per_step": dn["dec_ms"] / K * f, "achieved_gbs": dn["dec_gbs"]},
                 "prefill": {"ms_per_step": dn["pre_ms"] / K * f, "useful_tflops": dn["pre_tflops"]},
                 "speedup": (dn["ms"] * f) / ms,
                 "note": "dense K/V of all 32 layers (~292 GB) does not fit one GPU: measured on "
                         f"{dn['L']} layers, times scaled by {f:g}"}
    line = {
        "metric": "SP-KV mixed prefill + decode tokens/s (ragged batch 64)", "value": tokens / (ms * 1e-3),
        "unit": "tokens/s", "n_gpus": 1, "steps": K, "warmup": Wm, "ms_per_step": ms / K,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": name, "layers": L, "batch": B, "prefilling": NP, "chunk": C,
                   "contexts": "uniform[4096, 65536], seeded", "keep_rates": "beta(0.5, 2.0)",
                   "density": sp["density"], "resident_gb": sp["resident_gb"],
                   "l2": "inputs larger than L2", "cuda_graph": False},
        "clocks": sp["clocks"], "gpu_launches": K * (L * NP * 6 + (2 * L if args.per_layer else 2)),
        "decode": {"tokens_per_s": K * nd / (sp["dec_ms"] * 1e-3), "ms_per_step": sp["dec_ms"] / K,
                   "achieved_gbs": sp["dec_gbs"], "frac_of_measured_hbm": sp["dec_gbs"] / hbm_peak},
        "prefill": {"tokens_per_s": K * NP * C / (sp["pre_ms"] * 1e-3), "ms_per_step": sp["pre_ms"] / K,
                    "useful_tflops": sp["pre_tflops"], "frac_of_sustained_bf16": sp["pre_tflops"] / 1356.9,
                    "kernel": "prefill_attn_tc5x2h_kernel (tcgen05, P.V in fp16)"},
        "roofline": {"bound": "tensor", "kernel": "prefill_attn_tc5x2h_kernel", "achieved": sp["pre_tflops"],
                     "peak": 1356.9, "unit": "TFLOP/s", "frac": sp["pre_tflops"] / 1356.9,
                     "peak_kind": "of measured (sustained)", "traffic": None},
        "e2e": None, "dense": dense,
    }
    print(json.dumps(line))



def run_softgate(args):
    """Soft-gated whole-sequence forward (the paper's training-time attention, Eq. 6) on one
    sequence of --softgate-T tokens with the head shape of the 8 B model: useful TFLOP/s against the
    sustained bf16 peak, and beside it the hard-gated forward of the same sequence through
    spkv_prefill (kept pairs compacted, so its work shrinks with the density)."""
    import numpy as np
    import torch

    from paper_2605_14037_b200 import build as spkv_build
    spkv_build.build()
    from paper_2605_14037_b200 import spkv
    dev = torch.device("cuda:0")
    torch.cuda.set_device(dev)
    T, Hq, Hkv = args.softgate_T, 32, 8
    gen = torch.Generator(device=dev)
    gen.manual_seed(0)
    rnd = lambda *shape: torch.randn(shape, generator=gen, device=dev).to(torch.bfloat16)
    q, k, v = rnd(T, Hq, 128), rnd(T, Hkv, 128), rnd(T, Hkv, 128)
    # gates: logits N(b_h, 1) with b_h such that head h would keep a fraction r_h at tau = 0.5
    rates = np.random.default_rng(0).beta(0.5, 2.0, size=Hkv).clip(0.01, 0.99)
    from statistics import NormalDist
    bias = torch.tensor([NormalDist().inv_cdf(float(r)) for r in rates], dtype=torch.float32, device=dev)
    logits = torch.randn((T, Hkv), generator=gen, device=dev) + bias
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            peak, peak_kind = float(json.load(f)["bf16_tflops_sustained"]), "of measured (sustained)"
    except Exception:
        peak, peak_kind = 1400.0, "of fallback (sustained)"
    ev = lambda: torch.cuda.Event(enable_timing=True)

    def timed(fn):
        for _ in range(max(3, args.warmup)):
            fn()
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        while time.perf_counter() - t0 < args.settle_seconds:
            fn()
            torch.cuda.synchronize()
        times = []
        with ClockSampler(0) as clk:
            while len(times) < 5 or (sum(times) < 2000.0 and len(times) < 200):
                a, b = ev(), ev()
                a.record(); fn(); b.record()
                torch.cuda.synchronize()
                times.append(a.elapsed_time(b))
        return median(times), times, clk.result

    status = torch.zeros(1, dtype=torch.int32, device=dev)
    soft_out = torch.empty_like(q)
    soft_ms, soft_all, clocks = timed(lambda: spkv.spkv_softgate_forward(q, k, v, logits, window=W, out=soft_out,
                                                                       status=status))
    assert int(status.item()) == 0, "a bounded wait ran out in the soft-gated forward"
    flops = 4.0 * 128 * Hq * T * (T + 1) / 2
    # hard-gated forward of the same tokens: spkv_prefill on an empty sequence with C = T
    kept = int((logits >= 0).sum().item())
    cache = spkv.Cache(n_layers=1, max_seqs=1, n_q_heads=Hq, n_kv_heads=Hkv, max_context=T + 64,
                       pool_pages=kept // 64 + 2 * Hkv + 8, window=W, tau=TAU, device=dev)
    out = torch.empty_like(q)

    def hard():
        cache.spkv_cache_reset_seq(0)
        cache.spkv_prefill(0, 0, k, v, logits, q=q, out=out)

    hard_ms, _, _ = timed(hard)
    cache.check()
    st = cache.spkv_cache_stats()
    line = {
        "metric": "soft-gated whole-sequence forward (Eq. 6), useful TFLOP/s", "value": flops / (soft_ms * 1e-3) / 1e12,
        "unit": "TFLOP/s", "n_gpus": 1, "steps": len(soft_all), "warmup": max(3, args.warmup), "ms_per_step": soft_ms,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": f"softgate_forward_T{T}_q{Hq}_kv{Hkv}", "tokens": T, "q_heads": Hq, "kv_heads": Hkv,
                   "window": W, "alpha": 0.0, "l2": "q and out (2 x %.0f MB) stream from HBM; K/V pages are re-read from L2" % (T * Hq * 256 / 1e6)},
        "clocks": clocks,
        "repeats": {"n": len(soft_all), "min": min(soft_all), "median": soft_ms, "max": max(soft_all), "unit": "ms"},
        "gpu_launches": 3 + (1 if T < 4000 else 0),
        "roofline": {"bound": "tensor", "kernel": "prefill_attn_tc5x2h_kernel<.., soft>", "achieved": flops / (soft_ms * 1e-3) / 1e12,
                     "peak": peak, "unit": "TFLOP/s", "frac": flops / (soft_ms * 1e-3) / 1e12 / peak, "peak_kind": peak_kind,
                     "flops_per_launch": flops, "traffic": None},
        "hard_gated": {"ms": hard_ms, "density": st.density_cache, "speedup_over_soft": soft_ms / hard_ms,
                       "how": "spkv_prefill of the same tokens on an empty sequence, tau = 0.5 (reset + prefill timed)"},
        "e2e": None,
    }
    print(json.dumps(line))


def load_traffic(workload, launch_bytes):
    """DRAM bytes per decode launch from the committed ncu summary, if there is one."""
    try:
        with open(os.path.join(ROOT, "profiles", "decode_traffic.json")) as f:
            t = json.load(f)
        # measured on a smaller case; traffic grows in proportion to the algorithmic bytes
        return t["dram_bytes_per_launch"] / t["algorithmic_bytes_per_launch"] * launch_bytes
    except Exception:
        return None


def cpu_baseline(cfg, budget_s=20.0, steps=None):
    """The oracle, as it stands, on a bounded sample: the units of `n_seq` sequences of one
    layer at the configured context, a few decode steps; scaled to whole-job tokens/s."""
    import numpy as np

    import oracle
    from paper_2605_14037_b200 import synth
    rng = np.random.default_rng(1)
    Hq, Hkv, T, B, L = cfg["Hq"], cfg["Hkv"], cfg["T"], cfg["B"], cfg["L"]
    G = Hq // Hkv
    n_seq = 2 if B >= 2 else 1
    rates = (np.full(Hkv, cfg["rate"]) if cfg["beta"] is None
             else synth.keep_rates(np.random.default_rng(0), L, Hkv, *cfg["beta"])[0])
    units = [oracle.Unit(W, 128) for _ in range(n_seq * Hkv)]
    Tb = min(T, 32768)        # state built with min(T, 32768) pairs per unit to bound the set-up
    for i, u in enumerate(units):
        k, v = synth.normal_bf16(rng, (Tb, 128)), synth.normal_bf16(rng, (Tb, 128))
        lg = synth.logits_with_keep_rate(rng, (Tb,), float(rates[i % Hkv]) * T / Tb if Tb < T else float(rates[i % Hkv]), 0.0)
        u.prefill(k, v, lg, 0.0)
    n = len(units)
    scale = 1.0 / math.sqrt(128)
    t_used, done = 0.0, 0
    while (steps is None and t_used < budget_s and done < 512) or (steps is not None and done < steps):
        k, v = synth.normal_bf16(rng, (n, 128)), synth.normal_bf16(rng, (n, 128))
        q = synth.normal_bf16(rng, (n, G, 128))
        lg = rng.standard_normal(n).astype(np.float32)
        t0 = time.perf_counter()
        oracle.step_batch(units, k, v, lg, 0.0, q, scale)
        t_used += time.perf_counter() - t0
        done += 1
    per_step_full = (t_used / done) * (L * B * Hkv / n)
    kept = sum(len(u) for u in units)
    density = kept / max(1, sum(max(Tb + done - W, 0) for _ in units))
    return {"value": B / per_step_full, "unit": "tokens/s", "cores": oracle.threads(), "kind": "oracle",
            "sample": f"{n} units ({n_seq} sequences x {Hkv} KV heads of layer 0, context {T}), "
                      f"{done} decode steps (append + attend), scaled by units to {L} layers x batch {B}",
            "sample_density": density, "sample_kept_pairs": kept,
            "seconds": t_used}


def run_reference(args):
    """Reference arm = the CPU oracle on a bounded sample per step (rank 0 only)."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    cfg = CONFIGS[args.config]
    steps = max(1, min(args.steps, 16))
    cb = cpu_baseline(cfg, steps=steps + min(args.warmup, 2))
    L, B = cfg["L"], cfg["B"]
    line = {
        "impl": "reference",
        "metric": "SP-KV decode tokens/s at 32K ctx; achieved HBM GB/s vs peak (surviving bytes)",
        "value": cb["value"], "unit": "tokens/s", "n_gpus": int(os.environ.get("WORLD_SIZE", "1")),
        "steps": steps, "warmup": min(args.warmup, 2), "ms_per_step": 1e3 * B / cb["value"],
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic",
        "config": {"workload": cfg["name"], "layers": L, "batch": B, "context": cfg["T"], "window": W,
                   "tau": TAU},
        "cpu_baseline": {k: cb[k] for k in ("value", "unit", "cores", "kind", "sample", "sample_density")},
        "e2e": {"value": cb["value"], "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))


def replica_launch_command(n, argv, port=None):
    """The torchrun command line that runs this script as `n` replicas on one node."""
    if port is None:
        import socket
        with socket.socket() as sock:
            sock.bind(("127.0.0.1", 0))
            port = sock.getsockname()[1]
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(n),
            "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__), *argv]


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=256)
    ap.add_argument("--warmup", type=int, default=8)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=2, choices=sorted(CONFIGS))
    ap.add_argument("--no-graph", action="store_true", help="launch every kernel from the host")
    ap.add_argument("--no-dense", dest="dense", action="store_false", help="skip the dense baseline")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU-oracle baseline")
    ap.add_argument("--e2e-steps", type=int, default=32)
    ap.add_argument("--layers", type=int, default=0,
                    help="override the layer count (small profiling captures only; not a bench line)")
    ap.add_argument("--cpu-seconds", type=float, default=15.0)
    ap.add_argument("--settle-seconds", type=float, default=1.0,
                    help="untimed replay of the timed region before the first repeat (clocks settle under load)")
    ap.add_argument("--steps-per-graph", type=int, default=0,
                    help="steps captured in one CUDA graph (default: 1, and 16 for the tiny config 1, whose "
                         "step is shorter than the time the host needs to replay a graph)")
    ap.add_argument("--per-layer", action="store_true",
                    help="time the step as 2 L per-layer calls (spkv_score_append_evict, spkv_decode_attention) "
                         "instead of one spkv_decode_stack call (comparison run, not the bench line)")
    ap.add_argument("--stream-ordered", action="store_true",
                    help="create the cache without SPKV_FLAG_OVERLAP: every launch waits for the previous one, as "
                         "in a model whose layers depend on each other (comparison run, not the bench line)")
    ap.add_argument("--softgate-T", type=int, default=0,
                    help="measure the soft-gated whole-sequence forward on this many tokens instead (not the bench line)")
    ap.add_argument("--sweep-tau", default="",
                    help="comma-separated thresholds: one decode measurement per tau, nothing else")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # replicas only: N independent copies of the workload, one process per GPU; started here
        # the way a launcher would start them
        sys.exit(subprocess.call(replica_launch_command(args.gpus, sys.argv[1:])))
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3
    if args.steps_per_graph <= 0:
        args.steps_per_graph = 16 if args.config == 1 else 1
    if args.stream_ordered:
        CACHE_FLAGS[0] = 0
    if args.impl == "reference":
        run_reference(args)
    elif args.softgate_T > 0:
        if int(os.environ.get("RANK", "0")) == 0:
            run_softgate(args)
    elif args.config == 4:
        if int(os.environ.get("RANK", "0")) == 0:
            run_config4(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
