#!/usr/bin/env python
"""Benchmark of the compressed-KV streaming attention step.

A "step" is one frame through the whole hot path for all 24 layers: fused
dequant + attention, importance scores, top-k prune, quantise + pack
(configuration 2: 16 heads x 64, 1374 tokens/frame, budget 21984 tokens per
layer, 4-bit KV, bf16), in steady state (the cache is filled to its budget by
untimed prefill frames first).  Prints ONE JSON line.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]
  python bench.py --config 3      long horizon: 24 layers x 1000 frames, budget 10992, 2-bit, drifting means;
                                  per-frame latency p50 / p99 over frames 100-1000, its slope, bytes at start and end
  python bench.py --config 4      one layer: budgets {4096, 16384, 65536} x bits {2, 4, 8} x frames {32, 256}, and the
                                  uncompressed bf16 cache grown to a share of the free memory, timed at checkpoints
  python bench.py --batch B       B independent streams stepped together (xsv_step_batch) against the same B streams
                                  stepped one after the other, at the benchmark's budget and at a budget of 4096

N > 1 (under torchrun): the path does not shard -- every rank runs an independent
replica (its own stream of frames); value = all ranks' frames / max-over-ranks time.
--impl reference: the CPU oracle, as it stands, on the host cores (rank 0 only).
"""
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

H, D, F, LAYERS, L_MAX, BITS = 16, 64, 1374, 24, 21984, 4
PREFILL = 16                 # frames that fill the cache to the budget (untimed set-up)
TORCH_DTYPE = "bfloat16"     # input type of the generated frames; "float16" only in sweep cases (--dtype fp16)
POOL = 4                     # distinct frames per layer, cycled
METRIC = "frames/s of compressed-KV causal attention step (24 layers)"
WORKLOAD = ("config2: 24 layers x (16 heads x 64), 1374 tokens/frame, budget 21984 tokens/layer, 4-bit KV, bf16, "
            "steady state after a 16-frame prefill")


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        m = json.load(open(p))
        return dict(tflops=float(m.get("bf16_tflops_sustained", m.get("bf16_tflops"))),
                    tflops_burst=float(m.get("bf16_tflops", m.get("bf16_tflops_sustained"))), hbm=float(m["hbm_gbs"]),
                    source="measured (MEASURED_PEAKS.json, sustained bf16)")
    return dict(tflops=1400.0, tflops_burst=1590.0, hbm=6650.0, source="fallback (no MEASURED_PEAKS.json)")


TRAFFIC_FILE = os.path.join("profiles", "attention_config2_traffic.txt")


def attn_traffic():
    """DRAM bytes per attention launch from the committed ncu summary (with the capture it came from), if any."""
    out = {"bytes": None, "source": None}
    try:
        for line in open(os.path.join(ROOT, TRAFFIC_FILE)):
            if line.startswith("traffic_bytes_per_launch:"):
                out["bytes"] = float(line.split(":")[1])
            elif line.startswith("captured:"):
                out["source"] = f"{TRAFFIC_FILE} ({line.split(':', 1)[1].strip()})"
    except OSError:
        pass
    return out


class ClockSampler:
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.rows, self.proc, self.index = [], None, index

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-i", str(self.index), "-lms", "100"], stdout=subprocess.PIPE, text=True)
            self.th = threading.Thread(target=self._read, daemon=True)
            self.th.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([f.strip() for f in line.split(",")])

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.12)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
            except (ValueError, IndexError):
                continue
            for n, v in zip(names, r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def gen_frames(torch, dev, layers, pool, seed):
    """Synthetic device-resident inputs with the recipe of the parity streams: Q, V ~ N(0,1);
    K = (N(0,1) + mu) * m, mu ~ N(0, 0.5^2) per (layer, head, channel), m = 10 on 4 channels per head."""
    g = torch.Generator(device=dev)
    g.manual_seed(seed)
    frames = []
    for l in range(layers):
        mu = torch.randn(H, 1, D, device=dev, generator=g) * 0.5
        m = torch.ones(H, 1, D, device=dev)
        for h in range(H):
            idx = torch.randperm(D, device=dev, generator=g)[:4]
            m[h, 0, idx] = 10.0
        per = []
        for p in range(pool):
            dt = getattr(torch, TORCH_DTYPE)
            q = torch.randn(H, F, D, device=dev, generator=g).to(dt)
            k = ((torch.randn(H, F, D, device=dev, generator=g) + mu) * m).to(dt)
            v = torch.randn(H, F, D, device=dev, generator=g).to(dt)
            per.append((q.contiguous(), k.contiguous(), v.contiguous()))
        frames.append(per)
    return frames


def oracle_layer_step_seconds(repeats=1):
    """Time one steady-state layer-step of the CPU oracle (config-2 shape): 1/24 of a frame."""
    import numpy as np
    from oracle import xsv_oracle as orc
    from paper_2602_21780_b200 import synth
    st = synth.Stream(H=H, d=D, F=F, dtype="bf16")
    ref = orc.LayerCache(H, D, L_MAX, BITS)
    # a full cache built directly with the oracle's quantiser from 16 synthetic frames
    Ks, Vs = [], []
    for t in range(PREFILL):
        _, k, v = st.frame(t)
        Ks.append(k); Vs.append(v)
    K = np.concatenate(Ks, axis=1); V = np.concatenate(Vs, axis=1)
    T = K.shape[1]
    ng = -(-T // 64)
    pad = ng * 64 - T
    Kp = np.concatenate([K, np.repeat(K[:, -1:, :], pad, axis=1)], axis=1) if pad else K
    kc, ks, kz = orc.quantize_groups(Kp.reshape(H, ng, 64, D).transpose(0, 1, 3, 2), BITS)
    kc = kc.transpose(0, 1, 3, 2).reshape(H, ng * 64, D)[:, :T]
    vc, vs, vz = orc.quantize_groups(V.reshape(H, T, 1, D), BITS)
    ref.load_state(PREFILL, F, kc, ks, kz, vc.reshape(H, T, D), vs, vz, np.arange(T))
    best = None
    for r in range(repeats):
        q, k, v = st.frame(PREFILL + r)
        t0 = time.perf_counter()
        ref.step(q, k, v)
        dt = time.perf_counter() - t0
        best = dt if best is None else min(best, dt)
    return best


def oracle_config_times(max_seconds=60.0):
    """One steady-state layer-step of the oracle per configuration, on all BLAS threads and on one thread.
    The one-thread run takes a sample of the heads (scaled up by the head ratio; heads are independent in every
    step of the oracle except the head mean of the scores, which is a small share) so that it stays bounded."""
    import numpy as np
    from oracle import xsv_oracle as orc
    from paper_2602_21780_b200 import synth
    try:
        from threadpoolctl import threadpool_limits
    except Exception:
        threadpool_limits = None
    out = {}
    t_begin = time.perf_counter()
    shapes = {"config0": (16, 261, 1044, 4, "fp16", 1), "config1/2": (16, F, 21984, 4, "bf16", 1),
              "config3": (16, F, 10992, 2, "bf16", 1)}
    for name, (Hc, Fc, Lc, bc, dt, _) in shapes.items():
        entry = {}
        for threads, heads in (("all", Hc), ("one", 2)):
            if time.perf_counter() - t_begin > max_seconds:
                break
            st = synth.Stream(H=heads, d=D, F=Fc, dtype=dt)
            ref = orc.LayerCache(heads, D, Lc, bc)
            n_pre = Lc // Fc
            pre = [st.frame(t) for t in range(n_pre)]
            K, V = np.concatenate([f[1] for f in pre], axis=1), np.concatenate([f[2] for f in pre], axis=1)
            T = K.shape[1]
            ng = -(-T // 64)
            pad = ng * 64 - T
            Kp = np.concatenate([K, np.repeat(K[:, -1:, :], pad, axis=1)], axis=1) if pad else K
            kc, ks, kz = orc.quantize_groups(Kp.reshape(heads, ng, 64, D).transpose(0, 1, 3, 2), bc)
            kc = kc.transpose(0, 1, 3, 2).reshape(heads, ng * 64, D)[:, :T]
            vc, vs, vz = orc.quantize_groups(V.reshape(heads, T, 1, D), bc)
            ref.load_state(n_pre, Fc, kc, ks, kz, vc.reshape(heads, T, D), vs, vz, np.arange(T))
            q, k, v = st.frame(n_pre)
            ctx = threadpool_limits(limits=1) if (threads == "one" and threadpool_limits) else None
            t0 = time.perf_counter()
            if ctx:
                with ctx:
                    ref.step(q, k, v)
            else:
                ref.step(q, k, v)
            dt_s = (time.perf_counter() - t0) * (Hc / heads)
            entry[("all_threads_s" if threads == "all" else "one_thread_s")] = dt_s
            if threads == "one":
                entry["one_thread_sample"] = f"{heads} of {Hc} heads, scaled by {Hc // heads}"
        out[name] = entry
    return out


def replica_seed(base, rank):
    """Every rank streams its own frames: the path does not shard, ranks are independent replicas."""
    return base + rank


def job_throughput(ms_local, steps, world, dist=None, device=None):
    """Whole-job frames/s of `world` independent replicas: all ranks' frames over the slowest rank's time.
    Returns (frames_per_s, ms_max).  `dist` is torch.distributed (initialised) when world > 1."""
    ms = float(ms_local)
    if world > 1:
        import torch
        t = torch.tensor([ms], dtype=torch.float64, device=device)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms = float(t.item())
    return world * steps / (ms * 1e-3), ms


def blas_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [i.get("num_threads", 1) for i in threadpool_info() if i.get("user_api") == "blas"]
        return max(n) if n else os.cpu_count()
    except Exception:
        return os.cpu_count()


def run_reference(args, rank):
    if rank != 0:
        return
    import numpy  # noqa: F401  (loads the BLAS whose threads are reported)
    for _ in range(args.warmup and 1):
        oracle_layer_step_seconds()
    times = [oracle_layer_step_seconds() for _ in range(max(1, min(args.steps, 3)))]
    sec = sum(times) / len(times)
    fps = 1.0 / (LAYERS * sec)
    cores = blas_threads()
    line = {"impl": "reference", "metric": METRIC, "value": fps, "unit": "frames/s", "n_gpus": args.gpus,
            "steps": len(times), "warmup": 1 if args.warmup else 0, "ms_per_step": LAYERS * sec * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": {"workload": WORKLOAD},
            "cpu_baseline": {"value": fps, "unit": "frames/s", "cores": cores, "kind": "oracle",
                             "sample": "one steady-state layer-step (T_c=21984) per timed step = 1/24 frame, "
                                       "extrapolated x24"},
            "e2e": {"value": fps, "unit": "frames/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


class DriftFeed:
    """Per-layer inputs of configuration 3, drawn on the device: the recipe of gen_frames plus per-channel means of
    Q, K and V that follow an AR(1) process (rho = 0.95, stationary standard deviation 0.5), advanced frame by frame."""

    def __init__(self, torch, dev, layers, seed, rho=0.95):
        self.torch, self.dev, self.layers, self.rho = torch, dev, layers, rho
        self.g = torch.Generator(device=dev)
        self.g.manual_seed(seed)
        self.mu = torch.randn(layers, H, 1, D, device=dev, generator=self.g) * 0.5
        self.m = torch.ones(layers, H, 1, D, device=dev)
        for l in range(layers):
            for h in range(H):
                self.m[l, h, 0, torch.randperm(D, device=dev, generator=self.g)[:4]] = 10.0
        self.drift = [torch.randn(layers, H, 1, D, device=dev, generator=self.g) * 0.5 for _ in range(3)]
        self.innov = (1.0 - rho * rho) ** 0.5 * 0.5

    def frame(self):
        """(Q, K, V), each [layers, H, F, D] bf16, for the next frame."""
        t = self.torch
        for i in range(3):
            self.drift[i] = self.rho * self.drift[i] + self.innov * t.randn(self.layers, H, 1, D, device=self.dev, generator=self.g)
        shp = (self.layers, H, F, D)
        q = (t.randn(shp, device=self.dev, generator=self.g) + self.drift[0]).to(t.bfloat16)
        k = ((t.randn(shp, device=self.dev, generator=self.g) + self.mu + self.drift[1]) * self.m).to(t.bfloat16)
        v = (t.randn(shp, device=self.dev, generator=self.g) + self.drift[2]).to(t.bfloat16)
        return q, k, v


def run_config3(args, torch, binding, dev, stream):
    """24 layers x 1000 frames, budget 10992, 2-bit, drifting means: frames/s, per-frame latency distribution over
    frames 100-1000 and its slope, device bytes at the start of the steady state and at the end."""
    layers, frames, L, bits = args.layers, args.frames or 1000, 10992, 2
    feed = DriftFeed(torch, dev, layers, seed=20260221 + 3)
    out = torch.empty(H, F, D, device=dev, dtype=torch.bfloat16)
    cache = binding.Cache(layers, H, D, L, bits)
    cache.set_deferred_join(True)
    sp = stream.cuda_stream
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(frames)]
    bytes_at = {}
    sampler = ClockSampler(dev.index or 0)
    sampler.start()
    launches0 = binding.kernel_launches()
    t_wall = time.perf_counter()
    for f in range(frames):
        q, k, v = feed.frame()                           # drawn before the frame's clock starts
        ev[f][0].record(stream)
        for l in range(layers):
            rc = cache.step_raw(l, q[l].data_ptr(), k[l].data_ptr(), v[l].data_ptr(), F, binding.BF16, out.data_ptr(), sp)
            if rc != 0:
                raise RuntimeError(f"xsv_step failed: status {rc}")
        cache.join(stream)
        ev[f][1].record(stream)
        if f in (9, 99, frames - 1):
            bytes_at[f + 1] = cache.bytes()
        if f % 50 == 49:
            torch.cuda.synchronize()                     # bounds the queue of pending launches and inputs
    torch.cuda.synchronize()
    wall = time.perf_counter() - t_wall
    clocks = sampler.stop()
    assert cache.status() == 0, "device status word set"
    ms = [a.elapsed_time(b) for a, b in ev]
    lo = min(100, frames // 2)
    steady = sorted(ms[lo:])
    n = len(steady)
    xs = list(range(lo, frames))
    mx, my = sum(xs) / n, sum(ms[lo:]) / n
    slope = sum((x - mx) * (y - my) for x, y in zip(xs, ms[lo:])) / max(1e-9, sum((x - mx) ** 2 for x in xs))
    total_ms = sum(ms[lo:])
    line = {"metric": "frames/s of compressed-KV causal attention step (24 layers), long horizon", "value": n / (total_ms * 1e-3),
            "unit": "frames/s", "n_gpus": 1, "steps": n, "warmup": lo, "ms_per_step": total_ms / n, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": f"config3: {layers} layers x (16 heads x 64), 1374 tokens/frame, {frames} frames, budget {L} "
                                   f"tokens/layer, {bits}-bit KV, bf16, AR(1) drift (rho 0.95) of the per-channel means of Q, K, V "
                                   "drawn on the device", "deferred_join": True,
                       "l2": "each frame touches 203 MB of fresh inputs + 203 MB of cache (> 126 MB L2); no flush"},
            "clocks": clocks, "gpu_launches": binding.kernel_launches() - launches0,
            "latency_ms_per_frame": {"frames": f"{lo}-{frames}", "p50": steady[n // 2], "p99": steady[min(n - 1, int(n * 0.99))],
                                     "min": steady[0], "max": steady[-1], "slope_ms_per_frame": slope,
                                     "slope_over_run_fraction_of_p50": slope * n / steady[n // 2]},
            "cache_bytes_at_frame": bytes_at, "cache_bytes_constant": len(set(bytes_at.values())) == 1,
            "kv_bytes_per_layer": cache.layer_kv_bytes(0), "cache_len": cache.len(0), "wall_s_incl_input_generation": wall}
    cache.destroy()
    print(json.dumps(line), flush=True)


def run_config4(args, torch, binding, dev, stream):
    """One layer at paper shape: the budget x bits x frames sweep, then the uncompressed bf16 cache grown towards a
    share of the free device memory and timed at checkpoints (frames between checkpoints are appended without their
    attention, so the run does not pay for every step before a checkpoint)."""
    sp = stream.cuda_stream
    frames_pool = gen_frames(torch, dev, 1, POOL, seed=20260221 + 4)[0]
    out = torch.empty(H, F, D, device=dev, dtype=torch.bfloat16)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    peaks = measured_peaks()
    rows = []
    for budget in (4096, 16384, 65536):
        for bits in (2, 4, 8):
            for n_frames in (32, 256):
                c = binding.Cache(1, H, D, budget, bits)
                c.set_deferred_join(True)
                times = []
                for f in range(n_frames):
                    q, k, v = frames_pool[f % POOL]
                    timed = f >= n_frames - 8                       # the last 8 frames of the run
                    if timed:
                        e0.record(stream)
                    rc = c.step_raw(0, q.data_ptr(), k.data_ptr(), v.data_ptr(), F, binding.BF16, out.data_ptr(), sp)
                    if rc != 0:
                        raise RuntimeError(f"xsv_step failed: status {rc}")
                    if timed:
                        c.join(stream)
                        e1.record(stream)
                        torch.cuda.synchronize()
                        times.append(e0.elapsed_time(e1))
                assert c.status() == 0
                ms = sorted(times)[len(times) // 2]
                T = c.len(0) + F
                rows.append({"budget": budget, "bits": bits, "frames": n_frames, "cache_len": c.len(0),
                             "pruning": c.len(0) >= max(budget, 2 * F) and n_frames * F > budget,
                             "ms_per_layer_step": ms, "layer_steps_per_s": 1e3 / ms,
                             "attention_tflops_if_all_time_were_attention": 4.0 * F * T * D * H / (ms * 1e-3) / 1e12,
                             "kv_bytes": c.layer_kv_bytes(0), "device_bytes": c.bytes()})
                c.destroy()
    # ---- the uncompressed reference point: no pruning, no quantisation, cache as large as the memory allows
    free, total = torch.cuda.mem_get_info()
    tok_bytes = 2 * H * D * 2                                        # K and V rows, bf16
    limit = min(0.85 * free, args.max_gb * 1e9)
    max_frames = int((limit - 2e9) // (tok_bytes * F))               # 2 GB kept for scratch and inputs
    checkpoints = [n for n in (32, 256, 1000, 4000, 16000) if n < max_frames] + [max_frames]
    c = binding.Cache(1, H, D, 0, 16)
    c.set_options(max_frame_tokens=F, max_cache_tokens=(max_frames + 2) * F)
    grown = []
    done = 0
    for cp in checkpoints:
        while done < cp - 1:                                         # bulk append up to the frame before the checkpoint
            q, k, v = frames_pool[done % POOL]
            c.append(0, k, v, stream)
            done += 1
        torch.cuda.synchronize()
        times = []
        for r in range(3):                                           # the checkpoint's own step, timed; repeated on
            q, k, v = frames_pool[(done + r) % POOL]                 # the following frames (the cache grows by three)
            e0.record(stream)
            rc = c.step_raw(0, q.data_ptr(), k.data_ptr(), v.data_ptr(), F, binding.BF16, out.data_ptr(), sp)
            e1.record(stream)
            torch.cuda.synchronize()
            if rc != 0:
                raise RuntimeError(f"xsv_step failed: status {rc}")
            times.append(e0.elapsed_time(e1))
        done += 3
        ms = sorted(times)[1]
        T = done * F
        grown.append({"frames": done, "cache_tokens": c.len(0), "kv_bytes": c.layer_kv_bytes(0), "ms_per_layer_step": ms,
                      "attention_tflops": 4.0 * F * T * D * H / (ms * 1e-3) / 1e12,
                      "frac_of_bf16_sustained": 4.0 * F * T * D * H / (ms * 1e-3) / 1e12 / peaks["tflops"]})
    assert c.status() == 0
    dev_bytes = c.bytes()
    c.destroy()
    line = {"metric": "one-layer sweep: ms per layer-step over budget x bits x frames; uncompressed bf16 cache growth",
            "value": None, "unit": "ms per layer-step", "n_gpus": 1, "higher_is_better": False, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": "config4: one layer, 16 heads x 64, 1374 tokens/frame, bf16; median of the last 8 frames of "
                                   "each run; uncompressed run: bits = 16, no budget, frames between checkpoints appended "
                                   "without attention (xsv_cache_append)",
                       "uncompressed_memory_limit_bytes": limit, "free_bytes": free, "total_bytes": total},
            "sweep": rows, "uncompressed": grown, "uncompressed_device_bytes": dev_bytes}
    print(json.dumps(line), flush=True)


def run_batch_bench(args, torch, binding, dev, stream):
    """B independent streams, `layers` layers each, in steady state: frames/s of all streams together when every
    layer-step is one xsv_step_batch call over the B streams, against the same streams stepped one after the other."""
    B, layers, n_frames = args.batch, min(args.layers, 4), max(args.steps, 10)
    sp = stream.cuda_stream
    pools = [gen_frames(torch, dev, layers, 2, seed=20260221 + 10 + b) for b in range(B)]
    outs = [torch.empty(H, F, D, device=dev, dtype=torch.bfloat16) for _ in range(B)]
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    rows = []
    for budget in (L_MAX, 4096):
        res = {}
        for mode in ("sequential", "batched"):
            caches = [binding.Cache(layers, H, D, budget, BITS) for _ in range(B)]
            for c in caches:
                c.set_deferred_join(True)        # as the benchmark: the inputs stay untouched, joined before the clock stops

            def frame(f):
                if mode == "sequential":
                    for b in range(B):
                        for l in range(layers):
                            q, k, v = pools[b][l][f % 2]
                            rc = caches[b].step_raw(l, q.data_ptr(), k.data_ptr(), v.data_ptr(), F, binding.BF16, outs[b].data_ptr(), sp)
                            if rc != 0:
                                raise RuntimeError(f"xsv_step failed: status {rc}")
                else:
                    for l in range(layers):
                        qkv = [pools[b][l][f % 2] for b in range(B)]
                        binding.step_batch(caches, l, [x[0] for x in qkv], [x[1] for x in qkv], [x[2] for x in qkv], outs, stream)

            prefill = budget // F + 3
            for f in range(prefill):
                frame(f)
            torch.cuda.synchronize()
            e0.record(stream)
            for f in range(n_frames):
                frame(prefill + f)
            for c in caches:
                c.join(stream)
            e1.record(stream)
            torch.cuda.synchronize()
            ms = e0.elapsed_time(e1)
            for c in caches:
                assert c.status() == 0
                c.destroy()
            res[mode] = B * n_frames / (ms * 1e-3)          # frames of all streams per second (of a `layers`-layer stack)
        rows.append({"budget": budget, "streams": B, "layers": layers, "frames_per_s_sequential": res["sequential"],
                     "frames_per_s_batched": res["batched"], "ratio": res["batched"] / res["sequential"]})
    line = {"metric": f"frames/s of {B} streams stepped together vs one after the other ({layers}-layer stacks)", "value": rows[0]["ratio"],
            "unit": "ratio batched / sequential at the benchmark's budget", "n_gpus": 1, "steps": n_frames, "higher_is_better": True,
            "dtype": "bf16", "data": "synthetic",
            "config": {"workload": f"{B} streams x {layers} layers x (16 heads x 64), 1374 tokens/frame, {BITS}-bit KV, bf16, steady state"},
            "rows": rows}
    print(json.dumps(line), flush=True)


def main():
    global LAYERS, WORKLOAD, L_MAX, BITS, PREFILL, TORCH_DTYPE
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=40)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="xsv", choices=["xsv", "reference"])
    ap.add_argument("--attn", default="auto", choices=["auto", "mma", "tc5"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--layers", type=int, default=LAYERS,
                    help="layers in the stack (default 24 = the benchmark; fewer only for profiling a small case)")
    ap.add_argument("--budget-frames", type=int, default=L_MAX // F,
                    help="cache budget in frames (default 16 = the benchmark; other values: the cache-length sweep)")
    ap.add_argument("--bits", type=int, default=BITS, choices=[2, 4, 8, 16],
                    help="bits per cached element (default 4 = the benchmark; 16 = quantisation off, pruning only)")
    ap.add_argument("--dtype", default="bf16", choices=["bf16", "fp16"],
                    help="input type (default bf16 = the benchmark; fp16: a sweep case, e.g. with --bits 16 the copy-engine feed)")
    ap.add_argument("--config", type=int, default=2, choices=[2, 3, 4],
                    help="2: the benchmark (default); 3: the long-horizon run; 4: the one-layer sweep and the uncompressed cache")
    ap.add_argument("--frames", type=int, default=0, help="--config 3: frames to stream (default 1000)")
    ap.add_argument("--batch", type=int, default=0, help="streams stepped together (2-8): the batched-against-sequential comparison")
    ap.add_argument("--max-gb", type=float, default=120.0,
                    help="--config 4: cap in GB on the uncompressed cache (it also stays below 85 %% of the free memory)")
    args = ap.parse_args()
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.impl == "reference":
        run_reference(args, rank)
        return
    if args.layers != LAYERS:
        WORKLOAD = WORKLOAD.replace("24 layers", f"{args.layers} layers (profiling case, not the benchmark)")
        LAYERS = args.layers
    sweep = args.budget_frames * F != L_MAX or args.bits != BITS or args.dtype != "bf16"
    if args.dtype == "fp16":
        TORCH_DTYPE = "float16"
    if sweep:
        if args.budget_frames < 3:
            ap.error("--budget-frames must be at least 3")
        WORKLOAD = (WORKLOAD.replace("config2:", "sweep case (not the benchmark), config2 with")
                    .replace(f"budget {L_MAX} tokens/layer", f"budget {args.budget_frames * F} tokens/layer")
                    .replace(f"{BITS}-bit KV", f"{args.bits}-bit KV").replace("-bit KV, bf16,", f"-bit KV, {args.dtype},")
                    .replace(f"{PREFILL}-frame prefill", f"{args.budget_frames}-frame prefill"))
        L_MAX, BITS, PREFILL = args.budget_frames * F, args.bits, args.budget_frames
        args.no_cpu_baseline = True
    if args.warmup < 3:
        args.warmup = 3

    import torch
    import torch.distributed as dist
    import __graft_entry__ as ge
    ge.build()
    from paper_2602_21780_b200 import binding

    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if args.config in (3, 4) or args.batch:
        if rank == 0:
            fn = run_batch_bench if args.batch else (run_config3 if args.config == 3 else run_config4)
            fn(args, torch, binding, dev, torch.cuda.current_stream())
        return
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    frames = gen_frames(torch, dev, LAYERS, POOL, seed=replica_seed(20260221, rank))
    out = torch.empty(H, F, D, device=dev, dtype=getattr(torch, TORCH_DTYPE))
    xsv_dtype = binding.BF16 if TORCH_DTYPE == "bfloat16" else binding.F16
    stream = torch.cuda.current_stream()
    sp = stream.cuda_stream
    impl = {"auto": binding.ATTN_AUTO, "mma": binding.ATTN_MMA, "tc5": binding.ATTN_TC5}[args.attn]

    def make_cache():
        c = binding.Cache(LAYERS, H, D, L_MAX, BITS)
        c.set_attn_impl(impl)
        # the inputs of a frame stay untouched while the next layers run, so the end of a layer-step's selection and
        # re-quantisation may overlap the next layer-step (see xsv_cache_set_deferred_join); joined before the clock stops
        c.set_deferred_join(True)
        return c

    ptrs = [[(q.data_ptr(), k.data_ptr(), v.data_ptr()) for (q, k, v) in per] for per in frames]
    optr = out.data_ptr()

    def frame_step(cache, f):
        for l in range(LAYERS):
            q, k, v = ptrs[l][f % POOL]
            rc = cache.step_raw(l, q, k, v, F, xsv_dtype, optr, sp)
            if rc != 0:
                raise RuntimeError(f"xsv_step failed: status {rc}")

    cache = make_cache()
    for f in range(PREFILL):
        frame_step(cache, f)
    for f in range(args.warmup):
        frame_step(cache, PREFILL + f)
    torch.cuda.synchronize()
    assert cache.len(0) == L_MAX
    bytes_before = cache.bytes()

    # events around every seventh attention kernel (a sample that walks through the layers): its live duration for the
    # roofline; a pair of events costs the stream a few microseconds, around every launch they took 3-5 % off the step
    cache.set_profiling(3)
    cache.profile_read(reset=True)
    sampler = ClockSampler(local_rank)
    sampler.start()
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    launches0 = binding.kernel_launches()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for f in range(args.steps):
        frame_step(cache, PREFILL + args.warmup + f)
    cache.join(stream)
    e1.record(stream)
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    ms = e0.elapsed_time(e1)
    launches = binding.kernel_launches() - launches0
    clocks = sampler.stop()
    prof = cache.profile_read(reset=True)
    # the other phases, in short passes of their own after the timed region (events around every phase slow the step):
    # once as the step runs (selection and quantisation on the library's own streams: spans that include waiting for
    # free multiprocessors) and once with every kernel on the caller's stream in order (spans = kernel durations)
    n_phase_frames = max(1, min(3, args.steps))
    prof_all, prof_serial = None, None
    for mode in (1, 4):
        cache.set_profiling(mode)
        cache.profile_read(reset=True)
        for f in range(n_phase_frames):
            frame_step(cache, PREFILL + args.warmup + args.steps + f)
        cache.join(stream)
        torch.cuda.synchronize()
        if mode == 1:
            prof_all = cache.profile_read(reset=True)
        else:
            prof_serial = cache.profile_read(reset=True)
    cache.set_profiling(0)
    assert cache.status() == 0, "device status word set"
    assert cache.bytes() == bytes_before, "cache bytes changed in steady state"
    kv_layer = cache.layer_kv_bytes(0)
    total_bytes = cache.bytes()

    value, ms = job_throughput(ms, args.steps, world, dist if world > 1 else None, dev)

    # ---- roofline of the dominant kernel (attention), live CUDA-event durations
    peaks = measured_peaks()
    attn_ms, attn_launches = prof["attn"]
    attn_n = attn_launches                            # the timed sample: one attention kernel per timed phase
    T_all = L_MAX + F
    flops = 4.0 * F * T_all * D * H
    achieved = flops / (attn_ms / attn_n * 1e-3) / 1e12 if attn_n else None
    traffic = attn_traffic()
    roofline = {"bound": "tensor", "kernel": "fused dequant+attention", "achieved": achieved,
                "peak": peaks["tflops"], "unit": "TFLOP/s", "frac": achieved / peaks["tflops"] if achieved else None,
                "peak_burst": peaks["tflops_burst"], "frac_of_burst_peak": achieved / peaks["tflops_burst"] if achieved else None,
                "traffic": None if sweep else traffic["bytes"], "traffic_source": None if sweep else traffic["source"],
                "peak_source": peaks["source"],
                "flops_per_launch": flops, "avg_launch_ms": attn_ms / attn_n if attn_n else None,
                "launches_timed": attn_n, "launches_total": args.steps * LAYERS,
                "kernels_per_launch": attn_launches / attn_n if attn_n else None}
    # the bandwidth-bound phases: algorithmic bytes per layer-step / live duration
    k_keep = L_MAX - 2 * F
    n_mid = L_MAX - F
    tok_b = 2 * H * D * BITS // 8 + 2 * H * 8            # packed bytes per token incl. parameters
    score_bytes = n_mid * (H * D * BITS // 8 + H * 8) + H * F * D * 2
    quant_bytes = n_mid * tok_b + 2 * H * F * D * 2 + (L_MAX - F) * tok_b
    phases = {}
    steps_n = n_phase_frames * LAYERS
    for name, nbytes in (("score", score_bytes), ("select", n_mid * 4 + k_keep * 4), ("quant", quant_bytes)):
        pms, pn = prof_serial[name]
        oms, _ = prof_all[name]
        if steps_n and pms > 0:
            per = pms / steps_n
            phases[name] = {"avg_ms": per, "algorithmic_bytes": nbytes, "GB/s": nbytes / (per * 1e-3) / 1e9,
                            "frac_of_hbm": nbytes / (per * 1e-3) / 1e9 / peaks["hbm"], "launches_per_step": pn / steps_n,
                            "span_ms_when_overlapped": oms / steps_n if oms > 0 else None}
    phases["attn"] = {"avg_ms": attn_ms / attn_n if attn_n else None,
                      "avg_ms_serial_pass": prof_serial["attn"][0] / steps_n if steps_n else None}
    phases["note"] = (f"score/select/quant: {n_phase_frames} frames after the timed region with every kernel of the step on one "
                      "stream in order and events around each phase, so avg_ms is the duration of the phase's kernels "
                      "(24 layers x 700 MB of cache between two visits of a layer: nothing of it is still in the L2); "
                      "span_ms_when_overlapped is the same phase as the benchmark runs it, on the library's own streams "
                      "beside the attention kernel, where the span includes waiting for free multiprocessors")
    cache.destroy()

    # ---- end to end: same metric through the C ABI with HOST buffers (copies inside the timed region)
    e2e = None
    if not args.no_e2e:
        hq = [[tuple(t.cpu().pin_memory() for t in fr) for fr in per[:2]] for per in frames]
        houts = [torch.empty(H, F, D, dtype=getattr(torch, TORCH_DTYPE)).pin_memory() for _ in range(LAYERS)]
        c2 = make_cache()
        c2.set_host_pipelining(True)          # results travel back while the next layer computes
        for f in range(PREFILL + 3):
            frame_step(c2, f)
        n_e2e = max(3, min(args.steps, 10))

        def host_frame(f):
            for l in range(LAYERS):
                q, k, v = hq[l][f % 2]
                c2.step_host(l, q, k, v, houts[l], stream)
            c2.host_flush(stream)
            torch.cuda.synchronize()       # the frame's results are on the host

        host_frame(0)
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        e0.record(stream)
        for f in range(n_e2e):
            host_frame(1 + f)
        e1.record(stream)
        torch.cuda.synchronize()
        wall = (time.perf_counter() - t0) * 1e3
        ems = max(e0.elapsed_time(e1), wall)
        e2e_value, ems = job_throughput(ems, n_e2e, world, dist if world > 1 else None, dev)
        nb = H * F * D * 2
        e2e = {"value": e2e_value, "unit": "frames/s", "h2d_bytes_per_step": 3 * nb * LAYERS,
               "d2h_bytes_per_step": nb * LAYERS, "steps": n_e2e,
               "api": "xsv_step_host (pinned host Q/K/V in, host out back, per layer; copies overlap the kernels), xsv_cache_host_flush + synchronise per frame"}
        c2.destroy()

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        sec = oracle_layer_step_seconds()
        cpu = {"value": 1.0 / (LAYERS * sec), "unit": "frames/s", "cores": blas_threads(), "kind": "oracle",
               "nproc": os.cpu_count(),
               "sample": f"one steady-state layer-step (T_c={L_MAX}) = 1/24 frame: {sec:.2f} s on all threads, extrapolated x24",
               "layer_step_seconds_by_config": oracle_config_times()}

    if rank == 0:
        line = {"metric": METRIC, "value": value, "unit": "frames/s", "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": "bf16" if TORCH_DTYPE == "bfloat16" else "fp16", "data": "synthetic",
                "config": {"workload": WORKLOAD, "prefill_frames": PREFILL, "attn_impl": args.attn, "deferred_join": True,
                           "l2": "each step touches 203 MB of fresh inputs + 675 MB of cache (> 126 MB L2); no flush",
                           "multi_gpu": "replicas only"},
                "clocks": clocks, "e2e": e2e, "gpu_launches": launches, "roofline": roofline, "cpu_baseline": cpu,
                "phases": phases, "kv_bytes_per_layer": kv_layer, "cache_bytes_total": total_bytes,
                "latency_ms_per_layer_step": ms / args.steps / LAYERS}
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
