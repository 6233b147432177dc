#!/usr/bin/env python
"""Benchmark of the compressed-KV streaming attention step.

A "step" is one frame through the whole hot path for all 24 layers: fused
dequant + attention, importance scores, top-k prune, quantise + pack
(configuration 2: 16 heads x 64, 1374 tokens/frame, budget 21984 tokens per
layer, 4-bit KV, bf16), in steady state (the cache is filled to its budget by
untimed prefill frames first).  Prints ONE JSON line.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

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
POOL = 4                     # distinct frames per layer, cycled
METRIC = "frames/s of compressed-KV causal attention step (24 layers)"
WORKLOAD = ("config2: 24 layers x (16 heads x 64), 1374 tokens/frame, budget 21984 tokens/layer, 4-bit KV, bf16, "
            "steady state after a 16-frame prefill")


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        m = json.load(open(p))
        return dict(tflops=float(m.get("bf16_tflops_sustained", m.get("bf16_tflops"))), hbm=float(m["hbm_gbs"]),
                    source="measured (MEASURED_PEAKS.json, sustained bf16)")
    return dict(tflops=1400.0, hbm=6650.0, source="fallback (no MEASURED_PEAKS.json)")


def attn_traffic_bytes():
    """DRAM bytes per attention launch from the committed ncu summary, if any."""
    p = os.path.join(ROOT, "profiles", "attention_config2_traffic.txt")
    try:
        for line in open(p):
            if line.startswith("traffic_bytes_per_launch:"):
                return float(line.split(":")[1])
    except OSError:
        pass
    return None


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
            q = torch.randn(H, F, D, device=dev, generator=g).to(torch.bfloat16)
            k = ((torch.randn(H, F, D, device=dev, generator=g) + mu) * m).to(torch.bfloat16)
            v = torch.randn(H, F, D, device=dev, generator=g).to(torch.bfloat16)
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


def main():
    global LAYERS, WORKLOAD, L_MAX, BITS, PREFILL
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
    sweep = args.budget_frames * F != L_MAX or args.bits != BITS
    if sweep:
        if args.budget_frames < 3:
            ap.error("--budget-frames must be at least 3")
        WORKLOAD = (WORKLOAD.replace("config2:", "sweep case (not the benchmark), config2 with")
                    .replace(f"budget {L_MAX} tokens/layer", f"budget {args.budget_frames * F} tokens/layer")
                    .replace(f"{BITS}-bit KV", f"{args.bits}-bit KV")
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
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    frames = gen_frames(torch, dev, LAYERS, POOL, seed=replica_seed(20260221, rank))
    out = torch.empty(H, F, D, device=dev, dtype=torch.bfloat16)
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
            rc = cache.step_raw(l, q, k, v, F, binding.BF16, optr, sp)
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
    # the other phases, in a short pass of their own after the timed region (events around every phase slow the step)
    cache.set_profiling(1)
    n_phase_frames = max(1, min(3, args.steps))
    for f in range(n_phase_frames):
        frame_step(cache, PREFILL + args.warmup + args.steps + f)
    torch.cuda.synchronize()
    prof_all = cache.profile_read(reset=True)
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
    roofline = {"bound": "tensor", "kernel": "fused dequant+attention", "achieved": achieved,
                "peak": peaks["tflops"], "unit": "TFLOP/s", "frac": achieved / peaks["tflops"] if achieved else None,
                "traffic": None if sweep else attn_traffic_bytes(), "peak_source": peaks["source"],
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
    for name, nbytes in (("score", score_bytes), ("select", n_mid * 4 + k_keep * 4), ("quant", quant_bytes)):
        pms, pn = prof_all[name]
        steps_n = n_phase_frames * LAYERS
        if steps_n and pms > 0:
            per = pms / steps_n
            phases[name] = {"avg_ms": per, "algorithmic_bytes": nbytes, "GB/s": nbytes / (per * 1e-3) / 1e9,
                            "frac_of_hbm": nbytes / (per * 1e-3) / 1e9 / peaks["hbm"], "launches_per_step": pn / steps_n}
    phases["attn"] = {"avg_ms": attn_ms / attn_n if attn_n else None}
    phases["note"] = (f"score/select/quant: events around every phase, {n_phase_frames} frames after the timed region; "
                      "select and quant run on the library's second stream under the tail of the attention kernel, so "
                      "their spans start when the scores are ready and include the wait for free multiprocessors: the "
                      "phases overlap and do not add up to the step")
    cache.destroy()

    # ---- end to end: same metric through the C ABI with HOST buffers (copies inside the timed region)
    e2e = None
    if not args.no_e2e:
        hq = [[tuple(t.cpu().pin_memory() for t in fr) for fr in per[:2]] for per in frames]
        houts = [torch.empty(H, F, D, dtype=torch.bfloat16).pin_memory() for _ in range(LAYERS)]
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
               "sample": f"one steady-state layer-step (T_c={L_MAX}) = 1/24 frame: {sec:.2f} s, extrapolated x24"}

    if rank == 0:
        line = {"metric": METRIC, "value": value, "unit": "frames/s", "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
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
