"""Step-locked comparison of the CUDA path (through the C ABI) with the CPU oracle.

Before each checked step the GPU layer state is exported and loaded into the
oracle; both run the step on the same inputs; then the outputs are compared:
attention within 1e-2 * max|out_oracle|, scores within 1e-3 * max|S_oracle|,
the kept set exactly (the oracle's Eq. 8 evaluated on the GPU's own scores),
codes / scales / offsets bit for bit."""
import numpy as np
import torch

from oracle import xsv_oracle as orc
from paper_2602_21780_b200 import binding, synth

ATTN_TOL = 1e-2
SCORE_TOL = 1e-3


def torch_dtype(name):
    return torch.float16 if name == "fp16" else torch.bfloat16


def to_dev(x, dtype):
    return torch.from_numpy(np.ascontiguousarray(x)).to("cuda:0", torch_dtype(dtype)).contiguous()


def load_oracle_state(ref, st, frames_done, F):
    if ref.bits == 16:
        dt = "fp16" if ref._dtype == "fp16" else "bf16"
        ref.load_state(frames_done, F, synth.from_bits16(st["Kraw"], dt), np.zeros((ref.H, 0, ref.d)),
                       np.zeros((ref.H, 0, ref.d)), synth.from_bits16(st["Vraw"], dt),
                       np.zeros((ref.H, 0, 1)), np.zeros((ref.H, 0, 1)), st["origin"])
    else:
        ref.load_state(frames_done, F, st["Kc"], st["Ks"], st["Kz"], st["Vc"], st["Vs"][..., None],
                       st["Vz"][..., None], st["origin"])


def check_state_invariants(st, bits, F_first, F_last, tokens_seen, T_expected):
    """What must hold for any cache state, checked wherever a state is imported into the oracle: its length,
    ascending origins, the first and the latest frame present in full, codes in range, positive scales."""
    T = st["T"]
    assert T == T_expected
    o = st["origin"]
    assert np.all(np.diff(o) > 0)
    assert np.array_equal(o[:F_first], np.arange(F_first))
    assert np.array_equal(o[-F_last:], tokens_seen - F_last + np.arange(F_last))
    if bits < 16:
        n = (1 << bits) - 1
        assert st["Kc"].max() <= n and st["Vc"].max() <= n
        assert np.all(st["Ks"] > 0) and np.all(st["Vs"] > 0)
        assert np.all(np.isfinite(st["Ks"])) and np.all(np.isfinite(st["Vs"]))
        # every stored (s, z) reproduces its group's codes from the values they dequantise to (Eq. 9 after Eq. 12)
        grp = np.arange(T) // 64
        for codes, s, z in ((st["Kc"], st["Ks"][:, grp, :], st["Kz"][:, grp, :]),
                            (st["Vc"], st["Vs"][..., None], st["Vz"][..., None])):
            x = orc.dequantize(codes, s, z)
            with np.errstate(over="ignore", invalid="ignore"):
                back = np.clip(np.rint((x - z).astype(np.float32) / s.astype(np.float32)), 0, n)
            assert np.array_equal(back.astype(np.int64), codes)


def compare_states(st, ref, bits, tag):
    assert st["T"] == ref.T, f"{tag}: length {st['T']} vs {ref.T}"
    assert np.array_equal(st["origin"], ref.origin), f"{tag}: kept set differs"
    if bits == 16:
        dt = ref._dtype
        assert np.array_equal(synth.from_bits16(st["Kraw"], dt), ref.Kc), f"{tag}: raw K differs"
        assert np.array_equal(synth.from_bits16(st["Vraw"], dt), ref.Vc), f"{tag}: raw V differs"
        return
    bits32 = lambda a: np.ascontiguousarray(a, np.float32).view(np.uint32)
    for name, a, b in (("V codes", st["Vc"], ref.Vc), ("V offsets", bits32(st["Vz"]), bits32(ref.Vz[..., 0])),
                       ("K codes", st["Kc"], ref.Kc), ("K offsets", bits32(st["Kz"]), bits32(ref.Kz))):
        assert np.array_equal(a, b), f"{tag}: {name} differ at {np.argwhere(a != b)[:4].tolist()}"
    assert np.array_equal(st["Vs"].view(np.uint32), ref.Vs[..., 0].view(np.uint32)), f"{tag}: V scales differ"
    assert np.array_equal(st["Ks"].view(np.uint32), np.ascontiguousarray(ref.Ks).view(np.uint32)), f"{tag}: K scales differ"


def run_stream(stream, frames, L_max, bits, check_steps=None, impl=binding.ATTN_AUTO, n_special=5, g=16,
               frame_fn=None, max_cache_tokens=-1, layers=1, layer=0, deferred_join=False, max_frame_tokens=0,
               device_fn=None, key_magnitude_limit=None):
    """Run `frames` steps on the GPU; verify the steps in check_steps (0-based; None = all).
    frame_fn(t) may return frames of different sizes (then max_frame_tokens names the largest).
    device_fn(t), if given, supplies the inputs of the steps that are not checked as CUDA tensors (long streams:
    the state a checked step starts from is imported from the GPU, so those inputs need no CPU twin).
    key_magnitude_limit: if given, the attention output of a checked step is compared only while the dequantised
    cached keys stay below it in magnitude (see test_configs_2_and_3_mid_and_last_frames for why); everything
    else is compared regardless, and the steps left out are counted in "attn_skipped".
    Returns a dict of the worst errors seen."""
    H, d, dtype = stream.H, stream.d, stream.dtype
    cache = binding.Cache(layers, H, d, L_max, bits)
    cache.set_attn_impl(impl)
    cache.set_deferred_join(deferred_join)
    if (n_special, g) != (5, 16) or max_cache_tokens >= 0 or max_frame_tokens > 0:
        cache.set_options(n_special=n_special, pool_group=g, max_cache_tokens=max_cache_tokens,
                          max_frame_tokens=max_frame_tokens)
    ref = orc.LayerCache(H, d, L_max, bits, n_special=n_special, g=g)
    ref._dtype = dtype
    worst = dict(attn=0.0, score=0.0, pruned_steps=0, checked=0, attn_skipped=0, key_magnitude=0.0)
    F_first, F_prev, tokens_seen, T_expected = 0, 0, 0, 0
    for t in range(frames):
        checked = check_steps is None or t in check_steps
        if checked or device_fn is None:
            q, k, v = frame_fn(t) if frame_fn else stream.frame(t)
            Q, K, V = to_dev(q, dtype), to_dev(k, dtype), to_dev(v, dtype)
        else:
            Q, K, V = device_fn(t)
        F = Q.shape[1]
        out = torch.empty_like(Q)
        if checked:
            st0 = cache.export_layer(layer)
            if t > 0:
                check_state_invariants(st0, bits, F_first, F_prev, tokens_seen, T_expected)
            load_oracle_state(ref, st0, t, F_first)
        for l in range(layers):            # other layers take the same inputs; only `layer` is verified
            cache.step(l, Q, K, V, out)
        torch.cuda.synchronize()
        if t == 0:
            F_first = F
        T_expected = orc.next_cache_len(t + 1, T_expected, F_first, F, L_max)
        tokens_seen += F
        F_prev = F
        assert cache.len(layer) == T_expected
        if not checked:
            continue
        S_gpu = cache.last_scores()
        kmag = float(np.abs(ref.dequant_K()).max()) if ref.T else 0.0
        worst["key_magnitude"] = max(worst["key_magnitude"], kmag)
        o_ref = ref.step(q, k, v, select_on=S_gpu.astype(np.float64) if S_gpu.size else None)
        o_gpu = out.float().cpu().numpy().astype(np.float64)
        assert np.all(np.isfinite(o_gpu)), f"step {t}: non-finite attention output"
        if key_magnitude_limit is not None and kmag > key_magnitude_limit:
            worst["attn_skipped"] += 1
        else:
            e = float(np.max(np.abs(o_gpu - o_ref)) / np.max(np.abs(o_ref)))
            worst["attn"] = max(worst["attn"], e)
            assert e <= ATTN_TOL, f"step {t}: attention error {e:.3e} of max|out|"
        if ref.last_scores is not None and ref.last_scores.size == 0:
            assert S_gpu.size == 0                      # empty middle segment (budget below two frames)
            worst["pruned_steps"] += 1
        elif ref.last_scores is not None:
            assert S_gpu.shape == ref.last_scores.shape, f"step {t}: score count"
            es = float(np.max(np.abs(S_gpu - ref.last_scores)) / np.max(np.abs(ref.last_scores)))
            worst["score"] = max(worst["score"], es)
            worst["pruned_steps"] += 1
            assert es <= SCORE_TOL, f"step {t}: score error {es:.3e} of max|S|"
        else:
            assert S_gpu.size == 0, f"step {t}: GPU pruned but the oracle did not"
        compare_states(cache.export_layer(layer), ref, bits, f"step {t}")
        worst["checked"] += 1
    assert cache.status() == 0
    worst["bytes"] = cache.bytes()
    worst["kv_bytes"] = cache.layer_kv_bytes(layer)
    assert worst["kv_bytes"] == ref.kv_bytes_packed()
    cache.destroy()
    return worst


def device_stream(H, F, dtype, seed, d=64, pool=4, drift_rho=None):
    """Inputs for unchecked steps, drawn on the device with the recipe of synth.Stream (Q, V ~ N(0,1); K with a
    per-channel offset and four ten-fold channels per head; optionally AR(1) drifting means).  Returns device_fn."""
    g = torch.Generator(device="cuda:0")
    g.manual_seed(seed)
    td = torch_dtype(dtype)
    mu = torch.randn(H, 1, d, device="cuda:0", generator=g) * 0.5
    m = torch.ones(H, 1, d, device="cuda:0")
    for h in range(H):
        m[h, 0, torch.randperm(d, device="cuda:0", generator=g)[:4]] = 10.0
    state = {"t": -1, "dq": None, "dk": None, "dv": None}
    frames = []

    def fn(t):
        if drift_rho is None:
            if not frames:
                for _ in range(pool):
                    q = torch.randn(H, F, d, device="cuda:0", generator=g)
                    k = (torch.randn(H, F, d, device="cuda:0", generator=g) + mu) * m
                    v = torch.randn(H, F, d, device="cuda:0", generator=g)
                    frames.append(tuple(x.to(td).contiguous() for x in (q, k, v)))
            return frames[t % pool]
        rho, innov = drift_rho, (1.0 - drift_rho ** 2) ** 0.5 * 0.5
        while state["t"] < t:                                    # the means advance frame by frame
            for key in ("dq", "dk", "dv"):
                eps = torch.randn(H, 1, d, device="cuda:0", generator=g)
                state[key] = eps * 0.5 if state[key] is None else rho * state[key] + innov * eps
            state["t"] += 1
        q = torch.randn(H, F, d, device="cuda:0", generator=g) + state["dq"]
        k = (torch.randn(H, F, d, device="cuda:0", generator=g) + mu + state["dk"]) * m
        v = torch.randn(H, F, d, device="cuda:0", generator=g) + state["dv"]
        return tuple(x.to(td).contiguous() for x in (q, k, v))

    return fn


def run_batch(streams, frames, L_max, bits, starts=None, check_steps=None, deferred_join=False):
    """Several independent streams stepped together through xsv_step_batch, each verified against its own oracle
    with the step-locked protocol of run_stream.  streams: synth.Stream objects (same heads and dtype; frame sizes
    may differ); starts[i]: the frame at which stream i joins (so that lengths differ and some streams prune while
    others still append).  Returns the worst errors over all streams."""
    B = len(streams)
    starts = starts or [0] * B
    H, d, dtype = streams[0].H, streams[0].d, streams[0].dtype
    caches = [binding.Cache(1, H, d, L_max, bits) for _ in range(B)]
    for c in caches:
        c.set_deferred_join(deferred_join)
    refs = [orc.LayerCache(H, d, L_max, bits) for _ in range(B)]
    for r in refs:
        r._dtype = dtype
    track = [dict(F_first=0, F_prev=0, seen=0, T=0, t=0) for _ in range(B)]
    worst = dict(attn=0.0, score=0.0, pruned_steps=0, checked=0, batched_calls=0)
    for t in range(frames):
        active = [i for i in range(B) if t >= starts[i]]
        data = {i: streams[i].frame(t - starts[i]) for i in active}
        dev = {i: tuple(to_dev(x, dtype) for x in data[i]) for i in active}
        outs = {i: torch.empty_like(dev[i][0]) for i in active}
        checked = check_steps is None or t in check_steps
        if checked:
            for i in active:
                st0 = caches[i].export_layer(0)
                tr = track[i]
                if tr["t"] > 0:
                    check_state_invariants(st0, bits, tr["F_first"], tr["F_prev"], tr["seen"], tr["T"])
                load_oracle_state(refs[i], st0, tr["t"], tr["F_first"])
        binding.step_batch([caches[i] for i in active], 0, [dev[i][0] for i in active], [dev[i][1] for i in active],
                           [dev[i][2] for i in active], [outs[i] for i in active])
        worst["batched_calls"] += 1
        torch.cuda.synchronize()
        for i in active:
            tr = track[i]
            F = data[i][0].shape[1]
            if tr["t"] == 0:
                tr["F_first"] = F
            tr["T"] = orc.next_cache_len(tr["t"] + 1, tr["T"], tr["F_first"], F, L_max)
            tr["seen"] += F
            tr["F_prev"] = F
            tr["t"] += 1
            assert caches[i].len(0) == tr["T"]
        if not checked:
            continue
        for i in active:
            q, k, v = data[i]
            ref = refs[i]
            S_gpu = caches[i].last_scores()
            o_ref = ref.step(q, k, v, select_on=S_gpu.astype(np.float64) if S_gpu.size else None)
            o_gpu = outs[i].float().cpu().numpy().astype(np.float64)
            assert np.all(np.isfinite(o_gpu)), f"step {t}, stream {i}: non-finite attention output"
            e = float(np.max(np.abs(o_gpu - o_ref)) / np.max(np.abs(o_ref)))
            worst["attn"] = max(worst["attn"], e)
            assert e <= ATTN_TOL, f"step {t}, stream {i}: attention error {e:.3e} of max|out|"
            if ref.last_scores is not None and ref.last_scores.size:
                assert S_gpu.shape == ref.last_scores.shape
                es = float(np.max(np.abs(S_gpu - ref.last_scores)) / np.max(np.abs(ref.last_scores)))
                worst["score"] = max(worst["score"], es)
                assert es <= SCORE_TOL, f"step {t}, stream {i}: score error {es:.3e} of max|S|"
                worst["pruned_steps"] += 1
            compare_states(caches[i].export_layer(0), ref, bits, f"step {t}, stream {i}")
            worst["checked"] += 1
    for c in caches:
        assert c.status() == 0
        c.destroy()
    return worst
