"""CUDA path vs oracle, through the C ABI (run on the B200 machine: -m gpu)."""
import numpy as np
import pytest
import torch

from oracle import xsv_oracle as orc
from paper_2602_21780_b200 import binding, synth
from tests.gpu_harness import run_stream

pytestmark = pytest.mark.gpu

IMPLS = [binding.ATTN_MMA, binding.ATTN_AUTO]


@pytest.mark.parametrize("impl", IMPLS)
def test_config0_every_step(impl):
    c = synth.CONFIGS[0]
    st = synth.config_stream(0)
    w = run_stream(st, c["frames"], c["L_max"], c["bits"], impl=impl)
    assert w["checked"] == 8 and w["pruned_steps"] == 4


@pytest.mark.parametrize("bits", [2, 4, 8])
@pytest.mark.parametrize("dtype", ["fp16", "bf16"])
def test_small_ragged_shapes(bits, dtype):
    # F not a multiple of any tile, budget not a multiple of the group, ragged pooling tail
    st = synth.Stream(H=3, d=64, F=75, dtype=dtype, layer=2)
    w = run_stream(st, 7, 331, bits)
    assert w["pruned_steps"] == 3


@pytest.mark.parametrize("impl", IMPLS)
def test_budget_below_two_frames_and_exact_fit(impl):
    st = synth.Stream(H=2, d=64, F=130, dtype="bf16", layer=3)
    run_stream(st, 5, 200, 4, impl=impl)            # L_max < 2F: k = 0, cache = first + current
    st = synth.Stream(H=2, d=64, F=64, dtype="fp16", layer=4)
    w = run_stream(st, 7, 256, 4, impl=impl)        # T == L_max at step 4: no prune; step 5 prunes
    assert w["pruned_steps"] == 3


def test_ties_are_broken_by_position():
    # identical keys everywhere -> all scores equal -> the lowest positions of the middle are kept
    base = synth.Stream(H=2, d=64, F=40, dtype="fp16", layer=5)

    def frame(t):
        q, k, v = base.frame(t)
        k = np.broadcast_to(base.frame(0)[1][:, :1, :], k.shape).copy()
        return q, k, v

    w = run_stream(base, 6, 100, 4, frame_fn=frame)
    assert w["pruned_steps"] == 4


@pytest.mark.parametrize("L_max", [0, 150])
def test_quantisation_off(L_max):
    st = synth.Stream(H=2, d=64, F=50, dtype="bf16", layer=6)
    run_stream(st, 6, L_max, 16, max_cache_tokens=400 if L_max == 0 else -1)


def test_quantise_only_unbounded_cache():
    # ablation "quantisation without pruning": no budget, 4-bit cache growing up to its capacity
    st = synth.Stream(H=2, d=64, F=50, dtype="bf16", layer=10)
    w = run_stream(st, 6, 0, 4, max_cache_tokens=400)
    assert w["pruned_steps"] == 0


@pytest.mark.parametrize("bits", [4, 16])
def test_checkpoint_restore_continues_the_stream(bits):
    # export after 5 frames, import into a fresh cache, step both on: same outputs, same state
    st = synth.Stream(H=4, d=64, F=70, dtype="bf16", layer=11)
    a = binding.Cache(2, 4, 64, 260, bits)
    frames = [tuple(torch.from_numpy(x).to("cuda:0", torch.bfloat16).contiguous() for x in st.frame(t)) for t in range(8)]
    out_a, out_b = torch.empty_like(frames[0][0]), torch.empty_like(frames[0][0])
    for t in range(5):
        for l in range(2):
            a.step(l, *frames[t], out_a)
    b = binding.Cache(2, 4, 64, 260, bits)
    for l in range(2):
        b.import_layer(l, a.export_layer(l), frames_done=5, frame_tokens=70, dtype_code=binding.BF16)
    assert b.len(0) == a.len(0) and b.frames(1) == 5
    for t in range(5, 8):
        for l in range(2):
            a.step(l, *frames[t], out_a)
            b.step(l, *frames[t], out_b)
            torch.cuda.synchronize()
            assert torch.equal(out_a, out_b)
    for l in range(2):
        sa, sb = a.export_layer(l), b.export_layer(l)
        for key in sa:
            assert np.array_equal(sa[key], sb[key])
    assert a.status() == 0 and b.status() == 0
    a.destroy(); b.destroy()


@pytest.mark.parametrize("dtype", ["fp16", "bf16"])
def test_quantization_mse_matches_oracle(dtype):
    # the granularity study of Table 1 on the synthetic keys (outlier channels) and values; 300 tokens = 4 full groups
    # and a partial one
    st = synth.Stream(H=3, d=64, F=300, dtype=dtype, layer=12)
    _, K, V = st.frame(0)
    tdt = torch.float16 if dtype == "fp16" else torch.bfloat16
    for name, x in (("K", K), ("V", V)):
        xd = torch.from_numpy(x).to("cuda:0", tdt).contiguous()
        for bits in (2, 4, 8):
            for gran in ("channel", "token"):
                got = binding.quantization_mse(xd, bits, gran == "channel")
                want = orc.quantization_mse(x, bits, gran)
                assert got == pytest.approx(want, rel=1e-9), (name, bits, gran)


def test_deferred_join_parity_and_equality():
    # with the join deferred the side streams of one layer-step run under the next one's kernels: same results
    st = synth.Stream(H=4, d=64, F=261, dtype="fp16", layer=13)
    w = run_stream(st, 9, 1044, 4, layers=3, layer=1, deferred_join=True)
    assert w["pruned_steps"] >= 4
    frames = [tuple(torch.from_numpy(x).to("cuda:0", torch.float16).contiguous() for x in st.frame(t)) for t in range(10)]
    outs, states = [], []
    for deferred in (False, True):
        c = binding.Cache(3, 4, 64, 1044, 4)
        c.set_deferred_join(deferred)
        o = [[torch.empty_like(frames[0][0]) for _ in range(3)] for _ in range(10)]
        for t in range(10):
            for l in range(3):
                c.step(l, *frames[t], o[t][l])
        c.join()
        torch.cuda.synchronize()
        outs.append(o)
        states.append([c.export_layer(l) for l in range(3)])
        assert c.status() == 0
        c.destroy()
    for t in range(10):
        for l in range(3):
            assert torch.equal(outs[0][t][l], outs[1][t][l])
    for l in range(3):
        for key in states[0][l]:
            assert np.array_equal(states[0][l][key], states[1][l][key])


def test_pooling_options_and_multi_layer():
    st = synth.Stream(H=4, d=64, F=37, dtype="fp16", layer=7)
    run_stream(st, 6, 100, 4, n_special=1, g=4, layers=3, layer=2)


def test_drifting_stream_two_bits():
    st = synth.Stream(H=16, d=64, F=261, dtype="bf16", layer=1, drift_rho=0.95)
    w = run_stream(st, 8, 783, 2)
    assert w["pruned_steps"] == 5


@pytest.mark.parametrize("impl", IMPLS)
def test_config1_sampled_steps(impl):
    # paper shape: 1374 tokens/frame, budget 21984; verify the first step, the end of the ramp,
    # the first pruning steps and a later steady-state step
    c = synth.CONFIGS[1]
    st = synth.config_stream(1)
    w = run_stream(st, 20, c["L_max"], c["bits"], check_steps={0, 1, 15, 16, 17, 19}, impl=impl)
    assert w["pruned_steps"] == 3


def test_config3_shape_sampled_steps():
    # long-horizon shape: 1374 tokens/frame, budget 10992 (8 frames), 2-bit, drifting means; a deeper layer's
    # stream; verify the first step, the end of the ramp, the first pruning steps
    c = synth.CONFIGS[3]
    st = synth.config_stream(3, layer=17)
    w = run_stream(st, 11, c["L_max"], c["bits"], check_steps={0, 7, 8, 9, 10})
    assert w["pruned_steps"] == 3


def test_config2_multi_layer_cache_is_per_layer():
    # several layers in one cache object at paper shape: layers are independent caches; verify a middle one
    c = synth.CONFIGS[2]
    st = synth.config_stream(2, layer=5)
    w = run_stream(st, 18, c["L_max"], c["bits"], check_steps={0, 16, 17}, layers=3, layer=1)
    assert w["pruned_steps"] == 2


@pytest.mark.parametrize("dtype", ["fp16", "bf16"])
def test_importance_scores_entry_point(dtype):
    from oracle import xsv_oracle as orc
    from tests.gpu_harness import to_dev
    st = synth.Stream(H=16, d=64, F=1374, dtype=dtype, layer=9)
    q, k, _ = st.frame(0)
    keys = np.concatenate([k, st.frame(1)[1], st.frame(2)[1]], axis=1)[:, :3001]
    S = binding.importance_scores(to_dev(q, dtype), to_dev(keys, dtype)).cpu().numpy()
    ref = orc.importance_scores(q, keys, 5, 16)
    assert np.max(np.abs(S - ref)) <= 1e-3 * np.max(np.abs(ref))
    # pooling parameters reach the kernel
    S2 = binding.importance_scores(to_dev(q, dtype), to_dev(keys, dtype), n_special=1, pool_group=7).cpu().numpy()
    ref2 = orc.importance_scores(q, keys, 1, 7)
    assert np.max(np.abs(S2 - ref2)) <= 1e-3 * np.max(np.abs(ref2))


def test_api_errors_and_bytes_constant():
    c = binding.Cache(2, 16, 64, 600, 4)
    Q = torch.randn(16, 261, 64, device="cuda", dtype=torch.float16)
    out = torch.empty_like(Q)
    lib = binding.load()
    assert lib.xsv_step(c._h, 5, Q.data_ptr(), Q.data_ptr(), Q.data_ptr(), 261, 0, out.data_ptr(), None) == 1
    assert lib.xsv_step(c._h, 0, Q.data_ptr(), Q.data_ptr(), Q.data_ptr(), 261, 0, Q.data_ptr(), None) == 1
    assert lib.xsv_step(c._h, 0, Q.data_ptr() + 2, Q.data_ptr(), Q.data_ptr(), 261, 0, out.data_ptr(), None) == 2
    c.step(0, Q, Q, Q, out)
    with pytest.raises(binding.XsvError) as e:
        c.step(0, Q, Q, Q, out)                       # layer 0 twice before layer 1
    assert e.value.code == 3
    with pytest.raises(binding.XsvError) as e:
        c.set_options(n_special=3)                    # options after the first step
    assert e.value.code == 3
    Q2 = torch.randn(16, 300, 64, device="cuda", dtype=torch.float16)      # more tokens than the largest frame allowed
    assert lib.xsv_step(c._h, 1, Q2.data_ptr(), Q2.data_ptr(), Q2.data_ptr(), 300, 0, out.data_ptr(), None) == 2
    assert lib.xsv_step(c._h, 1, Q.data_ptr(), Q.data_ptr(), Q.data_ptr(), 261, 1, out.data_ptr(), None) == 2
    c.step(1, Q, Q, Q, out)
    b0 = c.bytes()
    for _ in range(6):
        for l in range(2):
            c.step(l, Q, Q, Q, out)
    torch.cuda.synchronize()
    assert c.bytes() == b0 and c.len(0) == 600 and c.status() == 0
    c.destroy()


@pytest.mark.parametrize("defer,deferred_join", [(False, False), (True, False), (True, True)])
def test_host_step_matches_device_step(defer, deferred_join):
    st = synth.Stream(H=4, d=64, F=90, dtype="bf16", layer=8)
    a = binding.Cache(1, 4, 64, 300, 4)
    b = binding.Cache(1, 4, 64, 300, 4)
    a.set_host_pipelining(defer)
    a.set_deferred_join(deferred_join)
    hosts, devs = [], []
    for t in range(7):
        q, k, v = (torch.from_numpy(x).to(torch.bfloat16) for x in st.frame(t))
        Qh, Kh, Vh = q.pin_memory(), k.pin_memory(), v.pin_memory()
        oh = torch.empty_like(Qh).pin_memory()
        a.step_host(0, Qh, Kh, Vh, oh)              # no synchronisation between calls: copies and kernels overlap
        hosts.append((Qh, Kh, Vh, oh))
        Q, K, V = q.cuda(), k.cuda(), v.cuda()
        od = torch.empty_like(Q)
        b.step(0, Q, K, V, od)
        devs.append(od)
    if defer:
        a.host_flush()
    torch.cuda.synchronize()
    for (_, _, _, oh), od in zip(hosts, devs):
        assert torch.equal(oh, od.cpu())
    sa, sb = a.export_layer(0), b.export_layer(0)
    for key in sa:
        assert np.array_equal(sa[key], sb[key])
    a.destroy(); b.destroy()


def test_bounded_wait_times_out_and_reports():
    # a wait that nothing satisfies returns after its limit with the timeout status; the context stays usable
    import time
    t0 = time.time()
    assert binding.selftest_bounded_wait() == 6
    assert 1.0 < time.time() - t0 < 30.0
    x = torch.ones(4, device="cuda")
    assert float(x.sum()) == 4.0


def test_long_horizon_stream_stays_flat():
    # config-3 shape (1374 tokens/frame, budget 10992, 2-bit, per-channel means drifting as an AR(1) process),
    # fewer layers and frames than the full run: once pruning has started the cache bytes and the cache length stay
    # constant and the per-frame time does not drift
    from tests.gpu_harness import device_stream
    H, F, L, bits, layers, frames = 16, 1374, 10992, 2, 4, 300
    feeds = [device_stream(H, F, "bf16", seed=40 + l, drift_rho=0.95) for l in range(layers)]
    out = torch.empty(H, F, 64, device="cuda", dtype=torch.bfloat16)
    c = binding.Cache(layers, H, 64, L, bits)
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(2 * frames)]
    bytes_seen = set()
    for t in range(frames):
        inputs = [feeds[l](t) for l in range(layers)]          # drawn before the clock starts
        ev[2 * t].record()
        for l in range(layers):
            c.step(l, *inputs[l], out)
        ev[2 * t + 1].record()
        if t >= 9:
            bytes_seen.add(c.bytes())
            assert c.len(layers - 1) == L
    torch.cuda.synchronize()
    assert c.status() == 0
    assert len(bytes_seen) == 1                                   # constant device memory
    assert torch.isfinite(out.float()).all()
    times = [ev[2 * t].elapsed_time(ev[2 * t + 1]) for t in range(frames)]
    med = lambda xs: sorted(xs)[len(xs) // 2]
    early, late = med(times[20:60]), med(times[-40:])
    assert abs(late - early) < 0.10 * early, (early, late)        # medians: robust against a neighbour's burst
    c.destroy()


def test_host_step_with_joins_between_calls():
    # deferred join + host buffers + xsv_cache_join between the calls and no device synchronisation: a staging slot
    # must not be refilled while the side-stream kernels of the step that read it are still running
    st = synth.Stream(H=4, d=64, F=200, dtype="bf16", layer=14)
    a = binding.Cache(1, 4, 64, 700, 4)
    b = binding.Cache(1, 4, 64, 700, 4)
    a.set_deferred_join(True)
    hosts, devs = [], []
    for t in range(9):
        q, k, v = (torch.from_numpy(x).to(torch.bfloat16) for x in st.frame(t))
        Qh, Kh, Vh = q.pin_memory(), k.pin_memory(), v.pin_memory()
        oh = torch.empty_like(Qh).pin_memory()
        a.step_host(0, Qh, Kh, Vh, oh)
        a.join()                                       # the caller's stream waits; the copy stream must still be held back
        hosts.append((Qh, Kh, Vh, oh))
        Q, K, V = q.cuda(), k.cuda(), v.cuda()
        od = torch.empty_like(Q)
        b.step(0, Q, K, V, od)
        devs.append(od)
    torch.cuda.synchronize()
    for (_, _, _, oh), od in zip(hosts, devs):
        assert torch.equal(oh, od.cpu())
    sa, sb = a.export_layer(0), b.export_layer(0)
    for key in sa:
        assert np.array_equal(sa[key], sb[key])
    a.destroy(); b.destroy()


def test_two_devices_in_one_process():
    # kernel attributes (opt-in shared memory) are set per device: a cache on a second GPU of the same process works
    if torch.cuda.device_count() < 2:
        pytest.skip("one GPU visible")
    st = synth.Stream(H=2, d=64, F=150, dtype="fp16", layer=15)
    outs = []
    for dev in (0, 1):
        torch.cuda.set_device(dev)
        c = binding.Cache(1, 2, 64, 400, 4)
        o = None
        for t in range(5):
            q, k, v = (torch.from_numpy(x).to(f"cuda:{dev}", torch.float16).contiguous() for x in st.frame(t))
            o = torch.empty_like(q)
            c.step(0, q, k, v, o)
        torch.cuda.synchronize()
        assert c.status() == 0
        outs.append(o.cpu())
        c.destroy()
    torch.cuda.set_device(0)
    assert torch.equal(outs[0], outs[1])
