"""CUDA path vs oracle on the kernel variants and input ranges that the main parity file does not reach
(run on the B200 machine: -m gpu).  Every case goes through the C ABI and the step-locked harness."""
import numpy as np
import pytest
import torch

from oracle import xsv_oracle as orc
from paper_2602_21780_b200 import binding, synth
from tests.gpu_harness import device_stream, run_batch, run_stream, to_dev

pytestmark = pytest.mark.gpu

F_PAPER = 1374


def test_selection_above_32768_keys_radix_path():
    # Eq. 8 on a middle segment of 34 350 keys (budget 26 frames): the selection kernel for more keys than
    # the register-resident variants hold; first two pruning steps, few heads to keep the oracle cheap
    st = synth.Stream(H=2, d=64, F=F_PAPER, dtype="bf16", layer=21)
    w = run_stream(st, 28, 26 * F_PAPER, 4, check_steps={26, 27}, device_fn=device_stream(2, F_PAPER, "bf16", 21))
    assert w["pruned_steps"] == 2


def test_selection_above_32768_keys_with_ties():
    # the same path with all scores equal: the lowest positions of the middle must be kept
    base = synth.Stream(H=1, d=64, F=F_PAPER, dtype="fp16", layer=22)
    k0 = base.frame(0)[1][:, :1, :]

    def frame(t):
        q, k, v = base.frame(t)
        return q, np.broadcast_to(k0, k.shape).copy(), v

    def dev(t):
        q, k, v = frame(t % 3)
        return to_dev(q, "fp16"), to_dev(k, "fp16"), to_dev(v, "fp16")

    w = run_stream(base, 27, 26 * F_PAPER, 4, check_steps={26}, frame_fn=frame, device_fn=dev)
    assert w["pruned_steps"] == 1


def test_selection_between_24577_and_32768_keys():
    # middle segment of 27 480 keys (budget 21 frames): the widest register-resident selection variant
    st = synth.Stream(H=2, d=64, F=F_PAPER, dtype="bf16", layer=23)
    w = run_stream(st, 23, 21 * F_PAPER, 4, check_steps={21, 22}, device_fn=device_stream(2, F_PAPER, "bf16", 23))
    assert w["pruned_steps"] == 2


def test_single_head_long_cache_many_parts_per_query_tile():
    # one head, 16 488 cached tokens: the six query-tile pairs are spread over all 148 CTAs, so every pair is
    # merged from about 25 parts (the general path of the merge kernel)
    st = synth.Stream(H=1, d=64, F=F_PAPER, dtype="bf16", layer=24)
    w = run_stream(st, 14, 12 * F_PAPER, 4, check_steps={0, 11, 12, 13}, device_fn=device_stream(1, F_PAPER, "bf16", 24))
    assert w["pruned_steps"] == 2


@pytest.mark.parametrize("bits", [2, 8])
def test_paper_shape_two_and_eight_bits(bits):
    # 16 heads x 1374 tokens with 2-bit and 8-bit caches (their own unpacking paths in the attention kernel):
    # first step, first cached step, first pruning step
    st = synth.Stream(H=16, d=64, F=F_PAPER, dtype="bf16", layer=25 + bits)
    w = run_stream(st, 4, 3 * F_PAPER, bits, check_steps={0, 1, 3})
    assert w["pruned_steps"] == 1


def test_paper_shape_fp16_inputs():
    # float16 inputs at the paper's frame size (the other paper-shape cases feed bfloat16): no conversion on the way
    # into the attention kernel, float16 rounding of the frame's rows in the quantiser's input
    st = synth.Stream(H=4, d=64, F=F_PAPER, dtype="fp16", layer=40)
    w = run_stream(st, 5, 3 * F_PAPER, 4)
    assert w["checked"] == 5 and w["pruned_steps"] == 2


@pytest.mark.parametrize("dtype,L_max", [("bf16", 2 * F_PAPER + 700), ("fp16", 0)])
def test_paper_shape_unquantised_cache(dtype, L_max):
    # bits = 16: raw rows staged through shared memory by the attention kernel's producers; paper-sized frames (a ragged
    # last tile of 94 rows in the frame, ragged cache ends after pruning), pruning on (bf16) and off (fp16)
    st = synth.Stream(H=4, d=64, F=F_PAPER, dtype=dtype, layer=41)
    w = run_stream(st, 4, L_max, 16, max_cache_tokens=-1 if L_max else 4 * F_PAPER)
    assert w["checked"] == 4 and w["pruned_steps"] == (2 if L_max else 0)


def test_unquantised_fp16_cache_fed_by_the_copy_engine():
    # fp16 inputs with bits = 16: K and V tiles reach shared memory by tensor-map bulk copies (rows past the end of the
    # cache or of the frame arrive as zeros).  Ragged sizes: 300-token frames (a 44-row last tile), a cache that ends
    # inside a tile after pruning, several heads; every step checked.  Then two such streams in one launch.
    st = synth.Stream(H=3, d=64, F=300, dtype="fp16", layer=43)
    w = run_stream(st, 7, 1000, 16)
    assert w["checked"] == 7 and w["pruned_steps"] >= 3
    streams = [synth.Stream(H=3, d=64, F=300 - 40 * i, dtype="fp16", layer=44 + i) for i in range(2)]
    w = run_batch(streams, 6, 900, 16, starts=[0, 1])
    assert w["pruned_steps"] >= 4


@pytest.mark.parametrize("bits", [2, 4])
def test_frames_of_alternating_size(bits):
    # frame sizes differ from step to step (inputs resized to a maximum edge have varying token counts):
    # Eq. 8 with T_first and T_current as separate quantities; every step checked
    sizes = [F_PAPER, 1029, F_PAPER, 1029, 1029, F_PAPER, 1029, F_PAPER]
    big = synth.Stream(H=2, d=64, F=F_PAPER, dtype="bf16", layer=30 + bits)

    def frame(t):
        q, k, v = big.frame(t)
        n = sizes[t]
        return q[:, :n].copy(), k[:, :n].copy(), v[:, :n].copy()

    w = run_stream(big, len(sizes), 4500, bits, frame_fn=frame, max_frame_tokens=F_PAPER)
    assert w["checked"] == len(sizes) and w["pruned_steps"] >= 4


def test_first_frame_smaller_than_later_ones():
    sizes = [300, 500, 420, 500, 300, 500]
    big = synth.Stream(H=3, d=64, F=500, dtype="fp16", layer=33)

    def frame(t):
        q, k, v = big.frame(t)
        n = sizes[t]
        return q[:, :n].copy(), k[:, :n].copy(), v[:, :n].copy()

    w = run_stream(big, len(sizes), 1300, 4, frame_fn=frame, max_frame_tokens=500)
    assert w["pruned_steps"] >= 2
    # beyond max_frame_tokens the step is refused and the cache is unchanged
    c = binding.Cache(1, 3, 64, 1300, 4)
    c.set_options(max_frame_tokens=400)
    Q = torch.zeros(3, 401, 64, device="cuda", dtype=torch.float16)
    out = torch.empty_like(Q)
    with pytest.raises(binding.XsvError) as e:
        c.step(0, Q, Q, Q, out)
    assert e.value.code == 2 and c.len(0) == 0
    c.destroy()


@pytest.mark.parametrize("centre,eps", [(1.0, 1e-3), (1.0, 1e-7), (100.0, 1e-5), (-100.0, 1e-7)])
def test_near_constant_key_channel_far_from_zero(centre, eps):
    # one key channel per head equal to centre + eps * N(0,1): its groups get a tiny scale beside a large offset.
    # fp16 keys cannot hold 1 + 1e-7, but re-quantised kept keys are float32 and reach such groups; bf16 inputs with
    # a spread below their resolution give exactly constant groups (the degenerate rule)
    base = synth.Stream(H=2, d=64, F=130, dtype="bf16", layer=34)
    rng = np.random.Generator(np.random.Philox(key=np.array([7, 34], dtype=np.uint64)))

    def frame(t):
        q, k, v = base.frame(t)
        k = k.copy()
        k[:, :, 9] = synth.round_to_dtype((centre + eps * rng.standard_normal(k[:, :, 9].shape)).astype(np.float32), "bf16")
        k[:, :, 40] = synth.round_to_dtype(np.full_like(k[:, :, 40], centre * 3), "bf16")
        return q, k, v

    w = run_stream(base, 7, 520, 4, frame_fn=frame)
    assert w["pruned_steps"] >= 3


def test_requantised_groups_with_tiny_scale_reach_the_attention_kernel():
    # a cache state built by hand and imported: float32 key groups 1 +- 1e-7 (scale about 1e-8 beside an offset of
    # 1, below what fp16 holds as a normal number) as re-quantised kept keys can form them; the attention over it
    # must match the oracle
    H, F, T, bits = 2, 64, 192, 4
    rng = np.random.Generator(np.random.Philox(key=np.array([8, 35], dtype=np.uint64)))
    Kv = rng.standard_normal((H, T, 64)).astype(np.float32)
    Kv[:, :, 5] = np.float32(1.0) + np.float32(1e-7) * rng.standard_normal((H, T)).astype(np.float32)
    Kv[:, :, 17] = np.float32(-250.0) + np.float32(3e-5) * rng.standard_normal((H, T)).astype(np.float32)
    Vv = rng.standard_normal((H, T, 64)).astype(np.float32)
    kc, ks, kz = orc.quantize_groups(Kv.reshape(H, T // 64, 64, 64).transpose(0, 1, 3, 2), bits)
    vc, vs, vz = orc.quantize_groups(Vv.reshape(H, T, 1, 64), bits)
    state = dict(T=T, Kc=np.ascontiguousarray(kc.transpose(0, 1, 3, 2).reshape(H, T, 64)), Ks=ks, Kz=kz,
                 Vc=vc.reshape(H, T, 64), Vs=vs.reshape(H, T), Vz=vz.reshape(H, T), origin=np.arange(T, dtype=np.int64))
    assert ks.min() < 1e-6 and np.abs(kz).max() > 200
    ref = orc.LayerCache(H, 64, 0, bits)
    ref.load_state(3, F, state["Kc"], ks, kz, state["Vc"], vs, vz, state["origin"])
    c = binding.Cache(1, H, 64, 0, bits)
    c.set_options(max_cache_tokens=512)
    c.import_layer(0, state, frames_done=3, frame_tokens=F, dtype_code=binding.F16)
    st = synth.Stream(H=H, d=64, F=F, dtype="fp16", layer=35)
    q, k, v = st.frame(0)
    out = torch.empty(H, F, 64, device="cuda", dtype=torch.float16)
    c.step(0, to_dev(q, "fp16"), to_dev(k, "fp16"), to_dev(v, "fp16"), out)
    o_ref = ref.step(q, k, v)
    e = float(np.max(np.abs(out.float().cpu().numpy() - o_ref)) / np.max(np.abs(o_ref)))
    assert e <= 1e-2, e
    assert c.status() == 0
    c.destroy()


def test_bf16_inputs_at_the_edges_of_the_fp16_range():
    # bf16 magnitudes up to 65 280 (the largest bf16 below the fp16 limit) and down to 2^-20 are inside the supported
    # range; a value of 2^16 is not and is reported through the status word
    H, F = 2, 140
    st = synth.Stream(H=H, d=64, F=F, dtype="bf16", layer=36)

    def frame(t):
        q, k, v = st.frame(t)
        q, k, v = q.copy(), k.copy(), v.copy()
        v[:, 3::17, 5] = 65280.0
        v[:, 5::19, 6] = -65280.0
        v[:, 1::7, 8] = 2.0 ** -20
        k[:, 2::11, 3] = 2.0 ** -18
        q[:, 4::13, 3] = 2.0 ** -16
        k[:, 7, 1] = 300.0
        return q, k, v

    w = run_stream(st, 6, 0, 16, frame_fn=frame, max_cache_tokens=1024)           # raw 16-bit cache: the inputs themselves
    assert w["checked"] == 6
    q, k, v = frame(0)
    v[0, 0, 0] = 65536.0
    out = torch.empty(H, F, 64, device="cuda", dtype=torch.bfloat16)
    c = binding.Cache(1, H, 64, 1000, 4)              # a quantised cache attends over fp16 operands: out of range
    c.step(0, to_dev(q, "bf16"), to_dev(k, "bf16"), to_dev(v, "bf16"), out)
    assert c.status() == 7                                                         # XSV_ERR_RANGE
    c.destroy()
    c = binding.Cache(1, H, 64, 0, 16)                # an unquantised bf16 cache attends over bf16 operands: no such limit
    c.step(0, to_dev(q, "bf16"), to_dev(k, "bf16"), to_dev(v, "bf16"), out)
    assert c.status() == 0 and bool(torch.isfinite(out.float()).all())
    c.destroy()


def test_config2_mid_and_last_frames():
    # configuration 2 (200 frames, 4-bit) at a middle and at the last frame of a deeper layer; the frames in between
    # are drawn on the device, the state before each checked step is held to the invariants
    c = synth.CONFIGS[2]
    st = synth.config_stream(2, layer=7)
    w = run_stream(st, 200, c["L_max"], c["bits"], check_steps={99, 199}, layers=2, layer=1,
                   device_fn=device_stream(c["H"], c["F"], c["dtype"], seed=102))
    assert w["checked"] == 2 and w["pruned_steps"] == 2


@pytest.mark.parametrize("bits", [2, 4])
def test_config3_long_horizon_samples(bits):
    # configuration 3 (1000 frames, budget 10 992, drifting means) at frames 100, 500 and the last one; once at its
    # own 2 bits and once at 4 bits.  Scores, kept sets, codes, scales and zero-points are compared at every sample.
    # Kept keys are quantised again after every pruning step; the minimum-offset quantiser reproduces a group's
    # extremes exactly, so key magnitudes must stay those of the inputs over all 1000 frames (with a rounded integer
    # zero-point they were measured to grow tenfold within a hundred frames at 2 bits).  The magnitude is asserted,
    # and with it every sample's attention output is compared.
    c = synth.CONFIGS[3]
    st = synth.config_stream(3, layer=4)
    w = run_stream(st, 1000, c["L_max"], bits, check_steps={100, 500, 999}, key_magnitude_limit=128.0,
                   device_fn=device_stream(c["H"], c["F"], c["dtype"], seed=103, drift_rho=c["drift_rho"]))
    assert w["checked"] == 3 and w["pruned_steps"] == 3
    assert w["attn_skipped"] == 0 and w["key_magnitude"] < 128.0


@pytest.mark.parametrize("B", [2, 4, 8])
def test_several_streams_in_one_launch(B):
    # B independent video streams stepped together: one attention launch for all of them, every stream compared with
    # its own oracle at every step.  The streams join one frame apart, so that their cache lengths differ and some
    # prune while others still append; frame sizes differ between streams as well
    streams = [synth.Stream(H=4, d=64, F=200 - 15 * (i % 3), dtype="bf16", layer=60 + i) for i in range(B)]
    w = run_batch(streams, 7 + B // 2, 640, 4, starts=[i // 2 for i in range(B)])
    assert w["pruned_steps"] >= 2 * B and w["checked"] >= 5 * B


def test_two_streams_at_paper_shape_and_two_bits():
    streams = [synth.Stream(H=16, d=64, F=F_PAPER, dtype="bf16", layer=70 + i) for i in range(2)]
    w = run_batch(streams, 5, 3 * F_PAPER, 2, starts=[0, 1], check_steps={3, 4}, deferred_join=True)
    assert w["pruned_steps"] >= 3


def test_eight_long_streams_are_launched_in_groups():
    # eight streams whose caches are long enough that the library splits the call into two attention launches of four
    # streams each (148 CTAs do not divide evenly by eight); the last step is compared with each stream's oracle
    streams = [synth.Stream(H=4, d=64, F=F_PAPER, dtype="bf16", layer=80 + i) for i in range(8)]
    w = run_batch(streams, 18, 16 * F_PAPER, 4, check_steps={17}, deferred_join=True)
    assert w["checked"] == 8 and w["pruned_steps"] == 8


def test_batch_rejects_mismatched_caches_before_launching():
    a, b = binding.Cache(1, 4, 64, 500, 4), binding.Cache(1, 4, 64, 500, 2)
    Q = torch.zeros(4, 100, 64, device="cuda", dtype=torch.float16)
    outs = [torch.empty_like(Q), torch.empty_like(Q)]
    with pytest.raises(binding.XsvError) as e:
        binding.step_batch([a, b], 0, [Q, Q], [Q, Q], [Q, Q], outs)
    assert e.value.code == 2 and a.len(0) == 0 and b.len(0) == 0           # different bit widths: nothing was stepped
    with pytest.raises(binding.XsvError) as e:
        binding.step_batch([a, a], 0, [Q, Q], [Q, Q], [Q, Q], outs)
    assert e.value.code == 1 and a.len(0) == 0
    a.destroy(); b.destroy()


def test_config1_every_step():
    # configuration 1 in full: 64 frames at paper shape, every step checked, so that each imported state was itself
    # verified by the step before it, back to the empty cache
    c = synth.CONFIGS[1]
    st = synth.config_stream(1)
    w = run_stream(st, c["frames"], c["L_max"], c["bits"])
    assert w["checked"] == 64 and w["pruned_steps"] == 48
