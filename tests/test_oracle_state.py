"""Invariants of the oracle's cache update (Fig. 2 steps 3-5; Eq. 8-11)."""
import numpy as np
import pytest

from oracle import xsv_oracle as orc
from paper_2602_21780_b200 import synth


def _stream(H=4, d=64, F=70, frames=7, dtype="fp16"):
    st = synth.Stream(H=H, d=d, F=F, dtype=dtype, layer=1)
    return [st.frame(t) for t in range(frames)]

def _old_state(cache):
    return dict(Kc=cache.Kc.copy(), Ks=cache.Ks.copy(), Kz=cache.Kz.copy(), Vc=cache.Vc.copy(),
                Vs=cache.Vs.copy(), Vz=cache.Vz.copy(), origin=cache.origin.copy(), T=cache.T,
                Kd=cache.dequant_K().copy())


def check_requantised_keys(old, new, K_fresh, F, G, bits):
    """Section 3.3 (quantisation is applied to the final cache, kept and fresh keys alike): every key group of the
    new order that is not frozen holds the Eq. 9-10 quantisation of its members' SOURCE values -- for a kept token
    the dequantised value it had in the old cache (found through its origin, not through the oracle's own gather),
    for a token of the current frame its input.  Checked: the per-element error bound s/2, and that the stored
    (s, z) and codes are what the quantiser gives on those source values."""
    T_new, H, d = new["T"], new["Kc"].shape[0], new["Kc"].shape[2]
    n_kept = T_new - F
    pos_old = {int(o): i for i, o in enumerate(old["origin"])}
    src = np.array([pos_old[int(o)] for o in new["origin"][:n_kept]], dtype=np.int64)
    source = np.concatenate([old["Kd"][:, src, :], np.asarray(K_fresh, np.float32)], axis=1)   # [H, T_new, d]
    grp = np.arange(T_new) // G
    dk_new = orc.dequantize(new["Kc"], new["Ks"][:, grp, :], new["Kz"][:, grp, :]).astype(np.float64)
    s_tok = new["Ks"][:, grp, :].astype(np.float64)
    fz = new["frozen"]
    lo = fz * G
    assert np.all(np.abs(dk_new[:, lo:] - source[:, lo:]) <= 0.5 * s_tok[:, lo:] * (1 + 2.0 ** -12))
    # frozen groups: values unchanged
    assert np.array_equal(dk_new[:, :lo].astype(np.float32), source[:, :lo])
    for gi in range(fz, -(-T_new // G)):
        a, b = gi * G, min((gi + 1) * G, T_new)
        c, s, z = orc.quantize_groups(source[:, a:b, :].transpose(0, 2, 1), bits)
        assert np.array_equal(s.view(np.uint32), np.ascontiguousarray(new["Ks"][:, gi]).view(np.uint32)), f"group {gi}: scale"
        assert np.array_equal(z, new["Kz"][:, gi]), f"group {gi}: zero-point"
        assert np.array_equal(c.transpose(0, 2, 1), new["Kc"][:, a:b]), f"group {gi}: codes"
        # the group's extremes are reproduced at the ends of the code range
        mn, mx = source[:, a:b].min(axis=1), source[:, a:b].max(axis=1)
        live = mx > mn
        assert np.all(new["Kc"][:, a:b].min(axis=1)[live] == 0)
        assert np.all(new["Kc"][:, a:b].max(axis=1)[live] >= (1 << bits) - 2)


def _new_state(cache):
    return dict(Kc=cache.Kc, Ks=cache.Ks, Kz=cache.Kz, origin=cache.origin, T=cache.T,
                frozen=cache.last_frozen_groups)


@pytest.mark.parametrize("bits", [2, 4, 8])
def test_kept_keys_are_requantised_from_their_dequantised_source(bits):
    H, d, F, G, L_max = 3, 64, 70, 64, 300
    cache = orc.LayerCache(H, d, L_max, bits)
    pruned = 0
    for t, (Q, K, V) in enumerate(_stream(H, d, F, frames=8)):
        old = _old_state(cache)
        cache.step(Q, K, V)
        check_requantised_keys(old, _new_state(cache), K, F, G, bits)
        pruned += cache.last_scores is not None
    assert pruned >= 3


def test_requantisation_pin_catches_a_wrong_gather():
    # plant mistakes in the oracle's result (never in the CUDA path): kept keys taken from the neighbouring slot,
    # and kept keys gathered in the wrong order inside one group; the pin must reject both
    H, d, F, G, bits, L_max = 3, 64, 70, 64, 4, 300
    cache = orc.LayerCache(H, d, L_max, bits)
    frames = _stream(H, d, F, frames=6)
    for Q, K, V in frames[:5]:
        cache.step(Q, K, V)
    old = _old_state(cache)
    Q, K, V = frames[5]
    cache.step(Q, K, V)
    assert cache.last_scores is not None
    good = _new_state(cache)
    check_requantised_keys(old, good, K, F, G, bits)
    fz, n_kept = good["frozen"], good["T"] - F
    assert fz * G + 2 < n_kept
    shifted = dict(good, Kc=good["Kc"].copy())
    shifted["Kc"][:, fz * G + 1:n_kept] = good["Kc"][:, fz * G:n_kept - 1]       # every kept key one slot late
    with pytest.raises(AssertionError):
        check_requantised_keys(old, shifted, K, F, G, bits)
    swapped = dict(good, Kc=good["Kc"].copy())
    a = fz * G
    swapped["Kc"][:, [a, a + 1]] = good["Kc"][:, [a + 1, a]]
    with pytest.raises(AssertionError):
        check_requantised_keys(old, swapped, K, F, G, bits)


def test_state_update_invariants_quantised():
    H, d, F, G, bits, L_max = 4, 64, 70, 64, 4, 300
    cache = orc.LayerCache(H, d, L_max, bits)
    for t, (Q, K, V) in enumerate(_stream(H, d, F)):
        old = dict(Kc=cache.Kc.copy(), Ks=cache.Ks.copy(), Kz=cache.Kz.copy(), Vc=cache.Vc.copy(),
                   Vs=cache.Vs.copy(), Vz=cache.Vz.copy(), origin=cache.origin.copy(), T=cache.T)
        cache.step(Q, K, V)
        T = cache.T
        assert T == orc.expected_cache_len(t + 1, F, L_max)
        assert cache.Kc.shape == (H, T, d) and cache.Ks.shape == (H, -(-T // G), d)
        assert cache.Vs.shape == (H, T, 1)
        assert np.all(np.diff(cache.origin) > 0)
        assert np.array_equal(cache.origin[:F], np.arange(F))
        assert np.array_equal(cache.origin[-F:], t * F + np.arange(F))
        # kept tokens: V codes and parameters carried verbatim
        pos_old = {int(o): i for i, o in enumerate(old["origin"])}
        src = np.array([pos_old[int(o)] for o in cache.origin[:-F]], dtype=np.int64)
        assert np.array_equal(cache.Vc[:, :T - F], old["Vc"][:, src])
        assert np.array_equal(cache.Vs[:, :T - F], old["Vs"][:, src])
        assert np.array_equal(cache.Vz[:, :T - F], old["Vz"][:, src])
        # fresh V rows: direct quantisation of the inputs, error <= s/2
        dv = cache.dequant_V()[:, -F:].astype(np.float64)
        assert np.all(np.abs(dv - V) <= 0.5 * cache.Vs[:, -F:].astype(np.float64) * (1 + 2.0 ** -12))
        # frozen K prefix: identical codes and parameters
        fz = cache.last_frozen_groups
        moved = np.nonzero(src != np.arange(src.shape[0]))[0]
        first_moved = int(moved[0]) if moved.size else old["T"]
        assert fz == min(first_moved, old["T"]) // G
        assert np.array_equal(cache.Kc[:, :fz * G], old["Kc"][:, :fz * G])
        assert np.array_equal(cache.Ks[:, :fz], old["Ks"][:, :fz])
        # requantised K: every value stays inside its old group's range, and the
        # fresh frame's keys are within s/2 of the inputs
        dk = cache.dequant_K().astype(np.float64)
        grp = np.arange(T) // G
        s_tok = cache.Ks[:, grp, :].astype(np.float64)
        assert np.all(np.abs(dk[:, -F:] - K) <= 0.5 * s_tok[:, -F:] * (1 + 2.0 ** -12) + 1e-6)
        if t >= 1:
            assert cache.last_scores is None or cache.last_scores.shape[0] == old["T"] - F
    assert cache.kv_bytes_packed() == 2 * H * T * d // 2 + H * (-(-T // G)) * d * 8 + H * T * 8


def test_scored_keys_are_the_dequantised_cache_middle():
    # the selection made inside step() equals Eq. 8 applied to Eq. 3-7 evaluated on the
    # dequantised cache as it stood before the step
    H, d, F, bits, L_max = 2, 64, 40, 2, 100
    cache = orc.LayerCache(H, d, L_max, bits)
    for t, (Q, K, V) in enumerate(_stream(H, d, F, frames=5)):
        Kd, T_c = cache.dequant_K().copy(), cache.T
        cache.step(Q, K, V)
        if t >= 1 and T_c + F > L_max:
            S = orc.importance_scores(Q, Kd[:, F:T_c], 5, 16)
            assert np.array_equal(S, cache.last_scores)
            keep = orc.keep_positions(S, F, F, T_c + F, L_max)
            assert np.array_equal(keep, cache.last_keep)
            worst_kept = S[keep[F:-F] - F].min()
            evicted = np.setdiff1d(np.arange(F, T_c), keep)
            assert S[evicted - F].max() <= worst_kept


def test_fp_cache_holds_gathered_inputs_exactly():
    H, d, F, L_max = 2, 64, 30, 80
    cache = orc.LayerCache(H, d, L_max, 16)
    hist = []
    for Q, K, V in _stream(H, d, F, frames=5):
        cache.step(Q, K, V)
        hist.append((K, V))
        Kh = np.concatenate([k for k, _ in hist], axis=1)
        assert np.array_equal(cache.Kc, Kh[:, cache.origin])
