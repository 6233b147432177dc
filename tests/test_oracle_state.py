"""Invariants of the oracle's cache update (Fig. 2 steps 3-5; Eq. 8-11)."""
import numpy as np

from oracle import xsv_oracle as orc
from paper_2602_21780_b200 import synth


def _stream(H=4, d=64, F=70, frames=7, dtype="fp16"):
    st = synth.Stream(H=H, d=d, F=F, dtype=dtype, layer=1)
    return [st.frame(t) for t in range(frames)]


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
