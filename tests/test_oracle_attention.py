"""Pins for the oracle's attention (Eq. 2) and for pruning's effect on it."""
import numpy as np
import torch

from oracle import xsv_oracle as orc


def _sdpa(q, k, v, mask=None):
    # library softmax attention, float64, default scale 1/sqrt(d)
    o = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(q), torch.from_numpy(k), torch.from_numpy(v),
        attn_mask=None if mask is None else torch.from_numpy(mask))
    return o.numpy()


def _frames(n, H, F, d, seed):
    rng = np.random.default_rng(seed)
    return [tuple(rng.standard_normal((H, F, d)).astype(np.float16).astype(np.float32)
                  for _ in range(3)) for _ in range(n)]


def test_unbounded_fp_cache_is_block_causal_attention():
    H, F, d, n = 3, 7, 8, 5
    fr = _frames(n, H, F, d, 0)
    cache = orc.LayerCache(H, d, L_max=0, bits=16, n_special=1, g=2, G=8)
    outs = [cache.step(*f) for f in fr]
    Qa = np.concatenate([f[0] for f in fr], axis=1).astype(np.float64)
    Ka = np.concatenate([f[1] for f in fr], axis=1).astype(np.float64)
    Va = np.concatenate([f[2] for f in fr], axis=1).astype(np.float64)
    fid = np.arange(n * F) // F
    mask = fid[:, None] >= fid[None, :]            # a query sees frames <= its own
    ref = _sdpa(Qa, Ka, Va, mask)
    got = np.concatenate(outs, axis=1)
    assert np.max(np.abs(got - ref)) < 1e-12
    assert cache.T == n * F and np.array_equal(cache.origin, np.arange(n * F))


def test_attention_rows_are_convex_combinations_and_permutation_invariant():
    rng = np.random.default_rng(1)
    Q = rng.standard_normal((2, 5, 8))
    K = rng.standard_normal((2, 11, 8))
    V = np.ones((2, 11, 8))
    assert np.allclose(orc.attention(Q, K, V), 1.0, atol=1e-13)
    V = rng.standard_normal((2, 11, 8))
    p = rng.permutation(11)
    assert np.allclose(orc.attention(Q, K, V), orc.attention(Q, K[:, p], V[:, p]), atol=1e-13)
    # one key only -> output is that value row
    assert np.allclose(orc.attention(Q, K[:, :1], V[:, :1]), np.broadcast_to(V[:, :1], (2, 5, 8)))


def test_pruned_fp_cache_equals_attention_over_kept_tokens():
    H, F, d, n = 2, 9, 8, 7
    L_max = 30
    fr = _frames(n, H, F, d, 2)
    cache = orc.LayerCache(H, d, L_max=L_max, bits=16, n_special=1, g=4, G=8)
    Kh = np.zeros((H, 0, d), np.float32)
    Vh = np.zeros((H, 0, d), np.float32)
    for t, (Q, K, V) in enumerate(fr):
        kept = cache.origin.copy()                  # tokens the step will attend to
        out = cache.step(Q, K, V)
        Kh = np.concatenate([Kh, K], axis=1)
        Vh = np.concatenate([Vh, V], axis=1)
        idx = np.concatenate([kept, t * F + np.arange(F)])
        ref = _sdpa(Q.astype(np.float64), Kh[:, idx].astype(np.float64), Vh[:, idx].astype(np.float64))
        assert np.max(np.abs(out - ref)) < 1e-12
        assert cache.T == orc.expected_cache_len(t + 1, F, L_max)
        # first and current frames always present, positions ascending
        assert np.array_equal(cache.origin[:F], np.arange(F))
        assert np.array_equal(cache.origin[-F:], t * F + np.arange(F))
        assert np.all(np.diff(cache.origin) > 0)
    assert cache.T == max(L_max, 2 * F)


def test_budget_below_two_frames_keeps_first_and_current_only():
    H, F, d = 1, 6, 8
    fr = _frames(4, H, F, d, 3)
    cache = orc.LayerCache(H, d, L_max=8, bits=16, n_special=1, g=2, G=8)
    for t, f in enumerate(fr):
        cache.step(*f)
        if t >= 1:
            assert np.array_equal(cache.origin, np.concatenate([np.arange(F), t * F + np.arange(F)]))
