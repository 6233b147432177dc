"""CPU oracle for the XStreamVGGT compressed-KV streaming attention step.

TEST INFRASTRUCTURE ONLY.  This module is the slow, plain statement of what the
hot path computes, written from the paper's equations.  It shares no code with
the CUDA library, imports nothing from it, and may be imported only by the
tests, by the smoke check and by the benchmark's cpu-baseline leg.

Notation follows the paper: H heads, d channels per head, F tokens per frame
(1 camera + R register + N patch tokens), L_max the cache budget, g the query
pooling group, G the quantisation group, b the bit width, n = 2^b - 1.

Arithmetic: attention, pooling, scoring are accumulated in float64.  The
quantiser (Eq. 9-10) and dequantiser (Eq. 12) are carried out in IEEE float32
with one operation per rounding, because their results are integer codes and
float32 scales and offsets that the GPU must reproduce bit for bit.

Pins (tests/test_oracle_*.py): block-causal attention against a library
softmax-attention routine; attention after pruning against attention over the
gathered kept tokens; scores against a hand-worked example, a closed form for
constant inputs and the linearity identity; selection against the pairwise
"beaten by fewer than k" definition; the quantiser against hand-worked codes,
the s/2 error bound, min->0, constant groups and an exhaustive two-element
sweep; the state update against its invariants.  The whole-stream numbers have
no printed counterpart in the paper (it gives no worked numeric example).
"""
from __future__ import annotations

import numpy as np

F32 = np.float32
TINY = F32(2.0 ** -126)


# --------------------------------------------------------------------------
# Eq. 9-10: asymmetric uniform quantiser, one group at a time (vectorised over
# leading axes; the group is the LAST axis of `x`).
#
# Form.  Section 3.3 prints the quantiser with an integer zero-point,
# code = round(x / s) + z with z = round(-x_min / s); section 4.1 says the
# quantisation is carried out with KIVI, whose quantiser subtracts the group
# minimum instead: code = round((x - x_min) / s), x~ = code * s + x_min.  The two
# differ by the rounding of the zero-point, i.e. by a shift of the whole grid of
# up to s/2.  The cache is quantised again after every pruning step (section
# 3.3: quantisation is applied to the final cache, kept and new entries alike),
# and under that repetition the difference decides: with the minimum subtracted
# a group's extremes are reproduced exactly, so ranges never outgrow the data;
# with the rounded zero-point every pass shifts them, the selection keeps the
# keys with the largest projections, and at 2 bits key magnitudes were measured
# to grow tenfold within a few hundred frames.  The minimum-offset form is the
# reading taken here; `z` below is that offset (a float32 in value units).
# --------------------------------------------------------------------------
def quantize_groups(x, bits):
    """Quantise each row of x[..., m] as one group (Eq. 9-10, minimum-offset form).

    s = (x_max - x_min) / (2^b - 1); z = x_min;
    code = clamp(round((x - z) / s), 0, 2^b - 1); round = nearest, ties to even.
    All in float32, one rounding per operation: one subtraction for the range,
    one true division for s, then per element one subtraction and one true
    division.  Degenerate group (s below the smallest normal float32, which
    includes x_max == x_min): s := 1, which gives code 0 everywhere and the
    dequantised value x_min exactly.
    Returns (codes uint8 [..., m], s float32 [...], z float32 [...]).
    """
    x = np.asarray(x, dtype=F32)
    n = (1 << bits) - 1
    mn = x.min(axis=-1).astype(F32)
    mx = x.max(axis=-1).astype(F32)
    with np.errstate(divide="ignore", invalid="ignore", over="ignore"):
        s = ((mx - mn).astype(F32) / F32(n)).astype(F32)
        s = np.where(s >= TINY, s, F32(1.0)).astype(F32)
        y = (x - mn[..., None]).astype(F32)
        q = np.rint((y / s[..., None]).astype(F32))
    codes = np.clip(q.astype(np.float64), 0, n).astype(np.uint8)
    return codes, s, mn


def dequantize(codes, s, z):
    """Eq. 12 (inverse of Eq. 9): x~ = code * s + z, a float32 multiply followed by a float32 add
    (two roundings; no fused multiply-add).

    codes [..., m]; s, z broadcastable to codes' shape."""
    prod = (codes.astype(F32) * np.asarray(s, dtype=F32)).astype(F32)
    return (prod + np.asarray(z, dtype=F32)).astype(F32)


def quantization_mse(x, bits, granularity, G=64):
    """Mean squared error of Eq. 9-12 under one of the two granularities of Eq. 11 (the quantity of Table 1).

    x [H, T, d] (d == G).  granularity "channel": one (s, z) per channel per group of G consecutive tokens (the
    scheme Eq. 11 assigns to keys; a last, partial group holds the remaining tokens); "token": one (s, z) per token
    over its d channels (the scheme for values).  Quantise, dequantise, and average (x - x~)^2 over all elements
    in float64.
    """
    x = np.asarray(x, dtype=F32)
    H, T, d = x.shape
    if granularity == "token":
        c, s, z = quantize_groups(x, bits)                       # groups along the channel axis
        xh = dequantize(c, s[..., None], z[..., None])
    elif granularity == "channel":
        xh = np.empty_like(x)
        for t0 in range(0, T, G):
            blk = x[:, t0:t0 + G, :].transpose(0, 2, 1)           # [H, d, tokens of the group]
            c, s, z = quantize_groups(blk, bits)
            xh[:, t0:t0 + G, :] = dequantize(c, s[..., None], z[..., None]).transpose(0, 2, 1)
    else:
        raise ValueError(granularity)
    e = x.astype(np.float64) - xh.astype(np.float64)
    return float(np.mean(e * e))


# --------------------------------------------------------------------------
# Eq. 2: attention of one frame's queries over [cache ; current frame].
# --------------------------------------------------------------------------
def attention(Q, K_all, V_all):
    """softmax(Q K_all^T / sqrt(d)) V_all per head, float64.

    Q [H, F, d]; K_all, V_all [H, T, d].  Causality is frame-granular: every
    query of the current frame sees every cached token and every token of its
    own frame, so inside one step there is no mask."""
    Q = np.asarray(Q, dtype=np.float64)
    K_all = np.asarray(K_all, dtype=np.float64)
    V_all = np.asarray(V_all, dtype=np.float64)
    H, Fq, d = Q.shape
    out = np.empty((H, Fq, d), dtype=np.float64)
    inv_sqrt_d = 1.0 / np.sqrt(float(d))
    for h in range(H):
        logits = (Q[h] @ K_all[h].T) * inv_sqrt_d
        logits -= logits.max(axis=1, keepdims=True)
        w = np.exp(logits)
        w /= w.sum(axis=1, keepdims=True)
        out[h] = w @ V_all[h]
    return out


# --------------------------------------------------------------------------
# Eq. 3-7: token-importance scores from pooled queries.
# --------------------------------------------------------------------------
def pooled_query(Q, n_special, g):
    """Eq. 3: keep the first n_special rows (camera + register tokens) as they
    are, average the patch rows in consecutive groups of g (a short last group
    is averaged over its own members), concatenate.  Q [H, F, d] ->
    [H, N_pooled, d] float64."""
    Q = np.asarray(Q, dtype=np.float64)
    H, Fq, d = Q.shape
    special = Q[:, :n_special, :]
    normal = Q[:, n_special:, :]
    n_norm = normal.shape[1]
    rows = [special]
    for a in range(0, n_norm, g):
        rows.append(normal[:, a:a + g, :].mean(axis=1, keepdims=True))
    return np.concatenate(rows, axis=1)


def importance_scores(Q, K_prunable, n_special, g):
    """Eq. 3-7 taken literally.

    Q [H, F, d] current frame's queries; K_prunable [H, T_p, d] the cached
    (dequantised) keys of the prunable middle segment.
    Q_bar = mean over heads of the pooled query (Eq. 4);
    K_bar = mean over heads of the prunable keys (Eq. 5);
    S_matrix = Q_bar K_bar^T (Eq. 6, plain inner product, no scaling, no
    softmax); S = mean over the pooled-query rows (Eq. 7).  float64 [T_p]."""
    Qp = pooled_query(Q, n_special, g)
    Q_bar = Qp.mean(axis=0)
    K_bar = np.asarray(K_prunable, dtype=np.float64).mean(axis=0)
    S_matrix = Q_bar @ K_bar.T
    return S_matrix.mean(axis=0)


def importance_scores_collapsed(Q, K_prunable, n_special, g):
    """Same scores through the linearity identity S[j] = q~ . K_bar[j] with
    q~ the mean of Q_bar's rows.  Used by a test as a cross-check only."""
    Qp = pooled_query(Q, n_special, g)
    q_tilde = Qp.mean(axis=0).mean(axis=0)
    K_bar = np.asarray(K_prunable, dtype=np.float64).mean(axis=0)
    return K_bar @ q_tilde


# --------------------------------------------------------------------------
# Eq. 8: keep set.
# --------------------------------------------------------------------------
def select_middle(S, k):
    """Top-k of the middle segment's scores.  Total order: higher score first,
    equal scores by lower position first.  Returns the selected positions
    (relative to the segment) in ascending order."""
    S = np.asarray(S)
    k = int(max(0, min(k, S.shape[0])))
    order = np.lexsort((np.arange(S.shape[0]), -S.astype(np.float64)))
    return np.sort(order[:k]).astype(np.int64)


def keep_positions(S, T_first, T_current, T, L_max):
    """Eq. 8: I_keep = first frame  U  top-k of the middle  U  current frame,
    k = max(0, L_max - T_first - T_current), as ascending positions in [0, T)."""
    T_p = T - T_first - T_current
    assert S.shape[0] == T_p
    k = max(0, L_max - T_first - T_current)
    mid = select_middle(S, k) + T_first
    return np.concatenate([np.arange(T_first, dtype=np.int64), mid,
                           np.arange(T - T_current, T, dtype=np.int64)])


# --------------------------------------------------------------------------
# One layer's compressed cache and its streaming step.
# --------------------------------------------------------------------------
class LayerCache:
    """State of one layer's cache in its logical (unpacked) form.

    bits in {2,4,8}: Kc/Vc uint8 codes [H,T,d]; Ks / Kz float32 (scale, offset)
    [H, ceil(T/G), d] (per channel, groups of G consecutive tokens, Eq. 11);
    Vs / Vz float32 [H, T, d/G] (per token, groups of G channels).
    bits == 16: quantisation off, Kc/Vc hold the 16-bit inputs as float32.
    origin[T] = running index of the token in the stream (tokens of all earlier frames + its index in its
    frame; frame_index * F + token_index when every frame holds F tokens) -- a label by which kept sets
    are compared, not part of the method's arithmetic.
    L_max <= 0 means unbounded (no pruning)."""

    def __init__(self, H, d, L_max, bits, n_special=5, g=16, G=64):
        assert bits in (2, 4, 8, 16)
        assert d % G == 0
        self.H, self.d, self.L_max, self.bits = H, d, int(L_max), bits
        self.n_special, self.g, self.G = n_special, g, G
        self.t = 0
        self.F_first = 0
        self.tokens_seen = 0
        self.T = 0
        cdt = F32 if bits == 16 else np.uint8
        self.Kc = np.zeros((H, 0, d), cdt)
        self.Vc = np.zeros((H, 0, d), cdt)
        self.Ks = np.zeros((H, 0, d), F32)
        self.Kz = np.zeros((H, 0, d), F32)
        self.Vs = np.zeros((H, 0, d // G), F32)
        self.Vz = np.zeros((H, 0, d // G), F32)
        self.origin = np.zeros((0,), np.int64)
        self.last_scores = None
        self.last_keep = None

    # ---- Eq. 12 over the whole cache ----
    def dequant_K(self):
        if self.bits == 16:
            return self.Kc
        grp = np.arange(self.T) // self.G
        return dequantize(self.Kc, self.Ks[:, grp, :], self.Kz[:, grp, :])

    def dequant_V(self):
        if self.bits == 16:
            return self.Vc
        H, T, d, G = self.H, self.T, self.d, self.G
        c = self.Vc.reshape(H, T, d // G, G)
        return dequantize(c, self.Vs[..., None], self.Vz[..., None]).reshape(H, T, d)

    def step(self, Q, K, V, select_on=None):
        """One streaming step (Fig. 2): attention over [cache ; frame], then,
        if the total length exceeds the budget, scoring + top-k pruning, then
        quantisation of the resulting cache.  Q, K, V [H, F, d] hold values
        exactly representable in the 16-bit input type.  Returns out float64.

        select_on: for step-locked comparisons only -- an externally supplied
        score vector on which Eq. 8 is evaluated instead of this step's own
        scores (which are still computed and kept in last_scores), so that the
        cache update can be compared for one and the same keep set."""
        H, d, G = self.H, self.d, self.G
        Q = np.asarray(Q, dtype=F32)
        K = np.asarray(K, dtype=F32)
        V = np.asarray(V, dtype=F32)
        Fc = Q.shape[1]
        T_c = self.T
        Kd = self.dequant_K()
        Vd = self.dequant_V()

        # Eq. 2
        K_all = np.concatenate([Kd, K], axis=1)
        V_all = np.concatenate([Vd, V], axis=1)
        out = attention(Q, K_all, V_all)

        # append, then decide whether pruning is triggered (T > L_max)
        self.t += 1
        if self.t == 1:
            self.F_first = Fc
        T = T_c + Fc
        T_first = self.F_first
        prune = self.t >= 2 and self.L_max > 0 and T > self.L_max
        self.last_scores = None
        if prune:
            S = importance_scores(Q, Kd[:, T_first:T_c, :], self.n_special, self.g)
            keep = keep_positions(S if select_on is None else np.asarray(select_on), T_first, Fc, T, self.L_max)
            self.last_scores = S
        else:
            keep = np.arange(T, dtype=np.int64)
        self.last_keep = keep

        from_cache = keep[keep < T_c]          # kept cached tokens, ascending
        n_old = from_cache.shape[0]
        T_new = keep.shape[0]
        assert np.all(keep[n_old:] == np.arange(T_c, T))
        origin_new = np.concatenate(
            [self.origin[from_cache], self.tokens_seen + np.arange(Fc, dtype=np.int64)])
        self.tokens_seen += Fc

        if self.bits == 16:
            self.Kc = np.concatenate([self.Kc[:, from_cache], K], axis=1)
            self.Vc = np.concatenate([self.Vc[:, from_cache], V], axis=1)
            self.origin, self.T = origin_new, T_new
            return out

        # ---- V: kept tokens carry codes and (s, z) verbatim; fresh rows are
        # quantised per token over groups of G channels (Eq. 9-11).
        vc, vs, vz = quantize_groups(V.reshape(H, Fc, d // G, G), self.bits)
        Vc_new = np.concatenate([self.Vc[:, from_cache], vc.reshape(H, Fc, d)], axis=1)
        Vs_new = np.concatenate([self.Vs[:, from_cache], vs], axis=1)
        Vz_new = np.concatenate([self.Vz[:, from_cache], vz], axis=1)

        # ---- K: groups of G consecutive tokens of the NEW order, per channel.
        # A group is frozen (carried verbatim) if it lies wholly before the
        # first evicted position and was a full group of the old cache;
        # every other group is quantised afresh from the float32 values of its
        # members (dequantised for kept tokens, the inputs for fresh ones).
        evicted = np.setdiff1d(np.arange(T_c, dtype=np.int64), from_cache)
        first_evicted = int(evicted[0]) if evicted.size else T_c
        frozen_groups = min(first_evicted, T_c) // G
        n_groups = -(-T_new // G)
        K_vals = np.concatenate([Kd[:, from_cache], K], axis=1)      # float32 [H,T_new,d]
        Kc_new = np.zeros((H, T_new, d), np.uint8)
        Ks_new = np.zeros((H, n_groups, d), F32)
        Kz_new = np.zeros((H, n_groups, d), F32)
        fz = frozen_groups
        Kc_new[:, :fz * G] = self.Kc[:, :fz * G]
        Ks_new[:, :fz] = self.Ks[:, :fz]
        Kz_new[:, :fz] = self.Kz[:, :fz]
        for gi in range(fz, n_groups):
            a, b_ = gi * G, min((gi + 1) * G, T_new)
            blk = K_vals[:, a:b_, :].transpose(0, 2, 1)            # [H, d, m]: group = last axis
            c, s, z = quantize_groups(blk, self.bits)
            Kc_new[:, a:b_, :] = c.transpose(0, 2, 1)
            Ks_new[:, gi], Kz_new[:, gi] = s, z
        self.Kc, self.Ks, self.Kz = Kc_new, Ks_new, Kz_new
        self.Vc, self.Vs, self.Vz = Vc_new, Vs_new, Vz_new
        self.origin, self.T = origin_new, T_new
        self.last_frozen_groups = frozen_groups
        return out

    # ---- state exchange for step-locked comparisons ----
    def load_state(self, t, F_first, Kc, Ks, Kz, Vc, Vs, Vz, origin):
        self.t, self.F_first = int(t), int(F_first)
        self.T = int(origin.shape[0])
        cdt = F32 if self.bits == 16 else np.uint8
        self.Kc, self.Vc = np.asarray(Kc, cdt), np.asarray(Vc, cdt)
        self.Ks, self.Kz = np.asarray(Ks, F32), np.asarray(Kz, F32)
        self.Vs, self.Vz = np.asarray(Vs, F32), np.asarray(Vz, F32)
        self.origin = np.asarray(origin, np.int64)
        self.tokens_seen = int(self.origin[-1]) + 1 if self.T else 0     # the last frame's last token is always kept

    def kv_bytes_packed(self):
        """Bytes of the packed representation: b-bit codes + float32 scale +
        float32 offset per group (the figure the memory claim is about)."""
        if self.bits == 16:
            return 2 * self.H * self.T * self.d * 2
        code = 2 * self.H * self.T * self.d * self.bits // 8
        kmeta = self.H * (-(-self.T // self.G)) * self.d * 8
        vmeta = self.H * self.T * (self.d // self.G) * 8
        return code + kmeta + vmeta


def expected_cache_len(t, F, L_max):
    """Closed-form cache length after step t (1-based) for constant F."""
    T = t * F
    if t == 1 or L_max <= 0 or T <= L_max:
        return T
    return max(L_max, 2 * F)


def next_cache_len(t, T_c, F_first, F_t, L_max):
    """Cache length after step t (1-based) that appends a frame of F_t tokens to a cache of T_c tokens whose
    first frame holds F_first: the trigger rule of section 3.2 and the size of Eq. 8's keep set."""
    T = T_c + F_t
    if t == 1 or L_max <= 0 or T <= L_max:
        return T
    return F_first + max(0, L_max - F_first - F_t) + F_t
