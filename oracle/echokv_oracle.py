"""EchoKV decode attention -- plain CPU oracle (numpy, fp64).

TEST INFRASTRUCTURE ONLY.  This module defines what the CUDA library must
compute; it is slow, un-blocked and un-fused on purpose.  It shares no code
with the CUDA path and imports nothing from it.  Only the test-suite, the
smoke check and the benchmark's CPU-baseline leg may import it.

Every function takes real-valued numpy arrays (any float dtype; values that
were stored as bf16 or fp32 are widened to float64 exactly by the helpers at
the bottom) and computes in float64 without intermediate rounding.

Notation (paper, Section 3.2 "Network Architecture"):
  L      tokens in the cache
  H_kv   KV heads, d head dim, D = H_kv * d  flattened per-token KV width
  S      group size: layer l is an anchor ("global") layer iff l % S == 0 (Eq. 1)
  m      retained local dims of a compressed layer: C_local = C[:, :m]  (Eq. 2)
  W      predictor, shape [D - m, D + m]; C_hat_drop = W [C_global ; C_local] (Eq. 3)
  C_drop = C[:, m:] is what W predicts (Eq. 4)
  X_tilde = Reshape([X_local ; X_hat_drop]), X in {K, V}            (Eq. 6)
  A(Q, K, V) = softmax(Q K^T / sqrt(d)) V                           (Eq. 7, App. D.1)

Readings of points the paper leaves open (all listed in the design notes):
  * K and V have separate predictors, each seeing only its own kind of cache
    (Table "Hyperparameter configurations": 1408 = 1024 + 384 inputs).
  * no bias unless one is passed (Eq. 3 has none).
  * predictor input order is [global ; local] as written in Eq. 3.
  * flattening is head-major: flat index = head * d + feature.
  * query head h attends KV head floor(h / (H_q / H_kv)) (contiguous groups).
  * every cached token, the newest included, is reconstructed alike, unless a
    sink / recent window is asked for (Section 4.1): those tokens keep all dims.
  * the predictors see keys BEFORE the rotary position embedding (Section 3.2), so a
    cache of such keys must be rotated when it is read: with rope_theta given, every
    row t of K_tilde (retained, predicted or full-precision alike) is rotated to
    position t (half-split pairing of feature j with j + d/2, frequencies
    rope_theta^(-2j/d)) before q . k; q arrives already rotated; V is untouched.
    Without rope_theta (all printed configurations) K_tilde is used as it is.

Pins (tests/test_oracle_*.py): hand-computed softmax case, pure-python brute
force, torch scaled_dot_product_attention (library routine) for the m = D and
selector-weight cases, zero-weight closed forms, linearity, softmax shift /
permutation / log-sum-exp merge invariants, the paper's printed predictor
shapes, ratios and parameter totals; for the rotation: hand values, the complex-
number form, a library rotary routine, and the relative-position property; for an m that splits a
head, whole keys with a window, and the prefill-shaped call with a sink / window: index-by-index brute
force, the windowed decode step on every prefix, causal library attention in the all-true limit, and a
planted mistake.  What stays "parity unpinned": nothing in
the paper prints a numeric attention output, and how well a *trained* W
approximates the dropped cache cannot be checked without trained weights (it is
not part of what the kernels compute).
"""
from __future__ import annotations

import math

import numpy as np

# ----------------------------------------------------------------------------
# Configuration arithmetic (Eq. 1, Eq. 2, Appendix "Compression-Ratio
# Configurations", Table "Hyperparameter configurations")
# ----------------------------------------------------------------------------


def is_anchor_layer(layer: int, group_size: int) -> bool:
    """Eq. 1: the first layer of each group of S layers keeps its full cache."""
    return layer % group_size == 0


def anchor_of(layer: int, group_size: int) -> int:
    """Eq. 1: C_global^(k) = C_{k*S}; the anchor of layer k*S+i is layer k*S."""
    return layer - layer % group_size


def predictor_shape(D: int, m: int) -> tuple[int, int]:
    """(input dim, output dim) of W: input [C_global ; C_local] has D + m
    features, output C_hat_drop has D - m (Eq. 2-4)."""
    if not 0 <= m <= D:
        raise ValueError("need 0 <= m <= D")
    return D + m, D - m


def effective_ratio(D: int, group_size: int, m: int) -> float:
    """Kept fraction of a group's cache: one full layer plus S-1 layers of m
    dims, over S full layers (Appendix "Compression-Ratio Configurations")."""
    return (D + (group_size - 1) * m) / (group_size * D)


def n_compressed_layers(n_layers: int, group_size: int) -> int:
    return sum(0 if is_anchor_layer(l, group_size) else 1 for l in range(n_layers))


def total_predictor_params(n_layers: int, group_size: int, D: int, m: int,
                           bias: bool = False) -> int:
    """Two predictors (one for K, one for V) per compressed layer."""
    d_in, d_out = predictor_shape(D, m)
    per = d_in * d_out + (d_out if bias else 0)
    return 2 * n_compressed_layers(n_layers, group_size) * per


# ----------------------------------------------------------------------------
# Reconstruction (Eq. 2, 3, 4, 6)
# ----------------------------------------------------------------------------


def retained_dims(c: np.ndarray, m: int) -> np.ndarray:
    """Eq. 2: C_local = C[:, :m], what a compressed layer keeps of each token ([L, D] -> [L, m]).
    Compression is nothing but this eviction (Section 3.1)."""
    c = np.asarray(c)
    if not 0 <= m <= c.shape[1]:
        raise ValueError("need 0 <= m <= D")
    return c[:, :m]


def dropped_dims(c: np.ndarray, m: int) -> np.ndarray:
    """Eq. 4: C_drop = C[:, m:], what is evicted and later predicted ([L, D] -> [L, D - m])."""
    c = np.asarray(c)
    if not 0 <= m <= c.shape[1]:
        raise ValueError("need 0 <= m <= D")
    return c[:, m:]


def predictor_input(c_global: np.ndarray, c_local: np.ndarray) -> np.ndarray:
    """[C_global ; C_local] per token (Eq. 3): [L, D] and [L, m] -> [L, D + m]."""
    c_global = np.asarray(c_global, dtype=np.float64)
    c_local = np.asarray(c_local, dtype=np.float64)
    if c_global.shape[0] != c_local.shape[0]:
        raise ValueError("token counts differ")
    return np.concatenate([c_global, c_local], axis=1)


def reconstruct_dropped(W: np.ndarray, c_global: np.ndarray, c_local: np.ndarray,
                        bias: np.ndarray | None = None) -> np.ndarray:
    """Eq. 3: C_hat_drop[t, :] = W [C_global[t] ; C_local[t]]  (+ bias if given).

    W is [D - m, D + m] (rows = dropped flat dims m..D-1, columns = the D global
    dims then the m local dims).  Returns [L, D - m].
    """
    W = np.asarray(W, dtype=np.float64)
    x = predictor_input(c_global, c_local)                     # [L, D + m]
    if W.shape[1] != x.shape[1]:
        raise ValueError("W has %d columns, input has %d features" % (W.shape[1], x.shape[1]))
    c_hat = x @ W.T                                            # [L, D - m]
    if bias is not None:
        c_hat = c_hat + np.asarray(bias, dtype=np.float64)[None, :]
    return c_hat


def assemble_cache(c_local: np.ndarray, c_hat_drop: np.ndarray, n_kv_heads: int,
                   head_dim: int) -> np.ndarray:
    """Eq. 6: X_tilde = Reshape([X_local ; X_hat_drop]) -> [L, H_kv, d]
    (head-major flattening: flat index = head * d + feature)."""
    c_local = np.asarray(c_local, dtype=np.float64)
    c_hat_drop = np.asarray(c_hat_drop, dtype=np.float64)
    flat = np.concatenate([c_local, c_hat_drop], axis=1)
    L, D = flat.shape
    if D != n_kv_heads * head_dim:
        raise ValueError("local + dropped widths do not add up to H_kv * d")
    return flat.reshape(L, n_kv_heads, head_dim)


# ----------------------------------------------------------------------------
# Rotary position embedding applied when the cache is read (Section 3.2: the
# predictor inputs, hence the cached keys, are keys prior to RoPE)
# ----------------------------------------------------------------------------


def rope_angles(L: int, d: int, rope_theta: float) -> np.ndarray:
    """angle[t, j] = t * rope_theta^(-2 j / d) for positions t = 0..L-1 and the d/2
    frequency indices j (RoFormer's frequencies; position = index in the cache)."""
    if d % 2:
        raise ValueError("head dim must be even")
    j = np.arange(d // 2, dtype=np.float64)
    inv_freq = np.power(float(rope_theta), -2.0 * j / d)
    return np.arange(L, dtype=np.float64)[:, None] * inv_freq[None, :]


def rotate_keys(K: np.ndarray, rope_theta: float) -> np.ndarray:
    """Rotate row t of every head of K [L, H, d] to position t.  Feature j < d/2 is
    paired with feature j + d/2 (the "rotate half" layout of the Llama family):
        out[j]       = k[j] cos(a_tj) - k[j + d/2] sin(a_tj)
        out[j + d/2] = k[j + d/2] cos(a_tj) + k[j] sin(a_tj)
    """
    K = np.asarray(K, dtype=np.float64)
    L, H, d = K.shape
    a = rope_angles(L, d, rope_theta)[:, None, :]              # [L, 1, d/2]
    lo, hi = K[:, :, :d // 2], K[:, :, d // 2:]
    return np.concatenate([lo * np.cos(a) - hi * np.sin(a), hi * np.cos(a) + lo * np.sin(a)], axis=2)


# ----------------------------------------------------------------------------
# Attention (Eq. 7; softmax as defined in the QK-KL appendix)
# ----------------------------------------------------------------------------


def attention_probabilities(q: np.ndarray, K: np.ndarray, scale: float | None = None,
                            rope_theta: float | None = None) -> np.ndarray:
    """softmax_t(q_h . K[t, kv(h)] * scale) -> [H_q, L], kv(h) = h // (H_q / H_kv).
    With rope_theta, K holds un-rotated keys and row t is rotated to position t first."""
    q = np.asarray(q, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    if rope_theta is not None:
        K = rotate_keys(K, rope_theta)
    H_q, d = q.shape
    L, H_kv, d2 = K.shape
    if d2 != d or H_q % H_kv != 0:
        raise ValueError("bad head shapes")
    if L == 0:
        raise ValueError("softmax over an empty cache is undefined")
    if scale is None:
        scale = 1.0 / math.sqrt(d)
    g = H_q // H_kv
    p = np.empty((H_q, L), dtype=np.float64)
    for h in range(H_q):
        s = (K[:, h // g, :] @ q[h]) * scale                   # [L]
        e = np.exp(s - s.max())
        p[h] = e / e.sum()
    return p


def attention(q: np.ndarray, K: np.ndarray, V: np.ndarray, scale: float | None = None,
              rope_theta: float | None = None) -> np.ndarray:
    """Eq. 7 for one decode query per head: out[h] = sum_t p[h, t] V[t, kv(h), :].

    q [H_q, d], K and V [L, H_kv, d] -> [H_q, d].
    """
    V = np.asarray(V, dtype=np.float64)
    p = attention_probabilities(q, K, scale, rope_theta)
    H_q = p.shape[0]
    g = H_q // V.shape[1]
    out = np.empty((H_q, V.shape[2]), dtype=np.float64)
    for h in range(H_q):
        out[h] = p[h] @ V[:, h // g, :]
    return out


def full_attention(q: np.ndarray, k_cache: np.ndarray, v_cache: np.ndarray,
                   n_kv_heads: int, scale: float | None = None,
                   rope_theta: float | None = None) -> np.ndarray:
    """Attention of an anchor layer / the uncompressed mode: the stored cache
    [L, D] is used as it is (Eq. 7 with K_tilde = K, V_tilde = V)."""
    k_cache = np.asarray(k_cache, dtype=np.float64)
    v_cache = np.asarray(v_cache, dtype=np.float64)
    L, D = k_cache.shape
    d = D // n_kv_heads
    return attention(q, k_cache.reshape(L, n_kv_heads, d), v_cache.reshape(L, n_kv_heads, d), scale,
                     rope_theta)


def decode_attention(q: np.ndarray,
                     k_global: np.ndarray, v_global: np.ndarray,
                     k_local: np.ndarray, v_local: np.ndarray,
                     Wk: np.ndarray, Wv: np.ndarray,
                     n_kv_heads: int, scale: float | None = None,
                     bk: np.ndarray | None = None, bv: np.ndarray | None = None,
                     rope_theta: float | None = None, k_true: np.ndarray | None = None) -> np.ndarray:
    """One decode step of a compressed layer for one sequence.

    k_global, v_global [L, D]  full cache of the group's anchor layer   (Eq. 1)
    k_local,  v_local  [L, m]  retained dims of this layer              (Eq. 2)
    Wk, Wv [D - m, D + m]      this layer's predictors                  (Eq. 3)
    q [H_q, d]                 the new token's queries
    Steps: predict the dropped dims (Eq. 3), rebuild K_tilde, V_tilde (Eq. 6),
    (rotate K_tilde by position if rope_theta is given), attend (Eq. 7).  Returns [H_q, d].
    k_true [L, D]: the "save K" setting of Section 5.2 -- the layer's keys are kept whole and
    used as they are (k_local, Wk, bk are ignored); reconstruction applies to the values only.
    """
    k_global = np.asarray(k_global, dtype=np.float64)
    D = k_global.shape[1]
    d = D // n_kv_heads
    v_hat = reconstruct_dropped(Wv, v_global, v_local, bv)
    if k_true is not None:
        K_t = np.asarray(k_true, dtype=np.float64).reshape(-1, n_kv_heads, d)
        if K_t.shape[0] != k_global.shape[0]:
            raise ValueError("token counts differ")
    else:
        K_t = assemble_cache(k_local, reconstruct_dropped(Wk, k_global, k_local, bk), n_kv_heads, d)
    V_t = assemble_cache(v_local, v_hat, n_kv_heads, d)
    return attention(q, K_t, V_t, scale, rope_theta)


def decode_attention_query_heads(q: np.ndarray,
                                 k_global: np.ndarray, v_global: np.ndarray,
                                 k_local: np.ndarray, v_local: np.ndarray,
                                 Wk: np.ndarray, Wv: np.ndarray,
                                 n_kv_heads: int, query_heads, scale: float | None = None,
                                 k_true_drop=None, v_true_drop=None, n_sink: int = 0, n_window: int = 0,
                                 rope_theta: float | None = None, k_true=None,
                                 bk=None, bv=None) -> dict[int, np.ndarray]:
    """The same quantity as decode_attention (or decode_attention_windowed, when a sink / window
    is given), for a chosen few query heads only.

    Heads are independent in Eq. 7 and each dropped flat dim is one row of W in
    Eq. 3, so for query head h only the rows of W that produce dims of KV head kv(h)
    are evaluated.  Eq. 6 concatenates at the flat index m, wherever that falls: of a
    head that m splits, the dims below m are the stored ones and the rest are predicted.
    k_true [L, D]: the "save K" setting (keys whole, used as they are).
    Used to check sampled outputs of workloads too large to run in full.  Returns {h: out[h] as [d]}.
    """
    q = np.asarray(q, dtype=np.float64)
    k_global = np.asarray(k_global, dtype=np.float64)
    v_global = np.asarray(v_global, dtype=np.float64)
    k_local = np.asarray(k_local, dtype=np.float64)
    v_local = np.asarray(v_local, dtype=np.float64)
    H_q, d = q.shape
    D = k_global.shape[1]
    m = v_local.shape[1]
    L = k_global.shape[0]
    g = H_q // n_kv_heads
    if scale is None:
        scale = 1.0 / math.sqrt(d)
    keep = full_precision_tokens(L, n_sink, n_window) if (n_sink or n_window) else None

    def head_dims(c_global, c_local, W, bias, c_true_drop, lo):
        """Flat dims [lo, lo + d) of the rebuilt cache: [L, d]."""
        n_stored = min(max(m - lo, 0), d)             # dims of this head below m: stored
        parts = [c_local[:, lo:lo + n_stored]]
        if n_stored < d:                              # the rest: rows of W (Eq. 3)
            rows = slice(lo + n_stored - m, lo + d - m)
            pred = predictor_input(c_global, c_local) @ np.asarray(W, dtype=np.float64)[rows].T
            if bias is not None:
                pred = pred + np.asarray(bias, dtype=np.float64)[rows]
            if keep is not None:                      # sink / window tokens keep their true dims
                pred = overlay_true_dims(pred, np.asarray(c_true_drop, dtype=np.float64)[:, rows], keep)
            parts.append(pred)
        return np.concatenate(parts, axis=1)

    out = {}
    for h in query_heads:
        kv = h // g
        lo = kv * d                                   # flat dims [lo, lo + d) of K_tilde
        if k_true is not None:
            K_h = np.asarray(k_true, dtype=np.float64)[:, lo:lo + d]
        else:
            K_h = head_dims(k_global, k_local, Wk, bk, k_true_drop, lo)
        V_h = head_dims(v_global, v_local, Wv, bv, v_true_drop, lo)
        if rope_theta is not None:
            K_h = rotate_keys(K_h[:, None, :], rope_theta)[:, 0, :]
        s = (K_h @ q[h]) * scale
        e = np.exp(s - s.max())
        out[h] = (e / e.sum()) @ V_h
    return out


# ----------------------------------------------------------------------------
# Sink and recent-window tokens kept at full precision (Section 4.1, "Implement
# details": 4 sink tokens and a local window of 128 tokens)
# ----------------------------------------------------------------------------


def full_precision_tokens(L: int, n_sink: int, n_window: int) -> np.ndarray:
    """Boolean [L]: token t keeps its whole K / V (nothing of it is predicted) iff it
    is one of the first n_sink tokens or one of the last n_window tokens."""
    if n_sink < 0 or n_window < 0:
        raise ValueError("negative sink / window size")
    t = np.arange(L)
    return (t < n_sink) | (t >= L - n_window)


def overlay_true_dims(c_hat_drop: np.ndarray, c_true_drop: np.ndarray, keep: np.ndarray) -> np.ndarray:
    """Dropped dims of every token: the stored true values where keep[t], the
    predicted ones elsewhere.  Rows of c_true_drop outside `keep` are never read."""
    out = np.array(c_hat_drop, dtype=np.float64, copy=True)
    keep = np.asarray(keep, dtype=bool)
    out[keep] = np.asarray(c_true_drop, dtype=np.float64)[keep]
    return out


def decode_attention_windowed(q, k_global, v_global, k_local, v_local, Wk, Wv, n_kv_heads: int,
                              k_true_drop, v_true_drop, n_sink: int, n_window: int,
                              scale: float | None = None, bk=None, bv=None,
                              rope_theta: float | None = None, k_true=None) -> np.ndarray:
    """decode_attention with the sink and recent-window tokens at full precision:
    for those tokens the dropped dims come from k_true_drop / v_true_drop ([L, D - m],
    the layer's own dims m..D-1), for all others from Eq. 3.  With k_true [L, D] (the
    "save K" setting of Section 5.2) the keys are whole anyway and used as they are
    (k_local, Wk, bk, k_true_drop are ignored); the window then matters to the values only.
    Returns [H_q, d]."""
    q = np.asarray(q, dtype=np.float64)
    d = q.shape[1]
    L = np.asarray(k_global).shape[0]
    if L < 1:
        raise ValueError("empty cache: softmax over no token is undefined")
    keep = full_precision_tokens(L, n_sink, n_window)
    if k_true is not None:
        K_t = np.asarray(k_true, dtype=np.float64).reshape(-1, n_kv_heads, d)
        if K_t.shape[0] != L:
            raise ValueError("token counts differ")
    else:
        k_drop = overlay_true_dims(reconstruct_dropped(Wk, k_global, k_local, bk), k_true_drop, keep)
        K_t = assemble_cache(k_local, k_drop, n_kv_heads, d)
    v_drop = overlay_true_dims(reconstruct_dropped(Wv, v_global, v_local, bv), v_true_drop, keep)
    return attention(q, K_t, assemble_cache(v_local, v_drop, n_kv_heads, d), scale, rope_theta)


# ----------------------------------------------------------------------------
# Prefill-shaped use: the last n_q tokens of a sequence are queries at once (Section 5.4: the
# dropped parts of the cache can be evicted already during the pre-filling phase)
# ----------------------------------------------------------------------------


def prefill_attention(q: np.ndarray, k_global, v_global, k_local, v_local, Wk, Wv, n_kv_heads: int,
                      scale: float | None = None, bk=None, bv=None, rope_theta: float | None = None,
                      k_true=None, k_true_drop=None, v_true_drop=None, n_sink: int = 0,
                      n_window: int = 0) -> np.ndarray:
    """q [n_q, H_q, d]: queries of the last n_q of the L cached tokens; query i sits at position
    L - n_q + i and attends the tokens up to and including its own (causal).  The cache of a
    compressed layer is rebuilt once (Eq. 3, Eq. 6) and each query evaluates Eq. 7 over its prefix.
    With Wk = Wv = None the layer holds its full cache (k_global, v_global are used as they are:
    an anchor layer).  k_true [L, D]: the "save K" setting of Section 5.2, as in decode_attention
    (keys whole and used as they are; only the values are predicted).
    With a sink / window (Section 4.1) every query is the decode step of the sequence cut off at its
    own position: of ITS prefix the first n_sink and the last n_window tokens are at full precision
    (k_true_drop, v_true_drop [L, D - m] as in decode_attention_windowed), so a token is read at full
    precision by the queries at most n_window - 1 positions after it and as predicted by the later ones.
    Returns [n_q, H_q, d]."""
    q = np.asarray(q, dtype=np.float64)
    n_q, H_q, d = q.shape
    k_global = np.asarray(k_global, dtype=np.float64)
    v_global = np.asarray(v_global, dtype=np.float64)
    L = k_global.shape[0]
    if n_q < 1 or n_q > L:
        raise ValueError("need 1 <= n_q <= L")
    windowed = (n_sink > 0 or n_window > 0) and not (Wk is None and Wv is None)
    if windowed:
        k_local = np.asarray(k_local, dtype=np.float64)
        v_local = np.asarray(v_local, dtype=np.float64)
    if Wk is None and Wv is None:
        K_t = k_global.reshape(L, n_kv_heads, d)
        V_t = v_global.reshape(L, n_kv_heads, d)
    else:
        v_hat = reconstruct_dropped(Wv, v_global, v_local, bv)
        if k_true is not None:
            K_t = np.asarray(k_true, dtype=np.float64).reshape(-1, n_kv_heads, d)
            if K_t.shape[0] != L:
                raise ValueError("token counts differ")
            k_hat = None
        else:
            k_hat = reconstruct_dropped(Wk, k_global, k_local, bk)
            K_t = assemble_cache(k_local, k_hat, n_kv_heads, d)
        V_t = assemble_cache(v_local, v_hat, n_kv_heads, d)
    if rope_theta is not None and not windowed:
        K_t = rotate_keys(K_t, rope_theta)
    out = np.empty((n_q, H_q, d), dtype=np.float64)
    for i in range(n_q):
        n_seen = L - n_q + i + 1
        if windowed:
            # this query's own sink and window, on its own prefix
            keep = full_precision_tokens(n_seen, n_sink, n_window)
            V_i = assemble_cache(v_local[:n_seen], overlay_true_dims(v_hat[:n_seen], np.asarray(v_true_drop)[:n_seen], keep),
                                 n_kv_heads, d)
            if k_hat is None:
                K_i = K_t[:n_seen]
            else:
                K_i = assemble_cache(k_local[:n_seen],
                                     overlay_true_dims(k_hat[:n_seen], np.asarray(k_true_drop)[:n_seen], keep), n_kv_heads, d)
            out[i] = attention(q[i], K_i, V_i, scale, rope_theta)
        else:
            out[i] = attention(q[i], K_t[:n_seen], V_t[:n_seen], scale)
    return out


# ----------------------------------------------------------------------------
# Multi-layer step (Eq. 1): which cache each layer attends over
# ----------------------------------------------------------------------------


def layer_step(layer: int, group_size: int, q: np.ndarray, caches_k, caches_v,
               weights_k, weights_v, n_kv_heads: int, m: int,
               scale: float | None = None, rope_theta: float | None = None) -> np.ndarray:
    """Decode attention of `layer` for one sequence.

    caches_k[l], caches_v[l]: [L, D] full (true) caches of every layer; a
    compressed layer only ever reads its first m dims, an anchor layer all D.
    weights_k[l], weights_v[l]: predictors of compressed layers.
    """
    if is_anchor_layer(layer, group_size):
        return full_attention(q, caches_k[layer], caches_v[layer], n_kv_heads, scale, rope_theta)
    a = anchor_of(layer, group_size)
    return decode_attention(q, caches_k[a], caches_v[a],
                            np.asarray(caches_k[layer])[:, :m], np.asarray(caches_v[layer])[:, :m],
                            weights_k[layer], weights_v[layer], n_kv_heads, scale, rope_theta=rope_theta)


# ----------------------------------------------------------------------------
# Stored-precision helpers (exact widening; no arithmetic of the method here)
# ----------------------------------------------------------------------------


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """uint16 bf16 bit patterns -> float64, exactly (bf16 is the top half of fp32)."""
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


def widen(x) -> np.ndarray:
    """Widen a stored tensor to float64: uint16 arrays are bf16 bit patterns,
    float arrays are taken by value."""
    x = np.asarray(x)
    if x.dtype == np.uint16:
        return bf16_bits_to_f64(x)
    return x.astype(np.float64)
