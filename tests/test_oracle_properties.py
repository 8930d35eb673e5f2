"""Randomised property checks of the oracle (hypothesis): shapes and seeds are drawn, the properties are ones the
mathematics fixes -- independence of heads, limits of the sink / window and "save K" settings, causality of the
prefill-shaped form, the split-K merge identity, and the relative-position property of the rotation."""
import math

import numpy as np
from hypothesis import given, settings, strategies as st

from oracle import echokv_oracle as O


def draw_case(seed, L, H_kv, g, d, r):
    rng = np.random.default_rng(seed)
    D, m = H_kv * d, r * d
    return dict(q=rng.standard_normal((H_kv * g, d)), kg=rng.standard_normal((L, D)), vg=rng.standard_normal((L, D)),
                kl=rng.standard_normal((L, m)), vl=rng.standard_normal((L, m)),
                Wk=rng.standard_normal((D - m, D + m)) / math.sqrt(D + m),
                Wv=rng.standard_normal((D - m, D + m)) / math.sqrt(D + m),
                kt=rng.standard_normal((L, D - m)), vt=rng.standard_normal((L, D - m)),
                H_kv=H_kv, H_q=H_kv * g, d=d, D=D, m=m, L=L, rng=rng)


shapes = dict(seed=st.integers(0, 2 ** 31 - 1), L=st.integers(1, 24), H_kv=st.integers(1, 4), g=st.sampled_from([1, 2, 4]),
              d=st.sampled_from([2, 4, 8]))


def args(c):
    return c["kg"], c["vg"], c["kl"], c["vl"], c["Wk"], c["Wv"], c["H_kv"]


@settings(max_examples=40, deadline=None)
@given(r_frac=st.floats(0, 1), rope=st.sampled_from([None, 100.0, 10000.0]), **shapes)
def test_heads_are_independent_and_the_per_head_form_agrees(seed, L, H_kv, g, d, r_frac, rope):
    c = draw_case(seed, L, H_kv, g, d, min(H_kv - 1, int(r_frac * H_kv)))
    full = O.decode_attention(c["q"], *args(c), rope_theta=rope)
    per = O.decode_attention_query_heads(c["q"], *args(c), range(c["H_q"]), rope_theta=rope)
    for h in range(c["H_q"]):
        np.testing.assert_allclose(per[h], full[h], rtol=1e-10, atol=1e-12)
    # changing one query head's vector changes that head's output only
    q2 = c["q"].copy()
    q2[0] += 1.0
    other = O.decode_attention(q2, *args(c), rope_theta=rope)
    np.testing.assert_array_equal(other[1:], full[1:])


@settings(max_examples=40, deadline=None)
@given(n_sink=st.integers(0, 6), n_window=st.integers(0, 30), **shapes)
def test_sink_and_window_limits(seed, L, H_kv, g, d, n_sink, n_window):
    c = draw_case(seed, L, H_kv, g, d, max(0, H_kv - 1))
    got = O.decode_attention_windowed(c["q"], *args(c), c["kt"], c["vt"], n_sink, n_window)
    if n_sink + n_window >= L:       # every token keeps all its dims: attention on the true cache
        K = np.concatenate([c["kl"], c["kt"]], axis=1).reshape(L, H_kv, d)
        V = np.concatenate([c["vl"], c["vt"]], axis=1).reshape(L, H_kv, d)
        np.testing.assert_allclose(got, O.attention(c["q"], K, V), rtol=1e-10, atol=1e-12)
    if n_sink == 0 and n_window == 0:
        np.testing.assert_array_equal(got, O.decode_attention(c["q"], *args(c)))
    keep = O.full_precision_tokens(L, n_sink, n_window)
    assert keep.sum() == min(L, n_sink + n_window) or n_sink + n_window > L
    assert keep[:min(n_sink, L)].all() and keep[max(0, L - n_window):].all()


@settings(max_examples=30, deadline=None)
@given(n_q=st.integers(1, 8), rope=st.sampled_from([None, 10000.0]), **shapes)
def test_prefill_rows_are_decode_steps_on_prefixes(seed, L, H_kv, g, d, n_q, rope):
    n_q = min(n_q, L)
    c = draw_case(seed, L, H_kv, g, d, max(0, H_kv - 1))
    q = c["rng"].standard_normal((n_q, c["H_q"], d))
    got = O.prefill_attention(q, *args(c), rope_theta=rope)
    i = int(c["rng"].integers(0, n_q))
    n = L - n_q + i + 1
    want = O.decode_attention(q[i], c["kg"][:n], c["vg"][:n], c["kl"][:n], c["vl"][:n], c["Wk"], c["Wv"], H_kv,
                              rope_theta=rope)
    np.testing.assert_allclose(got[i], want, rtol=1e-10, atol=1e-12)


@settings(max_examples=40, deadline=None)
@given(cut=st.floats(0.05, 0.95), **shapes)
def test_split_contexts_merge_by_log_sum_exp(seed, L, H_kv, g, d, cut):
    L = max(L, 2)
    c = draw_case(seed, L, H_kv, g, d, 0)
    K, V = c["kg"].reshape(L, H_kv, d), c["vg"].reshape(L, H_kv, d)
    n = min(L - 1, max(1, int(cut * L)))
    whole = O.attention(c["q"], K, V)
    scale = 1.0 / math.sqrt(d)
    for h in range(c["H_q"]):
        kv = h // g
        parts = []
        for sl in (slice(0, n), slice(n, L)):
            s = (K[sl, kv] @ c["q"][h]) * scale
            mx = s.max()
            e = np.exp(s - mx)
            parts.append((mx, e.sum(), e @ V[sl, kv]))
        M = max(p[0] for p in parts)
        den = sum(math.exp(p[0] - M) * p[1] for p in parts)
        num = sum(math.exp(p[0] - M) * p[2] for p in parts)
        np.testing.assert_allclose(num / den, whole[h], rtol=1e-10, atol=1e-12)


@settings(max_examples=40, deadline=None)
@given(seed=st.integers(0, 2 ** 31 - 1), d=st.sampled_from([2, 4, 8, 16]), p=st.integers(0, 500), t=st.integers(0, 500),
       shift=st.integers(0, 2000), theta=st.sampled_from([50.0, 10000.0, 500000.0]))
def test_rotation_depends_on_the_position_difference_only(seed, d, p, t, shift, theta):
    rng = np.random.default_rng(seed)
    qv, kv = rng.standard_normal(d), rng.standard_normal(d)

    def at(v, pos):
        buf = np.zeros((pos + 1, 1, d))
        buf[pos, 0] = v
        return O.rotate_keys(buf, theta)[pos, 0]
    a = at(qv, p) @ at(kv, t)
    b = at(qv, p + shift) @ at(kv, t + shift)
    assert abs(a - b) <= 1e-9 * (1.0 + abs(a)) + 1e-9 * np.linalg.norm(qv) * np.linalg.norm(kv)
    np.testing.assert_allclose(np.linalg.norm(at(kv, t)), np.linalg.norm(kv), rtol=1e-12)


@settings(max_examples=30, deadline=None)
@given(**shapes)
def test_save_k_with_exact_value_predictor_is_attention_on_the_true_cache(seed, L, H_kv, g, d):
    c = draw_case(seed, L, H_kv, g, d, max(0, H_kv - 1))
    D, m = c["D"], c["m"]
    k_true = np.concatenate([c["kl"], c["kt"]], axis=1)
    vg = c["vg"].copy()
    vg[:, m:] = c["vt"]
    Wv = np.zeros((D - m, D + m))
    Wv[np.arange(D - m), m + np.arange(D - m)] = 1.0
    got = O.decode_attention(c["q"], c["kg"], vg, c["kl"], c["vl"], None, Wv, H_kv, k_true=k_true)
    V = np.concatenate([c["vl"], c["vt"]], axis=1).reshape(L, H_kv, d)
    np.testing.assert_allclose(got, O.attention(c["q"], k_true.reshape(L, H_kv, d), V), rtol=1e-10, atol=1e-12)
