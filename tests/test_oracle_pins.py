"""Pins for the CPU oracle: everything here is independent of the oracle's own
formulas -- values the paper prints, hand-derived closed forms, a pure-python
brute force written index by index, torch library routines, and invariants."""
import math
import os

import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import echokv_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def rng(seed):
    return np.random.default_rng(seed)


def rand_case(seed, L=37, H_q=8, H_kv=4, d=8, r=1, m=None):
    """m, when given, is the retained width in flat dims and need not end on a head boundary."""
    g = rng(seed)
    D = H_kv * d
    m = r * d if m is None else m
    return dict(
        q=g.standard_normal((H_q, d)),
        kg=g.standard_normal((L, D)), vg=g.standard_normal((L, D)),
        kl=g.standard_normal((L, m)), vl=g.standard_normal((L, m)),
        Wk=g.standard_normal((D - m, D + m)) / math.sqrt(D + m),
        Wv=g.standard_normal((D - m, D + m)) / math.sqrt(D + m),
        H_kv=H_kv, d=d, m=m, D=D, L=L, H_q=H_q)


def run(c, **kw):
    return O.decode_attention(c["q"], c["kg"], c["vg"], c["kl"], c["vl"], c["Wk"], c["Wv"],
                              c["H_kv"], **kw)


# --------------------------------------------------------------------------
# P7: the paper's printed table (tests/golden/paper_predictor_table.txt)
# --------------------------------------------------------------------------
def load_table():
    rows = []
    with open(os.path.join(GOLDEN, "paper_predictor_table.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                t = line.split()
                rows.append((float(t[0]), int(t[1]), int(t[2]), int(t[3]), int(t[4]), float(t[5]), float(t[6])))
    return rows


def test_paper_predictor_shapes_ratios_and_param_totals():
    D, n_layers = 8 * 128, 32
    rows = load_table()
    assert len(rows) == 3
    for target, S, m, d_in, d_out, params_m, ratio_printed in rows:
        assert O.predictor_shape(D, m) == (d_in, d_out)
        assert round(O.effective_ratio(D, S, m), 2) == pytest.approx(ratio_printed, abs=0.0051)
        # two predictors (K and V) per compressed layer; the paper's totals round to one
        # decimal of a million either without bias (28.8, 33.6) or with it (50.2)
        nb = O.total_predictor_params(n_layers, S, D, m, bias=False) / 1e6
        wb = O.total_predictor_params(n_layers, S, D, m, bias=True) / 1e6
        assert min(abs(nb - params_m), abs(wb - params_m)) < 0.051
    # exact counts behind those roundings
    assert O.total_predictor_params(32, 2, 1024, 384) == 16 * 2 * 1408 * 640 == 28_835_840
    assert O.total_predictor_params(32, 2, 1024, 0) == 16 * 2 * 1024 * 1024 == 33_554_432
    assert O.total_predictor_params(32, 4, 1024, 64) == 24 * 2 * 1088 * 960 == 50_135_040
    assert O.total_predictor_params(32, 4, 1024, 64, bias=True) == 50_135_040 + 24 * 2 * 960
    assert O.effective_ratio(1024, 2, 384) == 0.6875
    assert O.effective_ratio(1024, 4, 64) == 0.296875


def test_eviction_eq2_eq4_matches_the_printed_shapes():
    # the table's rows: what is kept (m) plus the anchor's D dims is the predictor's input width, what is
    # dropped its output width; kept and dropped together are the token's cache again
    g = rng(77)
    for ratio, S, m, d_in, d_out, _, _ in load_table():
        D = 1024
        c = g.standard_normal((5, D))
        kept, dropped = O.retained_dims(c, m), O.dropped_dims(c, m)
        assert kept.shape == (5, m) and dropped.shape == (5, d_out)
        assert O.predictor_input(c, kept).shape == (5, d_in)
        np.testing.assert_array_equal(np.concatenate([kept, dropped], axis=1), c)
        np.testing.assert_array_equal(O.assemble_cache(kept, dropped, 8, 128).reshape(5, D), c)
    with pytest.raises(ValueError):
        O.retained_dims(np.zeros((2, 8)), 9)


def test_save_k_setting_uses_the_true_keys():
    # "save K" (Section 5.2): keys whole, values predicted.  Pins: with a selector W^V it is standard attention on
    # the true cache (library routine); with a selector W^K the ordinary path gives the same as handing over the
    # true keys; the K predictor and the retained key dims are not read at all
    c = rand_case(41, L=19, H_q=8, H_kv=4, d=8, r=1)
    g = rng(41)
    D, m, L = c["D"], c["m"], c["L"]
    k_true = np.concatenate([c["kl"], g.standard_normal((L, D - m))], axis=1)
    v_true_drop = g.standard_normal((L, D - m))
    # the anchor's V carries this layer's dropped V dims, and W^V selects them
    vg = c["vg"].copy()
    vg[:, m:] = v_true_drop
    Wv_sel = np.zeros((D - m, D + m))
    Wv_sel[np.arange(D - m), m + np.arange(D - m)] = 1.0
    got = O.decode_attention(c["q"], c["kg"], vg, c["kl"], c["vl"], None, Wv_sel, c["H_kv"], k_true=k_true)
    V_true = np.concatenate([c["vl"], v_true_drop], axis=1).reshape(L, c["H_kv"], c["d"])
    np.testing.assert_allclose(got, sdpa(c["q"], k_true.reshape(L, c["H_kv"], c["d"]), V_true), rtol=1e-12, atol=1e-13)
    # selector W^K on an anchor that carries the true dropped key dims: the ordinary path equals the save-K path
    kg = c["kg"].copy()
    kg[:, m:] = k_true[:, m:]
    ordinary = O.decode_attention(c["q"], kg, c["vg"], c["kl"], c["vl"], Wv_sel, c["Wv"], c["H_kv"])
    saved = O.decode_attention(c["q"], kg, c["vg"], np.full_like(c["kl"], np.nan), c["vl"], None, c["Wv"], c["H_kv"],
                               k_true=k_true)
    np.testing.assert_allclose(saved, ordinary, rtol=1e-12, atol=1e-13)
    # and it differs from predicting the keys with a random predictor
    assert np.abs(run(c) - O.decode_attention(c["q"], c["kg"], c["vg"], c["kl"], c["vl"], None, c["Wv"], c["H_kv"],
                                              k_true=k_true)).max() > 1e-3
    with pytest.raises(ValueError):
        O.decode_attention(c["q"], c["kg"], c["vg"], c["kl"], c["vl"], None, c["Wv"], c["H_kv"], k_true=k_true[:-1])


def test_prefill_shaped_attention():
    c = rand_case(51, L=21, H_q=8, H_kv=4, d=8, r=1)
    g = rng(51)
    n_q = 6
    q = g.standard_normal((n_q, c["H_q"], c["d"]))
    args = (c["kg"], c["vg"], c["kl"], c["vl"], c["Wk"], c["Wv"], c["H_kv"])
    got = O.prefill_attention(q, *args)
    # the last query sees the whole cache: the decode step; every other query: the decode step on its prefix
    np.testing.assert_allclose(got[-1], O.decode_attention(q[-1], *args), rtol=1e-12, atol=1e-14)
    for i in (0, 3):
        n = c["L"] - n_q + i + 1
        want = O.decode_attention(q[i], c["kg"][:n], c["vg"][:n], c["kl"][:n], c["vl"][:n], c["Wk"], c["Wv"], c["H_kv"])
        np.testing.assert_allclose(got[i], want, rtol=1e-12, atol=1e-14)
    # causal: what comes after a query's own token does not matter to it
    kg2, vg2 = c["kg"].copy(), c["vg"].copy()
    kg2[-2:] = 7.0
    vg2[-2:] = -3.0
    got2 = O.prefill_attention(q, kg2, vg2, c["kl"], c["vl"], c["Wk"], c["Wv"], c["H_kv"])
    np.testing.assert_array_equal(got2[: n_q - 2], got[: n_q - 2])
    assert np.abs(got2[-1] - got[-1]).max() > 1e-3
    # a full (anchor) cache with all tokens as queries: causal scaled-dot-product attention (library routine)
    L, H, d = c["L"], c["H_kv"], c["d"]
    qa = g.standard_normal((L, c["H_q"], d))
    full = O.prefill_attention(qa, c["kg"], c["vg"], None, None, None, None, H)
    tq = torch.from_numpy(qa).permute(1, 0, 2)[None]
    tk = torch.from_numpy(c["kg"].reshape(L, H, d)).permute(1, 0, 2)[None]
    tv = torch.from_numpy(c["vg"].reshape(L, H, d)).permute(1, 0, 2)[None]
    ref = F.scaled_dot_product_attention(tq, tk, tv, is_causal=True, enable_gqa=True)[0].permute(1, 0, 2).numpy()
    np.testing.assert_allclose(full, ref, rtol=1e-12, atol=1e-13)
    # rotation: position of key t is t whatever the query
    rot = O.prefill_attention(q, *args, rope_theta=10000.0)
    np.testing.assert_allclose(rot[-1], O.decode_attention(q[-1], *args, rope_theta=10000.0), rtol=1e-12, atol=1e-14)
    with pytest.raises(ValueError):
        O.prefill_attention(g.standard_normal((c["L"] + 1, c["H_q"], c["d"])), *args)
    # "save K" (Section 5.2): whole keys as they are; a query's row is the save-K decode step on its prefix, and with
    # the keys of a selector-predictor cache it is plain causal attention over those keys and the rebuilt values
    k_true = g.standard_normal((c["L"], c["H_kv"] * c["d"]))
    sk = O.prefill_attention(q, *args, k_true=k_true)
    for i in (0, n_q - 1):
        n = c["L"] - n_q + i + 1
        want = O.decode_attention(q[i], c["kg"][:n], c["vg"][:n], c["kl"][:n], c["vl"][:n], c["Wk"], c["Wv"], c["H_kv"],
                                  k_true=k_true[:n])
        np.testing.assert_allclose(sk[i], want, rtol=1e-12, atol=1e-14)
    assert np.abs(sk - got).max() > 1e-3            # the predicted keys are not used
    np.testing.assert_array_equal(O.prefill_attention(q, c["kg"], c["vg"], None, c["vl"], None, c["Wv"], c["H_kv"],
                                                      k_true=k_true), sk)       # k_local, Wk ignored


def test_anchor_assignment_eq1():
    S = 4
    assert [O.is_anchor_layer(l, S) for l in range(9)] == [True, False, False, False, True, False, False, False, True]
    assert [O.anchor_of(l, S) for l in range(9)] == [0, 0, 0, 0, 4, 4, 4, 4, 8]
    assert O.n_compressed_layers(32, 4) == 24 and O.n_compressed_layers(32, 2) == 16
    assert O.n_compressed_layers(30, 4) == 22      # last group shorter


# --------------------------------------------------------------------------
# P1a: a case worked out by hand (closed form, rational probabilities)
# --------------------------------------------------------------------------
def test_hand_computed_two_token_case():
    # d = 2, H_kv = 2 (D = 4), one retained head (m = 2), H_q = 2, L = 2.
    # Predictor inputs x_t = [global(4) ; local(2)], separately for K and V:
    #   K: x_0 = [1,0,0,0, 2,0]   x_1 = [0,1,0,0, 0,2]
    #   V: x_0 = [1,0,0,0, 3,0]   x_1 = [0,1,0,0, 0,3]
    # Wk picks x[0] and x[5]:  K_hat_0 = [1, 0], K_hat_1 = [0, 2]
    # head 1 (dropped): q = [c, c], c = sqrt(2) ln 3, scale 1/sqrt(2):
    #   s = [ln 3, 2 ln 3] -> p = [1/4, 3/4]
    # Wv: V_hat_t = [4 x[0], 8 x[0] + 2 x[5]]: V_hat_0 = [4, 8], V_hat_1 = [0, 6]
    #   -> out = 1/4 [4, 8] + 3/4 [0, 6] = [1, 6.5]
    # head 0 (retained): K = local rows [2,0],[0,2]; q = [0, ln2/sqrt(2)]:
    #   s = [0, ln 2] -> p = [1/3, 2/3]; V local rows [3,0],[0,3] -> out = [1, 2]
    kg = np.array([[1., 0, 0, 0], [0, 1., 0, 0]])
    vg = kg.copy()
    kl = np.array([[2., 0], [0, 2.]])
    vl = np.array([[3., 0], [0, 3.]])
    Wk = np.zeros((2, 6)); Wk[0, 0] = 1; Wk[1, 5] = 1
    Wv = np.zeros((2, 6)); Wv[0, 0] = 4; Wv[1, 0] = 8; Wv[1, 5] = 2
    c = math.sqrt(2) * math.log(3)
    q = np.array([[0.0, math.log(2) / math.sqrt(2)], [c, c]])
    out = O.decode_attention(q, kg, vg, kl, vl, Wk, Wv, n_kv_heads=2)
    np.testing.assert_allclose(out, [[1.0, 2.0], [1.0, 6.5]], rtol=0, atol=1e-14)
    p = O.attention_probabilities(q, O.assemble_cache(kl, O.reconstruct_dropped(Wk, kg, kl), 2, 2))
    np.testing.assert_allclose(p, [[1 / 3, 2 / 3], [1 / 4, 3 / 4]], atol=1e-15)


# --------------------------------------------------------------------------
# P1b: pure-python brute force, written index by index
# --------------------------------------------------------------------------
def brute_force(c, scale=None):
    q, kg, vg, kl, vl, Wk, Wv = (c[k].tolist() for k in ("q", "kg", "vg", "kl", "vl", "Wk", "Wv"))
    H_q, H_kv, d, m, D, L = c["H_q"], c["H_kv"], c["d"], c["m"], c["D"], c["L"]
    scale = 1.0 / math.sqrt(d) if scale is None else scale
    grp = H_q // H_kv

    def rebuilt(glob, loc, W, t, flat):          # flat dim `flat` of token t
        if flat < m:
            return loc[t][flat]
        row = W[flat - m]
        return math.fsum([row[i] * glob[t][i] for i in range(D)] +
                         [row[D + i] * loc[t][i] for i in range(m)])
    out = []
    for h in range(H_q):
        kv = h // grp
        s = [scale * math.fsum(q[h][j] * rebuilt(kg, kl, Wk, t, kv * d + j) for j in range(d))
             for t in range(L)]
        mx = max(s)
        e = [math.exp(v - mx) for v in s]
        z = math.fsum(e)
        out.append([math.fsum(e[t] / z * rebuilt(vg, vl, Wv, t, kv * d + j) for t in range(L))
                    for j in range(d)])
    return np.array(out)


@pytest.mark.parametrize("seed,L,H_q,H_kv,d,r", [(1, 3, 2, 2, 4, 1), (2, 5, 4, 2, 4, 0),
                                                   (3, 7, 6, 3, 2, 2), (4, 4, 2, 2, 4, 2), (5, 1, 4, 4, 2, 1)])
def test_brute_force_tiny(seed, L, H_q, H_kv, d, r):
    c = rand_case(seed, L, H_q, H_kv, d, r)
    np.testing.assert_allclose(run(c), brute_force(c), rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(run(c, scale=0.37), brute_force(c, 0.37), rtol=1e-12, atol=1e-13)


# --------------------------------------------------------------------------
# P2 / P8: library routines (torch SDPA, torch linear) as a second opinion
# --------------------------------------------------------------------------
def sdpa(q, K, V, scale=None):
    """torch scaled_dot_product_attention, fp64: q [H_q, d], K/V [L, H_kv, d]."""
    tq = torch.from_numpy(np.asarray(q))[None, :, None, :]
    tk = torch.from_numpy(np.asarray(K)).permute(1, 0, 2)[None]
    tv = torch.from_numpy(np.asarray(V)).permute(1, 0, 2)[None]
    o = F.scaled_dot_product_attention(tq, tk, tv, scale=scale, enable_gqa=True)
    return o[0, :, 0, :].numpy()


def test_nothing_dropped_equals_standard_attention():
    # m = D: the predictor has no rows; result must be plain attention on the stored cache
    c = rand_case(11, L=53, H_q=8, H_kv=4, d=8, r=4)
    assert c["Wk"].shape == (0, 2 * c["D"])
    out = run(c)
    K = c["kl"].reshape(c["L"], c["H_kv"], c["d"])
    V = c["vl"].reshape(c["L"], c["H_kv"], c["d"])
    np.testing.assert_allclose(out, sdpa(c["q"], K, V), rtol=1e-11, atol=1e-13)
    np.testing.assert_allclose(out, O.full_attention(c["q"], c["kl"], c["vl"], c["H_kv"]), rtol=0, atol=0)


@pytest.mark.parametrize("r", [0, 1, 3])
def test_against_torch_linear_and_sdpa(r):
    c = rand_case(20 + r, L=64, H_q=8, H_kv=4, d=8, r=r)
    xk = torch.from_numpy(np.concatenate([c["kg"], c["kl"]], axis=1))
    xv = torch.from_numpy(np.concatenate([c["vg"], c["vl"]], axis=1))
    k_hat = F.linear(xk, torch.from_numpy(c["Wk"]))
    v_hat = F.linear(xv, torch.from_numpy(c["Wv"]))
    K = torch.cat([torch.from_numpy(c["kl"]), k_hat], 1).reshape(c["L"], c["H_kv"], c["d"]).numpy()
    V = torch.cat([torch.from_numpy(c["vl"]), v_hat], 1).reshape(c["L"], c["H_kv"], c["d"]).numpy()
    np.testing.assert_allclose(run(c), sdpa(c["q"], K, V), rtol=1e-11, atol=1e-13)
    np.testing.assert_allclose(run(c, scale=0.2), sdpa(c["q"], K, V, scale=0.2), rtol=1e-11, atol=1e-13)


# --------------------------------------------------------------------------
# P4: selector weights -> exact reconstruction -> attention on the true layer
# --------------------------------------------------------------------------
def test_selector_weights_reduce_to_attention_on_true_cache():
    g = rng(31)
    L, H_q, H_kv, d, r = 29, 6, 3, 4, 1
    D, m = H_kv * d, r * d
    k_true, v_true = g.standard_normal((L, D)), g.standard_normal((L, D))
    # current layer identical to the anchor; W selects anchor dims m..D-1
    Wk = np.zeros((D - m, D + m)); Wv = np.zeros((D - m, D + m))
    for i in range(D - m):
        Wk[i, m + i] = 1.0
        Wv[i, m + i] = 1.0
    q = g.standard_normal((H_q, d))
    out = O.decode_attention(q, k_true, v_true, k_true[:, :m], v_true[:, :m], Wk, Wv, H_kv)
    ref = sdpa(q, k_true.reshape(L, H_kv, d), v_true.reshape(L, H_kv, d))
    np.testing.assert_allclose(out, ref, rtol=1e-11, atol=1e-13)
    # and selecting through the *local* columns: dropped dim i := local dim (i mod m)
    Wk2 = np.zeros_like(Wk); Wv2 = np.zeros_like(Wv)
    for i in range(D - m):
        Wk2[i, D + i % m] = 1.0
        Wv2[i, D + i % m] = 1.0
    kl, vl = g.standard_normal((L, m)), g.standard_normal((L, m))
    out2 = O.decode_attention(q, k_true, v_true, kl, vl, Wk2, Wv2, H_kv)
    ref2 = sdpa(q, np.tile(kl, (1, H_kv)).reshape(L, H_kv, d), np.tile(vl, (1, H_kv)).reshape(L, H_kv, d))
    np.testing.assert_allclose(out2, ref2, rtol=1e-11, atol=1e-13)


# --------------------------------------------------------------------------
# P3: linearity of the reconstruction, additivity over the two column blocks
# --------------------------------------------------------------------------
def test_reconstruction_is_linear_and_block_additive():
    g = rng(41)
    L, D, m = 9, 12, 4
    W = g.standard_normal((D - m, D + m))
    xg, yg = g.standard_normal((L, D)), g.standard_normal((L, D))
    xl, yl = g.standard_normal((L, m)), g.standard_normal((L, m))
    a, b = 1.75, -0.5
    lhs = O.reconstruct_dropped(W, a * xg + b * yg, a * xl + b * yl)
    rhs = a * O.reconstruct_dropped(W, xg, xl) + b * O.reconstruct_dropped(W, yg, yl)
    np.testing.assert_allclose(lhs, rhs, rtol=1e-12, atol=1e-12)
    z_g, z_l = np.zeros_like(xg), np.zeros_like(xl)
    parts = O.reconstruct_dropped(W, xg, z_l) + O.reconstruct_dropped(W, z_g, xl)
    np.testing.assert_allclose(O.reconstruct_dropped(W, xg, xl), parts, rtol=1e-12, atol=1e-12)
    # the global block is columns 0..D-1, the local block columns D..D+m-1
    np.testing.assert_allclose(O.reconstruct_dropped(W, xg, z_l), xg @ W[:, :D].T, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(O.reconstruct_dropped(W, z_g, xl), xl @ W[:, D:].T, rtol=1e-12, atol=1e-12)
    bias = g.standard_normal(D - m)
    np.testing.assert_allclose(O.reconstruct_dropped(W, xg, xl, bias) - O.reconstruct_dropped(W, xg, xl),
                               np.tile(bias, (L, 1)), rtol=1e-12, atol=1e-12)


# --------------------------------------------------------------------------
# P5: zero-weight closed forms
# --------------------------------------------------------------------------
def test_zero_key_predictor_gives_uniform_average():
    c = rand_case(51, L=33, H_q=8, H_kv=4, d=4, r=1)
    full = run(c)
    c0 = dict(c, Wk=np.zeros_like(c["Wk"]))
    out = run(c0)
    g = c["H_q"] // c["H_kv"]
    x_mean = np.concatenate([c["vg"], c["vl"]], axis=1).mean(axis=0)
    v_hat_mean = c["Wv"] @ x_mean                       # W^V mean_t(x_t)
    for h in range(c["H_q"]):
        kv = h // g
        if kv * c["d"] < c["m"]:
            np.testing.assert_allclose(out[h], full[h], rtol=0, atol=0)   # retained heads untouched
        else:
            lo = kv * c["d"] - c["m"]
            np.testing.assert_allclose(out[h], v_hat_mean[lo:lo + c["d"]], rtol=1e-12, atol=1e-13)


def test_zero_value_predictor_gives_zero_output_on_dropped_heads():
    c = rand_case(52, L=21, H_q=4, H_kv=4, d=4, r=2)
    out = run(dict(c, Wv=np.zeros_like(c["Wv"])))
    assert np.all(out[2:] == 0.0)
    np.testing.assert_allclose(out[:2], run(c)[:2], rtol=0, atol=0)


# --------------------------------------------------------------------------
# P6: softmax invariants
# --------------------------------------------------------------------------
def test_probabilities_sum_to_one_and_shift_invariance():
    c = rand_case(61, L=40, H_q=4, H_kv=2, d=8, r=1)
    K = O.assemble_cache(c["kl"], O.reconstruct_dropped(c["Wk"], c["kg"], c["kl"]), 2, 8)
    p = O.attention_probabilities(c["q"], K)
    np.testing.assert_allclose(p.sum(axis=1), 1.0, rtol=1e-13)
    # adding c * q_h / |q_h|^2 to every key of a head shifts all its scores by c
    out = run(c)
    V = O.assemble_cache(c["vl"], O.reconstruct_dropped(c["Wv"], c["vg"], c["vl"]), 2, 8)
    K2 = K.copy()
    K2[:, 0, :] += 3.0 * c["q"][0] / (c["q"][0] @ c["q"][0])
    out2 = O.attention(c["q"], K2, V)
    np.testing.assert_allclose(out2[0], out[0], rtol=1e-10, atol=1e-12)


def test_large_scores_do_not_overflow():
    q = np.array([[1000.0, 0.0]])
    K = np.array([[[1.0, 0.0]], [[2.0, 0.0]], [[-1.0, 0.0]]])
    V = np.array([[[1.0, 0.0]], [[0.0, 1.0]], [[5.0, 5.0]]])
    out = O.attention(q, K, V, scale=1.0)
    assert np.all(np.isfinite(out))
    np.testing.assert_allclose(out, [[0.0, 1.0]], atol=1e-300)


def test_token_permutation_leaves_output_unchanged():
    c = rand_case(62, L=31, H_q=4, H_kv=2, d=8, r=1)
    perm = rng(7).permutation(c["L"])
    cp = dict(c, kg=c["kg"][perm], vg=c["vg"][perm], kl=c["kl"][perm], vl=c["vl"][perm])
    np.testing.assert_allclose(run(cp), run(c), rtol=1e-12, atol=1e-14)


def test_concatenated_contexts_merge_by_log_sum_exp():
    c = rand_case(63, L=50, H_q=4, H_kv=2, d=8, r=1)
    cut = 19
    K = O.assemble_cache(c["kl"], O.reconstruct_dropped(c["Wk"], c["kg"], c["kl"]), 2, 8)
    scale = 1 / math.sqrt(8)
    whole = run(c)
    merged = np.zeros_like(whole)
    for h in range(4):
        parts = []
        for sl in (slice(0, cut), slice(cut, 50)):
            cc = dict(c, kg=c["kg"][sl], vg=c["vg"][sl], kl=c["kl"][sl], vl=c["vl"][sl])
            s = (K[sl, h // 2, :] @ c["q"][h]) * scale
            parts.append((run(cc)[h], math.log(np.exp(s - s.max()).sum()) + s.max()))
        w = np.array([math.exp(l - max(p[1] for p in parts)) for _, l in parts])
        merged[h] = (w[0] * parts[0][0] + w[1] * parts[1][0]) / w.sum()
    np.testing.assert_allclose(merged, whole, rtol=1e-11, atol=1e-13)


# --------------------------------------------------------------------------
# per-head evaluation, multi-layer routing, stored-precision helpers
# --------------------------------------------------------------------------
@pytest.mark.parametrize("r", [0, 1, 2, 4])
def test_per_head_evaluation_matches_full_evaluation(r):
    c = rand_case(70 + r, L=45, H_q=8, H_kv=4, d=8, r=r)
    full = run(c)
    some = O.decode_attention_query_heads(c["q"], c["kg"], c["vg"], c["kl"], c["vl"], c["Wk"], c["Wv"],
                                          c["H_kv"], query_heads=[0, 3, 4, 7])
    for h, v in some.items():
        np.testing.assert_allclose(v, full[h], rtol=1e-12, atol=1e-14)
    # and directly against the brute force
    bf = brute_force(c)
    for h, v in some.items():
        np.testing.assert_allclose(v, bf[h], rtol=1e-12, atol=1e-13)


def test_layer_step_routes_anchor_and_compressed_layers():
    g = rng(81)
    n_layers, S, L, H_q, H_kv, d, r = 6, 3, 17, 4, 2, 4, 1
    D, m = H_kv * d, r * d
    ck = [g.standard_normal((L, D)) for _ in range(n_layers)]
    cv = [g.standard_normal((L, D)) for _ in range(n_layers)]
    wk = [None if l % S == 0 else g.standard_normal((D - m, D + m)) for l in range(n_layers)]
    wv = [None if l % S == 0 else g.standard_normal((D - m, D + m)) for l in range(n_layers)]
    q = g.standard_normal((H_q, d))
    for l in range(n_layers):
        out = O.layer_step(l, S, q, ck, cv, wk, wv, H_kv, m)
        if l % S == 0:
            ref = sdpa(q, ck[l].reshape(L, H_kv, d), cv[l].reshape(L, H_kv, d))
        else:
            a = (l // S) * S
            c = dict(q=q, kg=ck[a], vg=cv[a], kl=ck[l][:, :m], vl=cv[l][:, :m], Wk=wk[l], Wv=wv[l],
                     H_q=H_q, H_kv=H_kv, d=d, m=m, D=D, L=L)
            ref = brute_force(c)
        np.testing.assert_allclose(out, ref, rtol=1e-11, atol=1e-13)


def test_bf16_widening_is_exact():
    x = torch.randn(1000, generator=torch.Generator().manual_seed(3)).to(torch.bfloat16)
    bits = x.view(torch.int16).numpy().view(np.uint16)
    np.testing.assert_array_equal(O.bf16_bits_to_f64(bits), x.to(torch.float64).numpy())
    np.testing.assert_array_equal(O.widen(bits), x.to(torch.float64).numpy())
    f = np.float32([1.5, -2.25])
    np.testing.assert_array_equal(O.widen(f), np.float64([1.5, -2.25]))


def test_empty_cache_is_rejected():
    with pytest.raises(ValueError):
        O.attention(np.ones((2, 4)), np.zeros((0, 1, 4)), np.zeros((0, 1, 4)))


# --------------------------------------------------------------------------
# Planted mistakes (on the CPU, in the oracle): each must be caught by a pin
# --------------------------------------------------------------------------
def _expect_caught(monkeypatch, attr, wrong, pins):
    monkeypatch.setattr(O, attr, wrong)
    caught = 0
    for pin in pins:
        try:
            pin()
        except AssertionError:
            caught += 1
        except ValueError:
            caught += 1
    monkeypatch.undo()
    assert caught > 0, "planted mistake in %s slipped through" % attr


def test_planted_mistakes_are_caught(monkeypatch):
    good_input = O.predictor_input
    good_probs = O.attention_probabilities
    good_recon = O.reconstruct_dropped

    def swapped_concat(c_global, c_local):                       # [local ; global]
        return np.concatenate([np.asarray(c_local, float), np.asarray(c_global, float)], axis=1)

    def no_scale(q, K, scale=None, rope_theta=None):                              # forgot 1/sqrt(d)
        return good_probs(q, K, 1.0 if scale is None else scale)

    def wrong_group(q, K, scale=None, rope_theta=None):                           # h % H_kv instead of h // g
        K = np.asarray(K, float)
        H_q, H_kv = np.asarray(q).shape[0], K.shape[1]
        g = H_q // H_kv
        idx = [(h % H_kv) for h in range(H_q)]
        K2 = np.stack([K[:, idx[h], :] for h in range(H_q)], axis=1)   # [L, H_q, d]
        return good_probs(q, K2, scale)

    def dropped_local_block(W, c_global, c_local, bias=None):    # ignores the local features
        return good_recon(W, c_global, np.zeros_like(np.asarray(c_local, float)), bias)

    def transposed_square_W(W, c_global, c_local, bias=None):
        W = np.asarray(W, float)
        return good_recon(W.T if W.shape[0] == W.shape[1] else W, c_global, c_local, bias)

    pins = [test_hand_computed_two_token_case,
            lambda: test_brute_force_tiny(2, 5, 4, 2, 4, 0),
            lambda: test_brute_force_tiny(3, 7, 6, 3, 2, 2),
            lambda: test_against_torch_linear_and_sdpa(1),
            test_selector_weights_reduce_to_attention_on_true_cache,
            test_reconstruction_is_linear_and_block_additive]
    _expect_caught(monkeypatch, "predictor_input", swapped_concat, pins)
    _expect_caught(monkeypatch, "attention_probabilities", no_scale, pins)
    _expect_caught(monkeypatch, "attention_probabilities", wrong_group, pins)
    _expect_caught(monkeypatch, "reconstruct_dropped", dropped_local_block, pins)
    _expect_caught(monkeypatch, "reconstruct_dropped", transposed_square_W, pins)


# --------------------------------------------------------------------------
# Sink and recent-window tokens at full precision (Section 4.1)
# --------------------------------------------------------------------------
def true_dropped(c, seed):
    """A layer's own dims m..D-1 (what the predictor stands in for), unrelated to W on purpose."""
    rng = np.random.default_rng(1000 + seed)
    return rng.standard_normal((c["L"], c["D"] - c["m"])), rng.standard_normal((c["L"], c["D"] - c["m"]))


def run_windowed(c, kt, vt, n_sink, n_window, scale=None):
    return O.decode_attention_windowed(c["q"], c["kg"], c["vg"], c["kl"], c["vl"], c["Wk"], c["Wv"], c["H_kv"],
                                       kt, vt, n_sink, n_window, scale)


def brute_force_windowed(c, kt, vt, n_sink, n_window, all_keys_true=False):
    """Index by index: a sink / window token reads its stored dims, any other token the predicted ones.
    all_keys_true: every token's key dims m..D-1 are read from kt (keys kept whole)."""
    q, kg, vg, kl, vl, Wk, Wv = (c[k].tolist() for k in ("q", "kg", "vg", "kl", "vl", "Wk", "Wv"))
    H_q, H_kv, d, m, D, L = c["H_q"], c["H_kv"], c["d"], c["m"], c["D"], c["L"]
    grp = H_q // H_kv

    def value(glob, loc, W, true, t, flat, always_true=False):
        if flat < m:
            return loc[t][flat]
        if always_true or t < n_sink or t > L - 1 - n_window:
            return true[t][flat - m]
        row = W[flat - m]
        return math.fsum([row[i] * glob[t][i] for i in range(D)] + [row[D + i] * loc[t][i] for i in range(m)])
    out = []
    for h in range(H_q):
        kv = h // grp
        s = [math.fsum(q[h][j] * value(kg, kl, Wk, kt.tolist(), t, kv * d + j, all_keys_true) for j in range(d))
             / math.sqrt(d) for t in range(L)]
        mx = max(s)
        e = [math.exp(v - mx) for v in s]
        z = math.fsum(e)
        out.append([math.fsum(e[t] / z * value(vg, vl, Wv, vt.tolist(), t, kv * d + j) for t in range(L))
                    for j in range(d)])
    return np.array(out)


@pytest.mark.parametrize("seed,L,H_q,H_kv,d,r,n_sink,n_window", [
    (11, 9, 4, 2, 4, 1, 2, 3), (12, 7, 2, 2, 4, 0, 1, 0), (13, 8, 6, 3, 2, 2, 0, 2), (14, 5, 2, 2, 4, 1, 4, 4)])
def test_windowed_brute_force_tiny(seed, L, H_q, H_kv, d, r, n_sink, n_window):
    c = rand_case(seed, L, H_q, H_kv, d, r)
    kt, vt = true_dropped(c, seed)
    np.testing.assert_allclose(run_windowed(c, kt, vt, n_sink, n_window),
                               brute_force_windowed(c, kt, vt, n_sink, n_window), rtol=1e-12, atol=1e-13)


def test_windowed_limits():
    c = rand_case(21, 10, 4, 2, 4, 1)
    kt, vt = true_dropped(c, 21)
    # no sink, no window: the plain method
    np.testing.assert_array_equal(run_windowed(c, kt, vt, 0, 0), run(c))
    # everything inside sink + window: standard attention on the layer's true cache (library routine)
    K = np.concatenate([c["kl"], kt], axis=1).reshape(c["L"], c["H_kv"], c["d"])
    V = np.concatenate([c["vl"], vt], axis=1).reshape(c["L"], c["H_kv"], c["d"])
    for n_sink, n_window in ((4, 6), (0, 10), (10, 0), (3, 128)):
        np.testing.assert_allclose(run_windowed(c, kt, vt, n_sink, n_window), sdpa(c["q"], K, V), rtol=1e-12, atol=1e-13)
    # rows of the true dims outside sink / window are never read
    poisoned_k, poisoned_v = kt.copy(), vt.copy()
    poisoned_k[2:7] = np.nan
    poisoned_v[2:7] = np.nan
    np.testing.assert_array_equal(run_windowed(c, poisoned_k, poisoned_v, 2, 3), run_windowed(c, kt, vt, 2, 3))
    # the per-head evaluation agrees
    per = O.decode_attention_query_heads(c["q"], c["kg"], c["vg"], c["kl"], c["vl"], c["Wk"], c["Wv"], c["H_kv"],
                                         range(c["H_q"]), k_true_drop=kt, v_true_drop=vt, n_sink=2, n_window=3)
    full = run_windowed(c, kt, vt, 2, 3)
    for h in range(c["H_q"]):
        np.testing.assert_allclose(per[h], full[h], rtol=1e-12, atol=1e-14)


def test_windowed_planted_mistakes_are_caught(monkeypatch):
    good = O.full_precision_tokens

    def window_at_the_front(L, n_sink, n_window):               # the window must be the LAST tokens
        t = np.arange(L)
        return (t < n_sink) | ((t >= n_sink) & (t < n_sink + n_window))

    def off_by_one(L, n_sink, n_window):
        t = np.arange(L)
        return (t < n_sink) | (t > L - n_window)

    def sink_forgotten(L, n_sink, n_window):
        return good(L, 0, n_window)

    pins = [lambda: test_windowed_brute_force_tiny(11, 9, 4, 2, 4, 1, 2, 3),
            lambda: test_windowed_brute_force_tiny(13, 8, 6, 3, 2, 2, 0, 2)]
    for bad in (window_at_the_front, off_by_one, sink_forgotten):
        _expect_caught(monkeypatch, "full_precision_tokens", bad, pins)


# --------------------------------------------------------------------------
# m that splits a head (the paper's m = 64 and m = 384 with d = 128: Appendix
# "Compression-Ratio Configurations"): Eq. 6 concatenates at the flat index
# --------------------------------------------------------------------------
@pytest.mark.parametrize("seed,L,H_q,H_kv,d,m", [(31, 5, 4, 2, 4, 2), (32, 6, 4, 2, 4, 6), (33, 4, 6, 3, 4, 5),
                                                   (34, 7, 2, 2, 8, 12)])
def test_brute_force_with_a_split_head(seed, L, H_q, H_kv, d, m):
    c = rand_case(seed, L, H_q, H_kv, d, m=m)
    assert c["m"] % d != 0 and c["Wk"].shape == (c["D"] - m, c["D"] + m)
    bf = brute_force(c)
    np.testing.assert_allclose(run(c), bf, rtol=1e-12, atol=1e-13)
    # the per-head evaluation takes the stored dims of the split head from the cache and the rest from W
    per = O.decode_attention_query_heads(c["q"], c["kg"], c["vg"], c["kl"], c["vl"], c["Wk"], c["Wv"], c["H_kv"],
                                         query_heads=range(H_q))
    for h in range(H_q):
        np.testing.assert_allclose(per[h], bf[h], rtol=1e-12, atol=1e-13)
    # a selector predictor makes the split head exact: standard attention on the true cache (library routine)
    g = rng(seed + 100)
    D = c["D"]
    k_true = np.concatenate([c["kl"], g.standard_normal((L, D - m))], axis=1)
    v_true = np.concatenate([c["vl"], g.standard_normal((L, D - m))], axis=1)
    sel = np.zeros((D - m, D + m))
    sel[np.arange(D - m), m + np.arange(D - m)] = 1.0
    kg, vg = c["kg"].copy(), c["vg"].copy()
    kg[:, m:], vg[:, m:] = k_true[:, m:], v_true[:, m:]
    got = O.decode_attention(c["q"], kg, vg, c["kl"], c["vl"], sel, sel, c["H_kv"])
    np.testing.assert_allclose(got, sdpa(c["q"], k_true.reshape(L, H_kv, d), v_true.reshape(L, H_kv, d)),
                               rtol=1e-12, atol=1e-13)


def test_per_head_evaluation_with_biases_whole_keys_and_a_window():
    for m in (8, 12):                           # head-aligned and head-splitting (d = 8)
        c = rand_case(90 + m, L=23, H_q=8, H_kv=4, d=8, m=m)
        g = rng(90 + m)
        bk, bv = g.standard_normal(c["D"] - m), g.standard_normal(c["D"] - m)
        args = (c["q"], c["kg"], c["vg"], c["kl"], c["vl"], c["Wk"], c["Wv"], c["H_kv"])
        heads = range(c["H_q"])
        full = O.decode_attention(*args, bk=bk, bv=bv)
        per = O.decode_attention_query_heads(*args, query_heads=heads, bk=bk, bv=bv)
        k_true = g.standard_normal((c["L"], c["D"]))
        full_sk = O.decode_attention(*args, bv=bv, k_true=k_true, rope_theta=500.0)
        per_sk = O.decode_attention_query_heads(*args, query_heads=heads, bv=bv, k_true=k_true, rope_theta=500.0)
        kt, vt = true_dropped(c, m)
        full_w = O.decode_attention_windowed(*args, kt, vt, 2, 5, bk=bk, bv=bv, rope_theta=500.0)
        per_w = O.decode_attention_query_heads(*args, query_heads=heads, k_true_drop=kt, v_true_drop=vt, n_sink=2,
                                               n_window=5, bk=bk, bv=bv, rope_theta=500.0)
        full_wsk = O.decode_attention_windowed(*args, None, vt, 2, 5, bv=bv, k_true=k_true)
        per_wsk = O.decode_attention_query_heads(*args, query_heads=heads, v_true_drop=vt, n_sink=2, n_window=5, bv=bv,
                                                 k_true=k_true)
        for h in heads:
            np.testing.assert_allclose(per[h], full[h], rtol=1e-12, atol=1e-13)
            np.testing.assert_allclose(per_sk[h], full_sk[h], rtol=1e-12, atol=1e-13)
            np.testing.assert_allclose(per_w[h], full_w[h], rtol=1e-12, atol=1e-13)
            np.testing.assert_allclose(per_wsk[h], full_wsk[h], rtol=1e-12, atol=1e-13)
        # the bias is a plain shift of the predicted dims: the same as one more input feature that is always 1
        ones = np.ones((c["L"], 1))
        kl1, vl1 = np.concatenate([c["kl"], ones], axis=1), np.concatenate([c["vl"], ones], axis=1)
        Wk1 = np.concatenate([c["Wk"], bk[:, None]], axis=1)
        Wv1 = np.concatenate([c["Wv"], bv[:, None]], axis=1)
        K1 = O.reconstruct_dropped(Wk1, c["kg"], kl1)
        np.testing.assert_allclose(K1, O.reconstruct_dropped(c["Wk"], c["kg"], c["kl"], bk), rtol=1e-12, atol=1e-13)
        V1 = O.reconstruct_dropped(Wv1, c["vg"], vl1)
        np.testing.assert_allclose(V1, O.reconstruct_dropped(c["Wv"], c["vg"], c["vl"], bv), rtol=1e-12, atol=1e-13)


def test_window_with_whole_keys():
    """"Save K" with a sink / window: the keys are whole, so the window changes the values only."""
    c = rand_case(61, L=11, H_q=4, H_kv=2, d=4, m=4)
    g = rng(61)
    L, D, m, H, d = c["L"], c["D"], c["m"], c["H_kv"], c["d"]
    k_true = g.standard_normal((L, D))
    kt, vt = true_dropped(c, 61)
    args = (c["q"], c["kg"], c["vg"], c["kl"], c["vl"], c["Wk"], c["Wv"], H)
    got = O.decode_attention_windowed(*args, kt, vt, 2, 3, k_true=k_true)
    # brute force: the keys of a cache whose K predictor is never consulted = every token's keys "true"
    c2 = dict(c)
    c2["kl"] = k_true[:, :m]
    bf = brute_force_windowed(c2, k_true[:, m:], vt, 2, 3, all_keys_true=True)
    np.testing.assert_allclose(got, bf, rtol=1e-12, atol=1e-13)
    # no window: the plain save-K step; everything inside the window: standard attention on the true cache
    np.testing.assert_array_equal(O.decode_attention_windowed(*args, kt, vt, 0, 0, k_true=k_true),
                                  O.decode_attention(*args, k_true=k_true))
    V = np.concatenate([c["vl"], vt], axis=1).reshape(L, H, d)
    np.testing.assert_allclose(O.decode_attention_windowed(*args, kt, vt, 0, L, k_true=k_true),
                               sdpa(c["q"], k_true.reshape(L, H, d), V), rtol=1e-12, atol=1e-13)
    # k_local, Wk and k_true_drop are not read
    bad = (c["q"], c["kg"], c["vg"], np.full_like(c["kl"], np.nan), c["vl"], None, c["Wv"], H)
    np.testing.assert_array_equal(O.decode_attention_windowed(*bad, None, vt, 2, 3, k_true=k_true), got)


def test_prefill_shaped_attention_with_sink_and_window():
    """Every query is the windowed decode step of the sequence cut off at its own position."""
    for m, rope in ((8, None), (12, 700.0)):
        c = rand_case(71 + m, L=19, H_q=8, H_kv=4, d=8, m=m)
        g = rng(71 + m)
        n_q, n_sink, n_window = 9, 2, 4
        L, H, d = c["L"], c["H_kv"], c["d"]
        q = g.standard_normal((n_q, c["H_q"], d))
        kt, vt = true_dropped(c, m)
        args = (c["kg"], c["vg"], c["kl"], c["vl"], c["Wk"], c["Wv"], H)
        got = O.prefill_attention(q, *args, k_true_drop=kt, v_true_drop=vt, n_sink=n_sink, n_window=n_window,
                                  rope_theta=rope)
        for i in range(n_q):
            n = L - n_q + i + 1
            want = O.decode_attention_windowed(q[i], c["kg"][:n], c["vg"][:n], c["kl"][:n], c["vl"][:n], c["Wk"],
                                               c["Wv"], H, kt[:n], vt[:n], n_sink, n_window, rope_theta=rope)
            np.testing.assert_allclose(got[i], want, rtol=1e-12, atol=1e-13)
        if rope is None:
            # index by index, for a query in the middle of the chunk: ITS last n_window tokens are the true ones
            i = 4
            n = L - n_q + i + 1
            cut = dict(c, q=q[i], kg=c["kg"][:n], vg=c["vg"][:n], kl=c["kl"][:n], vl=c["vl"][:n], L=n)
            np.testing.assert_allclose(got[i], brute_force_windowed(cut, kt[:n], vt[:n], n_sink, n_window),
                                       rtol=1e-12, atol=1e-13)
        # a token is read as stored by the queries close behind it and as predicted by the later ones: what is
        # stored for token L - n_q (the first query's own) reaches the queries 0 .. n_window - 1 only
        kt2, vt2 = kt.copy(), vt.copy()
        kt2[L - n_q] += 1.0
        vt2[L - n_q] -= 1.0
        got2 = O.prefill_attention(q, *args, k_true_drop=kt2, v_true_drop=vt2, n_sink=n_sink, n_window=n_window,
                                   rope_theta=rope)
        assert all(np.abs(got2[i] - got[i]).max() > 1e-6 for i in range(n_window))
        np.testing.assert_array_equal(got2[n_window:], got[n_window:])
        # no sink, no window: the plain prefill-shaped call; a window as long as the cache: causal attention on
        # the true cache (library routine)
        np.testing.assert_array_equal(O.prefill_attention(q, *args, k_true_drop=kt, v_true_drop=vt, rope_theta=rope),
                                      O.prefill_attention(q, *args, rope_theta=rope))
        if rope is None:
            allq = g.standard_normal((L, c["H_q"], d))
            full = O.prefill_attention(allq, *args, k_true_drop=kt, v_true_drop=vt, n_sink=0, n_window=L)
            K = np.concatenate([c["kl"], kt], axis=1).reshape(L, H, d)
            V = np.concatenate([c["vl"], vt], axis=1).reshape(L, H, d)
            tq = torch.from_numpy(allq).permute(1, 0, 2)[None]
            tk = torch.from_numpy(K).permute(1, 0, 2)[None]
            tv = torch.from_numpy(V).permute(1, 0, 2)[None]
            ref = F.scaled_dot_product_attention(tq, tk, tv, is_causal=True, enable_gqa=True)[0].permute(1, 0, 2).numpy()
            np.testing.assert_allclose(full, ref, rtol=1e-12, atol=1e-13)


def test_prefill_window_planted_mistake_is_caught(monkeypatch):
    good = O.full_precision_tokens

    def window_of_the_whole_cache(L, n_sink, n_window):          # one window for all queries, at the end of the cache
        return good(19, n_sink, n_window)[:L]

    _expect_caught(monkeypatch, "full_precision_tokens", window_of_the_whole_cache,
                   [test_prefill_shaped_attention_with_sink_and_window])
