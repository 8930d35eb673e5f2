"""Pins of the oracle's rotate-on-read path (Section 3.2: the predictors, hence the cache, hold keys
prior to the rotary position embedding) against things other than the oracle itself: values worked
out by hand, the complex-number form of the rotation, a library rotary routine (the Llama layout), the
relative-position property, and planted mistakes."""
import math

import numpy as np
import pytest
import torch

from oracle import echokv_oracle as O
from tests.test_oracle_pins import _expect_caught, rand_case, run, sdpa, true_dropped

THETA = 10000.0


def test_hand_values_pairing_and_frequencies():
    # d = 4: two frequencies, 1 and theta^(-2/4) = 0.01; feature 0 pairs with 2, feature 1 with 3.
    K = np.zeros((101, 1, 4))
    K[1, 0] = [1, 0, 0, 0]          # position 1, first pair: angle 1
    K[100, 0] = [0, 1, 0, 0]        # position 100, second pair: angle 100 * 0.01 = 1
    K[0, 0] = [3, -2, 5, 7]         # position 0: untouched
    K[50, 0] = [0, 0, 1, 0]         # position 50, first pair, starting on the second axis
    R = O.rotate_keys(K, THETA)
    c1, s1 = math.cos(1.0), math.sin(1.0)
    np.testing.assert_allclose(R[1, 0], [c1, 0, s1, 0], atol=1e-15)
    np.testing.assert_allclose(R[100, 0], [0, c1, 0, s1], atol=1e-13)
    np.testing.assert_array_equal(R[0, 0], [3, -2, 5, 7])
    np.testing.assert_allclose(R[50, 0], [-math.sin(50.0), 0, math.cos(50.0), 0], atol=1e-13)
    a = O.rope_angles(3, 8, THETA)
    np.testing.assert_allclose(a[2], [2.0, 0.2, 0.02, 0.002], rtol=1e-14)


def test_complex_number_form():
    # (k_j + i k_{j+d/2}) * exp(i t w_j), w_j = theta^(-2j/d)
    g = np.random.default_rng(3)
    L, H, d = 29, 3, 16
    K = g.standard_normal((L, H, d))
    z = K[:, :, :d // 2] + 1j * K[:, :, d // 2:]
    w = np.array([THETA ** (-(2 * j) / d) for j in range(d // 2)])
    zr = z * np.exp(1j * np.arange(L)[:, None, None] * w[None, None, :])
    want = np.concatenate([zr.real, zr.imag], axis=2)
    np.testing.assert_allclose(O.rotate_keys(K, THETA), want, rtol=1e-12, atol=1e-13)


def test_library_rotary_routine_llama_layout():
    llama = pytest.importorskip("transformers.models.llama.modeling_llama")
    g = np.random.default_rng(4)
    L, H, d = 33, 2, 8
    K = g.standard_normal((L, H, d))
    inv_freq = 1.0 / (THETA ** (torch.arange(0, d, 2, dtype=torch.float64) / d))
    ang = torch.arange(L, dtype=torch.float64)[:, None] * inv_freq[None, :]
    emb = torch.cat([ang, ang], dim=-1)[None]                         # [1, L, d]
    k = torch.from_numpy(K).permute(1, 0, 2)[None]                    # [1, H, L, d]
    _, k_rot = llama.apply_rotary_pos_emb(k, k, emb.cos(), emb.sin())
    np.testing.assert_allclose(O.rotate_keys(K, THETA), k_rot[0].permute(1, 0, 2).numpy(), rtol=1e-12, atol=1e-13)


def test_rotation_keeps_norms_and_relative_position_property():
    g = np.random.default_rng(5)
    L, d = 40, 8
    K = g.standard_normal((L, 1, d))
    R = O.rotate_keys(K, THETA)
    np.testing.assert_allclose(np.linalg.norm(R, axis=2), np.linalg.norm(K, axis=2), rtol=1e-13)
    # a query rotated to position p against a key rotated to position t depends on p - t only
    q0, k0 = g.standard_normal(d), g.standard_normal(d)

    def at(v, pos):
        buf = np.zeros((pos + 1, 1, d))
        buf[pos, 0] = v
        return O.rotate_keys(buf, THETA)[pos, 0]
    ref = at(q0, 17) @ at(k0, 5)
    for shift in (1, 9, 300):
        assert abs(at(q0, 17 + shift) @ at(k0, 5 + shift) - ref) < 1e-11
    assert abs(at(q0, 18) @ at(k0, 5) - ref) > 1e-3


def test_attention_entry_points_rotate_the_assembled_cache():
    c = rand_case(31, L=23, H_q=8, H_kv=4, d=8, r=1)
    K_t = O.assemble_cache(c["kl"], O.reconstruct_dropped(c["Wk"], c["kg"], c["kl"]), c["H_kv"], c["d"])
    V_t = O.assemble_cache(c["vl"], O.reconstruct_dropped(c["Wv"], c["vg"], c["vl"]), c["H_kv"], c["d"])
    want = sdpa(c["q"], O.rotate_keys(K_t, THETA), V_t)               # library attention on rotated keys
    np.testing.assert_allclose(run(c, rope_theta=THETA), want, rtol=1e-12, atol=1e-13)
    assert np.abs(run(c, rope_theta=THETA) - run(c)).max() > 1e-3     # and it is not a no-op
    per = O.decode_attention_query_heads(c["q"], c["kg"], c["vg"], c["kl"], c["vl"], c["Wk"], c["Wv"], c["H_kv"],
                                         range(c["H_q"]), rope_theta=THETA)
    for h in range(c["H_q"]):
        np.testing.assert_allclose(per[h], want[h], rtol=1e-12, atol=1e-13)
    # uncompressed / anchor layers
    L, H, d = c["L"], c["H_kv"], c["d"]
    full = O.full_attention(c["q"], c["kg"], c["vg"], H, rope_theta=THETA)
    np.testing.assert_allclose(full, sdpa(c["q"], O.rotate_keys(c["kg"].reshape(L, H, d), THETA), c["vg"].reshape(L, H, d)),
                               rtol=1e-12, atol=1e-13)
    # sink / window tokens are rotated like every other row
    kt, vt = true_dropped(c, 31)
    keep = O.full_precision_tokens(L, 2, 3)
    K_w = O.assemble_cache(c["kl"], O.overlay_true_dims(O.reconstruct_dropped(c["Wk"], c["kg"], c["kl"]), kt, keep), H, d)
    V_w = O.assemble_cache(c["vl"], O.overlay_true_dims(O.reconstruct_dropped(c["Wv"], c["vg"], c["vl"]), vt, keep), H, d)
    got = O.decode_attention_windowed(c["q"], c["kg"], c["vg"], c["kl"], c["vl"], c["Wk"], c["Wv"], H, kt, vt, 2, 3,
                                      rope_theta=THETA)
    np.testing.assert_allclose(got, sdpa(c["q"], O.rotate_keys(K_w, THETA), V_w), rtol=1e-12, atol=1e-13)
    # a one-token cache sits at position 0: rotation changes nothing
    one = rand_case(32, L=1, H_q=4, H_kv=2, d=8, r=1)
    np.testing.assert_array_equal(run(one, rope_theta=THETA), run(one))
    # layer_step passes it on to both kinds of layer
    g = np.random.default_rng(33)
    caches_k = [g.standard_normal((L, c["D"])) for _ in range(2)]
    caches_v = [g.standard_normal((L, c["D"])) for _ in range(2)]
    for layer in (0, 1):
        a = O.layer_step(layer, 2, c["q"], caches_k, caches_v, [None, c["Wk"]], [None, c["Wv"]], H, c["m"], rope_theta=THETA)
        b = O.layer_step(layer, 2, c["q"], caches_k, caches_v, [None, c["Wk"]], [None, c["Wv"]], H, c["m"])
        assert np.abs(a - b).max() > 1e-3


def test_planted_rotation_mistakes_are_caught(monkeypatch):
    good_angles = O.rope_angles

    def interleaved_pairs(K, rope_theta):                  # pairs (2j, 2j+1) instead of (j, j + d/2)
        K = np.asarray(K, dtype=np.float64)
        L, H, d = K.shape
        a = good_angles(L, d, rope_theta)[:, None, :]
        out = np.empty_like(K)
        out[:, :, 0::2] = K[:, :, 0::2] * np.cos(a) - K[:, :, 1::2] * np.sin(a)
        out[:, :, 1::2] = K[:, :, 1::2] * np.cos(a) + K[:, :, 0::2] * np.sin(a)
        return out

    def wrong_direction(K, rope_theta):                    # rotates by -angle
        K = np.asarray(K, dtype=np.float64)
        L, H, d = K.shape
        a = good_angles(L, d, rope_theta)[:, None, :]
        lo, hi = K[:, :, :d // 2], K[:, :, d // 2:]
        return np.concatenate([lo * np.cos(a) + hi * np.sin(a), hi * np.cos(a) - lo * np.sin(a)], axis=2)

    def one_sign_dropped(K, rope_theta):                   # not a rotation any more
        K = np.asarray(K, dtype=np.float64)
        L, H, d = K.shape
        a = good_angles(L, d, rope_theta)[:, None, :]
        lo, hi = K[:, :, :d // 2], K[:, :, d // 2:]
        return np.concatenate([lo * np.cos(a) + hi * np.sin(a), hi * np.cos(a) + lo * np.sin(a)], axis=2)

    pins = [test_hand_values_pairing_and_frequencies, test_complex_number_form,
            test_rotation_keeps_norms_and_relative_position_property]
    for bad in (interleaved_pairs, wrong_direction, one_sign_dropped):
        _expect_caught(monkeypatch, "rotate_keys", bad, pins)

    def exponent_j_over_d(L, d, rope_theta):               # theta^(-j/d) instead of theta^(-2j/d)
        j = np.arange(d // 2, dtype=np.float64)
        return np.arange(L, dtype=np.float64)[:, None] * np.power(float(rope_theta), -j / d)[None, :]

    def positions_from_one(L, d, rope_theta):
        return good_angles(L + 1, d, rope_theta)[1:]

    for bad in (exponent_j_over_d, positions_from_one):
        _expect_caught(monkeypatch, "rope_angles", bad, pins)
