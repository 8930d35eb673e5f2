"""GPU parity with rotate-on-read (Section 3.2: the predictors, hence the cache, hold keys prior to the
rotary position embedding): every kernel family that computes q . k against the oracle's rotation."""
import ctypes as C

import numpy as np
import pytest
import torch

from paper_2603_22910_b200 import binding, build, synth
from tests.harness import Case, assert_parity, errors

pytestmark = pytest.mark.gpu

THETA = 10000.0


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    binding.lib()


CASES = [
    # name, base, overrides, lens, window
    ("tiny_fp32_d64", synth.C0, {}, None, None),
    ("fp32_d128_gqa2", synth.C0, dict(n_q_heads=8, n_kv_heads=4, head_dim=128, n_retained_heads=1, batch=2,
                                      context=150), [150, 64], None),
    ("c2_shape", synth.C2, dict(batch=3, context=1000), [1000, 517, 256], None),
    ("c1_shape", synth.C1, dict(batch=2, context=700), [700, 333], None),
    ("c2_pages64_random", synth.C2, dict(batch=2, context=600, page_tokens=64, random_pages=True), [600, 65], None),
    ("gqa8", synth.C2, dict(n_q_heads=32, n_kv_heads=4, n_retained_heads=1, batch=1, context=300), [300], None),
    ("ragged_many_tiles", synth.C2, dict(batch=5, context=2000, random_pages=True), [2000, 129, 128, 1153, 1], None),
    ("c2_window", synth.C2, dict(batch=3, context=1000, random_pages=True), [1000, 517, 100], (4, 128)),
    ("fp32_d64_window", synth.C0, dict(batch=2, context=200), [200, 50], (2, 16)),
    ("bf16_d64", synth.C0, dict(dtype="bf16", batch=2, context=200), [200, 77], None),
]


@pytest.mark.parametrize("name,base,over,lens,window", CASES, ids=[c[0] for c in CASES])
def test_rope_against_oracle(name, base, over, lens, window):
    w = base.replace(**over)
    case = Case(w, lens=lens, layers=[0, 1], window=window, rope=THETA)
    assert case.ctx.rope_enabled()
    paths = ([1, 2, 3] + (([4, 5] if w.page_tokens <= 32 else [4]) if w.n_q_heads // w.n_kv_heads <= 2 else [])) if case.ctx.decode_path() >= 2 else [1]
    stored_paths = [0, 1] if case.ctx.stored_path() == 1 else [0]
    ref0, ref1 = case.oracle(0), case.oracle(1)
    for stored_path in stored_paths:
        case.ctx.set_stored_path(stored_path)
        out0 = case.run(0)
        assert_parity(out0, ref0, w.dtype, "%s anchor stored_path %d" % (name, stored_path))
        np.testing.assert_array_equal(case.run(0, full=True), out0)
        for path in paths:
            case.ctx.set_decode_path(path)
            assert_parity(case.run(1), ref1, w.dtype, "%s path %d stored_path %d" % (name, path, stored_path))
    assert case.ctx.device_status() == binding.ECHOKV_OK
    # switched off again, the context computes the un-rotated result
    case.ctx.set_rope(0)
    assert not case.ctx.rope_enabled()
    case.rope = None
    assert_parity(case.run(1), case.oracle(1), w.dtype, name + " rope off")
    assert errors(case.oracle(1), ref1)[1] > 1e-2          # (and the rotation is no small change)
    case.close()


@pytest.mark.parametrize("base,over,lens,window", [
    (synth.C2, dict(batch=2, context=600), [600, 131], None),
    (synth.C0, dict(batch=2, context=200), [200, 50], None),
    (synth.C2, dict(batch=2, context=600, n_q_heads=16, n_retained_heads=5, page_tokens=64), [600, 107], (0, 16)),
    (synth.C0, dict(batch=2, context=200), [200, 50], (2, 16)),
], ids=["bf16_gqa", "fp32_d64", "bf16_gqa2_window", "fp32_d64_window"])
def test_rope_with_predictor_biases(base, over, lens, window):
    # a bias on the K predictor is rotated with the predicted keys: it does not cancel in the softmax any more
    # (with sink / window tokens a V bias reaches the output only with the predicted tokens' share of the probability)
    w = base.replace(**over)
    case = Case(w, lens=lens, layers=[0, 1], biases=True, rope=THETA, window=window)
    ref = case.oracle(1)
    for path in (([1, 2, 3] + (([4, 5] if w.page_tokens <= 32 else [4]) if w.n_q_heads // w.n_kv_heads <= 2 else [])) if case.ctx.decode_path() >= 2 else [1]):
        case.ctx.set_decode_path(path)
        assert_parity(case.run(1), ref, w.dtype, "biases path %d" % path)
    Wk, Wv, bk, bv = case.weights[1]
    case.ctx.set_weights(1, Wk, Wv, None, bv)
    assert errors(case.run(1), ref)[1] > 1e-3          # without the K bias the result is another one
    assert case.ctx.device_status() == binding.ECHOKV_OK
    case.close()


MIXED = [
    # name, base, overrides, lens, window, biases
    ("c2_shape", synth.C2, dict(batch=3, context=1000), [1000, 517, 256], None, False),
    ("c1_shape", synth.C1, dict(batch=2, context=700), [700, 333], None, False),
    ("pages64_random", synth.C2, dict(batch=2, context=600, page_tokens=64, random_pages=True), [600, 65], None, False),
    ("ragged_many_tiles", synth.C2, dict(batch=5, context=2000, random_pages=True), [2000, 129, 128, 1153, 1], None, True),
    ("window", synth.C2, dict(batch=3, context=1000, random_pages=True), [1000, 517, 100], (4, 128), False),
    ("window_biases", synth.C2, dict(batch=2, context=700), [700, 150], (4, 128), True),
    ("nothing_retained", synth.C2, dict(batch=2, context=700, n_retained_heads=0), [700, 300], None, True),
    ("one_dropped_head", synth.C2, dict(batch=2, context=400, n_retained_heads=7), [400, 258], (2, 40), False),
]


@pytest.mark.parametrize("name,base,over,lens,window,biases", MIXED, ids=[c[0] for c in MIXED])
def test_rotated_keys_with_the_absorbed_value_side(name, base, over, lens, window, biases):
    # with rotated keys the absorbed mode keeps the K side explicit and absorbs the V side only
    w = base.replace(**over)
    case = Case(w, lens=lens, layers=[0, 1], window=window, biases=biases, rope=THETA)
    ref = case.oracle(1)
    assert_parity(case.run(1), ref, w.dtype, name + " explicit")
    case.ctx.enable_absorbed()
    assert case.ctx.decode_mode() == 1 and case.ctx.rope_enabled()
    out = case.run(1)
    assert_parity(out, ref, w.dtype, name + " K explicit, V absorbed")
    np.testing.assert_array_equal(case.run(1), out)             # and it is repeatable
    assert_parity(case.run(0), case.oracle(0), w.dtype, name + " anchor")
    # the order of the two switches does not matter, and without the table the mode is the fully absorbed one
    case.ctx.set_rope(0)
    case.rope = None
    assert_parity(case.run(1), case.oracle(1), w.dtype, name + " absorbed, no rotation")
    case.ctx.set_rope(THETA)
    case.rope = THETA
    assert_parity(case.run(1), ref, w.dtype, name + " table set after the mode")
    assert case.ctx.device_status() == binding.ECHOKV_OK
    case.close()


def test_rope_with_a_retained_width_that_splits_a_head():
    # the paper's m = 64 keeps half of head 0: the split head is predicted whole (its stored dims passed through),
    # so the rotation, which pairs feature j with j + 64 of a head, finds both halves in one place
    w = synth.C2.replace(batch=2, context=300, n_retained_dims=64, n_retained_heads=0)
    case = Case(w, lens=[300, 77], layers=[0, 1], rope=THETA)
    assert_parity(case.run(1), case.oracle(1), w.dtype, "m = 64, rotated")
    assert case.ctx.device_status() == binding.ECHOKV_OK
    case.close()


def test_rope_argument_checks():
    w = synth.C0
    case = Case(w, layers=[1])
    lib, h = binding.lib(), case.ctx.handle
    n = C.c_uint64(0)
    assert lib.echokv_rope_table_bytes(C.byref(case.cfg), C.byref(n)) == binding.ECHOKV_OK
    cap, half = w.pages_per_seq * w.page_tokens, w.head_dim // 2
    assert n.value == (cap * half + (cap // 16) * half + 16 * half) * 8     # full, every 16th position, offsets 0..15
    buf = torch.empty(n.value + 16, dtype=torch.uint8, device="cuda")
    assert lib.echokv_set_rope(h, 10000.0, buf.data_ptr(), n.value - 1, None) == binding.ECHOKV_ECAPACITY
    assert lib.echokv_set_rope(h, 0.5, buf.data_ptr(), n.value, None) == binding.ECHOKV_EINVAL
    assert lib.echokv_set_rope(h, float("nan"), buf.data_ptr(), n.value, None) == binding.ECHOKV_EINVAL
    assert lib.echokv_set_rope(h, 10000.0, buf.data_ptr() + 8, n.value, None) == binding.ECHOKV_EINVAL
    assert lib.echokv_set_rope(h, 10000.0, None, 0, None) == binding.ECHOKV_EINVAL
    assert not case.ctx.rope_enabled()
    assert lib.echokv_set_rope(h, 10000.0, buf.data_ptr(), n.value, None) == binding.ECHOKV_OK
    assert case.ctx.rope_enabled()
    # the table the library wrote: (cos, sin)(t * theta^(-2j/d)), [d/2][capacity]
    torch.cuda.synchronize()
    flat = buf[: n.value].view(torch.float32).view(-1, 2).cpu().numpy().astype(np.float64)
    tab = flat[: cap * half].reshape(half, cap, 2)
    coarse = flat[cap * half: cap * half + (cap // 16) * half].reshape(cap // 16, half, 2)
    fine = flat[cap * half + (cap // 16) * half:].reshape(16, half, 2)
    t = np.arange(cap, dtype=np.float64)
    for j in (0, 1, half - 1):
        wj = 10000.0 ** (-2.0 * j / w.head_dim)
        np.testing.assert_allclose(tab[j, :, 0], np.cos(t * wj), atol=1e-7)
        np.testing.assert_allclose(tab[j, :, 1], np.sin(t * wj), atol=1e-7)
        np.testing.assert_allclose(coarse[:, j, 0], np.cos(t[::16] * wj), atol=1e-7)
        np.testing.assert_allclose(coarse[:, j, 1], np.sin(t[::16] * wj), atol=1e-7)
        np.testing.assert_allclose(fine[:, j, 1], np.sin(t[:16] * wj), atol=1e-7)
    case.close()


# ---- the rotating stored-head kernel (anchor layer 0 and the retained heads of layer 1) on its own edge cases ----
STORED_ROPE = [
    # name, base, overrides, lens
    ("mha_many_items", synth.C1, dict(batch=3, context=2100), [2100, 1025, 64]),
    ("gqa4_one_token", synth.C2, dict(batch=3, context=1500, n_retained_heads=3, random_pages=True), [1500, 257, 1]),
    ("gqa2_pages32", synth.C2, dict(n_q_heads=16, batch=2, context=900, page_tokens=32, random_pages=True), [900, 33]),
    ("gqa8_pages64", synth.C2, dict(n_q_heads=32, n_kv_heads=4, n_retained_heads=2, batch=2, context=700,
                                    page_tokens=64), [700, 65]),
    ("gqa8_long", synth.C2, dict(n_q_heads=32, n_kv_heads=4, n_retained_heads=1, batch=2, context=5000,
                                 random_pages=True), [5000, 4097]),
    ("gqa4_pages128", synth.C2, dict(batch=2, context=1000, page_tokens=128, n_retained_heads=5,
                                     random_pages=True), [1000, 129]),
]


@pytest.mark.parametrize("name,base,over,lens", STORED_ROPE, ids=[s[0] for s in STORED_ROPE])
def test_rotating_stored_head_kernel_against_oracle(name, base, over, lens):
    w = base.replace(**over)
    case = Case(w, lens=lens, layers=[0, 1], rope=THETA)
    assert case.ctx.stored_path() == 1 and case.ctx.rope_enabled()
    for layer in (0, 1):
        out = case.run(layer)
        assert_parity(out, case.oracle(layer), w.dtype, "%s layer %d" % (name, layer))
        np.testing.assert_array_equal(case.run(layer), out)            # repeatable bit for bit
    np.testing.assert_array_equal(case.run(0, full=True), case.run(0))
    assert case.ctx.device_status() == binding.ECHOKV_OK
    case.close()


def test_rotating_stored_head_kernel_more_sequences_than_one_launch_indexes():
    w = synth.C2.replace(batch=600, context=48, n_kv_heads=2, n_q_heads=8, n_retained_heads=1)
    rng = np.random.default_rng(5)
    lens = [int(v) for v in rng.integers(1, 49, size=w.batch)]
    case = Case(w, lens=lens, layers=[0, 1], rope=THETA)
    assert_parity(case.run(0), case.oracle(0), w.dtype, "batch 600, anchor, rotated")
    assert_parity(case.run(1), case.oracle(1), w.dtype, "batch 600, compressed, rotated")
    assert case.ctx.device_status() == binding.ECHOKV_OK
    case.close()


def test_rotating_stored_head_kernel_ignores_what_unused_slots_hold_and_reports_bad_input():
    w = synth.C2.replace(batch=2, context=600, n_retained_heads=3, random_pages=True)
    lens = [600, 70]
    n_pages = 2 * w.pages_per_seq + 9
    case = Case(w, lens=lens, layers=[0, 1], n_pages=n_pages, rope=THETA)
    clean = {l: case.run(l) for l in (0, 1)}
    used = torch.zeros((n_pages, w.page_tokens), dtype=torch.bool)
    for b, L in enumerate(lens):
        for t in range(L):
            used[int(case.table[b, t // w.page_tokens]), t % w.page_tokens] = True
    junk = torch.tensor([float("nan"), float("inf"), -3.0e38, 1.0e30], dtype=torch.float32)
    for l in (0, 1):
        for pool in (case.ctx.k_pools[l], case.ctx.v_pools[l]):
            fill = junk[torch.arange(pool.shape[-1]) % 4].to(pool.dtype).to(pool.device)
            pool[(~used).to(pool.device)] = fill
    for l in (0, 1):
        np.testing.assert_array_equal(case.run(l), clean[l])
    assert case.ctx.device_status() == binding.ECHOKV_OK
    # a length of zero and a page id outside the pool: reported, the other sequence untouched, nothing faults
    dev = case.ctx.device
    q = case.q[0].to(dev)
    out = case.ctx.decode_attention(0, q, torch.tensor([600, 0], dtype=torch.int32, device=dev)).cpu().numpy()
    assert case.ctx.device_status() == binding.ECHOKV_EBADLENGTH
    np.testing.assert_array_equal(out[0], clean[0][0])
    assert np.all(out[1] == 0.0)
    saved = case.ctx.block_table.clone()
    case.ctx.block_table[1, 1] = 10 ** 6
    out = case.ctx.decode_attention(0, q, case.seq_lens).cpu().numpy()
    assert case.ctx.device_status() == binding.ECHOKV_EBADPAGE
    np.testing.assert_array_equal(out[0], clean[0][0])
    assert np.all(np.isfinite(out))
    case.ctx.block_table.copy_(saved)
    np.testing.assert_array_equal(case.run(0), clean[0])
    assert case.ctx.device_status() == binding.ECHOKV_OK
    case.close()
