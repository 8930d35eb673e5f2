"""GPU parity of the absorbed-predictor decode mode: the same oracle (Eq. 3, 6, 7 evaluated as the
paper writes them, fp64) must be matched when the library folds the predictors into the queries
and the output instead of reconstructing K and V."""
import ctypes as C

import numpy as np
import pytest
import torch

from paper_2603_22910_b200 import binding, build, synth
from tests.harness import Case, assert_parity, errors

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    binding.lib()


SHAPES = [
    # name, base, overrides, lens
    ("c1_shape", synth.C1, dict(batch=2, context=700), [700, 333]),
    ("c2_shape", synth.C2, dict(batch=3, context=1000), [1000, 517, 256]),
    ("c2_ranges_ragged", synth.C2, dict(batch=4, context=2500, random_pages=True), [2500, 1025, 64, 1]),
    ("c4_25pct", synth.c4_point(25, 4096, 1), dict(batch=2, context=530), [530, 17]),
    ("c4_50pct_pages32", synth.c4_point(50, 4096, 1), dict(batch=2, context=300, page_tokens=32, random_pages=True),
     [300, 299]),
    ("odd_retained_pages64", synth.C2, dict(n_retained_heads=3, batch=2, context=600, page_tokens=64,
                                            random_pages=True), [600, 65]),
    ("nothing_retained_pages128", synth.C2, dict(n_retained_heads=0, batch=2, context=700, page_tokens=128,
                                                 random_pages=True), [700, 129]),
    ("one_dropped_head", synth.C2, dict(n_retained_heads=7, batch=2, context=300), [300, 258]),
    ("gqa8_64_query_heads", synth.C2, dict(n_q_heads=64, n_kv_heads=8, n_retained_heads=4, batch=2, context=400),
     [400, 130]),
    ("gqa2_16_query_heads", synth.C2, dict(n_q_heads=16, n_kv_heads=8, n_retained_heads=2, batch=2, context=400),
     [400, 63]),
    ("mha_16_heads", synth.C1, dict(n_q_heads=16, n_kv_heads=16, n_retained_heads=5, batch=2, context=300),
     [300, 200]),
]


@pytest.mark.parametrize("name,base,over,lens", SHAPES, ids=[s[0] for s in SHAPES])
def test_absorbed_mode_against_oracle(name, base, over, lens):
    w = base.replace(**over)
    case = Case(w, lens=lens, layers=[0, 1])
    explicit = case.run(1)
    case.ctx.enable_absorbed()
    assert case.ctx.decode_mode() == 1
    out = case.run(1)
    ref = case.oracle(1)
    assert_parity(out, ref, w.dtype, name + " absorbed")
    # and the two evaluation orders agree with one another far inside the tolerance
    assert errors(out, explicit)[1] < 1e-3
    # the anchor layer is served as before
    assert_parity(case.run(0), case.oracle(0), w.dtype, name + " anchor")
    case.ctx.set_decode_mode(0)
    np.testing.assert_array_equal(case.run(1), explicit)
    assert case.ctx.device_status() == binding.ECHOKV_OK
    case.close()


RAGGED = [
    # the paper's own settings for 8 KV heads x 128 (Appendix "Compression-Ratio Configurations"): m need not end
    # on a head boundary.  name, overrides, lens
    ("paper_S4_m64", dict(n_retained_dims=64, n_retained_heads=0, batch=2, context=700, group_size=4, n_layers=4),
     [700, 129]),
    ("paper_S2_m384", dict(n_retained_dims=384, n_retained_heads=3, batch=2, context=400, random_pages=True), [400, 65]),
    ("m320_pages64", dict(n_retained_dims=320, n_retained_heads=2, batch=2, context=500, page_tokens=64), [500, 64]),
    ("m960_one_half_head_dropped", dict(n_retained_dims=960, n_retained_heads=7, batch=2, context=300), [300, 7]),
]


@pytest.mark.parametrize("name,over,lens", RAGGED, ids=[r[0] for r in RAGGED])
def test_retained_dims_that_split_a_head(name, over, lens):
    w = synth.C2.replace(**over)
    layers = [l for l in range(w.n_layers) if not w.is_anchor(l)][:2]
    case = Case(w, lens=lens, layers=layers)
    # the explicit kernels work on whole heads: a head that m splits is predicted whole, its stored dims passed
    # through by one-hot rows in front of the predictors (exactly)
    assert case.ctx.decode_path() in (2, 3)
    for l in layers:
        assert_parity(case.run(l), case.oracle(l), w.dtype, "%s explicit, layer %d" % (name, l))
    case.ctx.enable_absorbed()
    for l in layers:
        assert_parity(case.run(l), case.oracle(l), w.dtype, "%s layer %d" % (name, l))
    assert case.ctx.device_status() == binding.ECHOKV_OK
    case.close()


def test_absorbed_multi_layer_random_pages():
    w = synth.C3.replace(n_layers=8, batch=2, context=420)
    case = Case(w, lens=[420, 131], n_pages=2 * w.pages_per_seq + 13)
    case.ctx.enable_absorbed()
    for l in case.layers:
        assert_parity(case.run(l), case.oracle(l), w.dtype, "layer %d" % l)
    assert case.ctx.device_status() == binding.ECHOKV_OK
    case.close()


def test_absorbed_predictor_bias():
    w = synth.C2.replace(batch=2, context=200)
    case = Case(w, lens=[200, 31], layers=[1], biases=True)
    case.ctx.enable_absorbed()
    assert_parity(case.run(1), case.oracle(1), w.dtype, "bias")
    case.close()


def test_absorbed_slots_that_hold_no_token_may_contain_anything():
    w = synth.C2.replace(batch=2, context=600, n_retained_heads=2, random_pages=True)
    lens = [600, 70]
    n_pages = 2 * w.pages_per_seq + 9
    case = Case(w, lens=lens, layers=[1], n_pages=n_pages)
    case.ctx.enable_absorbed()
    clean = case.run(1)
    used = torch.zeros((n_pages, w.page_tokens), dtype=torch.bool)
    for b, L in enumerate(lens):
        for t in range(L):
            used[int(case.table[b, t // w.page_tokens]), t % w.page_tokens] = True
    junk = torch.tensor([float("nan"), float("inf"), -3.0e38, 1.0e30], dtype=torch.float32)
    for l in (0, 1):
        for pool in (case.ctx.k_pools[l], case.ctx.v_pools[l]):
            fill = junk[torch.arange(pool.shape[-1]) % 4].to(pool.dtype).to(pool.device)
            pool[(~used).to(pool.device)] = fill
    np.testing.assert_array_equal(case.run(1), clean)
    assert_parity(case.run(1), case.oracle(1), w.dtype, "junk in unused slots")
    case.close()


def test_absorbed_bad_length_is_reported_and_zeroed():
    w = synth.C2.replace(batch=2, context=100)
    case = Case(w, lens=[100, 60], layers=[1])
    case.ctx.enable_absorbed()
    good = case.run(1)
    dev = case.ctx.device
    bad = torch.tensor([100, 0], dtype=torch.int32, device=dev)
    out = case.ctx.decode_attention(1, case.q[1].to(dev), bad)
    assert case.ctx.device_status() == binding.ECHOKV_EBADLENGTH
    out = out.cpu().numpy()
    np.testing.assert_array_equal(out[0], good[0])
    assert np.all(out[1] == 0.0)
    case.close()


def test_absorbed_mode_status_codes():
    L = binding.lib()
    # fp32 / head_dim 64: the mode is not offered
    n = C.c_uint64(0)
    cfg0 = binding.config_for(synth.C0)
    assert L.echokv_absorbed_workspace_bytes(C.byref(cfg0), C.byref(n)) == binding.ECHOKV_EUNSUPPORTED
    w = synth.C2.replace(batch=2, context=64)
    case = Case(w, lens=[64, 64], layers=[1])
    ctx = case.ctx
    assert L.echokv_set_decode_mode(ctx.handle, 1) == binding.ECHOKV_EUNSUPPORTED     # before the workspace exists
    assert L.echokv_set_decode_mode(ctx.handle, 2) == binding.ECHOKV_EINVAL
    assert L.echokv_absorbed_workspace_bytes(C.byref(case.cfg), C.byref(n)) == binding.ECHOKV_OK and n.value > 0
    buf = torch.empty(n.value, dtype=torch.uint8, device=ctx.device)
    assert L.echokv_enable_absorbed(ctx.handle, buf.data_ptr(), n.value - 1) == binding.ECHOKV_ECAPACITY
    assert L.echokv_enable_absorbed(ctx.handle, None, n.value) == binding.ECHOKV_EINVAL
    assert L.echokv_enable_absorbed(ctx.handle, buf.data_ptr(), n.value) == binding.ECHOKV_OK
    assert L.echokv_decode_mode(ctx.handle) == 1
    case.close()
