"""GPU parity of the "save K" setting (Section 5.2 of the paper: keys kept whole, reconstruction applied to the
values only): compressed layers hold K pools of full width and V pools of m dims; served by the absorbed mode."""
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
    # name, base, overrides, lens, biases
    ("c2_shape", synth.C2, dict(batch=3, context=1000), [1000, 517, 256], False),
    ("c1_shape", synth.C1, dict(batch=2, context=700), [700, 333], True),
    ("pages64_random", synth.C2, dict(batch=2, context=600, page_tokens=64, random_pages=True), [600, 65], False),
    ("ragged_many_tiles", synth.C2, dict(batch=5, context=2000, random_pages=True), [2000, 129, 128, 1153, 1], True),
    ("nothing_of_v_retained", synth.C2, dict(batch=2, context=700, n_retained_heads=0), [700, 300], False),
    ("m_64", synth.C2, dict(batch=2, context=500, n_retained_dims=64), [500, 130], False),
    ("gqa2", synth.C2, dict(n_q_heads=16, batch=2, context=400, n_retained_heads=3), [400, 77], False),
]


@pytest.mark.parametrize("name,base,over,lens,biases", CASES, ids=[c[0] for c in CASES])
@pytest.mark.parametrize("rope", [None, THETA], ids=["plain", "rotated"])
def test_save_k_against_oracle(name, base, over, lens, biases, rope):
    w = base.replace(save_k=True, **over)
    case = Case(w, lens=lens, layers=[0, 1], biases=biases, rope=rope)
    ctx = case.ctx
    # the K pool of the compressed layer has the anchor's width, the V pool m dims
    assert ctx.k_pools[1].shape[-1] == w.D and (ctx.v_pools[1] is None or ctx.v_pools[1].shape[-1] == w.m)
    assert ctx.decode_path() == 0
    q = case.q[1].to(ctx.device)
    with pytest.raises(binding.EchoKVError) as e:        # the explicit kernels predict K as well
        ctx.decode_attention(1, q, case.seq_lens)
    assert e.value.status == binding.ECHOKV_EUNSUPPORTED
    ctx.enable_absorbed()
    ref = case.oracle(1)
    assert_parity(case.run(1), ref, w.dtype, name)
    assert_parity(case.run(0), case.oracle(0), w.dtype, name + " anchor")
    # the result differs from the method with predicted keys (same stored values otherwise)
    w2 = base.replace(**over)
    if w2.m % w2.head_dim == 0 or rope is None:
        other = Case(w2, lens=lens, layers=[1], biases=biases, rope=rope)
        other.ctx.enable_absorbed()
        assert errors(other.run(1), ref)[1] > 1e-2
        other.close()
    assert ctx.device_status() == binding.ECHOKV_OK
    case.close()


WINDOW_CASES = [
    ("c2_shape", synth.C2, dict(batch=3, context=900, random_pages=True), [900, 517, 100], (4, 128), True),
    ("m_384_short_window", synth.C2, dict(batch=2, context=500, n_retained_dims=384, n_retained_heads=3), [500, 20],
     (2, 33), False),
    ("nothing_of_v_retained", synth.C2, dict(batch=2, context=400, n_retained_heads=0), [400, 131], (4, 128), False),
]


@pytest.mark.parametrize("name,base,over,lens,window,biases", WINDOW_CASES, ids=[c[0] for c in WINDOW_CASES])
@pytest.mark.parametrize("rope", [None, THETA], ids=["plain", "rotated"])
def test_save_k_with_sink_and_window(name, base, over, lens, window, biases, rope):
    """Whole keys with sink / window tokens (Section 5.2 with Section 4.1): the keys are all stored, so the window
    matters to the values only; decode and the prefill-shaped call."""
    w = base.replace(save_k=True, **over)
    case = Case(w, lens=lens, layers=[0, 1], biases=biases, window=window, rope=rope)
    ctx = case.ctx
    ctx.enable_absorbed()
    assert_parity(case.run(1), case.oracle(1), w.dtype, name)
    assert_parity(case.run(0), case.oracle(0), w.dtype, name + " anchor")
    assert ctx.device_status() == binding.ECHOKV_OK
    case.close()


def test_save_k_limits():
    w = synth.C2.replace(batch=1, context=300, save_k=True)
    cfg = binding.config_for(w)
    sizes = binding.echokv_query_sizes(cfg)
    assert sizes.compressed_pool_bytes == cfg.n_pages * w.page_tokens * w.m * 2       # the V pool
    assert sizes.anchor_pool_bytes == cfg.n_pages * w.page_tokens * w.D * 2           # the K pool in this setting
    ctx = binding.Context(cfg)
    # Wv is still required, Wk is not
    lib = binding.lib()
    wv = torch.zeros((w.d_drop, w.d_in), dtype=torch.bfloat16, device=ctx.device)
    assert lib.echokv_set_weights(ctx.handle, 1, None, None, None, None) == binding.ECHOKV_EINVAL
    assert lib.echokv_set_weights(ctx.handle, 1, None, wv.data_ptr(), None, None) == binding.ECHOKV_OK
    ctx.close()
    # a shape the absorbed mode does not take cannot be created in this setting
    small = synth.C0.replace(save_k=True)
    with pytest.raises(binding.EchoKVError) as e:
        binding.Context(binding.config_for(small))
    assert e.value.status == binding.ECHOKV_EUNSUPPORTED
