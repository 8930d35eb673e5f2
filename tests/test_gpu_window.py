"""GPU parity with sink and recent-window tokens kept at full precision (Section 4.1 of the paper:
4 sink tokens and a local window of 128 tokens): those tokens' dropped dims come from the side buffers,
every other token is predicted."""
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


CASES = [
    # name, base, overrides, lens, (n_sink, n_window)
    ("paper_setting_gqa", synth.C2, dict(batch=3, context=1000, random_pages=True), [1000, 517, 256], (4, 128)),
    ("paper_setting_mha", synth.C1, dict(batch=2, context=700), [700, 333], (4, 128)),
    ("shorter_than_the_window", synth.C2, dict(batch=3, context=140), [140, 100, 3], (4, 128)),
    ("window_only", synth.C2, dict(batch=2, context=400, n_retained_heads=4), [400, 129], (0, 64)),
    ("sink_only", synth.C2, dict(batch=2, context=300), [300, 2], (8, 0)),
    ("odd_sizes", synth.C2, dict(batch=2, context=600, n_retained_heads=7, page_tokens=64), [600, 259], (3, 37)),
    ("fp32_d64", synth.C0, dict(batch=2, context=200), [200, 50], (2, 16)),
]


# biases: Eq. 3 with the optional bias vectors.  With sink / window tokens a K bias no longer cancels in the softmax
# (it shifts the scores of the predicted tokens only) and a V bias reaches the output only with the predicted
# tokens' share of the probability.
@pytest.mark.parametrize("biases", [False, True], ids=["no_bias", "biases"])
@pytest.mark.parametrize("name,base,over,lens,window", CASES, ids=[c[0] for c in CASES])
def test_window_against_oracle(name, base, over, lens, window, biases):
    w = base.replace(**over)
    case = Case(w, lens=lens, layers=[0, 1], window=window, biases=biases)
    paths = ([1, 2, 3] + (([4, 5] if w.page_tokens <= 32 else [4]) if w.n_q_heads // w.n_kv_heads <= 2 else [])) if case.ctx.decode_path() >= 2 else [1]
    for path in paths:
        case.ctx.set_decode_path(path)
        assert_parity(case.run(1), case.oracle(1), w.dtype, "%s path %d" % (name, path))
    # the anchor layer is served as before
    assert_parity(case.run(0), case.oracle(0), w.dtype, name + " anchor")
    # and the absorbed-predictor mode gives the same, where the shape has it
    n = C.c_uint64(0)
    if binding.lib().echokv_absorbed_workspace_bytes(C.byref(case.cfg), C.byref(n)) == binding.ECHOKV_OK:
        case.ctx.enable_absorbed()
        assert_parity(case.run(1), case.oracle(1), w.dtype, name + " absorbed")
    assert case.ctx.device_status() == binding.ECHOKV_OK
    case.close()


def test_window_changes_the_result_and_everything_in_the_window_is_exact():
    # random predictors are poor: the output must move towards the true-cache result when the
    # window grows, and equal it once every token is inside sink + window
    w = synth.C2.replace(batch=1, context=130)
    plain = Case(w, lens=[130], layers=[1])
    base = plain.run(1)
    plain.close()
    case = Case(w, lens=[130], layers=[1], window=(4, 128))
    out = case.run(1)
    assert errors(out, base)[0] > 1e-3
    # all 130 tokens are inside 4 + 128 only if the window also covers tokens 2..3: it does (t >= 2)
    from oracle import echokv_oracle as O
    st = synth.to_numpy_stored
    k = np.concatenate([O.widen(st(case.host[(1, "k", 0)])), O.widen(st(case.true_drop[(1, "k", 0)]))], axis=1)
    v = np.concatenate([O.widen(st(case.host[(1, "v", 0)])), O.widen(st(case.true_drop[(1, "v", 0)]))], axis=1)
    ref = O.full_attention(O.widen(st(case.q[1]))[0], k, v, w.n_kv_heads)
    assert_parity(out[0], ref, w.dtype, "every token at full precision")
    case.close()


def test_appended_tokens_enter_sink_and_ring():
    # drive the cache only through the library's append: 7 tokens with sink 2 / window 3
    w = synth.C2.replace(batch=1, context=16)
    case = Case(w, lens=[1], layers=[1], window=(2, 3))
    dev = case.ctx.device
    full_k = synth.layer_cache(w, 1, "k", 0, width=w.D)
    full_v = synth.layer_cache(w, 1, "v", 0, width=w.D)
    for pos in range(1, 7):
        for l in (0, 1):
            fk = synth.layer_cache(w, l, "k", 0, width=w.D)[pos:pos + 1].to(dev)
            fv = synth.layer_cache(w, l, "v", 0, width=w.D)[pos:pos + 1].to(dev)
            case.ctx.append_kv(l, fk, fv, torch.tensor([pos], dtype=torch.int32, device=dev))
    torch.cuda.synchronize()
    side = case.ctx.k_side[1][0].cpu()
    for t in (0, 1):                                   # the sink
        assert torch.equal(side[t], full_k[t, w.m:])
    for t in (4, 5, 6):                                # the last three tokens, at ring slot 2 + t % 3
        assert torch.equal(side[2 + t % 3], full_k[t, w.m:])
    assert torch.equal(case.ctx.v_side[1][0].cpu()[2 + 6 % 3], full_v[6, w.m:])
    case.close()


def test_window_status_codes():
    L = binding.lib()
    w = synth.C2.replace(batch=2, context=64)
    case = Case(w, lens=[64, 64], layers=[1])
    n = C.c_uint64(0)
    assert L.echokv_side_buffer_bytes(C.byref(case.cfg), 4, 128, C.byref(n)) == binding.ECHOKV_OK
    assert n.value == 2 * 132 * w.d_drop * 2
    assert L.echokv_side_buffer_bytes(C.byref(case.cfg), 4, 5000, C.byref(n)) == binding.ECHOKV_EUNSUPPORTED
    assert L.echokv_side_buffer_bytes(C.byref(case.cfg), -1, 0, C.byref(n)) == binding.ECHOKV_EINVAL
    assert L.echokv_set_full_precision_window(case.ctx.handle, 4, 128, None, None) == binding.ECHOKV_EINVAL
    assert L.echokv_set_full_precision_window(case.ctx.handle, 0, 0, None, None) == binding.ECHOKV_OK
    case.close()
