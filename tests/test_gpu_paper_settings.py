"""The paper's own operating points, end to end against the oracle.

Appendix "Compression-Ratio Configurations" / Table "Hyperparameter configurations": on the GQA backbones
(8 KV heads of 128 dims, D = 1024) the three settings are (S = 2, m = 384), (S = 2, m = 0) and (S = 4, m = 64);
m = 64 and m = 384 split a head.  Section 3.2 feeds the predictors keys cached before the rotary embedding, and
Section 4.1 keeps 4 sink tokens and a window of 128 recent tokens at full precision.  Every combination of
{m} x {rotation} x {sink / window} x {bias} runs through the explicit decode path, the absorbed decode path and the
prefill-shaped call, at the decode tolerance."""
import itertools

import numpy as np
import pytest
import torch

from oracle import echokv_oracle as O
from paper_2603_22910_b200 import binding, build, synth
from tests.harness import TOL, Case, errors

pytestmark = pytest.mark.gpu

THETA = 10000.0
SETTINGS = {0: dict(group_size=2, n_retained_heads=0, n_retained_dims=0),
            64: dict(group_size=4, n_retained_heads=0, n_retained_dims=64),
            384: dict(group_size=2, n_retained_heads=3, n_retained_dims=384)}
GRID = list(itertools.product([0, 64, 384], [None, THETA], [None, (4, 128)], [False, True]))
IDS = ["m%d-%s-%s-%s" % (m, "rope" if r else "norope", "window" if win else "nowindow", "bias" if b else "nobias")
       for m, r, win, b in GRID]


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    binding.lib()


def workload(m):
    # the paper's backbone shape (32 query heads, 8 KV heads of 128 dims), three sequences of ragged lengths on
    # 16-token pages in a random order; layer 1 is compressed, layer 0 its anchor
    return synth.C2.replace(batch=3, context=700, random_pages=True, name="paper_m%d" % m, **SETTINGS[m])


def check(out, ref, what):
    max_abs, rel_l2 = errors(out, ref)
    tol = TOL["bf16"]
    assert np.all(np.isfinite(out)), "non-finite output " + what
    assert max_abs <= tol["max_abs"] and rel_l2 <= tol["rel_l2"], "%s: max_abs %.3e rel_l2 %.3e" % (what, max_abs, rel_l2)


@pytest.mark.parametrize("m,rope,window,biases", GRID, ids=IDS)
@pytest.mark.parametrize("mode", ["explicit", "absorbed"])
def test_decode_at_the_papers_settings(m, rope, window, biases, mode):
    w = workload(m)
    case = Case(w, lens=[700, 333, 130], layers=[0, 1], biases=biases, window=window, rope=rope)
    ctx = case.ctx
    if mode == "absorbed":
        ctx.enable_absorbed()
    else:
        assert ctx.decode_path() in (2, 3), "the tensor-core kernels serve a retained width that splits a head"
    for layer in (1, 0):
        check(case.run(layer), case.oracle(layer), "%s m=%d layer %d" % (mode, m, layer))
    assert ctx.device_status() == binding.ECHOKV_OK
    case.close()


def oracle_prefill(case, layer, q, b):
    w = case.w
    qn = O.widen(synth.to_numpy_stored(q))[b]
    a = w.anchor_of(layer)
    kg, vg = case._stored(a, "k", b), case._stored(a, "v", b)
    if w.is_anchor(layer):
        return O.prefill_attention(qn, kg, vg, None, None, None, None, w.n_kv_heads, rope_theta=case.rope)
    L = kg.shape[0]
    kl = case._stored(layer, "k", b) if w.m else np.zeros((L, 0))
    vl = case._stored(layer, "v", b) if w.m else np.zeros((L, 0))
    Wk, Wv, bk, bv = (None if t is None else O.widen(synth.to_numpy_stored(t)) for t in case.host_w[layer])
    kw = {}
    if case.window:
        kw = dict(k_true_drop=O.widen(synth.to_numpy_stored(case.true_drop[(layer, "k", b)])),
                  v_true_drop=O.widen(synth.to_numpy_stored(case.true_drop[(layer, "v", b)])),
                  n_sink=case.window[0], n_window=case.window[1])
    if w.save_k:                 # keys kept whole (Section 5.2): the stored K rows are the whole keys
        kw["k_true"] = case._stored(layer, "k", b)
        kl = kw["k_true"][:, :w.m]
    return O.prefill_attention(qn, kg, vg, kl, vl, Wk, Wv, w.n_kv_heads, bk=bk, bv=bv, rope_theta=case.rope, **kw)


@pytest.mark.parametrize("m,rope,window,biases", GRID, ids=IDS)
def test_prefill_at_the_papers_settings(m, rope, window, biases):
    w = workload(m)
    lens = [700, 333, 170]
    case = Case(w, lens=lens, layers=[0, 1], biases=biases, window=window, rope=rope)
    ctx, dev = case.ctx, case.ctx.device
    n_q = 150                     # more queries than the window is long: tokens of the chunk fall out of later windows
    q = synth.normal((w.batch, n_q, w.n_q_heads, w.head_dim), w.seed, 77, 5).to(synth.torch_dtype(w))
    recent = case.recent_rows(1, n_q) if window else (None, None)
    out = ctx.prefill_attention(1, q.to(dev), case.seq_lens, k_recent=recent[0], v_recent=recent[1])
    torch.cuda.synchronize()
    out = out.cpu().numpy().astype(np.float64)
    for b in range(w.batch):
        check(out[b], oracle_prefill(case, 1, q, b), "prefill m=%d seq %d" % (m, b))
    assert ctx.device_status() == binding.ECHOKV_OK
    case.close()


@pytest.mark.parametrize("rope", [None, THETA], ids=["norope", "rope"])
def test_prefill_with_whole_keys_and_a_window(rope):
    """Section 5.2 ("save K") with Section 4.1: the keys are stored whole, the window matters to the values only."""
    w = workload(384).replace(save_k=True, name="paper_m384_saveK")
    lens = [700, 333, 170]
    case = Case(w, lens=lens, layers=[0, 1], biases=True, window=(4, 128), rope=rope)
    ctx, dev = case.ctx, case.ctx.device
    n_q = 140
    q = synth.normal((w.batch, n_q, w.n_q_heads, w.head_dim), w.seed, 77, 6).to(synth.torch_dtype(w))
    recent = case.recent_rows(1, n_q)
    out = ctx.prefill_attention(1, q.to(dev), case.seq_lens, k_recent=recent[0], v_recent=recent[1])
    torch.cuda.synchronize()
    out = out.cpu().numpy().astype(np.float64)
    for b in range(w.batch):
        check(out[b], oracle_prefill(case, 1, q, b), "prefill, whole keys, seq %d" % b)
    assert ctx.device_status() == binding.ECHOKV_OK
    case.close()


BAND = [
    # name, overrides of the backbone shape, window, queries: the sink / window pass of the prefill-shaped call
    ("gqa4_no_sink_short_window", dict(), (0, 5), 37),
    ("gqa4_sink_only", dict(), (6, 0), 9),
    ("mha_window_longer_than_the_chunk", dict(n_q_heads=8, n_kv_heads=8, n_retained_heads=3, n_retained_dims=384), (2, 70), 33),
    ("gqa2", dict(n_q_heads=16, n_kv_heads=8, n_retained_heads=3, n_retained_dims=384), (4, 128), 130),
    ("gqa8", dict(n_q_heads=32, n_kv_heads=4, group_size=2, n_retained_heads=1, n_retained_dims=128), (4, 128), 131),
    ("gqa4_very_long_window", dict(), (3, 1500), 70),        # (too long for four queries per block)
]


@pytest.mark.parametrize("name,over,window,n_q", BAND, ids=[c[0] for c in BAND])
@pytest.mark.parametrize("rope", [None, THETA], ids=["norope", "rope"])
def test_prefill_window_shapes(name, over, window, n_q, rope):
    """Windows shorter and longer than the chunk of queries, sink only, window only, every group size."""
    L = max(1700, n_q + 10)
    w = synth.C2.replace(batch=2, context=L, random_pages=True, name="band_" + name,
                         **{**SETTINGS[384], **over})
    lens = [L, max(n_q, L // 2 + 3)]
    case = Case(w, lens=lens, layers=[0, 1], biases=True, window=window, rope=rope)
    ctx, dev = case.ctx, case.ctx.device
    q = synth.normal((w.batch, n_q, w.n_q_heads, w.head_dim), w.seed, 77, 8).to(synth.torch_dtype(w))
    recent = case.recent_rows(1, n_q)
    out = ctx.prefill_attention(1, q.to(dev), case.seq_lens, k_recent=recent[0], v_recent=recent[1])
    torch.cuda.synchronize()
    out = out.cpu().numpy().astype(np.float64)
    for b in range(w.batch):
        check(out[b], oracle_prefill(case, 1, q, b), "prefill %s seq %d" % (name, b))
    assert ctx.device_status() == binding.ECHOKV_OK
    case.close()
