"""Parity at the benchmark's full sizes, in the launch configuration bench.py times: the workloads
are too large for the oracle to evaluate whole, so a seeded sample of (layer, sequence, query head)
outputs is recomputed one by one (heads are independent in Eq. 7, and a predicted head needs only
its own rows of W in Eq. 3).  Inputs are drawn on the device by the seeded generators and read back
from the pools for the oracle."""
import numpy as np
import pytest
import torch

import bench
from oracle import echokv_oracle as O
from paper_2603_22910_b200 import binding, build, synth
from tests.harness import TOL

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    binding.lib()


def sampled_check(w, mode, samples, absorbed, seed=7):
    """`samples` outputs, stratified (bench.stratified_picks): every sequence of the batch, the first, a middle
    and the last compressed layer and the first and last anchor layer, and every KV head -- so every pair of
    dropped heads a fused-kernel work item handles, and with whole sequences the first and the last (partial)
    token tile of each -- instead of a handful drawn at random."""
    resident, step_layers = bench.plan_layers(w, mode)
    st = bench.State(w, 0, resident)
    ctx = st.ctx
    if absorbed:
        ctx.enable_absorbed()
    for l, attend in step_layers:          # exactly bench.py's step
        ctx.append_kv(l, st.new_dev[(l, "k")], st.new_dev[(l, "v")], st.positions)
        if attend:
            if mode == "full" or w.is_anchor(l):
                ctx.full_attention(l, st.q_dev[l], st.lens, out=st.out[l])
            else:
                ctx.decode_attention(l, st.q_dev[l], st.lens, out=st.out[l])
    torch.cuda.synchronize()
    assert ctx.device_status() == binding.ECHOKV_OK
    attend_layers = [l for l, a in step_layers if a]
    picks = bench.stratified_picks(w, attend_layers, samples, seed=seed)
    assert {b for _, b, _ in picks} == set(range(min(w.batch, len(picks))))
    res = bench.parity_sample(st, picks)
    tol = TOL[w.dtype]
    ctx.close()
    del st
    torch.cuda.empty_cache()
    assert res["outputs"] >= min(samples, w.batch * w.n_q_heads) * 0.9, res
    assert res["max_abs"] <= tol["max_abs"] and res["rel_l2"] <= tol["rel_l2"], res
    return res["max_abs"], res["rel_l2"]


@pytest.mark.parametrize("absorbed", [False, True], ids=["explicit", "absorbed"])
def test_config1_full_size_sampled(absorbed):
    sampled_check(synth.C1, "compressed", samples=64, absorbed=absorbed)


@pytest.mark.parametrize("absorbed", [False, True], ids=["explicit", "absorbed"])
def test_config2_full_size_sampled(absorbed):
    sampled_check(synth.C2, "compressed", samples=64, absorbed=absorbed)


@pytest.mark.parametrize("absorbed", [False, True], ids=["explicit", "absorbed"])
def test_config3_full_size_32_layers_sampled(absorbed):
    sampled_check(synth.C3, "compressed", samples=64, absorbed=absorbed)


def test_config4_sweep_points_sampled():
    # one point per compression ratio, at the long-context end that still keeps the run short
    for ratio, context, batch in ((25, 65536, 4), (50, 131072, 2), (75, 16384, 32)):
        sampled_check(synth.c4_point(ratio, context, batch), "compressed", samples=16, absorbed=False)
    sampled_check(synth.c4_point(75, 131072, 2), "compressed", samples=16, absorbed=True)


def test_uncompressed_path_full_size_sampled():
    sampled_check(synth.C1, "full", samples=32, absorbed=False)
    sampled_check(synth.C2, "full", samples=32, absorbed=False)


def test_prefill_call_config2_full_size_sampled():
    """The prefill-shaped call at the C2 shape with 512 causal queries per sequence (the configuration
    `bench.py --prefill-queries 512` times): query i of the chunk attends the cached prefix up to its own
    position, which is the decode step of a sequence cut off there, so sampled (sequence, query, head)
    outputs are recomputed with the single-head decode oracle on the truncated cache."""
    w, n_q, layer = synth.C2, 512, 1
    st = bench.State(w, 0, [0, 1])
    ctx = st.ctx
    q = synth.normal((w.batch, n_q, w.n_q_heads, w.head_dim), w.seed, 77, 1, device=st.dev).to(torch.bfloat16)
    out = ctx.prefill_attention(layer, q, st.lens)
    torch.cuda.synchronize()
    assert ctx.device_status() == binding.ECHOKV_OK
    rng = np.random.default_rng(11)
    picks = [(0, 0, 0), (w.batch - 1, n_q - 1, w.n_q_heads - 1)]           # first and last query of the chunk
    picks += [(int(rng.integers(w.batch)), int(rng.integers(n_q)), int(rng.integers(w.n_q_heads))) for _ in range(4)]
    worst = num = den = 0.0
    for b, i, h in picks:
        _, kg, vg, kl, vl, Wk, Wv = st.oracle_inputs(layer, b)
        n_seen = w.context - n_q + i + 1
        qi = O.widen(synth.to_numpy_stored(q[b, i].cpu()))
        ref = O.decode_attention_query_heads(qi, kg[:n_seen], vg[:n_seen], kl[:n_seen], vl[:n_seen], Wk, Wv,
                                             n_kv_heads=w.n_kv_heads, query_heads=[h])[h]
        got = out[b, i, h].cpu().numpy().astype(np.float64)
        assert np.all(np.isfinite(got))
        worst = max(worst, float(np.max(np.abs(got - ref))))
        num += float(np.sum((got - ref) ** 2))
        den += float(np.sum(ref ** 2))
    rel = (num / max(den, 1e-300)) ** 0.5
    ctx.close()
    del st
    torch.cuda.empty_cache()
    # (the tolerance of the decode calls)
    assert worst <= 2e-2 and rel <= 5e-3, (worst, rel)
