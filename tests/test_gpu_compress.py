"""The switch from full-cache generation to compressed inference (Section 3.1, Section 5.4 of the paper): a
layer cached at full width is evicted down to its retained dims by the library; the copies must be bit-exact
and the layer must then decode exactly as if it had been cached compressed all along."""
import numpy as np
import pytest
import torch

from oracle import echokv_oracle as O
from paper_2603_22910_b200 import binding, build, synth
from tests.harness import Case, assert_parity

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    binding.lib()


CASES = [
    # name, base, overrides, lens, window, chunk boundaries of a prefill done in pieces
    ("gqa_window", synth.C2, dict(batch=3, context=1000, random_pages=True), [1000, 517, 100], (4, 128), [0, 300, 301]),
    ("mha_no_window", synth.C1, dict(batch=2, context=700), [700, 333], None, [0, 64]),
    ("fp32_d64_window", synth.C0, dict(batch=2, context=200), [200, 50], (2, 16), [0, 17]),
    ("nothing_retained", synth.C2, dict(batch=2, context=300, n_retained_heads=0), [300, 140], (4, 128), [0, 200]),
    ("pages128", synth.C2, dict(batch=2, context=700, page_tokens=128, random_pages=True), [700, 129], (3, 37), [0, 128]),
    ("split_head_window", synth.C2, dict(batch=2, context=500, n_retained_dims=64, n_retained_heads=0, group_size=4,
                                         n_layers=4), [500, 131], (4, 128), [0, 250]),
    ("keys_whole_window", synth.C2, dict(batch=2, context=600, save_k=True, random_pages=True), [600, 140], (4, 128),
     [0, 333]),
    ("keys_whole", synth.C2, dict(batch=2, context=300, save_k=True, n_retained_dims=384, n_retained_heads=3), [300, 17],
     None, [0, 100]),
]


@pytest.mark.parametrize("name,base,over,lens,window,chunks", CASES, ids=[c[0] for c in CASES])
def test_evicted_layer_equals_a_layer_cached_compressed(name, base, over, lens, window, chunks):
    w = base.replace(**over)
    case = Case(w, lens=lens, layers=[0, 1], window=window)
    ctx, dev = case.ctx, case.ctx.device
    if w.save_k:
        ctx.enable_absorbed()           # (keys kept whole: decode calls are served by the absorbed mode)
    want_out = case.run(1)
    assert_parity(want_out, case.oracle(1), w.dtype, name + " before")
    n_pages = case.cfg.n_pages
    # the layer's full-width cache, as a backbone generating with the full cache would hold it
    full = {kind: [synth.layer_cache(w, 1, kind, b, width=w.D)[: lens[b]] for b in range(w.batch)] for kind in "kv"}
    pools = {kind: synth.paged_pool(w, full[kind], case.table, n_pages, w.D).to(dev) for kind in "kv"}
    keep = {}
    for kind, mine in (("k", ctx.k_pools), ("v", ctx.v_pools)):
        if mine[1] is not None:
            keep[kind] = mine[1].clone()
            mine[1].zero_()
    side_keep = None
    if window and w.D > w.m:
        side_keep = (ctx.k_side[1].clone(), ctx.v_side[1].clone())
        ctx.k_side[1].zero_()
        ctx.v_side[1].zero_()

    def check():
        for kind, mine in (("k", ctx.k_pools), ("v", ctx.v_pools)):
            if mine[1] is not None:
                assert torch.equal(mine[1], keep[kind]), kind + " pool differs"
                # and it is Eq. 2 of the full-width cache, token by token
                for b in range(w.batch):
                    got = torch.stack([mine[1][int(case.table[b, t // w.page_tokens]), t % w.page_tokens]
                                       for t in (0, lens[b] // 2, lens[b] - 1)]).cpu()
                    ref = O.retained_dims(full[kind][b][[0, lens[b] // 2, lens[b] - 1]].float().numpy(),
                                          w.mk if kind == "k" else w.m)
                    np.testing.assert_array_equal(got.float().numpy(), ref)
        if side_keep is not None:
            assert torch.equal(ctx.v_side[1], side_keep[1])
            if not w.save_k:               # (whole keys are in the pool: their side buffer is neither written nor read)
                assert torch.equal(ctx.k_side[1], side_keep[0])
        np.testing.assert_array_equal(case.run(1), want_out)
        assert ctx.device_status() == binding.ECHOKV_OK

    ctx.compress_layer(1, pools["k"], pools["v"], case.seq_lens)
    check()
    # the same in pieces, as a chunked prefill would do it (the window is taken relative to each call's length,
    # later calls overwrite the ring slots)
    for mine in (ctx.k_pools[1], ctx.v_pools[1]):
        if mine is not None:
            mine.zero_()
    if side_keep is not None:
        ctx.k_side[1].zero_()
        ctx.v_side[1].zero_()
    bounds = chunks + [max(lens)]
    for lo, hi in zip(bounds[:-1], bounds[1:]):
        begins = torch.tensor([min(lo, L) for L in lens], dtype=torch.int32, device=dev)
        ends = torch.tensor([min(hi, L) for L in lens], dtype=torch.int32, device=dev)
        live = [b for b in range(w.batch) if min(hi, lens[b]) >= 1]
        if len(live) != w.batch:       # sequences that have nothing cached yet are left out of the call
            slots = torch.tensor(live, dtype=torch.int32, device=dev)
            ctx.compress_layer(1, pools["k"], pools["v"], ends[live].contiguous(), begins[live].contiguous(), slots)
        else:
            ctx.compress_layer(1, pools["k"], pools["v"], ends, begins)
    check()
    case.close()


def test_compress_argument_checks_and_device_status():
    w = synth.C2.replace(batch=2, context=300)
    case = Case(w, lens=[300, 100], layers=[0, 1])
    ctx, dev = case.ctx, case.ctx.device
    pool = torch.zeros((case.cfg.n_pages, w.page_tokens, w.D), dtype=torch.bfloat16, device=dev)
    with pytest.raises(binding.EchoKVError) as e:
        ctx.compress_layer(0, pool, pool, case.seq_lens)            # an anchor layer keeps everything
    assert e.value.status == binding.ECHOKV_ENOTCOMPRESSED
    lib = binding.lib()
    assert lib.echokv_compress_layer(ctx.handle, 1, None, pool.data_ptr(), None, None, case.seq_lens.data_ptr(), 2,
                                     None) == binding.ECHOKV_EINVAL
    assert lib.echokv_compress_layer(ctx.handle, 1, pool.data_ptr() + 2, pool.data_ptr(), None, None,
                                     case.seq_lens.data_ptr(), 2, None) == binding.ECHOKV_EINVAL
    assert lib.echokv_compress_layer(ctx.handle, 1, pool.data_ptr(), pool.data_ptr(), None, None,
                                     case.seq_lens.data_ptr(), 3, None) == binding.ECHOKV_ECAPACITY
    before = ctx.k_pools[1].clone()
    bad_begin = torch.tensor([301, 0], dtype=torch.int32, device=dev)
    ctx.compress_layer(1, pool, pool, case.seq_lens, bad_begin)
    assert ctx.device_status() == binding.ECHOKV_EBADLENGTH
    # the sequence with the bad range was left alone, the other one was evicted (to zeros, here)
    t = case.table
    assert torch.equal(ctx.k_pools[1][int(t[0, 0])], before[int(t[0, 0])])
    assert int(ctx.k_pools[1][int(t[1, 0])].abs().sum()) == 0
    case.close()
