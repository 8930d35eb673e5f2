"""GPU parity: the CUDA library (through the C-ABI) against the CPU oracle, element by
element, on the same seeded stored values."""
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


def check_layers(case, what):
    w = case.w
    worst = (0.0, 0.0)
    for l in case.layers:
        out = case.run(l)
        ref = case.oracle(l)
        e = assert_parity(out, ref, w.dtype, "%s layer %d" % (what, l))
        worst = max(worst, e, key=lambda t: t[1])
        if w.is_anchor(l):
            np.testing.assert_array_equal(case.run(l, full=True), out)
    assert case.ctx.device_status() == binding.ECHOKV_OK
    return worst


def test_config0_tiny_fp32_full():
    case = Case(synth.C0, layers=[0, 1])
    assert case.ctx.decode_path() == 1
    check_layers(case, "c0")
    case.close()


SMALL = [
    # name, base, overrides, lens
    ("c1_shape", synth.C1, dict(batch=2, context=700), [700, 333]),
    ("c2_shape", synth.C2, dict(batch=3, context=1000), [1000, 517, 256]),
    ("c2_shape_pages64", synth.C2, dict(batch=2, context=600, page_tokens=64, random_pages=True), [600, 65]),
    ("c4_25pct", synth.c4_point(25, 4096, 1), dict(batch=2, context=530), [530, 17]),
    ("c4_50pct", synth.c4_point(50, 4096, 1), dict(batch=2, context=300, random_pages=True), [300, 299]),
    ("mha_d64_bf16", synth.C0, dict(dtype="bf16", batch=2, context=200), [200, 77]),
    ("gqa2_fp32_d128", synth.C0, dict(n_q_heads=8, n_kv_heads=4, head_dim=128, n_retained_heads=1,
                                      batch=2, context=150), [150, 64]),
    ("one_dropped_head", synth.C2, dict(n_retained_heads=7, batch=2, context=300), [300, 258]),
    ("pages128", synth.C2, dict(batch=2, context=700, page_tokens=128, random_pages=True), [700, 129]),
    ("gqa8_bf16", synth.C2, dict(n_q_heads=32, n_kv_heads=4, n_retained_heads=1, batch=1, context=300), [300]),
    ("many_tiles_ragged", synth.C2, dict(batch=5, context=2000, random_pages=True), [2000, 129, 128, 1153, 1]),
    ("mha_three_dropped", synth.C1.replace(n_q_heads=4, n_kv_heads=4), dict(n_retained_heads=1, batch=2, context=600),
     [600, 385]),
    ("gqa2_six_dropped", synth.C2, dict(n_q_heads=16, batch=3, context=900, random_pages=True), [900, 257, 130]),
    ("mha_m64", synth.C1.replace(n_q_heads=8, n_kv_heads=8), dict(n_retained_heads=0, n_retained_dims=64, batch=2,
                                                                 context=400, random_pages=True), [400, 33]),
]


@pytest.mark.parametrize("name,base,over,lens", SMALL, ids=[s[0] for s in SMALL])
@pytest.mark.parametrize("path", [1, 2, 3, 4])
def test_small_shapes_against_oracle(name, base, over, lens, path):
    w = base.replace(**over)
    case = Case(w, lens=lens, layers=[0, 1])
    if path >= 2 and case.ctx.decode_path() < 2:
        case.close()
        pytest.skip("shape is served by the CUDA-core kernel only")
    if path == 4 and w.n_q_heads // w.n_kv_heads > 2:
        case.close()
        pytest.skip("the four-heads-per-item kernel takes at most two query heads per KV head")
    assert case.ctx.decode_path() in (1, 2, 3, 4, 5)  # a context starts on the family its shape runs fastest on
    case.ctx.set_decode_path(path)
    check_layers(case, name)
    case.close()


STORED = [
    # name, base, overrides, lens: shapes of the stored-head attention (anchor layer 0, retained heads of layer 1)
    ("mha", synth.C1, dict(batch=3, context=2100), [2100, 1025, 64]),
    ("gqa4", synth.C2, dict(batch=3, context=1500, n_retained_heads=3, random_pages=True), [1500, 257, 1]),
    ("gqa2_pages32", synth.C2, dict(n_q_heads=16, batch=2, context=900, page_tokens=32, random_pages=True), [900, 33]),
    ("gqa8_pages64", synth.C2, dict(n_q_heads=32, n_kv_heads=4, n_retained_heads=2, batch=2, context=700,
                                    page_tokens=64), [700, 65]),
    ("gqa4_pages128", synth.C2, dict(batch=2, context=1000, page_tokens=128, n_retained_heads=5,
                                     random_pages=True), [1000, 129]),
]


@pytest.mark.parametrize("name,base,over,lens", STORED, ids=[s[0] for s in STORED])
@pytest.mark.parametrize("stored_path", [0, 1])
def test_stored_head_kernels_against_oracle(name, base, over, lens, stored_path):
    w = base.replace(**over)
    case = Case(w, lens=lens, layers=[0, 1])
    assert case.ctx.stored_path() == 1        # bf16, head_dim 128: the TMA + tensor-core kernel by default
    case.ctx.set_stored_path(stored_path)
    check_layers(case, "%s stored_path %d" % (name, stored_path))
    case.close()


def test_slots_that_hold_no_token_may_contain_anything():
    # cache slots past a sequence's length, and pages no sequence uses, were never written: fill
    # them with NaN and huge values; the result must not change
    w = synth.C2.replace(batch=2, context=600, n_retained_heads=3, random_pages=True)
    lens = [600, 70]
    n_pages = 2 * w.pages_per_seq + 9
    case = Case(w, lens=lens, layers=[0, 1], n_pages=n_pages)
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
        assert_parity(case.run(l), case.oracle(l), w.dtype, "junk in unused slots, layer %d" % l)
    assert case.ctx.device_status() == binding.ECHOKV_OK
    case.close()


def test_config3_shape_multi_layer_random_pages():
    # 8 layers = two groups of S = 4; ragged lengths; pool larger than needed, random page order
    w = synth.C3.replace(n_layers=8, batch=2, context=420)
    case = Case(w, lens=[420, 131], n_pages=2 * w.pages_per_seq + 13)
    check_layers(case, "c3_shape")
    case.close()


@pytest.mark.parametrize("r", [0, 8])
def test_nothing_retained_and_nothing_dropped(r):
    w = synth.C2.replace(batch=2, context=300, n_retained_heads=r)
    case = Case(w, lens=[300, 40], layers=[0, 1])
    assert case.ctx.decode_path() == (0 if r == 8 else case.ctx.decode_path())
    check_layers(case, "r=%d" % r)
    if r == 8:   # a layer that drops nothing also serves echokv_full_attention
        np.testing.assert_array_equal(case.run(1, full=True), case.run(1))
    case.close()


@pytest.mark.parametrize("L", [1, 15, 16, 17, 255, 256, 257])
def test_short_and_boundary_lengths(L):
    w = synth.C2.replace(batch=2, context=L + 3, n_retained_heads=4)
    case = Case(w, lens=[L, L + 3], layers=[0, 1])
    check_layers(case, "L=%d" % L)
    case.close()


def test_predictor_bias():
    w = synth.C2.replace(batch=2, context=200)
    case = Case(w, lens=[200, 31], layers=[1], biases=True)
    check_layers(case, "bias")
    nb = Case(w, lens=[200, 31], layers=[1], biases=False)
    assert errors(case.run(1), nb.run(1))[0] > 1e-3      # the bias is not a no-op
    case.close(); nb.close()


def test_page_order_does_not_change_the_result():
    w = synth.C2.replace(batch=2, context=333)
    a = Case(w, lens=[333, 90], layers=[0, 1])
    b = Case(w.replace(random_pages=True), lens=[333, 90], layers=[0, 1], n_pages=2 * w.pages_per_seq + 5)
    for l in (0, 1):
        np.testing.assert_array_equal(a.run(l), b.run(l))
    a.close(); b.close()


def test_sequence_slots_select_block_table_rows():
    w = synth.C2.replace(batch=3, context=200)
    case = Case(w, lens=[200, 150, 99], layers=[1])
    base = case.run(1)
    dev = case.ctx.device
    order = [2, 0, 1]
    slots = torch.tensor(order, dtype=torch.int32, device=dev)
    q = case.q[1][order].contiguous().to(dev)
    lens = case.seq_lens[order].contiguous()
    out = case.ctx.decode_attention(1, q, lens, seq_slots=slots)
    torch.cuda.synchronize()
    np.testing.assert_array_equal(out.cpu().numpy(), base[order])
    case.close()


def test_append_writes_only_what_the_layer_keeps():
    w = synth.C2.replace(batch=2, context=40)
    case = Case(w, lens=[40, 23], layers=[0, 1])
    for b, L in enumerate(case.lens):
        page = int(case.table[b, (L - 1) // w.page_tokens])
        slot = (L - 1) % w.page_tokens
        for l, width in ((0, w.D), (1, w.m)):
            got = case.ctx.k_pools[l][page, slot].cpu()
            assert got.shape[0] == width
            assert torch.equal(got, case.host[(l, "k", "new")][b, :width])
            assert not (got == 777.0).any()
    case.close()


def test_bad_length_and_bad_page_are_reported_not_fatal():
    w = synth.C2.replace(batch=2, context=100)
    case = Case(w, lens=[100, 60], layers=[1])
    good = case.run(1)
    dev = case.ctx.device
    q = case.q[1].to(dev)
    bad_lens = torch.tensor([100, 0], dtype=torch.int32, device=dev)
    out = case.ctx.decode_attention(1, q, bad_lens)
    assert case.ctx.device_status() == binding.ECHOKV_EBADLENGTH
    out = out.cpu().numpy()
    np.testing.assert_array_equal(out[0], good[0])
    assert np.all(out[1] == 0.0)
    too_long = torch.tensor([100, 10 ** 6], dtype=torch.int32, device=dev)
    case.ctx.decode_attention(1, q, too_long)
    assert case.ctx.device_status() == binding.ECHOKV_EBADLENGTH
    # a page id outside the pool: reported, no fault
    saved = case.ctx.block_table.clone()
    case.ctx.block_table[1, 1] = 10 ** 6
    out = case.ctx.decode_attention(1, q, case.seq_lens)
    assert case.ctx.device_status() == binding.ECHOKV_EBADPAGE
    assert np.all(np.isfinite(out.cpu().numpy()))
    case.ctx.block_table.copy_(saved)
    np.testing.assert_array_equal(case.run(1), good)
    assert case.ctx.device_status() == binding.ECHOKV_OK
    case.close()


def test_host_status_codes_on_gpu():
    w = synth.C2.replace(batch=2, context=64)
    case = Case(w, lens=[64, 64], layers=[0, 1])
    ctx, L = case.ctx, binding.lib()
    q = case.q[1].to(ctx.device)
    out = torch.empty(q.shape, dtype=torch.float32, device=ctx.device)
    args = (q.data_ptr(), out.data_ptr(), None, case.seq_lens.data_ptr())
    assert L.echokv_full_attention(ctx.handle, 1, *args, 2, None) == binding.ECHOKV_ENOTANCHOR
    assert L.echokv_decode_attention(ctx.handle, 2, *args, 2, None) == binding.ECHOKV_EINVAL
    assert L.echokv_decode_attention(ctx.handle, 1, *args, 3, None) == binding.ECHOKV_ECAPACITY
    assert L.echokv_set_weights(ctx.handle, 0, q.data_ptr(), q.data_ptr(), None, None) == binding.ECHOKV_ENOTCOMPRESSED
    fresh = binding.Context(case.cfg)
    assert L.echokv_decode_attention(fresh.handle, 1, *args, 2, None) == binding.ECHOKV_ENOWEIGHTS
    fresh.close(); case.close()


def test_layer_step_from_host_memory_matches_device_calls():
    w = synth.C2.replace(batch=2, context=129)
    case = Case(w, lens=[129, 70], layers=[0, 1])
    ref = case.run(1)
    # replay the last token through the host entry point on a second context
    other = Case(w, lens=[129, 70], layers=[0, 1])
    lens_host = torch.tensor(case.lens, dtype=torch.int32).pin_memory()
    out_host = torch.empty((w.batch, w.n_q_heads, w.head_dim), dtype=torch.float32).pin_memory()
    for l, attend in ((0, False), (1, True)):
        other.ctx.layer_step_host(l, other.q[1].pin_memory(), other.host[(l, "k", "new")].pin_memory(),
                                  other.host[(l, "v", "new")].pin_memory(), out_host, lens_host, attend=attend)
    np.testing.assert_array_equal(out_host.numpy(), ref)
    case.close(); other.close()


@pytest.mark.parametrize("absorbed", [False, True, "by_page_order"], ids=["explicit", "absorbed", "by_page_order"])
def test_layer_step_replayed_from_a_cuda_graph(absorbed):
    # every call only enqueues kernels on the caller's stream, so a whole step can be captured once and replayed
    # (by_page_order: the kernel family is decided on the device inside the captured step, decode path 5)
    w = synth.C2.replace(batch=2, context=600)
    if absorbed == "by_page_order":
        w = synth.C1.replace(batch=2, context=600, random_pages=True)
    case = Case(w, lens=[600, 333], layers=[0, 1])
    ctx, dev = case.ctx, case.ctx.device
    if absorbed == "by_page_order":
        assert ctx.decode_path() == 5
    elif absorbed:
        ctx.enable_absorbed()
    q = {l: case.q[l].to(dev) for l in (0, 1)}
    out = {l: torch.empty(q[l].shape, dtype=torch.float32, device=dev) for l in (0, 1)}
    new = {(l, kind): case.host[(l, kind, "new")].to(dev) for l in (0, 1) for kind in ("k", "v")}

    def step():
        for l in (0, 1):
            ctx.append_kv(l, new[(l, "k")], new[(l, "v")], case.positions)
            ctx.decode_attention(l, q[l], case.seq_lens, out=out[l])

    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        step()                       # first-use set-up happens here, outside the capture
        side.synchronize()
        eager = {l: out[l].clone() for l in (0, 1)}
        with torch.cuda.graph(graph, stream=side):
            step()
    torch.cuda.current_stream().wait_stream(side)
    for l in (0, 1):
        out[l].fill_(float("nan"))
    graph.replay()
    torch.cuda.synchronize()
    for l in (0, 1):
        assert torch.equal(out[l], eager[l])
    # new queries through the same graph: the captured kernels read the tensors, not copies of them
    q2 = synth.queries(w.replace(seed=w.seed + 5), 1).to(dev)
    q[1].copy_(q2)
    graph.replay()
    torch.cuda.synchronize()
    replayed = out[1].clone()
    direct = ctx.decode_attention(1, q2, case.seq_lens)
    torch.cuda.synchronize()
    assert torch.equal(replayed, direct)
    assert ctx.device_status() == binding.ECHOKV_OK
    case.close()


def test_more_sequences_than_one_launch_indexes():
    # the tcgen05 kernels index at most 256 sequences per launch and the stored-head kernel 512: a larger
    # batch is split over several launches
    w = synth.C2.replace(batch=600, context=48, n_kv_heads=2, n_q_heads=8, n_retained_heads=1)
    rng = np.random.default_rng(3)
    lens = [int(v) for v in rng.integers(1, 49, size=w.batch)]
    case = Case(w, lens=lens, layers=[0, 1])
    for path in (2, 3):
        case.ctx.set_decode_path(path)
        assert_parity(case.run(1), case.oracle(1), w.dtype, "batch 600, path %d" % path)
    wide = synth.C1.replace(batch=300, context=40, n_kv_heads=8, n_q_heads=8, n_retained_heads=2)
    lens_w = [int(v) for v in rng.integers(1, 41, size=wide.batch)]
    case_w = Case(wide, lens=lens_w, layers=[0, 1])
    case_w.ctx.set_decode_path(4)
    assert_parity(case_w.run(1), case_w.oracle(1), wide.dtype, "batch 300, path 4")
    case_w.close()
    assert_parity(case.run(0), case.oracle(0), w.dtype, "batch 600, anchor")
    assert case.ctx.device_status() == binding.ECHOKV_OK
    case.close()


def test_every_sequence_unusable_gives_zeros_and_a_status():
    w = synth.C2.replace(batch=2, context=64)
    case = Case(w, lens=[64, 64], layers=[0, 1])
    dev = case.ctx.device
    bad = torch.tensor([0, -5], dtype=torch.int32, device=dev)
    for l in (0, 1):
        out = case.ctx.decode_attention(l, case.q[l].to(dev), bad)
        assert case.ctx.device_status() == binding.ECHOKV_EBADLENGTH
        assert np.all(out.cpu().numpy() == 0.0)
    case.close()


def test_a_bounded_wait_that_runs_out_reports_a_timeout_and_leaves_the_context_usable():
    """The give-up path of the kernels' waits (a limit, a status, an abort flag that releases the other roles),
    driven by a probe that waits on a barrier nothing arrives on: no fault, no hang, nothing left in flight."""
    import time
    w = synth.C2.replace(batch=2, context=300)
    case = Case(w, lens=[300, 77], layers=[0, 1])
    ctx = case.ctx
    before = case.run(1)
    assert ctx.device_status() == binding.ECHOKV_OK
    t0 = time.perf_counter()
    left = ctx.diag_bounded_wait(200000)            # ~0.1 ms of SM cycles
    torch.cuda.synchronize()
    assert time.perf_counter() - t0 < 5.0
    assert left.cpu().tolist() == [1, 1]            # the waiting warp gave up; the other one was released by its flag
    assert ctx.device_status() == binding.ECHOKV_ETIMEOUT
    assert ctx.device_status() == binding.ECHOKV_OK          # read and cleared
    np.testing.assert_array_equal(case.run(1), before)       # the context works as before
    assert ctx.device_status() == binding.ECHOKV_OK
    assert binding.lib().echokv_diag_bounded_wait(ctx.handle, 0, left.data_ptr(), None) == binding.ECHOKV_EINVAL
    case.close()


@pytest.mark.parametrize("mode", ["explicit", "absorbed"])
def test_a_page_outside_the_pool_is_reported_and_harms_no_other_sequence(mode):
    """A page id outside the pool is a caller's error: it is reported, nothing is read through it (no fault), and
    the other sequences of the call come out bit for bit as without it."""
    w = synth.C2.replace(batch=3, context=200)
    case = Case(w, lens=[200, 100, 77], layers=[0, 1])
    ctx = case.ctx
    if mode == "absorbed":
        ctx.enable_absorbed()
    good = case.run(1)
    saved = ctx.block_table.clone()
    ctx.block_table[1, 2] = 10 ** 6                     # tokens 32 .. 47 of sequence 1
    out = case.run(1)
    assert ctx.device_status() == binding.ECHOKV_EBADPAGE
    np.testing.assert_array_equal(out[0], good[0])
    np.testing.assert_array_equal(out[2], good[2])
    ctx.block_table.copy_(saved)
    np.testing.assert_array_equal(case.run(1), good)
    assert ctx.device_status() == binding.ECHOKV_OK
    case.close()


def test_the_kernel_family_follows_the_page_order_found_in_the_block_table():
    """Decode path 5: both fused kernels are launched and a word written on the device (pages of the batch in order
    or not) says which of them runs; the merge and the sink / window partial follow the partial size of that kernel."""
    base = synth.C1.replace(batch=3, context=1500)
    lens = [1500, 700, 64]
    for window in (None, (4, 128)):
        flags = {}
        for random_pages in (False, True):
            w = base.replace(random_pages=random_pages)
            case = Case(w, lens=lens, layers=[0, 1], window=window)
            assert case.ctx.decode_path() == 5            # long contraction, one query head per KV head, 16-token pages
            out = case.run(1)
            flags[random_pages] = case.ctx.diag_page_order()
            assert_parity(out, case.oracle(1), w.dtype, "path 5, random_pages=%s, window=%s" % (random_pages, window))
            # the same numbers as the kernel family it chose, run on its own
            case.ctx.set_decode_path(2 if flags[random_pages] == 1 else 4)
            np.testing.assert_array_equal(case.run(1), out)
            case.ctx.set_decode_path(5)
            np.testing.assert_array_equal(case.run(1), out)
            assert case.ctx.device_status() == binding.ECHOKV_OK
            case.close()
        assert flags == {False: 1, True: 0}
    # pages of 64 tokens: nothing to decide
    case = Case(synth.C1.replace(batch=2, context=300, page_tokens=64), lens=[300, 100], layers=[0, 1])
    assert case.ctx.decode_path() == 2
    with pytest.raises(Exception):
        case.ctx.set_decode_path(5)
    case.close()
