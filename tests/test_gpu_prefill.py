"""GPU parity of the prefill-shaped call: the last n_q cached tokens of every sequence as causal queries over the
rebuilt cache (rebuilt once per call into a bf16 scratch, then a causal attention kernel)."""
import numpy as np
import pytest
import torch

from oracle import echokv_oracle as O
from paper_2603_22910_b200 import binding, build, synth
from tests.harness import Case, errors

pytestmark = pytest.mark.gpu

THETA = 10000.0

# This call materialises the rebuilt K~ / V~ rows in 16 bits (the decode calls keep them in fp32).  A query that attends
# a handful of tokens returns nearly a single V~ row, so the value rows (and the probabilities) are fp16, whose rounding
# of |v| up to ~5 stays near 1e-3; the tolerance is that of the decode calls.
TOL_PREFILL = dict(max_abs=2e-2, rel_l2=5e-3)


def assert_parity(out, ref, dtype, what=""):
    max_abs, rel_l2 = errors(out, ref)
    assert np.all(np.isfinite(out)), "non-finite output " + what
    assert max_abs <= TOL_PREFILL["max_abs"] and rel_l2 <= TOL_PREFILL["rel_l2"], \
        "%s: max_abs %.3e, rel_l2 %.3e" % (what, max_abs, rel_l2)
    return max_abs, rel_l2


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    binding.lib()


def queries(w, n_q, seed):
    return (synth.normal((w.batch, n_q, w.n_q_heads, w.head_dim), w.seed, 77, seed)).to(synth.torch_dtype(w))


def oracle_prefill(case, layer, q, b, rope):
    w = case.w
    qn = O.widen(synth.to_numpy_stored(q))[b]
    a = w.anchor_of(layer)
    kg, vg = case._stored(a, "k", b), case._stored(a, "v", b)
    if w.is_anchor(layer):
        return O.prefill_attention(qn, kg, vg, None, None, None, None, w.n_kv_heads, rope_theta=rope)
    L = kg.shape[0]
    kl = case._stored(layer, "k", b) if w.m else np.zeros((L, 0))
    vl = case._stored(layer, "v", b) if w.m else np.zeros((L, 0))
    Wk, Wv, bk, bv = (None if t is None else O.widen(synth.to_numpy_stored(t)) for t in case.host_w[layer])
    k_true = None
    if w.save_k:                 # keys kept whole (Section 5.2): the stored K rows are the whole keys
        k_true = case._stored(layer, "k", b)
        kl = k_true[:, :w.m]
    return O.prefill_attention(qn, kg, vg, kl, vl, Wk, Wv, w.n_kv_heads, bk=bk, bv=bv, rope_theta=rope, k_true=k_true)


CASES = [
    # name, base, overrides, lens, n_q, biases, rope
    ("gqa_one_tile", synth.C2, dict(batch=2, context=700), [700, 333], 37, False, None),
    ("gqa_three_tiles", synth.C2, dict(batch=2, context=600, random_pages=True), [600, 200], 150, True, None),
    ("mha", synth.C1, dict(batch=2, context=500), [500, 257], 64, False, None),
    ("gqa_rope", synth.C2, dict(batch=2, context=700, page_tokens=64, random_pages=True), [700, 130], 65, True, THETA),
    ("one_query_is_the_decode_step", synth.C2, dict(batch=2, context=300), [300, 17], 1, False, None),
    ("every_token_a_query", synth.C2, dict(batch=1, context=200, n_retained_heads=6), [200], 200, False, THETA),
    ("nothing_retained", synth.C2, dict(batch=2, context=400, n_retained_heads=0), [400, 129], 70, False, None),
    ("two_heads_per_cta_128_queries", synth.C2, dict(batch=2, context=400, random_pages=True), [400, 128], 128, False, THETA),
    ("eight_heads_per_cta", synth.C2, dict(batch=2, context=300, n_q_heads=64), [300, 33], 20, False, None),
    ("mha_two_ctas_per_head", synth.C1, dict(batch=1, context=600), [600], 300, False, None),
    ("second_cta_half_empty", synth.C2, dict(batch=2, context=700), [700, 300], 300, False, None),
    ("keys_whole", synth.C2, dict(batch=2, context=500, save_k=True), [500, 260], 130, True, None),
    ("keys_whole_rope", synth.C1, dict(batch=2, context=300, save_k=True), [300, 77], 40, False, THETA),
]


@pytest.mark.parametrize("name,base,over,lens,n_q,biases,rope", CASES, ids=[c[0] for c in CASES])
def test_prefill_against_oracle(name, base, over, lens, n_q, biases, rope):
    w = base.replace(**over)
    case = Case(w, lens=lens, layers=[0, 1], biases=biases, rope=rope)
    ctx = case.ctx
    for layer in (1, 0):
        q = queries(w, n_q, layer)
        # the scratch starts as NaN patterns: rows past a sequence's end must never reach a result
        ctx.prefill_attention(layer, q.to(ctx.device), case.seq_lens)
        ctx.prefill_scratch.fill_(0xFF)
        out = ctx.prefill_attention(layer, q.to(ctx.device), case.seq_lens)
        torch.cuda.synchronize()
        out = out.cpu().numpy().astype(np.float64)
        for b in range(w.batch):
            ref = oracle_prefill(case, layer, q, b, rope)
            assert_parity(out[b], ref, w.dtype, "%s layer %d seq %d" % (name, layer, b))
    if n_q == 1:     # a single query per sequence: the same function as the decode call
        q = queries(w, 1, 1)
        dec = ctx.decode_attention(1, q[:, 0].contiguous().to(ctx.device), case.seq_lens).cpu().numpy()
        pre = ctx.prefill_attention(1, q.to(ctx.device), case.seq_lens).cpu().numpy()[:, 0]
        assert_parity(pre, dec.astype(np.float64), w.dtype, name + " vs decode")
    assert ctx.device_status() == binding.ECHOKV_OK
    case.close()


def test_prefill_short_sequences_and_argument_checks():
    w = synth.C2.replace(batch=3, context=300)
    case = Case(w, lens=[300, 20, 64], layers=[0, 1])
    ctx, dev = case.ctx, case.ctx.device
    n_q = 64
    q = queries(w, n_q, 3)
    out = ctx.prefill_attention(1, q.to(dev), case.seq_lens).cpu().numpy().astype(np.float64)
    assert ctx.device_status() == binding.ECHOKV_EBADLENGTH       # sequence 1 holds fewer tokens than queries
    assert not out[1].any()
    for b in (0, 2):
        assert_parity(out[b], oracle_prefill(case, 1, q, b, None), w.dtype, "seq %d" % b)
    lib, h = binding.lib(), ctx.handle
    o = torch.empty(q.shape, dtype=torch.float32, device=dev)
    qd = q.to(dev)
    scratch = ctx.prefill_scratch
    args = (qd.data_ptr(), o.data_ptr())
    assert lib.echokv_prefill_attention(h, 1, *args, 0, None, case.seq_lens.data_ptr(), 3, None, None,
                                        scratch.data_ptr(), scratch.numel(), None) == binding.ECHOKV_EINVAL
    assert lib.echokv_prefill_attention(h, 1, *args, n_q, None, case.seq_lens.data_ptr(), 3, None, None,
                                        scratch.data_ptr(), 1024, None) == binding.ECHOKV_ECAPACITY
    assert lib.echokv_prefill_attention(h, 1, *args, n_q, None, case.seq_lens.data_ptr(), 3, None, None, None, 0,
                                        None) == binding.ECHOKV_EINVAL
    # with a window set the call needs the recent tokens' rows from the caller
    ctx.set_full_precision_window(4, 128)
    assert lib.echokv_prefill_attention(h, 1, *args, n_q, None, case.seq_lens.data_ptr(), 3, None, None,
                                        scratch.data_ptr(), scratch.numel(), None) == binding.ECHOKV_EINVAL
    case.close()
    small = Case(synth.C0, layers=[1])
    n = torch.zeros(1, dtype=torch.int64)
    import ctypes as C
    nbytes = C.c_uint64(0)
    assert lib.echokv_prefill_scratch_bytes(C.byref(small.cfg), C.byref(nbytes)) == binding.ECHOKV_EUNSUPPORTED
    small.close()


@pytest.mark.parametrize("window", [None, (4, 128), (3, 20)], ids=["plain", "window_4_128", "window_3_20"])
def test_chunk_append_equals_token_by_token(window):
    # a chunk of n new tokens per sequence appended in one call: the cache (pools and side buffers) and the decode
    # result are those of a context that held the longer sequences from the start
    w = synth.C2.replace(batch=3, context=700, random_pages=True)
    n = 150
    long_lens = [700, 333, 151]
    ref = Case(w, lens=long_lens, layers=[0, 1], window=window)
    short = Case(w, lens=[L - n for L in long_lens], layers=[0, 1], window=window)
    dev = short.ctx.device
    first = torch.tensor([L - n for L in long_lens], dtype=torch.int32, device=dev)
    for layer in (0, 1):
        rows = {}
        for kind in "kv":
            full = torch.stack([synth.layer_cache(w, layer, kind, b, width=w.D)[long_lens[b] - n: long_lens[b]]
                                for b in range(w.batch)])                      # [B][n][D]
            if not w.is_anchor(layer) and not window:
                full[:, :, w.m:] = 777.0                                         # must never reach the cache
            rows[kind] = full.to(dev)
        short.ctx.append_kv_chunk(layer, rows["k"], rows["v"], first)
    torch.cuda.synchronize()
    assert short.ctx.device_status() == binding.ECHOKV_OK
    short.seq_lens = ref.seq_lens.clone()
    for layer in (0, 1):
        for b, L in enumerate(long_lens):
            for t in (0, L - n - 1, L - n, L - 75, L - 1):
                page, r = int(ref.table[b, t // w.page_tokens]), t % w.page_tokens
                for pa, pb in ((ref.ctx.k_pools, short.ctx.k_pools), (ref.ctx.v_pools, short.ctx.v_pools)):
                    assert torch.equal(pa[layer][page, r], pb[layer][page, r]), (layer, b, t)
    if window:
        n_sink, n_window = window
        for b, L in enumerate(long_lens):
            live = [t for t in range(L) if t < n_sink or t >= L - n_window]
            slots = [t if t < n_sink else n_sink + t % n_window for t in live]
            assert torch.equal(ref.ctx.k_side[1][b, slots], short.ctx.k_side[1][b, slots])
            assert torch.equal(ref.ctx.v_side[1][b, slots], short.ctx.v_side[1][b, slots])
    np.testing.assert_array_equal(short.run(1), ref.run(1))
    np.testing.assert_array_equal(short.run(0), ref.run(0))
    ref.close()
    short.close()


def test_prefill_scores_that_jump_mid_sequence():
    """A few keys in the middle of the cache score far above everything before them (2^46 and more above the running
    reference, some beyond what 2^x can hold in fp32): the kernel, which keeps a lazy reference maximum, must notice,
    move it and rescale what it has accumulated."""
    w = synth.C2.replace(batch=1, context=1000)
    case = Case(w, lens=[1000], layers=[0])
    ctx = case.ctx
    hot = slice(400, 421)
    rows = case.host[(0, "k", 0)]
    rows[hot] = rows[hot] * 32                       # (a power of two: exact in bf16)
    ctx.k_pools[0].view(-1, w.D)[hot] = rows[hot].to(ctx.device)       # identity page order: pool row = token
    n_q = 300
    q = queries(w, n_q, 5)
    out = ctx.prefill_attention(0, q.to(ctx.device), case.seq_lens).cpu().numpy().astype(np.float64)
    assert ctx.device_status() == binding.ECHOKV_OK
    ref = oracle_prefill(case, 0, q, 0, None)
    assert_parity(out[0], ref, w.dtype, "jumping scores")
    case.close()


def test_prefill_sequence_slots_select_block_table_rows():
    w = synth.C2.replace(batch=3, context=300)
    case = Case(w, lens=[300, 150, 99], layers=[0, 1])
    ctx, dev = case.ctx, case.ctx.device
    n_q = 70
    q = queries(w, n_q, 9).to(dev)
    base = ctx.prefill_attention(1, q, case.seq_lens).cpu().numpy()
    order = [2, 0, 1]
    slots = torch.tensor(order, dtype=torch.int32, device=dev)
    out = ctx.prefill_attention(1, q[order].contiguous(), case.seq_lens[order].contiguous(), seq_slots=slots)
    torch.cuda.synchronize()
    np.testing.assert_array_equal(out.cpu().numpy(), base[order])
    assert ctx.device_status() == binding.ECHOKV_OK
    case.close()
