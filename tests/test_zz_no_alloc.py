"""echokv_full_attention_noalloc: the entry point for callers that cannot allocate device
memory (no context, no workspace; partial results live in a fixed array inside the library).
It must give what echokv_full_attention gives, call after call, although every call reuses
the same scratch array and finds the previous call's leftovers in it.

Collected last on purpose (file name): a failure here must not hide any other test."""
import ctypes as C

import numpy as np
import pytest
import torch

from paper_2603_22910_b200 import binding, build, synth
from tests.harness import TOL, Case, errors


@pytest.mark.gpu
def test_noalloc_matches_full_attention_on_two_calls_in_a_row():
    build.build()
    assert torch.cuda.is_available()
    w = synth.C2.replace(batch=3, context=700, random_pages=True)
    case = Case(w, lens=[700, 333, 16], layers=[0])
    ctx, dev = case.ctx, case.ctx.device
    tol = TOL["bf16"]
    status = torch.full((1,), 99, dtype=torch.int32, device=dev)
    # call 1: the whole batch; call 2: other queries and shorter sequences, so that whatever call 1
    # left in the scratch array would show if it were read
    q1 = case.q[0].to(dev)
    q2 = synth.queries(w.replace(seed=w.seed + 1), 0).to(dev)
    lens1 = case.seq_lens
    lens2 = torch.tensor([130, 333, 1], dtype=torch.int32, device=dev)
    for q, lens in ((q1, lens1), (q2, lens2)):
        ref = ctx.full_attention(0, q, lens)
        out = torch.full_like(ref, float("nan"))
        binding.echokv_full_attention_noalloc(case.cfg, ctx.k_pools[0], ctx.v_pools[0], ctx.block_table,
                                              q, out, lens, status_out=status)
        torch.cuda.synchronize()
        assert int(status.item()) == binding.ECHOKV_OK
        max_abs, rel_l2 = errors(out.cpu().numpy(), ref.cpu().numpy())
        assert np.all(np.isfinite(out.cpu().numpy()))
        assert max_abs <= tol["max_abs"] and rel_l2 <= tol["rel_l2"], (max_abs, rel_l2)
    # and against the oracle, for the first call's inputs
    out = torch.empty_like(ref)
    binding.echokv_full_attention_noalloc(case.cfg, ctx.k_pools[0], ctx.v_pools[0], ctx.block_table,
                                          q1, out, lens1)
    torch.cuda.synchronize()
    max_abs, rel_l2 = errors(out.cpu().numpy(), case.oracle(0))
    assert max_abs <= tol["max_abs"] and rel_l2 <= tol["rel_l2"], (max_abs, rel_l2)
    # a device-side problem is reported through the status output, not by a fault
    bad = torch.tensor([700, 0, 16], dtype=torch.int32, device=dev)
    binding.echokv_full_attention_noalloc(case.cfg, ctx.k_pools[0], ctx.v_pools[0], ctx.block_table,
                                          q1, out, bad, status_out=status)
    torch.cuda.synchronize()
    assert int(status.item()) == binding.ECHOKV_EBADLENGTH
    assert np.all(out[1].cpu().numpy() == 0.0)
    case.close()


def test_noalloc_rejects_what_does_not_fit_the_fixed_scratch():
    build.build()
    lib = binding.lib()
    assert lib.echokv_noalloc_scratch_bytes() == 8 << 20
    w = synth.C2.replace(batch=1024, context=64)
    cfg = binding.config_for(w)
    # B * n_q_heads = 32768 partial rows of 520 bytes > 8 MiB: refused before any CUDA call
    rc = lib.echokv_full_attention_noalloc(C.byref(cfg), 0x1000, 0x1000, 0x1000, 0x1000, 0x1000, None, 0x1000,
                                           1024, None, None)
    assert rc == binding.ECHOKV_ESCRATCH
    assert "scratch" in binding.echokv_strerror(rc)
    assert lib.echokv_full_attention_noalloc(C.byref(cfg), None, None, None, None, None, None, None, 1, None,
                                             None) == binding.ECHOKV_EINVAL
    assert lib.echokv_full_attention_noalloc(C.byref(cfg), 0x1000, 0x1000, 0x1000, 0x1000, 0x1000, None, 0x1000,
                                             2048, None, None) == binding.ECHOKV_ECAPACITY


def test_noalloc_rejects_misaligned_pointers_and_overflowing_geometry_on_the_host():
    """Fake pointers only: every one of these must be refused before any CUDA call is made."""
    build.build()
    lib = binding.lib()
    cfg = binding.config_for(synth.C2.replace(batch=2, context=64))
    ok = [0x1000, 0x1000, 0x1000, 0x1000, 0x1000]          # k_pool, v_pool, table, q, out
    for i in (0, 1, 3, 4):                                 # a pointer aligned to 4 bytes only
        args = list(ok)
        args[i] = 0x1004
        rc = lib.echokv_full_attention_noalloc(C.byref(cfg), *args, None, 0x1000, 1, None, None)
        assert rc == binding.ECHOKV_EINVAL, i
    big = binding.config_for(synth.C2.replace(batch=2, context=64))
    big.max_pages_per_seq = (1 << 30) // big.page_tokens + 1       # capacity beyond 2^30 tokens
    assert lib.echokv_full_attention_noalloc(C.byref(big), *ok, None, 0x1000, 1, None, None) == binding.ECHOKV_EINVAL
    inf = binding.config_for(synth.C2.replace(batch=2, context=64))
    inf.softmax_scale = float("inf")
    assert lib.echokv_full_attention_noalloc(C.byref(inf), *ok, None, 0x1000, 1, None, None) == binding.ECHOKV_EINVAL


@pytest.mark.gpu
def test_noalloc_with_fewer_splits_than_it_would_like():
    """Many short sequences: 4 * SMs / (B * H_kv) splits do not fit the 8 MiB, so the split count is cut."""
    build.build()
    w = synth.C2.replace(batch=400, context=64)
    lens = [1 + (7 * i) % 64 for i in range(w.batch)]
    case = Case(w, lens=lens, layers=[0])
    ctx, dev = case.ctx, case.ctx.device
    tol = TOL["bf16"]
    q = case.q[0].to(dev)
    ref = ctx.full_attention(0, q, case.seq_lens)
    status = torch.full((1,), 99, dtype=torch.int32, device=dev)
    for _ in range(2):
        out = torch.full_like(ref, float("nan"))
        binding.echokv_full_attention_noalloc(case.cfg, ctx.k_pools[0], ctx.v_pools[0], ctx.block_table,
                                              q, out, case.seq_lens, status_out=status)
        torch.cuda.synchronize()
        assert int(status.item()) == binding.ECHOKV_OK
        max_abs, rel_l2 = errors(out.cpu().numpy(), ref.cpu().numpy())
        assert max_abs <= tol["max_abs"] and rel_l2 <= tol["rel_l2"], (max_abs, rel_l2)
    max_abs, rel_l2 = errors(out.cpu().numpy(), case.oracle(0))
    assert max_abs <= tol["max_abs"] and rel_l2 <= tol["rel_l2"], (max_abs, rel_l2)
    case.close()


@pytest.mark.gpu
def test_noalloc_fp32_head_dim_64_with_sequence_slots():
    build.build()
    w = synth.C0.replace(batch=3, context=200)
    case = Case(w, lens=[200, 77, 130], layers=[0])
    ctx, dev = case.ctx, case.ctx.device
    tol = TOL["fp32"]
    # rows of the block table taken in another order: sequence i of the call lives in slot slots[i]
    slots = torch.tensor([2, 0, 1], dtype=torch.int32, device=dev)
    q = case.q[0].to(dev)[slots.long()].contiguous()
    lens = case.seq_lens[slots.long()].contiguous()
    ref = ctx.full_attention(0, q, lens, seq_slots=slots)
    for _ in range(2):
        out = torch.full_like(ref, float("nan"))
        binding.echokv_full_attention_noalloc(case.cfg, ctx.k_pools[0], ctx.v_pools[0], ctx.block_table,
                                              q, out, lens, seq_slots=slots)
        torch.cuda.synchronize()
        max_abs, rel_l2 = errors(out.cpu().numpy(), ref.cpu().numpy())
        assert max_abs <= tol["max_abs"] and rel_l2 <= tol["rel_l2"], (max_abs, rel_l2)
    want = case.oracle(0)[slots.cpu().numpy()]
    max_abs, rel_l2 = errors(out.cpu().numpy(), want)
    assert max_abs <= tol["max_abs"] and rel_l2 <= tol["rel_l2"], (max_abs, rel_l2)
    case.close()
